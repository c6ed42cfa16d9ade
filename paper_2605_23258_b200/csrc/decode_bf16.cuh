// Split-KV decode attention over the mixed cache for bf16, head_dim 128.
//
// HBM-bound streaming kernel: every K/V row is read once.  A block owns a slice
// of a unit's 64-row tiles (retained tiles carry K and V, key-only tiles K),
// stages them with 16-byte cp.async into XOR-swizzled shared memory through a
// 3-deep ring, and each of its 4 warps takes 16 keys of every tile:
//   S = Q K^T      m16n8k16 bf16 MMA, the g query heads padded to the 16 MMA rows
//   online softmax in fp32 registers (exp2 with the scale folded in)
//   O += P V       (retained tile)   or   A += P K   (key-only tile: the
//                  p-weighted key sum that the merge step multiplies by W)
// P is fed to the second MMA as a bf16 hi + lo pair so that its rounding stays
// near 2^-17 relative.  The MMAs only keep the FP32 pipe out of the way of the
// memory stream; the kernel's roofline is HBM bandwidth.
#ifndef VECTOR_DECODE_BF16_CUH_
#define VECTOR_DECODE_BF16_CUH_

#include "common.cuh"

namespace vec {
namespace dbf {

constexpr int TILE = 64;              // keys per tile
constexpr int STAGES = 3;
constexpr int ROW_BYTES = 256;        // 128 bf16
constexpr int MAT_BYTES = TILE * ROW_BYTES;          // 16 KB
constexpr int STAGE_BYTES = 2 * MAT_BYTES;           // K tile + V tile
constexpr int STASH_BYTES = 4 * 32 * 32 * 4;         // one accumulator set per warp, parked at the pool switch
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STASH_BYTES;     // 112 KB
constexpr int REC = 2 + 2 * 128;                     // partial record floats per head

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes));
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8) += A(16x16) B(16x8); only rows 0..7 of A are non-zero, so the upper
// accumulator half stays zero and is parked in a scratch pair.
__device__ __forceinline__ void mma_lo8(float& c0, float& c1, float& z0, float& z1, uint32_t a0, uint32_t a2,
                                        uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%10,%10};\n"
        : "+f"(c0), "+f"(c1), "=f"(z0), "=f"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// byte offset of 16-byte chunk `chunk` of row `row` inside a swizzled 64x256-byte tile
__device__ __forceinline__ uint32_t swz(int row, int chunk) { return row * ROW_BYTES + ((chunk ^ (row & 7)) << 4); }

struct TileDesc {
    const __nv_bfloat16* k;   // first row of the tile's keys
    const __nv_bfloat16* v;   // first row of its values, or nullptr for a key-only tile
    int nrows;
};

__device__ __forceinline__ TileDesc tile_desc(int t, int n_rt, int u, const __nv_bfloat16* ret_k,
                                              const __nv_bfloat16* ret_v, const __nv_bfloat16* apx_k,
                                              int64_t cap_ret, int64_t cap_apx, int n_ret, int n_apx) {
    TileDesc d;
    if (t < n_rt) {
        int row0 = t * TILE;
        d.k = ret_k + ((size_t)u * cap_ret + row0) * 128;
        d.v = ret_v + ((size_t)u * cap_ret + row0) * 128;
        d.nrows = min(TILE, n_ret - row0);
    } else {
        int row0 = (t - n_rt) * TILE;
        d.k = apx_k + ((size_t)u * cap_apx + row0) * 128;
        d.v = nullptr;
        d.nrows = min(TILE, n_apx - row0);
    }
    return d;
}

__device__ __forceinline__ void issue_tile(const TileDesc& d, unsigned char* stage, int tid) {
    const uint32_t ks = smem_u32(stage), vs = ks + MAT_BYTES;
#pragma unroll
    for (int i = 0; i < (TILE * 16) / 128; ++i) {
        int c = tid + 128 * i, row = c >> 4, chunk = c & 15;
        bool ok = row < d.nrows;
        int srow = ok ? row : 0;                      // rows past the end are zero-filled, never read
        cp_async16(ks + swz(row, chunk), (const char*)d.k + (size_t)srow * ROW_BYTES + chunk * 16, ok ? 16 : 0);
        if (d.v) cp_async16(vs + swz(row, chunk), (const char*)d.v + (size_t)srow * ROW_BYTES + chunk * 16, ok ? 16 : 0);
    }
}

// grid (n_splits, U), 128 threads, SMEM_BYTES dynamic shared memory.
__global__ void __launch_bounds__(128, 2)
decode_split_bf16_d128(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ ret_k,
                       const __nv_bfloat16* __restrict__ ret_v, const __nv_bfloat16* __restrict__ apx_k,
                       int64_t cap_ret, int64_t cap_apx, int n_ret, int n_apx, int g, float scale_log2e,
                       float* __restrict__ partial) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int u = blockIdx.y, split = blockIdx.x, n_splits = gridDim.x;
    const int tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3;
    const int n_rt = (n_ret + TILE - 1) / TILE, n_at = (n_apx + TILE - 1) / TILE, n_tiles = n_rt + n_at;
    const int t_lo = (int)((int64_t)split * n_tiles / n_splits);
    const int t_hi = (int)((int64_t)(split + 1) * n_tiles / n_splits);

    // Q fragments of head row `gid` (zero for padding rows): 8 k-steps x {dims 2tig.., dims 8+2tig..}
    uint32_t qa[8][2];
    {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)u * g + min(gid, g - 1)) * 128);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = gid < g ? qrow[ks * 8 + tig] : 0u;
            qa[ks][1] = gid < g ? qrow[ks * 8 + 4 + tig] : 0u;
        }
    }
    // One accumulator set.  A block's tiles are ordered retained first, key-only second, so the
    // set collects sum p v until the first key-only tile, is parked in shared memory there (its
    // later rescaling tracked by one factor), and then collects sum p k.
    float acc[16][2];
#pragma unroll
    for (int n = 0; n < 16; ++n) { acc[n][0] = acc[n][1] = 0.f; }
    float* stash = reinterpret_cast<float*>(smem + STAGES * STAGE_BYTES) + wq * 32 * 32 + lane;
    bool stashed = false;
    float stash_scale = 1.f;
    float zz[4][2];                    // write-only parking for the unused accumulator halves
    float m = -INFINITY, l = 0.f;      // running max (scaled log2 units) and this thread's share of the sum

    // prologue: STAGES-1 tiles in flight
#pragma unroll
    for (int s = 0; s < STAGES - 1; ++s) {
        int t = t_lo + s;
        if (t < t_hi)
            issue_tile(tile_desc(t, n_rt, u, ret_k, ret_v, apx_k, cap_ret, cap_apx, n_ret, n_apx),
                       smem + s * STAGE_BYTES, tid);
        cp_commit();
    }
    for (int t = t_lo; t < t_hi; ++t) {
        cp_wait<STAGES - 2>();
        __syncthreads();
        {   // refill the stage consumed one iteration ago
            int tn = t + STAGES - 1;
            if (tn < t_hi)
                issue_tile(tile_desc(tn, n_rt, u, ret_k, ret_v, apx_k, cap_ret, cap_apx, n_ret, n_apx),
                           smem + ((tn - t_lo) % STAGES) * STAGE_BYTES, tid);
            cp_commit();
        }
        const bool retained = t < n_rt;
        const int nrows = retained ? min(TILE, n_ret - t * TILE) : min(TILE, n_apx - (t - n_rt) * TILE);
        const int kr0 = wq * 16;
        if (kr0 >= nrows) continue;            // this warp's 16 keys lie past the end of the pool
        const uint32_t ks_base = smem_u32(smem + ((t - t_lo) % STAGES) * STAGE_BYTES);
        const uint32_t vs_base = retained ? ks_base + MAT_BYTES : ks_base;

        // ---- S = Q K^T for 16 keys (two 8-key column tiles)
        float s0[2], s1[2];
        {
            // four independent accumulation chains (even / odd k-steps x two key tiles)
            float e0[2] = {0.f, 0.f}, e1[2] = {0.f, 0.f}, o0[2] = {0.f, 0.f}, o1[2] = {0.f, 0.f};
            const int mat = lane >> 3, r = lane & 7;
            const int key = kr0 + r + (mat >> 1) * 8;
#pragma unroll
            for (int ks = 0; ks < 8; ks += 2) {
                uint32_t b0, b1, b2, b3, c0, c1, c2, c3;
                ldsm_x4(ks_base + swz(key, ks * 2 + (mat & 1)), b0, b1, b2, b3);
                ldsm_x4(ks_base + swz(key, ks * 2 + 2 + (mat & 1)), c0, c1, c2, c3);
                mma_lo8(e0[0], e0[1], zz[0][0], zz[0][1], qa[ks][0], qa[ks][1], b0, b1);
                mma_lo8(e1[0], e1[1], zz[1][0], zz[1][1], qa[ks][0], qa[ks][1], b2, b3);
                mma_lo8(o0[0], o0[1], zz[2][0], zz[2][1], qa[ks + 1][0], qa[ks + 1][1], c0, c1);
                mma_lo8(o1[0], o1[1], zz[3][0], zz[3][1], qa[ks + 1][0], qa[ks + 1][1], c2, c3);
            }
            s0[0] = e0[0] + o0[0]; s0[1] = e0[1] + o0[1];
            s1[0] = e1[0] + o1[0]; s1[1] = e1[1] + o1[1];
        }
        // ---- online softmax over these 16 keys (row = head gid, shared by the 4 threads of a quad)
        const int kc = kr0 + 2 * tig;
        float t00 = kc < nrows ? s0[0] * scale_log2e : -INFINITY;
        float t01 = kc + 1 < nrows ? s0[1] * scale_log2e : -INFINITY;
        float t10 = kc + 8 < nrows ? s1[0] * scale_log2e : -INFINITY;
        float t11 = kc + 9 < nrows ? s1[1] * scale_log2e : -INFINITY;
        float mx = fmaxf(fmaxf(t00, t01), fmaxf(t10, t11));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (!retained && !stashed) {               // first key-only tile this warp works on
#pragma unroll
            for (int n = 0; n < 16; ++n) {
                stash[(2 * n) * 32] = acc[n][0];
                stash[(2 * n + 1) * 32] = acc[n][1];
                acc[n][0] = acc[n][1] = 0.f;
            }
            stashed = true;
            stash_scale = 1.f;
        }
        const float m_new = fmaxf(m, mx);          // finite: key kr0 is valid for every row
        const float alpha = exp2f(m - m_new);      // 0 on the first tile
        const float p00 = exp2f(t00 - m_new), p01 = exp2f(t01 - m_new);
        const float p10 = exp2f(t10 - m_new), p11 = exp2f(t11 - m_new);
        l = l * alpha + (p00 + p01) + (p10 + p11);
        m = m_new;
        stash_scale *= alpha;
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
            for (int n = 0; n < 16; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; }
        }
        // P as bf16 hi + lo
        const __nv_bfloat16 h00 = __float2bfloat16_rn(p00), h01 = __float2bfloat16_rn(p01);
        const __nv_bfloat16 h10 = __float2bfloat16_rn(p10), h11 = __float2bfloat16_rn(p11);
        const uint32_t pa_hi0 = pack_bf16(__bfloat162float(h00), __bfloat162float(h01));
        const uint32_t pa_hi2 = pack_bf16(__bfloat162float(h10), __bfloat162float(h11));
        const uint32_t pa_lo0 = pack_bf16(p00 - __bfloat162float(h00), p01 - __bfloat162float(h01));
        const uint32_t pa_lo2 = pack_bf16(p10 - __bfloat162float(h10), p11 - __bfloat162float(h11));
        // ---- accumulate P x (V tile | K tile) over the 16 column tiles of 8 dims
        {
            const int mat = lane >> 3, r = lane & 7;
            const int key = kr0 + r + (mat & 1) * 8;
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vs_base + swz(key, np * 2 + (mat >> 1)), b0, b1, b2, b3);
                mma_lo8(acc[2 * np][0], acc[2 * np][1], zz[0][0], zz[0][1], pa_hi0, pa_hi2, b0, b1);
                mma_lo8(acc[2 * np + 1][0], acc[2 * np + 1][1], zz[1][0], zz[1][1], pa_hi0, pa_hi2, b2, b3);
                mma_lo8(acc[2 * np][0], acc[2 * np][1], zz[2][0], zz[2][1], pa_lo0, pa_lo2, b0, b1);
                mma_lo8(acc[2 * np + 1][0], acc[2 * np + 1][1], zz[3][0], zz[3][1], pa_lo0, pa_lo2, b2, b3);
            }
        }
    }
    cp_wait<0>();
    __syncthreads();                    // every stage is free: reuse it for the cross-warp combine
    float* sm = reinterpret_cast<float*>(smem);          // [4 warps][8 heads][REC]
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    {
        float* rec = sm + ((size_t)wq * 8 + gid) * REC;
        if (tig == 0) { rec[0] = m; rec[1] = l; }
#pragma unroll
        for (int n = 0; n < 16; ++n) {
            // value part: the parked set if the switch happened, else the live set; key part: the rest
            float v0 = stashed ? stash[(2 * n) * 32] * stash_scale : acc[n][0];
            float v1 = stashed ? stash[(2 * n + 1) * 32] * stash_scale : acc[n][1];
            rec[2 + n * 8 + 2 * tig] = v0;
            rec[2 + n * 8 + 2 * tig + 1] = v1;
            rec[2 + 128 + n * 8 + 2 * tig] = stashed ? acc[n][0] : 0.f;
            rec[2 + 128 + n * 8 + 2 * tig + 1] = stashed ? acc[n][1] : 0.f;
        }
    }
    __syncthreads();
    float* out = partial + ((size_t)u * n_splits + split) * g * REC;
    for (int a = 0; a < g; ++a) {
        const float m0 = sm[(0 * 8 + a) * REC], m1 = sm[(1 * 8 + a) * REC], m2 = sm[(2 * 8 + a) * REC],
                    m3 = sm[(3 * 8 + a) * REC];
        const float M = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
        const float f0 = m0 > -INFINITY ? exp2f(m0 - M) : 0.f, f1 = m1 > -INFINITY ? exp2f(m1 - M) : 0.f;
        const float f2 = m2 > -INFINITY ? exp2f(m2 - M) : 0.f, f3 = m3 > -INFINITY ? exp2f(m3 - M) : 0.f;
        for (int c = tid; c < REC; c += 128) {
            float v;
            if (c == 0) v = M * 0.69314718055994531f;       // back to natural-log units for the merge step
            else v = f0 * sm[(0 * 8 + a) * REC + c] + f1 * sm[(1 * 8 + a) * REC + c] +
                     f2 * sm[(2 * 8 + a) * REC + c] + f3 * sm[(3 * 8 + a) * REC + c];
            out[a * REC + c] = v;
        }
    }
}

}  // namespace dbf
}  // namespace vec
#endif
