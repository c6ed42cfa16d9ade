// Reconstruction residual of Step 2 on the tensor cores (bf16, head_dim 128):
//   eps[p] = || v_i - W k~_i ||^2,  i = idx[p],  k~ = the key, or under RoPE decoupling the key
//   turned back by its position (the token index itself), channel c pairing with c + 64.
// The gather of the listed K and V rows is what costs (64 flop per byte: HBM-bound), so the
// kernel is built around keeping row loads in flight.  Per 128-row tile the accumulator in tensor
// memory is D = K_tile W^T (one chain of 8 tcgen05.mma); the epilogue subtracts the value row,
// which it reads from the tile's copy in shared memory, squares and adds along its TMEM lane.
//
// Persistent blocks (one per SM) own equal contiguous ranges of the global tile sequence.
//   warps 0-7   loaders: cp.async gathers of K and V rows into the stages, written directly in the
//               128-byte-swizzled layout the MMA reads; row indices are fetched one tile ahead.
//               Each thread gathers, for its rows, the 16-byte chunk qc of both key halves
//               (channels 8 qc.. and 64 + 8 qc..) and the same two chunks of V.
//   warp  8     MMA issuer, TMEM owner; also TMA-loads the unit's W when the range enters a new unit
//   warps 9-12  epilogue: thread = row
// Without RoPE: three stages of K | V (64 KB each), tiles published two behind the one being issued.
// With RoPE: the turned key is no longer a bf16 number, so it goes to the tensor cores as a bf16
// pair hi + lo (two chains over the same W), which keeps it to 2^-17 relative; two stages of
// K hi | K lo | V (96 KB each).  A loader thread turns its own eight channel pairs of each of its
// rows back once its own copies of the previous tile have landed (no cross-thread hand-over),
// writes hi in place and lo into the second operand tile.
#ifndef VECTOR_RESIDUAL_TC_CUH_
#define VECTOR_RESIDUAL_TC_CUH_

#include "common.cuh"
#include "internal.h"
#include "tcgen05.cuh"
#include "tma.cuh"

namespace vec {
namespace rtc {

constexpr int BOX_BYTES = 16384;                           // 128 rows x 128 bytes
constexpr int TILE = 128;
constexpr int OPERAND_BYTES = 2 * BOX_BYTES;               // 128 rows x 256 B as two swizzled halves
constexpr int EPI_WARPS = 4;

struct Params {
    int U, LH, n_idx, tpu;       // units, maps, rows per unit, tiles per unit
    long long N, n_tiles;        // keys per unit, U * tpu
};

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }

__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ long long range_begin(int b, long long n_tiles, int B) { return (long long)b * n_tiles / B; }

constexpr int R_LOADER_WARPS = 8;
constexpr int R_THREADS = 32 * (R_LOADER_WARPS + 1 + EPI_WARPS);
template <bool ROPE> struct RCfg {
    static constexpr int STAGES = ROPE ? 2 : 3;
    static constexpr int STAGE_BYTES = (ROPE ? 3 : 2) * OPERAND_BYTES;
    static constexpr int V_OFFSET = (ROPE ? 2 : 1) * OPERAND_BYTES;
    static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OPERAND_BYTES + 1024;     // + W
    static constexpr int TMEM_COLS = ROPE ? 256 : 512;          // one 128-column accumulator per stage
};
struct RSync {
    uint64_t full[3], done[3], empty[3];
    uint64_t w_full, w_empty;
    uint32_t tmem_base;
};

// grid: min(multiprocessors, n_tiles) blocks, R_THREADS threads, RCfg<ROPE>::SMEM_BYTES dynamic shared memory.
template <bool ROPE>
__global__ void __launch_bounds__(R_THREADS, 1)
residual_tc(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                 const __grid_constant__ CUtensorMap mapW, const int32_t* __restrict__ idx, const Params P,
                 const __grid_constant__ RopePhases rope, float* __restrict__ eps, int* __restrict__ fault) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ RSync sy;
    constexpr int STAGES = RCfg<ROPE>::STAGES, R_STAGE_BYTES = RCfg<ROPE>::STAGE_BYTES, TMEM_COLS = RCfg<ROPE>::TMEM_COLS;
    __shared__ unsigned long long phase_s[64];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* stage0 = smem;
    unsigned char* Ws = smem + STAGES * R_STAGE_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long gt_lo = range_begin(blockIdx.x, P.n_tiles, gridDim.x);
    const long long gt_hi = range_begin(blockIdx.x + 1, P.n_tiles, gridDim.x);
    const int n_my = (int)(gt_hi - gt_lo);

    // Programmatic launches on both sides (inside vector_route): the kernel after this one may be
    // scheduled as blocks here finish, and this one may have started before the kernel that writes
    // idx has drained -- the loaders, the only readers of idx, wait for it below.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid < 64) phase_s[tid] = rope.phase[tid];
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            tma::mbar_init(&sy.full[s], 32 * R_LOADER_WARPS);
            tma::mbar_init(&sy.done[s], 1);
            tma::mbar_init(&sy.empty[s], EPI_WARPS);
        }
        tma::mbar_init(&sy.w_full, 1);
        tma::mbar_init(&sy.w_empty, 1);
        tma::mbar_fence_init();
    }
    if (warp == R_LOADER_WARPS) {
        tc::tmem_alloc(&sy.tmem_base, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();

    if (warp < R_LOADER_WARPS) {
        // ------------------------------------------------------------------ loaders
        const int qc = tid & 7, rsub = tid >> 3;                    // chunk of each half, row inside a pass of 32 rows
        const uint32_t dst_thread = (uint32_t)rsub * 128u + (uint32_t)((qc ^ (rsub & 7)) << 4);   // + half * BOX + pass * 4096
        uint2 fr[8];                                                 // phases of this thread's eight channel pairs
#pragma unroll
        for (int e = 0; e < 8; ++e) fr[e] = reinterpret_cast<const uint2*>(phase_s)[qc * 8 + e];
        int32_t prev[4], cur[4], nxt[4];
        auto fetch_idx = [&](int i, int32_t (&out)[4]) {
            const long long gt = gt_lo + i;
            const int u = (int)(gt / P.tpu), t = (int)(gt - (long long)u * P.tpu);
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const int row = t * TILE + p * 32 + rsub;
                const int32_t v = row < P.n_idx ? idx[(size_t)u * P.n_idx + row] : -1;
                out[p] = (unsigned long long)v < (unsigned long long)P.N ? v : -1;   // an index outside the unit reads as a row of zeros
            }
        };
        // Turns this thread's pairs of the tile in stage s (rows listed in pos) and publishes the tile.
        auto turn_back = [&](int s, const int32_t (&pos)[4]) {
            const uint32_t hi0 = tma::smem_u32(stage0 + s * R_STAGE_BYTES) + dst_thread, lo0 = hi0 + OPERAND_BYTES;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                uint32_t xs[4], ys[4], xl[4], yl[4];
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(xs[0]), "=r"(xs[1]), "=r"(xs[2]), "=r"(xs[3]) : "r"(hi0 + p * 4096));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(ys[0]), "=r"(ys[1]), "=r"(ys[2]), "=r"(ys[3]) : "r"(hi0 + BOX_BYTES + p * 4096));
                const uint32_t tok = pos[p] >= 0 ? (uint32_t)pos[p] : 0u;      // rows past the list are zeros
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float x[2], y[2], cs[2], sn[2], xo[2], yo[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        x[h] = __uint_as_float(h ? (xs[e] & 0xffff0000u) : (xs[e] << 16));
                        y[h] = __uint_as_float(h ? (ys[e] & 0xffff0000u) : (ys[e] << 16));
                        rope_phase_cos_sin(tok, fr[2 * e + h], cs[h], sn[h]);
                    }
                    // both pairs of the word at once on the packed FMA path
                    const uint64_t x2 = tc::pack2(x[0], x[1]), y2 = tc::pack2(y[0], y[1]);
                    const uint64_t c2 = tc::pack2(cs[0], cs[1]), s2 = tc::pack2(sn[0], sn[1]);
                    tc::unpack2(tc::fma2(x2, c2, tc::mul2(y2, s2)), xo[0], xo[1]);
                    tc::unpack2(tc::fma2(y2, c2, tc::mul2(x2, tc::pack2(-sn[0], -sn[1]))), yo[0], yo[1]);
                    // hi = the pair rounded to bf16, lo = what the rounding left, again as bf16
                    xs[e] = pack2_bf16(xo[0], xo[1]);
                    ys[e] = pack2_bf16(yo[0], yo[1]);
                    xl[e] = pack2_bf16(xo[0] - __uint_as_float(xs[e] << 16), xo[1] - __uint_as_float(xs[e] & 0xffff0000u));
                    yl[e] = pack2_bf16(yo[0] - __uint_as_float(ys[e] << 16), yo[1] - __uint_as_float(ys[e] & 0xffff0000u));
                }
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(hi0 + p * 4096), "r"(xs[0]), "r"(xs[1]), "r"(xs[2]), "r"(xs[3]) : "memory");
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(hi0 + BOX_BYTES + p * 4096), "r"(ys[0]), "r"(ys[1]), "r"(ys[2]), "r"(ys[3]) : "memory");
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(lo0 + p * 4096), "r"(xl[0]), "r"(xl[1]), "r"(xl[2]), "r"(xl[3]) : "memory");
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(lo0 + BOX_BYTES + p * 4096), "r"(yl[0]), "r"(yl[1]), "r"(yl[2]), "r"(yl[3]) : "memory");
            }
            fence_async_proxy();
            tma::mbar_arrive(&sy.full[s]);
        };
        bool ok = true;
        asm volatile("griddepcontrol.wait;\n" ::: "memory");      // idx is complete and visible from here on
        if (n_my > 0) fetch_idx(0, cur);
#pragma unroll
        for (int p = 0; p < 4; ++p) prev[p] = -1;
        for (int i = 0; i < n_my && ok; ++i) {
            const int s = i % STAGES, round = i / STAGES;
            if (i + 1 < n_my) fetch_idx(i + 1, nxt);
            if (round > 0 && !tma::mbar_wait(&sy.empty[s], (round - 1) & 1, fault, 46)) { ok = false; break; }
            const int u = (int)((gt_lo + i) / P.tpu);
            const uint32_t kdst = tma::smem_u32(stage0 + s * R_STAGE_BYTES) + dst_thread;
            const uint32_t vdst = kdst + RCfg<ROPE>::V_OFFSET;
            const __nv_bfloat16* Ku = K + (size_t)u * P.N * 128 + qc * 8;
            const __nv_bfloat16* Vu = V + (size_t)u * P.N * 128 + qc * 8;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const bool valid = cur[p] >= 0;
                const size_t ro = valid ? (size_t)cur[p] * 128 : 0;
                const uint32_t nb = valid ? 16u : 0u;                  // zero fill past the end of the list
                cp_async16(kdst + p * 4096, Ku + ro, nb);
                cp_async16(kdst + BOX_BYTES + p * 4096, Ku + ro + 64, nb);
                cp_async16(vdst + p * 4096, Vu + ro, nb);
                cp_async16(vdst + BOX_BYTES + p * 4096, Vu + ro + 64, nb);
            }
            cp_async_commit();
            if (ROPE) {
                if (i > 0) {                             // this thread's copies of the previous tile have landed
                    cp_async_wait<1>();
                    turn_back((i - 1) % STAGES, prev);
                }
            } else if (i >= 2) {                         // ... of the tile before the previous one
                cp_async_wait<2>();
                fence_async_proxy();
                tma::mbar_arrive(&sy.full[(i - 2) % STAGES]);
            }
#pragma unroll
            for (int p = 0; p < 4; ++p) { prev[p] = cur[p]; cur[p] = nxt[p]; }
        }
        if (ROPE) {
            cp_async_wait<0>();
            if (ok && n_my > 0) turn_back((n_my - 1) % STAGES, prev);
        } else if (ok) {
            if (n_my > 1) { cp_async_wait<1>(); fence_async_proxy(); tma::mbar_arrive(&sy.full[(n_my - 2) % STAGES]); }
            cp_async_wait<0>();
            if (n_my > 0) { fence_async_proxy(); tma::mbar_arrive(&sy.full[(n_my - 1) % STAGES]); }
        } else {
            cp_async_wait<0>();
        }
    } else if (warp == R_LOADER_WARPS) {
        // ------------------------------------------------------------------ W loads and MMA issue
        if (lane == 0) {
            tma::prefetch_map(&mapW);
            const uint32_t w_addr = tma::smem_u32(Ws);
            const uint32_t idesc = tc::instr_desc(128, 128);
            int cur_u = -1;
            uint32_t n_units = 0;
            for (int i = 0; i < n_my; ++i) {
                const int s = i % STAGES, round = i / STAGES;
                const long long gt = gt_lo + i;
                const int u = (int)(gt / P.tpu);
                if (u != cur_u) {
                    if (n_units > 0 && !tma::mbar_wait(&sy.w_empty, (n_units - 1) & 1, fault, 47)) break;
                    tma::mbar_expect_tx(&sy.w_full, OPERAND_BYTES);
                    tma::load_3d(Ws, &mapW, 0, 0, u % P.LH, &sy.w_full);
                    tma::load_3d(Ws + BOX_BYTES, &mapW, 64, 0, u % P.LH, &sy.w_full);
                    if (!tma::mbar_wait(&sy.w_full, n_units & 1, fault, 48)) break;
                    cur_u = u;
                    ++n_units;
                }
                // the loaders start only once the kernel that writes idx has drained: do not spend this
                // thread's bounded polls on that kernel's run time (W, loaded above, is nobody's output)
                if (i == 0) asm volatile("griddepcontrol.wait;\n" ::: "memory");
                if (!tma::mbar_wait(&sy.full[s], round & 1, fault, 49)) break;
                tc::fence_after_sync();
                const uint32_t hi_addr = tma::smem_u32(stage0 + s * R_STAGE_BYTES), lo_addr = hi_addr + OPERAND_BYTES;
                const uint32_t d = sy.tmem_base + s * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t o = (ks >> 2) * BOX_BYTES + (ks & 3) * 32;
                    tc::mma_bf16(d, tc::smem_desc(hi_addr + o), tc::smem_desc(w_addr + o), idesc, ks > 0);
                }
                if (ROPE) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t o = (ks >> 2) * BOX_BYTES + (ks & 3) * 32;
                        tc::mma_bf16(d, tc::smem_desc(lo_addr + o), tc::smem_desc(w_addr + o), idesc, 1u);
                    }
                }
                tc::mma_commit(&sy.done[s]);
                const bool last_of_unit = (i + 1 == n_my) || (int)((gt + 1) / P.tpu) != u;
                if (last_of_unit) tc::mma_commit(&sy.w_empty);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                       // TMEM lanes this warp may read: 32 (warp % 4) ..
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = sy.tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t v_thread = (uint32_t)r * 128u;
        asm volatile("griddepcontrol.wait;\n" ::: "memory");      // as in the MMA thread: the waits below time this kernel only
        for (int i = 0; i < n_my; ++i) {
            const int s = i % STAGES, round = i / STAGES;
            // the value rows were written by the loaders: observe their barrier, then the MMA's
            if (!tma::mbar_wait_warp(&sy.full[s], round & 1, fault, 50)) break;
            if (!tma::mbar_wait_warp(&sy.done[s], round & 1, fault, 51)) break;
            tc::fence_after_sync();
            const long long gt = gt_lo + i;
            const int u = (int)(gt / P.tpu), t = (int)(gt - (long long)u * P.tpu);
            const uint32_t v_addr = tma::smem_u32(stage0 + s * R_STAGE_BYTES) + RCfg<ROPE>::V_OFFSET + v_thread;
            uint32_t ra[32], rb[32];
            const uint32_t taddr = lane_addr + s * 128;
            tc::tmem_ld32(taddr, ra);
            float e0 = 0.f, e1 = 0.f, e2 = 0.f, e3 = 0.f;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                uint32_t (&cur)[32] = (ch & 1) ? rb : ra;
                uint32_t (&nxt)[32] = (ch & 1) ? ra : rb;
                uint32_t vv[16];                           // columns 32 ch .. 32 ch + 31 of the value row
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int c16 = ch * 4 + q;            // 16-byte chunk of the 256-byte row
                    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                                 : "=r"(vv[4 * q]), "=r"(vv[4 * q + 1]), "=r"(vv[4 * q + 2]), "=r"(vv[4 * q + 3])
                                 : "r"(v_addr + (c16 >> 3) * BOX_BYTES + (((c16 & 7) ^ (r & 7)) << 4)));
                }
                tc::tmem_ld_wait(cur);
                if (ch < 3) tc::tmem_ld32(taddr + (ch + 1) * 32, nxt);
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float a = __uint_as_float(cur[j]) - __uint_as_float(vv[j >> 1] << 16);
                    const float b = __uint_as_float(cur[j + 1]) - __uint_as_float(vv[j >> 1] & 0xffff0000u);
                    const float c2 = __uint_as_float(cur[j + 2]) - __uint_as_float(vv[(j >> 1) + 1] << 16);
                    const float d2 = __uint_as_float(cur[j + 3]) - __uint_as_float(vv[(j >> 1) + 1] & 0xffff0000u);
                    e0 = fmaf(a, a, e0); e1 = fmaf(b, b, e1); e2 = fmaf(c2, c2, e2); e3 = fmaf(d2, d2, e3);
                }
            }
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) tma::mbar_arrive(&sy.empty[s]);
            const int row = t * TILE + r;
            if (row < P.n_idx) eps[(size_t)u * P.n_idx + row] = (e0 + e1) + (e2 + e3);
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == R_LOADER_WARPS) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(sy.tmem_base, TMEM_COLS);
    }
}

}  // namespace rtc
}  // namespace vec
#endif
