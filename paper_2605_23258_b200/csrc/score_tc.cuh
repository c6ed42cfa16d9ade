// Base importance score on the 5th-generation tensor cores (bf16, head_dim 128).
//
// The score of a key is the softmax mass it receives from the observation-window
// rows (causal inside the window), so the logits Q K^T are needed twice: once
// for the per-row normaliser, once for the per-key sum.  Both passes are
// persistent, warp-specialised kernels around tcgen05.mma with the accumulator
// in tensor memory; the orientation of the product is chosen per pass so that
// the reduction a thread performs runs along its own TMEM lane:
//
//   pass 1   D[row][key] = Q K^T   lane = window row  -> running (max, sum exp2) per row
//   pass 2   D[key][row] = K Q^T   lane = key         -> sum over rows of exp2(logit - lse[row])
//
// A work item is (unit, group of up to 256 rows, contiguous chunk of 128-key
// tiles); items are dealt round-robin to one block per SM with the row groups of
// a key chunk on neighbouring blocks, so that a chunk is fetched from HBM once
// and found in L2 by the other row groups.
//
// Roles inside a block (576 threads):
//   warps 0-15 softmax: two groups of two warpgroups; group 0 takes the block's even tiles,
//              group 1 the odd ones, so that while one group waits for its accumulator to be
//              refilled the other keeps the exponential unit busy; each thread owns one TMEM lane
//   warp  16   producer: TMA loads of the Q row group (once per item) and of the
//              K tiles into a 4-stage ring (128-byte swizzle, zero fill past the end)
//   warp  17   MMA issuer (one thread) and owner of the TMEM allocation
// All hand-offs are mbarriers; every wait is bounded and records a fault code.
#ifndef VECTOR_SCORE_TC_CUH_
#define VECTOR_SCORE_TC_CUH_

#include "common.cuh"
#include "tcgen05.cuh"
#include "tma.cuh"

namespace vec {
namespace stc {

using namespace tc;

constexpr int KT = 128;                    // keys per tile
constexpr int STAGES = 4;                  // K ring depth
constexpr int RG_ROWS = 256;               // window rows per row group
constexpr int BOX_BYTES = 16384;           // 128 rows x 128 bytes (64 bf16 of the head dimension)
constexpr int Q_BYTES = 4 * BOX_BYTES;     // [k half][256 rows][128 B]
constexpr int K_STAGE_BYTES = 2 * BOX_BYTES;   // [k half][128 keys][128 B]
constexpr int SMEM_BYTES = Q_BYTES + STAGES * K_STAGE_BYTES + 1024;
constexpr int SOFTMAX_WARPS = 16;
constexpr int THREADS = 32 * (SOFTMAX_WARPS + 2);
constexpr int TMEM_COLS = 512;

struct Params {
    int U, R, RG, w;            // units, rows per unit, row groups per unit, window
    long long N;                // keys per unit
    int nt, tpc, n_chunks;      // key tiles per unit, tiles per chunk, chunks per unit
    int n_items;                // U * n_chunks * RG
    float c;                    // logit scale * log2(e)
};

struct Item { int u, chunk, rg, t0, t1; };
__device__ __forceinline__ Item decode_item(int it, const Params& P) {
    Item i;
    i.rg = it % P.RG;
    const int uc = it / P.RG;
    i.chunk = uc % P.n_chunks;
    i.u = uc / P.n_chunks;
    i.t0 = i.chunk * P.tpc;
    i.t1 = min(P.nt, i.t0 + P.tpc);
    return i;
}

// Barriers and the TMEM base of one block.
struct Sync {
    uint64_t q_full, q_empty;
    uint64_t k_full[STAGES], k_empty[STAGES];
    uint64_t acc_full[4], acc_empty[4];
    uint32_t tmem_base;
};

// Producer and MMA roles are the same in both passes up to which operand is A and the tile shape.
//   PASS 1: per key tile two MMAs  D[buf = 2 (tile & 1) + rb] (128 x 128) = Q[rb] K^T
//   PASS 2: per key tile one MMA   D[buf = tile & 1]         (128 x 256) = K Q^T
template <int PASS>
__device__ __forceinline__ void producer_role(const CUtensorMap* mapQ, const CUtensorMap* mapK, const Params& P,
                                              Sync& sy, unsigned char* Qs, unsigned char* Ks, int* fault) {
    tma::prefetch_map(mapQ);
    tma::prefetch_map(mapK);
    uint32_t kcount = 0, icount = 0;
    for (int it = blockIdx.x; it < P.n_items; it += gridDim.x, ++icount) {
        const Item im = decode_item(it, P);
        if (icount > 0 && !tma::mbar_wait(&sy.q_empty, (icount - 1) & 1, fault, 11)) return;
        tma::mbar_expect_tx(&sy.q_full, Q_BYTES);
#pragma unroll
        for (int kh = 0; kh < 2; ++kh)
#pragma unroll
            for (int rb = 0; rb < 2; ++rb)
                tma::load_3d(Qs + kh * 2 * BOX_BYTES + rb * BOX_BYTES, mapQ, kh * 64, im.rg * RG_ROWS + rb * 128, im.u,
                             &sy.q_full);
        for (int t = im.t0; t < im.t1; ++t, ++kcount) {
            const uint32_t s = kcount % STAGES, round = kcount / STAGES;
            if (round > 0 && !tma::mbar_wait(&sy.k_empty[s], (round - 1) & 1, fault, 12)) return;
            tma::mbar_expect_tx(&sy.k_full[s], K_STAGE_BYTES);
            tma::load_3d(Ks + s * K_STAGE_BYTES, mapK, 0, t * KT, im.u, &sy.k_full[s]);
            tma::load_3d(Ks + s * K_STAGE_BYTES + BOX_BYTES, mapK, 64, t * KT, im.u, &sy.k_full[s]);
        }
    }
}

template <int PASS>
__device__ __forceinline__ void mma_role(const Params& P, Sync& sy, unsigned char* Qs, unsigned char* Ks, int* fault) {
    const uint32_t q_addr = tma::smem_u32(Qs), k_addr = tma::smem_u32(Ks);
    const uint32_t tmem = sy.tmem_base;
    uint32_t kcount = 0, icount = 0;
    for (int it = blockIdx.x; it < P.n_items; it += gridDim.x, ++icount) {
        const Item im = decode_item(it, P);
        if (!tma::mbar_wait(&sy.q_full, icount & 1, fault, 21)) return;
        fence_after_sync();
        for (int t = im.t0; t < im.t1; ++t, ++kcount) {
            const uint32_t s = kcount % STAGES, round = kcount / STAGES;
            if (!tma::mbar_wait(&sy.k_full[s], round & 1, fault, 22)) return;
            fence_after_sync();
            const uint32_t ks_addr = k_addr + s * K_STAGE_BYTES;
            if (PASS == 1) {
#pragma unroll
                for (int rb = 0; rb < 2; ++rb) {
                    const uint32_t buf = (kcount & 1) * 2 + rb, use = kcount >> 1;
                    if (use > 0 && !tma::mbar_wait(&sy.acc_empty[buf], (use - 1) & 1, fault, 23)) return;
                    fence_after_sync();
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t kh = ks >> 2, ko = (ks & 3) * 32;
                        mma_bf16(tmem + buf * 128, smem_desc(q_addr + kh * 2 * BOX_BYTES + rb * BOX_BYTES + ko),
                                 smem_desc(ks_addr + kh * BOX_BYTES + ko), instr_desc(128, 128), ks > 0);
                    }
                    mma_commit(&sy.acc_full[buf]);
                }
            } else {
                const uint32_t buf = kcount & 1, use = kcount >> 1;
                if (use > 0 && !tma::mbar_wait(&sy.acc_empty[buf], (use - 1) & 1, fault, 24)) return;
                fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t kh = ks >> 2, ko = (ks & 3) * 32;
                    mma_bf16(tmem + buf * 256, smem_desc(ks_addr + kh * BOX_BYTES + ko),
                             smem_desc(q_addr + kh * 2 * BOX_BYTES + ko), instr_desc(128, 256), ks > 0);
                }
                mma_commit(&sy.acc_full[buf]);
            }
            mma_commit(&sy.k_empty[s]);       // the stage is free once these MMAs have read it
        }
        mma_commit(&sy.q_empty);
    }
}

__device__ __forceinline__ void block_setup(Sync& sy, int empty_count) {
    if (threadIdx.x == 0) {
        tma::mbar_init(&sy.q_full, 1);
        tma::mbar_init(&sy.q_empty, 1);
#pragma unroll
        for (int s = 0; s < STAGES; ++s) { tma::mbar_init(&sy.k_full[s], 1); tma::mbar_init(&sy.k_empty[s], 1); }
#pragma unroll
        for (int b = 0; b < 4; ++b) { tma::mbar_init(&sy.acc_full[b], 1); tma::mbar_init(&sy.acc_empty[b], empty_count); }
        tma::mbar_fence_init();
    }
    if ((threadIdx.x >> 5) == SOFTMAX_WARPS + 1) {
        tmem_alloc(&sy.tmem_base, TMEM_COLS);
        tmem_relinquish();
    }
    fence_before_sync();
    __syncthreads();
    fence_after_sync();
}
__device__ __forceinline__ void block_teardown(Sync& sy) {
    fence_before_sync();
    __syncthreads();
    if ((threadIdx.x >> 5) == SOFTMAX_WARPS + 1) {
        __syncwarp();
        fence_after_sync();
        tmem_dealloc(sy.tmem_base, TMEM_COLS);
    }
}

// sum_i exp2(v[i] * c + n[i]) over 32 accumulator columns; n is either one value for all columns
// (pass 1: minus the row's reference) or a table in shared memory (pass 2: minus the rows' lse).
// Written in three stages (all FMAs, all exponentials, a tree of adds) so that the 32 MUFU
// operations issue back to back and nothing waits on the result of the one just before it.
__device__ __forceinline__ void sum_tree32(const float (&e)[32], uint64_t& acc) {
    uint64_t p[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) p[i] = pack2(e[2 * i], e[2 * i + 1]);
#pragma unroll
    for (int w = 8; w >= 1; w >>= 1)
#pragma unroll
        for (int i = 0; i < w; ++i) p[i] = add2(p[i], p[i + w]);
    acc = add2(acc, p[0]);
}
// The exponential unit (16 results per clock per SM) is what bounds both passes, so POLY16 of every
// 16 exponentials are evaluated on the FMA pipe instead: 2^x = 2^n p(f) with n = round(x),
// f = x - n in [-1/2, 1/2] and p the degree-4 minimax polynomial of 2^f (relative error 2.7e-6);
// n is added to the exponent field.  x is clamped to [-126, 128]: results below 2^-126 do not
// matter to a sum whose largest term is of order one, and at the upper end the exponent field must
// not wrap -- 2^128 comes out as about 3.4e38 (or a NaN), which the overflow test of the first pass
// (sum above 2^64, or not finite) catches, whereas a wrapped exponent would pass as a tiny term.
#ifndef VECTOR_SCORE_POLY16
#define VECTOR_SCORE_POLY16 4
#endif
constexpr int POLY16 = VECTOR_SCORE_POLY16;
__device__ __forceinline__ void exp2_poly_pair(float x0, float x1, float& e0, float& e1) {
    const float magic = 12582912.f;                    // 1.5 * 2^23: adding it leaves round(x) in the low mantissa bits
    x0 = fminf(fmaxf(x0, -126.f), 128.f);
    x1 = fminf(fmaxf(x1, -126.f), 128.f);
    const uint64_t x2 = pack2(x0, x1);
    const uint64_t t2 = add2(x2, pack2(magic, magic));
    const uint64_t n2 = add2(t2, pack2(-magic, -magic));
    const uint64_t f2 = fma2(n2, pack2(-1.f, -1.f), x2);
    uint64_t p2 = pack2(0.009570101276040077f, 0.009570101276040077f);
    p2 = fma2(p2, f2, pack2(0.05591785907745361f, 0.05591785907745361f));
    p2 = fma2(p2, f2, pack2(0.240247443318367f, 0.240247443318367f));
    p2 = fma2(p2, f2, pack2(0.6931217908859253f, 0.6931217908859253f));
    p2 = fma2(p2, f2, pack2(0.9999992847442627f, 0.9999992847442627f));
    float p0, p1, t0, t1;
    unpack2(p2, p0, p1);
    unpack2(t2, t0, t1);
    e0 = __uint_as_float(__float_as_uint(p0) + (__float_as_uint(t0) << 23));
    e1 = __uint_as_float(__float_as_uint(p1) + (__float_as_uint(t1) << 23));
}
// e[i] = 2^x[i] for 32 exponents: the first POLY16 of every 16 by polynomial, the rest by MUFU.
__device__ __forceinline__ void exp2_32(const float (&x)[32], float (&e)[32]) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) {
        if ((i & 15) < POLY16) exp2_poly_pair(x[i], x[i + 1], e[i], e[i + 1]);
        else { e[i] = ex2(x[i]); e[i + 1] = ex2(x[i + 1]); }
    }
}
__device__ __forceinline__ float exp2_sum32(const uint32_t (&v)[32], float c, float n) {
    const uint64_t c2 = pack2(c, c), n2 = pack2(n, n);
    float x[32], e[32];
#pragma unroll
    for (int i = 0; i < 32; i += 2) unpack2(fma2(pack2(v[i], v[i + 1]), c2, n2), x[i], x[i + 1]);
    exp2_32(x, e);
    uint64_t acc = pack2(0.f, 0.f);
    sum_tree32(e, acc);
    float s0, s1;
    unpack2(acc, s0, s1);
    return s0 + s1;
}
__device__ __forceinline__ void exp2_acc32(const uint32_t (&v)[32], float c, const float4* __restrict__ n, uint64_t& acc) {
    const uint64_t c2 = pack2(c, c);
    float x[32], e[32];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float4 n4 = n[i];
        unpack2(fma2(pack2(v[4 * i], v[4 * i + 1]), c2, pack2(n4.x, n4.y)), x[4 * i], x[4 * i + 1]);
        unpack2(fma2(pack2(v[4 * i + 2], v[4 * i + 3]), c2, pack2(n4.z, n4.w)), x[4 * i + 2], x[4 * i + 3]);
    }
    exp2_32(x, e);
    sum_tree32(e, acc);
}
__device__ __forceinline__ float max32(const uint32_t (&v)[32]) {
    float a = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
    float b = max3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
#pragma unroll
    for (int i = 6; i < 30; i += 4) {
        a = max3(a, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
        b = max3(b, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
    }
    return max3(a, b, fmaxf(__uint_as_float(v[30]), __uint_as_float(v[31])));
}

// One accumulator tile of pass 1 for this thread's row: 128 columns in four TMEM loads.  The
// buffer is handed back to the MMA warp as soon as the last load has completed.  The running sum l
// is kept against a reference m that lags behind the true maximum: the exponentials of a chunk do
// not wait for the chunk's maximum, and only when their sum exceeds 2^64 (always on an item's first
// chunk, where m = -inf) is the maximum taken, the reference moved and the chunk summed again.
template <bool MASKED>
__device__ __forceinline__ void softmax_tile_pass1(uint32_t taddr, float c, long long key0, long long last_visible,
                                                   float& m, float& l, uint64_t& empty_bar, int lane) {
    uint32_t ra[32], rb[32];
    tmem_ld32(taddr, ra);
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        uint32_t (&cur)[32] = (ch & 1) ? rb : ra;
        uint32_t (&nxt)[32] = (ch & 1) ? ra : rb;
        tmem_ld_wait(cur);
        if (ch < 3) {
            tmem_ld32(taddr + (ch + 1) * 32, nxt);
        } else {
            fence_before_sync();
            __syncwarp();
            if (lane == 0) tma::mbar_arrive(&empty_bar);
        }
        if (!MASKED) {
            // the sum itself tells whether a logit ran far ahead of the reference: only then is the
            // chunk's maximum looked for and the chunk summed again against it
            float s = exp2_sum32(cur, c, -m);
            if (!(s <= 1.8446744e19f)) {           // above 2^64, infinite (first chunk: m = -inf) or not a number
                const float cm = max32(cur) * c;
                l *= ex2(m - cm);
                m = cm;
                s = exp2_sum32(cur, c, -m);
            }
            l += s;
        } else {
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = key0 + ch * 32 + i > last_visible ? -INFINITY : __uint_as_float(cur[i]);
            float cm = v[0];
#pragma unroll
            for (int i = 1; i < 32; ++i) cm = fmaxf(cm, v[i]);
            const float m_new = fmaxf(m, cm * c);
            if (m_new > -INFINITY) {     // false only while every key so far is masked
                l *= ex2(m - m_new);     // exp2(-inf) = 0 on the first visible chunk
                float s0 = 0.f;
#pragma unroll
                for (int i = 0; i < 32; ++i) s0 += ex2(fmaf(v[i], c, -m_new));
                l += s0;
                m = m_new;
            }
        }
    }
}

// One accumulator tile of pass 2 for this thread's key: sum over 128 rows of exp2(logit2 - lse2[row]).
// Masked tiles: row j of the window (j0 = window index of the tile's first row, advancing cyclically
// with period w) sees this key only if key - (N - w) <= j.
template <bool MASKED>
__device__ __forceinline__ float softmax_tile_pass2(uint32_t taddr, float c, const float* nl_w, long long key_rel,
                                                    int j0, int w, uint64_t& empty_bar, int lane) {
    uint32_t ra[32], rb[32];
    tmem_ld32(taddr, ra);
    uint64_t acc = pack2(0.f, 0.f);
    float sm = 0.f;
    int j = j0;
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
        uint32_t (&cur)[32] = (ch & 1) ? rb : ra;
        uint32_t (&nxt)[32] = (ch & 1) ? ra : rb;
        tmem_ld_wait(cur);
        if (ch < 3) {
            tmem_ld32(taddr + (ch + 1) * 32, nxt);
        } else {
            fence_before_sync();
            __syncwarp();
            if (lane == 0) tma::mbar_arrive(&empty_bar);
        }
        if (!MASKED) {
            exp2_acc32(cur, c, reinterpret_cast<const float4*>(nl_w + ch * 32), acc);
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const float p = ex2(fmaf(__uint_as_float(cur[i]), c, nl_w[ch * 32 + i]));
                if (key_rel <= j) sm += p;
                if (++j == w) j = 0;
            }
        }
    }
    float s0, s1;
    unpack2(acc, s0, s1);
    return (s0 + s1) + sm;
}

// ---- pass 1 -----------------------------------------------------------------
// partial[((u * n_chunks + chunk) * 2 + group) * R + row] = (reference, sum of exp2 against it) of the
// row over the visible keys of the chunk's even (group 0) or odd (group 1) tiles, in units of log2 (logit * scale * log2 e).  grid: one block per SM.
__global__ void __launch_bounds__(THREADS, 1)
score_pass1_tc(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK, const Params P,
               float2* __restrict__ partial, int* __restrict__ fault) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ Sync sy;
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* Qs = smem;
    unsigned char* Ks = smem + Q_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    block_setup(sy, 4);

    if (warp == SOFTMAX_WARPS) {
        if (lane == 0) producer_role<1>(&mapQ, &mapK, P, sy, Qs, Ks, fault);
    } else if (warp == SOFTMAX_WARPS + 1) {
        if (lane == 0) mma_role<1>(P, sy, Qs, Ks, fault);
    } else {
        const int grp = warp >> 3, wg = (warp >> 2) & 1, quarter = warp & 3;
        const uint32_t lane_addr = sy.tmem_base + ((uint32_t)(quarter * 32) << 16);
        const long long vis0 = P.N - P.w;               // keys below this index are visible to every row
        uint32_t tcount = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < P.n_items && ok; it += gridDim.x) {
            const Item im = decode_item(it, P);
            const int row = im.rg * RG_ROWS + wg * 128 + quarter * 32 + lane;
            const bool wg_active = im.rg * RG_ROWS + wg * 128 < P.R;
            const long long last_visible = vis0 + (row % P.w);
            float m = -INFINITY, l = 0.f;
            for (int t = im.t0; t < im.t1; ++t, ++tcount) {
                if ((int)(tcount & 1) != grp) continue;
                const uint32_t buf = (tcount & 1) * 2 + wg, use = tcount >> 1;
                if (!tma::mbar_wait_warp(&sy.acc_full[buf], use & 1, fault, 31)) { ok = false; break; }
                fence_after_sync();
                if (wg_active) {
                    const uint32_t taddr = lane_addr + buf * 128;
                    const long long key0 = (long long)t * KT;
                    if (key0 + KT <= vis0) softmax_tile_pass1<false>(taddr, P.c, 0, 0, m, l, sy.acc_empty[buf], lane);
                    else softmax_tile_pass1<true>(taddr, P.c, key0, last_visible, m, l, sy.acc_empty[buf], lane);
                } else {
                    __syncwarp();
                    if (lane == 0) tma::mbar_arrive(&sy.acc_empty[buf]);
                }
            }
            if (ok && row < P.R)
                partial[(((size_t)im.u * P.n_chunks + im.chunk) * 2 + grp) * P.R + row] = make_float2(m, l);
        }
    }
    block_teardown(sy);
}

// lse2[u][row] = log2 sum over all visible keys of exp2(logit2), from the chunk partials.  grid (U).
__global__ void score_lse2_combine(const float2* __restrict__ partial, int R, int n_chunks, float* __restrict__ lse2) {
    const int u = blockIdx.x;
    for (int row = threadIdx.x; row < R; row += blockDim.x) {
        float M = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, partial[((size_t)u * n_chunks + c) * R + row].x);
        float L = 0.f;
        for (int c = 0; c < n_chunks; ++c) {
            const float2 p = partial[((size_t)u * n_chunks + c) * R + row];
            if (p.x > -INFINITY) L += p.y * exp2f(p.x - M);
        }
        lse2[(size_t)u * R + row] = M + log2f(L);
    }
}

// ---- pass 2 -----------------------------------------------------------------
// raw_part[(u * 2 RG + 2 rg + h) * N + key] = sum over rows [rg*256 + h*128, +128) of the softmax
// probability of `key`; the parts are added up by the pooling kernel.  grid: one block per SM.
__global__ void __launch_bounds__(THREADS, 1)
score_pass2_tc(const __grid_constant__ CUtensorMap mapQ, const __grid_constant__ CUtensorMap mapK, const Params P,
               const float* __restrict__ lse2, float* __restrict__ raw_part, int* __restrict__ fault) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ Sync sy;
    __shared__ __align__(16) float neg_lse[SOFTMAX_WARPS][128];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* Qs = smem;
    unsigned char* Ks = smem + Q_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    block_setup(sy, 8);

    if (warp == SOFTMAX_WARPS) {
        if (lane == 0) producer_role<2>(&mapQ, &mapK, P, sy, Qs, Ks, fault);
    } else if (warp == SOFTMAX_WARPS + 1) {
        if (lane == 0) mma_role<2>(P, sy, Qs, Ks, fault);
    } else {
        const int grp = warp >> 3, wg = (warp >> 2) & 1, quarter = warp & 3;
        const uint32_t lane_addr = sy.tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int key_in_tile = quarter * 32 + lane;
        const long long vis0 = P.N - P.w;
        float* nl_w = neg_lse[warp];                   // this warp's copy of -lse2 of its 128 rows
        uint32_t tcount = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < P.n_items && ok; it += gridDim.x) {
            const Item im = decode_item(it, P);
            const bool wg_active = im.rg * RG_ROWS + wg * 128 < P.R;
            const int row_base = im.rg * RG_ROWS + wg * 128;
            __syncwarp();
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int row = row_base + k * 32 + lane;
                nl_w[k * 32 + lane] = row < P.R ? -lse2[(size_t)im.u * P.R + row] : -INFINITY;   // -inf: padding rows add 0
            }
            __syncwarp();
            float* out = raw_part + ((size_t)im.u * 2 * P.RG + 2 * im.rg + wg) * P.N;
            for (int t = im.t0; t < im.t1; ++t, ++tcount) {
                if ((int)(tcount & 1) != grp) continue;
                const uint32_t buf = tcount & 1, use = tcount >> 1;
                if (!tma::mbar_wait_warp(&sy.acc_full[buf], use & 1, fault, 32)) { ok = false; break; }
                fence_after_sync();
                const long long key = (long long)t * KT + key_in_tile;
                float colsum = 0.f;
                if (wg_active) {
                    const uint32_t taddr = lane_addr + buf * 256 + wg * 128;
                    if ((long long)t * KT + KT <= vis0)
                        colsum = softmax_tile_pass2<false>(taddr, P.c, nl_w, 0, 0, 0, sy.acc_empty[buf], lane);
                    else
                        colsum = softmax_tile_pass2<true>(taddr, P.c, nl_w, key - vis0, row_base % P.w, P.w, sy.acc_empty[buf], lane);
                } else {
                    __syncwarp();
                    if (lane == 0) tma::mbar_arrive(&sy.acc_empty[buf]);
                }
                if (key < P.N) out[key] = colsum;           // zero for a row block past the last row
            }
        }
    }
    block_teardown(sy);
}

// raw[i] = sum of the parts; score[i] = max of raw over the centred window restricted to the
// prefix i < N - w; +inf for the window tokens.  grid (ceil(N / 1024), U), 256 threads.
constexpr int POOL_TILE = 1024;
__global__ void __launch_bounds__(256)
score_pool_parts(const float* __restrict__ raw_part, int parts, long long N, int w, int r, float* __restrict__ raw_out,
                 float* __restrict__ score) {
    __shared__ float rs[POOL_TILE + 16];
    const int u = blockIdx.y;
    const long long i0 = (long long)blockIdx.x * POOL_TILE;
    const float* base = raw_part + (size_t)u * parts * N;
    const long long P = N - w;
    for (int e = threadIdx.x; e < POOL_TILE + 2 * r; e += 256) {
        const long long i = i0 - r + e;
        float v = -INFINITY;
        if (i >= 0 && i < N) {
            v = 0.f;
            for (int p = 0; p < parts; ++p) v += base[(size_t)p * N + i];
            if (raw_out && e >= r && e < POOL_TILE + r) raw_out[(size_t)u * N + i] = v;
            if (i >= P) v = -INFINITY;           // pooling looks at the prefix only
        }
        rs[e] = v;
    }
    __syncthreads();
    for (int e = threadIdx.x; e < POOL_TILE; e += 256) {
        const long long i = i0 + e;
        if (i >= N) break;
        float best = INFINITY;
        if (i < P) {
            best = rs[e];
            for (int k = 1; k <= 2 * r; ++k) best = fmaxf(best, rs[e + k]);
        }
        score[(size_t)u * N + i] = best;
    }
}

// The same for N a multiple of 4: 16-byte loads and stores, four keys per thread.
__global__ void __launch_bounds__(256)
score_pool_parts_v4(const float* __restrict__ raw_part, int parts, long long N, int w, int r, float* __restrict__ raw_out,
                    float* __restrict__ score) {
    __shared__ __align__(16) float rs[POOL_TILE + 16];          // keys i0 - 8 .. i0 + POOL_TILE + 8
    const int u = blockIdx.y;
    const long long i0 = (long long)blockIdx.x * POOL_TILE;
    const float* base = raw_part + (size_t)u * parts * N;
    const long long P = N - w;
    for (int e4 = threadIdx.x; e4 < (POOL_TILE + 16) / 4; e4 += 256) {
        const long long i = i0 - 8 + 4 * e4;
        float4 v = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
        if (i >= 0 && i < N) {
            v = *reinterpret_cast<const float4*>(base + i);
            for (int p = 1; p < parts; ++p) {
                const float4 x = *reinterpret_cast<const float4*>(base + (size_t)p * N + i);
                v.x += x.x; v.y += x.y; v.z += x.z; v.w += x.w;
            }
            if (raw_out && e4 >= 2 && e4 < 2 + POOL_TILE / 4) *reinterpret_cast<float4*>(raw_out + (size_t)u * N + i) = v;
            if (i + 0 >= P) v.x = -INFINITY;           // pooling looks at the prefix only
            if (i + 1 >= P) v.y = -INFINITY;
            if (i + 2 >= P) v.z = -INFINITY;
            if (i + 3 >= P) v.w = -INFINITY;
        }
        *reinterpret_cast<float4*>(rs + 4 * e4) = v;
    }
    __syncthreads();
    const long long i = i0 + 4 * threadIdx.x;
    if (i >= N) return;
    float x[20];                                                // keys i - 8 .. i + 11
#pragma unroll
    for (int k = 0; k < 5; ++k) {
        const float4 v = *reinterpret_cast<const float4*>(rs + 4 * threadIdx.x + 4 * k);
        x[4 * k] = v.x; x[4 * k + 1] = v.y; x[4 * k + 2] = v.z; x[4 * k + 3] = v.w;
    }
    float o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float best = x[8 + j];
#pragma unroll
        for (int k = 1; k <= 7; ++k)
            if (k <= r) best = fmaxf(best, fmaxf(x[8 + j - k], x[8 + j + k]));
        o[j] = i + j < P ? best : INFINITY;
    }
    *reinterpret_cast<float4*>(score + (size_t)u * N + i) = make_float4(o[0], o[1], o[2], o[3]);
}

}  // namespace stc
}  // namespace vec
#endif
