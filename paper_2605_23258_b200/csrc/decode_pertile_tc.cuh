// Decode attention over the mixed cache with the reconstruction formed tile by tile on the
// 5th-generation tensor cores (bf16, head_dim 128, stored keys): the alternative form
//   o = sum_R p_i v_i + sum_A p_i (W k_i)
// of the generation-time attention (paper Section 3.2, Step 3: the value of an approximated token
// is rebuilt as W k).  For every tile of 128 key-only keys the reconstructed values are
// materialised as  V^T = W K_tile^T  (128 dims x 128 keys x 128) by tcgen05.mma with the accumulator
// in tensor memory -- W and K are bf16 data, so the products are exact -- brought back to shared
// memory as fp16 (eleven mantissa bits: a reconstructed value of size 25 is off by at most 0.006, a
// bf16 rounding would cost four times that) over the keys they came from, and then weighted like
// stored values, with the probabilities as an fp16 pair hi + lo.
//
// The mixed cache is streamed once, as in the factored kernel: 32 KB tiles (64 retained keys + their
// 64 values, or 128 key-only keys) dealt in equal contiguous ranges to one persistent block per
// multiprocessor.  Roles inside a block (256 threads):
//   warps 0-1  consumers: tile i belongs to warp i % 2.  Scores S = Q K^T with warp-level MMAs (the g
//              query heads padded to the MMA rows), online softmax, O += P V with P as bf16 hi + lo.
//              For a key-only tile V is the reconstructed tile: the warp says when it has read the
//              keys for the last time, waits for the conversion, and adds P V
//   warp  2    producer: TMA loads of the tiles into four 32 KB slots
//   warp  3    MMA issuer, owner of tensor memory; TMA-loads the unit's W when the range enters a unit
//   warps 4-7  conversion: thread = output dim (its TMEM lane).  Per key-only tile: reads its row of
//              V^T from tensor memory and writes it as fp16 over the tile's keys (the slot is a
//              [128 dims][128 keys] tile from then on)
// Per unit every consumer warp leaves one partial record (m, l, sum p v + sum p (W k)); the merge
// kernel combines the records without applying W.
// All hand-offs are mbarriers; every wait is bounded and records a fault code.
#ifndef VECTOR_DECODE_PERTILE_TC_CUH_
#define VECTOR_DECODE_PERTILE_TC_CUH_

#include "common.cuh"
#include "decode_bf16.cuh"
#include "internal.h"
#include "tcgen05.cuh"
#include "tma.cuh"

namespace vec {
namespace dpt {

using dbf::Plan;
using dbf::REC;

constexpr int KEYS = 64;
constexpr int CONSUMERS = 2;
constexpr int SLOTS = 4;                     // a multiple of CONSUMERS: a slot always serves the same warp
constexpr int SLOT_BYTES = 32768;
constexpr int HALF_BYTES = 16384;
constexpr int W_BYTES = 32768;
constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + W_BYTES + 1024;
constexpr int NB = 3;                        // V^T accumulators in tensor memory (128 columns each)
constexpr int TMEM_COLS = 512;
constexpr int THREADS = 256;
constexpr int RECON_WARPS = 4;
static_assert(SLOTS % CONSUMERS == 0, "a slot must always be consumed by the same warp");

struct Maps {
    CUtensorMap ret_k, ret_v;            // rank 3: (128 dims, pool rows, U units), box 64 x 64 x 1, 128B swizzle
    CUtensorMap apx_k;                   // the same tensor, box 64 x 128 x 1: 128 keys per half of the head dimension
    CUtensorMap w;                       // rank 3: (128 in, 128 out, L*Hkv maps), box 64 x 128 x 1
};

struct Sync {
    uint64_t full[SLOTS], empty[SLOTS];
    uint64_t vhat_full[NB], vhat_empty[NB];
    uint64_t keys_read[SLOTS];           // the consumer has formed its scores: the slot's keys may be overwritten
    uint64_t vt_ready[SLOTS];            // the slot holds V^T
    uint64_t w_full, w_empty;
    uint32_t tmem_base;
};

// grid (plan.B), THREADS threads, SMEM_BYTES dynamic shared memory.
// partial: [U][s_max][CONSUMERS][g][REC]; slot of (unit u, block b) = b - block_of_tile(first tile of u).
__global__ void __launch_bounds__(THREADS, 1)
decode_stream_pertile_tc(const __nv_bfloat16* __restrict__ q, const __grid_constant__ Maps maps, Plan pl, int n_ret, int n_apx,
                         int g, int LH, float scale_log2e, float* __restrict__ partial, int* __restrict__ fault) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ Sync sy;
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* Ws = smem + SLOTS * SLOT_BYTES;
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
    const long long gt_lo = dbf::tile_begin(b, pl), gt_hi = dbf::tile_begin(b + 1, pl);
    const int n_my = (int)(gt_hi - gt_lo);
    const int u0 = n_my > 0 ? (int)(gt_lo / pl.n_tiles) : 0;
    const int u_last = n_my > 0 ? (int)((gt_hi - 1) / pl.n_tiles) : -1;

    // the merge kernel is a programmatic dependent: it reads the records after its own wait
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) { tma::mbar_init(&sy.full[s], 1); tma::mbar_init(&sy.empty[s], 1); }
#pragma unroll
        for (int k = 0; k < NB; ++k) { tma::mbar_init(&sy.vhat_full[k], 1); tma::mbar_init(&sy.vhat_empty[k], RECON_WARPS); }
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) { tma::mbar_init(&sy.keys_read[s], 1); tma::mbar_init(&sy.vt_ready[s], RECON_WARPS); }
        tma::mbar_init(&sy.w_full, 1);
        tma::mbar_init(&sy.w_empty, 1);
        tma::mbar_fence_init();
    }
    if (wq == 3) {
        tc::tmem_alloc(&sy.tmem_base, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();

    // A slot is released by the consumer warp that owns it, for a key-only tile after it has weighted
    // the reconstructed values that took the keys' place.
    if (wq == 2) {
        // ------------------------------------------------------------------ producer
        if (lane == 0 && n_my > 0) {
            tma::prefetch_map(&maps.ret_k); tma::prefetch_map(&maps.ret_v); tma::prefetch_map(&maps.apx_k);
            const uint64_t pol = tma::policy_evict_first();      // the cache is read once per step
            int u = u0, t = (int)(gt_lo - (long long)u0 * pl.n_tiles);
            for (int i = 0; i < n_my; ++i) {
                const int s = i % SLOTS, round = i / SLOTS;
                if (round > 0 && !tma::mbar_wait(&sy.empty[s], (round - 1) & 1, fault, 61)) break;
                unsigned char* st = smem + s * SLOT_BYTES;
                tma::mbar_expect_tx(&sy.full[s], SLOT_BYTES);
                if (t < pl.n_rt) {
                    const int row0 = t * KEYS;
                    tma::load_3d_hint(st, &maps.ret_k, 0, row0, u, &sy.full[s], pol);
                    tma::load_3d_hint(st + 8192, &maps.ret_k, 64, row0, u, &sy.full[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES, &maps.ret_v, 0, row0, u, &sy.full[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES + 8192, &maps.ret_v, 64, row0, u, &sy.full[s], pol);
                } else {
                    const int row0 = (t - pl.n_rt) * 2 * KEYS;
                    tma::load_3d_hint(st, &maps.apx_k, 0, row0, u, &sy.full[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES, &maps.apx_k, 64, row0, u, &sy.full[s], pol);
                }
                if (++t == pl.n_tiles) { t = 0; ++u; }
            }
        }
    } else if (wq == 3) {
        // ------------------------------------------------------------------ W loads and MMA issue
        if (lane == 0 && n_my > 0) {
            tma::prefetch_map(&maps.w);
            const uint32_t w_addr = tma::smem_u32(Ws);
            const uint32_t idesc = tc::instr_desc(128, 128);
            int cur_u = -1;
            uint32_t n_units = 0, j = 0;               // units whose W was loaded; key-only tiles issued
            int u = u0, t = (int)(gt_lo - (long long)u0 * pl.n_tiles);
            for (int i = 0; i < n_my; ++i) {
                const int s = i % SLOTS, round = i / SLOTS;
                // every phase of a slot's barrier is observed, retained tiles included: a parity wait must not skip one
                if (!tma::mbar_wait(&sy.full[s], round & 1, fault, 62)) break;
                if (t >= pl.n_rt) {
                    if (u != cur_u) {
                        if (n_units > 0 && !tma::mbar_wait(&sy.w_empty, (n_units - 1) & 1, fault, 63)) break;
                        tma::mbar_expect_tx(&sy.w_full, W_BYTES);
                        tma::load_3d(Ws, &maps.w, 0, 0, u % LH, &sy.w_full);
                        tma::load_3d(Ws + W_BYTES / 2, &maps.w, 64, 0, u % LH, &sy.w_full);
                        if (!tma::mbar_wait(&sy.w_full, n_units & 1, fault, 64)) break;
                        cur_u = u;
                        ++n_units;
                    }
                    const uint32_t vb = j % NB, use = j / NB;
                    if (use > 0 && !tma::mbar_wait(&sy.vhat_empty[vb], (use - 1) & 1, fault, 65)) break;
                    tc::fence_after_sync();
                    const uint32_t k_addr = tma::smem_u32(smem + s * SLOT_BYTES);
                    const uint32_t d = sy.tmem_base + vb * 128;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t o = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                        tc::mma_bf16(d, tc::smem_desc(w_addr + o), tc::smem_desc(k_addr + o), idesc, ks > 0);
                    }
                    tc::mma_commit(&sy.vhat_full[vb]);
                    ++j;
                    const bool last_of_unit = t + 1 == pl.n_tiles || i + 1 == n_my;
                    if (last_of_unit) tc::mma_commit(&sy.w_empty);
                }
                if (++t == pl.n_tiles) { t = 0; ++u; }
            }
        }
    } else if (wq >= 4) {
        // ------------------------------------------------------------------ conversion warps
        const int quarter = wq & 3, c = quarter * 32 + lane;          // this thread's output dim = its TMEM lane = its row of V^T
        const uint32_t lane_addr = sy.tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t row_off = (uint32_t)c * 128u;                   // rows of 128 bytes, 16-byte chunk index XOR (row & 7)
        uint32_t j = 0, kcount[SLOTS] = {};
        bool ok = n_my > 0;
        int t = n_my > 0 ? (int)(gt_lo - (long long)u0 * pl.n_tiles) : 0;
        for (int i = 0; i < n_my && ok; ++i) {
            if (t >= pl.n_rt) {
                const int s = i % SLOTS;
                const uint32_t vb = j % NB, use = j / NB;
                // the MMA has read the keys and left V^T; the consumer has formed its scores
                if (!tma::mbar_wait_warp(&sy.vhat_full[vb], use & 1, fault, 72)) { ok = false; break; }
                if (!tma::mbar_wait_warp(&sy.keys_read[s], kcount[s] & 1, fault, 71)) { ok = false; break; }
                tc::fence_after_sync();
                const uint32_t hi_base = tma::smem_u32(smem + s * SLOT_BYTES) + row_off;
                const uint32_t taddr = lane_addr + vb * 128;
                // 16 keys = two 16-byte chunks of this row at a time, in a loop that stays rolled
                auto split16 = [&](const uint32_t (&v16)[16], int chunk0) {
                    uint32_t hi[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) hi[e] = dbf::pack_f16(__uint_as_float(v16[2 * e]), __uint_as_float(v16[2 * e + 1]));
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int chunk = chunk0 + h;                  // keys 8 chunk .. 8 chunk + 7: box chunk / 8, chunk % 8 inside the row
                        const uint32_t off = (uint32_t)(chunk >> 3) * HALF_BYTES + (uint32_t)(((chunk & 7) ^ (c & 7)) << 4);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(hi_base + off), "r"(hi[4 * h]), "r"(hi[4 * h + 1]), "r"(hi[4 * h + 2]), "r"(hi[4 * h + 3]) : "memory");
                    }
                };
                uint32_t ra[16], rb[16];
                tc::tmem_ld16(taddr, ra);
#pragma unroll 1
                for (int c2 = 0; c2 < 8; c2 += 2) {
                    tc::tmem_ld_wait16(ra);
                    tc::tmem_ld16(taddr + (c2 + 1) * 16, rb);
                    split16(ra, 2 * c2);
                    tc::tmem_ld_wait16(rb);
                    if (c2 + 2 < 8) tc::tmem_ld16(taddr + (c2 + 2) * 16, ra);
                    split16(rb, 2 * c2 + 2);
                }
                // the slot is refilled by a bulk copy once released: order these stores ahead of it
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                tc::fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    tma::mbar_arrive(&sy.vhat_empty[vb]);
                    tma::mbar_arrive(&sy.vt_ready[s]);
                }
                ++j;
                ++kcount[s];
            }
            if (++t == pl.n_tiles) t = 0;
        }
    } else if (n_my > 0) {
        // ------------------------------------------------------------------ consumers (warps 0 and 1)
        const int gid = lane >> 2, tig = lane & 3;
        // per-lane ldmatrix geometry (swizzle: 16-byte chunk index XOR (row & 7), rows are 128 bytes)
        const int mat = lane >> 3, r8 = lane & 7;
        const uint32_t qk_row = (uint32_t)(r8 + (mat >> 1) * 8) * 128u;      // QK: matrices = (keys 0-7|8-15) x (chunk lo|hi)
        const uint32_t qk_x = (uint32_t)(((mat & 1) ^ r8) << 4);
        const uint32_t pv_row = (uint32_t)(r8 + (mat & 1) * 8) * 128u;       // PV: matrices = (chunk lo|hi) x (keys 0-7|8-15)
        const uint32_t pv_x = (uint32_t)(((mat >> 1) ^ r8) << 4);
        uint32_t qa[8][2];
        float acc[16][4];                  // sum p v: [dim tile][c0,c1: P_hi rows | c2,c3: P_lo rows]
        float m = -INFINITY, l = 0.f;
        uint32_t vcount[SLOTS / CONSUMERS] = {0u, 0u};      // key-only tiles this warp has had in each of its two slots

        auto record_of = [&](int unit) -> float* {
            int slot = b - dbf::block_of_tile((long long)unit * pl.n_tiles, pl);
            if (slot < 0 || slot >= pl.s_max) { atomicCAS(fault, 0, 66); slot = 0; }     // cannot happen; never write out of bounds
            return partial + ((((size_t)unit * pl.s_max + slot) * CONSUMERS + wq) * g + gid) * REC;
        };
        auto load_q = [&](int unit) {
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)unit * g + min(gid, g - 1)) * 128);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                qa[ks][0] = gid < g ? qrow[ks * 8 + tig] : 0u;
                qa[ks][1] = gid < g ? qrow[ks * 8 + 4 + tig] : 0u;
            }
        };
        auto store_acc = [&](float* dst) {       // dims n*8 + 2 tig + {0,1} of head row gid
#pragma unroll
            for (int n = 0; n < 16; ++n)
                *reinterpret_cast<float2*>(dst + n * 8 + 2 * tig) = make_float2(acc[n][0] + acc[n][2], acc[n][1] + acc[n][3]);
        };
        auto zero_acc = [&]() {
#pragma unroll
            for (int n = 0; n < 16; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
        };
        // S = Q K^T for the 64 keys at kbase: two boxes `box` bytes apart hold the halves of the head dimension
        auto qk64 = [&](uint32_t kbase, uint32_t box, float (&sc)[8][2]) {
            float zz[2];
#pragma unroll
            for (int n = 0; n < 8; ++n) { sc[n][0] = 0.f; sc[n][1] = 0.f; }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {          // 16 keys per ldmatrix
                    uint32_t b0, b1, b2, b3;
                    dbf::ldsm_x4(kbase + (ks >> 2) * box + jj * 16 * 128 + qk_row + ((((2 * ks) & 7) << 4) ^ qk_x), b0, b1, b2, b3);
                    dbf::mma_lo8(sc[2 * jj][0], sc[2 * jj][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b0, b1);
                    dbf::mma_lo8(sc[2 * jj + 1][0], sc[2 * jj + 1][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b2, b3);
                }
            }
        };
        // P (this thread: head gid, keys 8 n + 2 tig, + 1 of 64) times the 64 rows at vbase (two boxes `box`
        // bytes apart: rows = keys of stored values, `trans`; or rows = dims of a reconstructed tile, keys
        // along the row).  P enters as bf16 hi in MMA rows 0-7 and, with `with_lo`, its bf16 remainder in rows 8-15.
        auto weigh64_values = [&](uint32_t vbase, const float (&sc)[8][2]) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const float p00 = sc[2 * kk][0], p01 = sc[2 * kk][1], p10 = sc[2 * kk + 1][0], p11 = sc[2 * kk + 1][1];
                const float h00 = __bfloat162float(__float2bfloat16_rn(p00)), h01 = __bfloat162float(__float2bfloat16_rn(p01));
                const float h10 = __bfloat162float(__float2bfloat16_rn(p10)), h11 = __bfloat162float(__float2bfloat16_rn(p11));
                const uint32_t a0 = dbf::pack_bf16(h00, h01), a2 = dbf::pack_bf16(h10, h11);
                const uint32_t a1 = dbf::pack_bf16(p00 - h00, p01 - h01), a3 = dbf::pack_bf16(p10 - h10, p11 - h11);
#pragma unroll
                for (int np = 0; np < 8; ++np) {
                    uint32_t b0, b1, b2, b3;
                    dbf::ldsm_x4_t(vbase + (np >> 2) * 8192 + kk * 16 * 128 + pv_row + ((((2 * np) & 7) << 4) ^ pv_x), b0, b1, b2, b3);
                    dbf::mma_16(acc[2 * np], a0, a1, a2, a3, b0, b1);
                    dbf::mma_16(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        };
        // The same for 64 keys of a reconstructed tile: V^T as fp16 at vbase, [128 dims][keys] in boxes of 128
        // rows; the probabilities as fp16 hi (MMA rows 0-7) + lo (rows 8-15).
        auto weigh64_rebuilt = [&](uint32_t vbase, const float (&sc)[8][2]) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const float p00 = sc[2 * kk][0], p01 = sc[2 * kk][1], p10 = sc[2 * kk + 1][0], p11 = sc[2 * kk + 1][1];
                const uint32_t a0 = dbf::pack_f16(p00, p01), a2 = dbf::pack_f16(p10, p11);
                const uint32_t a1 = dbf::pack_f16(p00 - dbf::f16_lo(a0), p01 - dbf::f16_hi(a0));
                const uint32_t a3 = dbf::pack_f16(p10 - dbf::f16_lo(a2), p11 - dbf::f16_hi(a2));
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) {        // 16 dims per ldmatrix: rows 16 jj .. of V^T, keys 16 kk .. along the row
                    uint32_t b0, b1, b2, b3;
                    dbf::ldsm_x4(vbase + jj * 16 * 128 + qk_row + ((((2 * kk) & 7) << 4) ^ qk_x), b0, b1, b2, b3);
                    dbf::mma_16_f16(acc[2 * jj], a0, a1, a2, a3, b0, b1);
                    dbf::mma_16_f16(acc[2 * jj + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        };
        auto flush = [&](int unit) {
            float lt = l;
            lt += __shfl_xor_sync(0xffffffffu, lt, 1);
            lt += __shfl_xor_sync(0xffffffffu, lt, 2);
            if (gid < g) {
                float* rec = record_of(unit);
                if (tig == 0) *reinterpret_cast<float4*>(rec) = make_float4(m * 0.69314718055994531f, lt, 1.f, 0.f);
                store_acc(rec + 4);
#pragma unroll
                for (int n = 0; n < 16; ++n) *reinterpret_cast<float2*>(rec + 4 + 128 + n * 8 + 2 * tig) = make_float2(0.f, 0.f);
            }
            zero_acc();
            m = -INFINITY; l = 0.f;
        };

        zero_acc();
        int i = wq;                                        // index into the block's tile sequence
        bool ok = true;                                    // false once a wait gave up: keep walking, touch nothing
        for (int u = u0; u <= u_last; ++u) {
            const long long unit_end = (long long)(u + 1) * pl.n_tiles - gt_lo;     // first sequence index past the unit
            bool loaded = false;
            for (; i < n_my && i < unit_end; i += CONSUMERS) {
                const int s = i % SLOTS, round = i / SLOTS;
                const int t = (int)(gt_lo + i - (long long)u * pl.n_tiles);
                if (ok) {
                    if (!loaded) { load_q(u); loaded = true; }
                    ok = tma::mbar_wait_warp(&sy.full[s], round & 1, fault, 67);
                }
                if (!ok) continue;
                const uint32_t base = tma::smem_u32(smem + s * SLOT_BYTES);
                if (t < pl.n_rt) {
                    // ---- retained tile: 64 keys at base, their values at base + HALF_BYTES
                    const int nrows = min(KEYS, n_ret - t * KEYS);
                    float sc[8][2];
                    qk64(base, 8192u, sc);
                    float mx = -INFINITY;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        const int kc = n * 8 + 2 * tig;
                        sc[n][0] = kc < nrows ? sc[n][0] * scale_log2e : -INFINITY;
                        sc[n][1] = kc + 1 < nrows ? sc[n][1] * scale_log2e : -INFINITY;
                        mx = fmaxf(mx, fmaxf(sc[n][0], sc[n][1]));
                    }
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m, mx);      // finite: key 0 of the tile is valid for every row
                    const float alpha = exp2f(m - m_new);  // 0 on the first step
                    float ls = 0.f;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        sc[n][0] = exp2f(sc[n][0] - m_new);
                        sc[n][1] = exp2f(sc[n][1] - m_new);
                        ls += sc[n][0] + sc[n][1];
                    }
                    l = l * alpha + ls;
                    m = m_new;
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                        for (int n = 0; n < 16; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; acc[n][2] *= alpha; acc[n][3] *= alpha; }
                    }
                    weigh64_values(base + HALF_BYTES, sc);
                    __syncwarp();
                    if (lane == 0) tma::mbar_arrive(&sy.empty[s]);
                } else {
                    // ---- key-only tile: 128 keys, each half of the head dimension in a box of 128 rows
                    const int r0 = (t - pl.n_rt) * 2 * KEYS;
                    const int nrows = min(2 * KEYS, n_apx - r0);
                    float sa[8][2], sb[8][2];
                    qk64(base, (uint32_t)HALF_BYTES, sa);
                    qk64(base + 64 * 128, (uint32_t)HALF_BYTES, sb);
                    // every lane is past its last read of the keys: the conversion warps may put V^T in their place
                    __syncwarp();
                    if (lane == 0) tma::mbar_arrive(&sy.keys_read[s]);
                    float mx = -INFINITY;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        const int kc = n * 8 + 2 * tig;
                        sa[n][0] = kc < nrows ? sa[n][0] * scale_log2e : -INFINITY;
                        sa[n][1] = kc + 1 < nrows ? sa[n][1] * scale_log2e : -INFINITY;
                        sb[n][0] = 64 + kc < nrows ? sb[n][0] * scale_log2e : -INFINITY;
                        sb[n][1] = 64 + kc + 1 < nrows ? sb[n][1] * scale_log2e : -INFINITY;
                        mx = fmaxf(fmaxf(mx, fmaxf(sa[n][0], sa[n][1])), fmaxf(sb[n][0], sb[n][1]));
                    }
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
                    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
                    const float m_new = fmaxf(m, mx);
                    const float alpha = exp2f(m - m_new);
                    float ls = 0.f;
#pragma unroll
                    for (int n = 0; n < 8; ++n) {
                        sa[n][0] = exp2f(sa[n][0] - m_new); sa[n][1] = exp2f(sa[n][1] - m_new);
                        sb[n][0] = exp2f(sb[n][0] - m_new); sb[n][1] = exp2f(sb[n][1] - m_new);
                        ls += (sa[n][0] + sa[n][1]) + (sb[n][0] + sb[n][1]);
                    }
                    l = l * alpha + ls;
                    m = m_new;
                    if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                        for (int n = 0; n < 16; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; acc[n][2] *= alpha; acc[n][3] *= alpha; }
                    }
                    // the reconstructed values, where the keys were
                    const int sl = (i / CONSUMERS) % (SLOTS / CONSUMERS);
                    ok = tma::mbar_wait_warp(&sy.vt_ready[s], vcount[sl] & 1, fault, 68);
                    ++vcount[sl];
                    if (ok) {
                        weigh64_rebuilt(base, sa);
                        weigh64_rebuilt(base + HALF_BYTES, sb);
                    }
                    __syncwarp();
                    if (lane == 0) tma::mbar_arrive(&sy.empty[s]);
                }
            }
            flush(u);
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (wq == 3) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(sy.tmem_base, TMEM_COLS);
    }
}

}  // namespace dpt
}  // namespace vec
#endif
