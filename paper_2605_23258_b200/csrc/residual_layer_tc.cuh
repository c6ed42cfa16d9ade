// Reconstruction residual of Step 2 for ONE map per layer (bf16, head_dim 128): the map is
// calibrated layer-wise (paper Section 5.1) on the keys and values concatenated over the layer's
// KV heads, so
//   eps[p] = sum_h || v_{i,h} - sum_h' W[h][h'] k_{i,h'} ||^2,   i = idx[p],
// with W[h][h'] the 128 x 128 block (output head h, input head h') of the [Hkv d][Hkv d] map.
// A dense contraction with K = Hkv d: for a tile of 128 listed tokens and an output head h the
// accumulator in tensor memory collects D_h = sum_h' K_h' W[h][h']^T over Hkv steps of 8
// tcgen05.mma each; the epilogue subtracts the value rows of head h, squares and adds along its
// TMEM lane, and carries the sum over the Hkv output heads.
//
// Persistent blocks (one per multiprocessor) own equal contiguous ranges of the tile sequence.
// A step is (tile, h, h'); per step a stage receives the gathered key rows of head h' (cp.async,
// written in the 128-byte-swizzled operand layout) and the block W[h][h'] (TMA).
//   warps 0-7   loaders: gathers of the K rows of a step; on the last h' of an output head also
//               the V rows of that head into the value buffer; thread 0 also issues the W loads
//   warp  8     MMA issuer, TMEM owner (two 128-column accumulators: the epilogue of head h runs
//               under the products of head h + 1)
//   warps 9-12  epilogue: thread = row
// What this first version costs: every step fetches 64 KB (keys and a W block, mostly from L2) for
// 0.27 us of tensor work, so it runs at the L2 rate, not the tensor rate.
#ifndef VECTOR_RESIDUAL_LAYER_TC_CUH_
#define VECTOR_RESIDUAL_LAYER_TC_CUH_

#include "common.cuh"
#include "internal.h"
#include "residual_tc.cuh"
#include "tcgen05.cuh"
#include "tma.cuh"

namespace vec {
namespace rlt {

using rtc::BOX_BYTES;
using rtc::OPERAND_BYTES;
using rtc::TILE;

constexpr int STAGES = 3;
constexpr int STAGE_BYTES = 2 * OPERAND_BYTES;            // K rows of one head | one W block
constexpr int LOADER_WARPS = 8;
constexpr int EPI_WARPS = 4;
constexpr int THREADS = 32 * (LOADER_WARPS + 1 + EPI_WARPS);
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + OPERAND_BYTES + 1024;      // + the value buffer
constexpr int TMEM_COLS = 256;

struct Params {
    int UL, L, Hkv, n_idx, tpu;      // (sequence, layer) units, layers, KV heads, rows per unit, tiles per unit
    long long N, n_tiles;            // keys per head, UL * tpu
};
struct Sync {
    uint64_t full[STAGES], w_full[STAGES], empty[STAGES];
    uint64_t v_full, v_empty;
    uint64_t acc_full[2], acc_empty[2];
    uint32_t tmem_base;
};

// grid: min(multiprocessors, n_tiles) blocks, THREADS threads, SMEM_BYTES dynamic shared memory.
// K, V: [UL][Hkv][N][128]; idx: [UL][n_idx]; eps: [UL][n_idx]; mapW: (Hkv*128 in, Hkv*128 out, L), box 64 x 128.
__global__ void __launch_bounds__(THREADS, 1)
residual_layer_tc(const __nv_bfloat16* __restrict__ K, const __nv_bfloat16* __restrict__ V,
                  const __grid_constant__ CUtensorMap mapW, const int32_t* __restrict__ idx, const Params P,
                  float* __restrict__ eps, int* __restrict__ fault) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ Sync sy;
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    unsigned char* stage0 = smem;
    unsigned char* Vs = smem + STAGES * STAGE_BYTES;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long gt_lo = rtc::range_begin(blockIdx.x, P.n_tiles, gridDim.x);
    const long long gt_hi = rtc::range_begin(blockIdx.x + 1, P.n_tiles, gridDim.x);
    const int H = P.Hkv, H2 = H * H;
    const long long n_steps = (gt_hi - gt_lo) * H2;

    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) {
            tma::mbar_init(&sy.full[s], 32 * LOADER_WARPS);
            tma::mbar_init(&sy.w_full[s], 1);
            tma::mbar_init(&sy.empty[s], 1);
        }
        tma::mbar_init(&sy.v_full, 32 * LOADER_WARPS);
        tma::mbar_init(&sy.v_empty, EPI_WARPS);
#pragma unroll
        for (int k = 0; k < 2; ++k) { tma::mbar_init(&sy.acc_full[k], 1); tma::mbar_init(&sy.acc_empty[k], EPI_WARPS); }
        tma::mbar_fence_init();
    }
    if (warp == LOADER_WARPS) {
        tc::tmem_alloc(&sy.tmem_base, TMEM_COLS);
        tc::tmem_relinquish();
    }
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();

    if (warp < LOADER_WARPS) {
        // ------------------------------------------------------------------ loaders
        const int qc = tid & 7, rsub = tid >> 3;                    // chunk of each half, row inside a pass of 32 rows
        const uint32_t dst_thread = (uint32_t)rsub * 128u + (uint32_t)((qc ^ (rsub & 7)) << 4);   // + half * BOX + pass * 4096
        int32_t rows[4];                                             // this thread's four rows of the tile at hand
        long long cur_tile = -1;
        uint32_t v_loads = 0;
        bool ok = true;
        if (tid == 0) tma::prefetch_map(&mapW);
        asm volatile("griddepcontrol.wait;\n" ::: "memory");      // idx is complete and visible from here on
        for (long long i = 0; i < n_steps && ok; ++i) {
            const int s = (int)(i % STAGES);
            const long long round = i / STAGES;
            const long long gt = gt_lo + i / H2;
            const int rem = (int)(i % H2), h = rem / H, hp = rem % H;
            const int ul = (int)(gt / P.tpu), t = (int)(gt - (long long)ul * P.tpu);
            if (gt != cur_tile) {
                cur_tile = gt;
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const int row = t * TILE + p * 32 + rsub;
                    const int32_t v = row < P.n_idx ? idx[(size_t)ul * P.n_idx + row] : -1;
                    rows[p] = (unsigned long long)v < (unsigned long long)P.N ? v : -1;     // an index outside the unit reads as zeros
                }
            }
            if (round > 0 && !tma::mbar_wait(&sy.empty[s], (uint32_t)(round - 1) & 1, fault, 81)) { ok = false; break; }
            unsigned char* st = stage0 + s * STAGE_BYTES;
            if (tid == 0) {                                         // the block (h, hp) of this layer's map
                tma::mbar_expect_tx(&sy.w_full[s], OPERAND_BYTES);
                tma::load_3d(st + OPERAND_BYTES, &mapW, hp * 128, h * 128, ul % P.L, &sy.w_full[s]);
                tma::load_3d(st + OPERAND_BYTES + BOX_BYTES, &mapW, hp * 128 + 64, h * 128, ul % P.L, &sy.w_full[s]);
            }
            const uint32_t kdst = tma::smem_u32(st) + dst_thread;
            const __nv_bfloat16* Ku = K + ((size_t)ul * H + hp) * P.N * 128 + qc * 8;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const bool valid = rows[p] >= 0;
                const size_t ro = valid ? (size_t)rows[p] * 128 : 0;
                const uint32_t nb = valid ? 16u : 0u;                  // zero fill past the end of the list
                rtc::cp_async16(kdst + p * 4096, Ku + ro, nb);
                rtc::cp_async16(kdst + BOX_BYTES + p * 4096, Ku + ro + 64, nb);
            }
            const bool with_v = hp == H - 1;
            if (with_v) {
                // the value rows of output head h, once its last product is on its way
                if (v_loads > 0 && !tma::mbar_wait(&sy.v_empty, (v_loads - 1) & 1, fault, 82)) { ok = false; break; }
                const uint32_t vdst = tma::smem_u32(Vs) + dst_thread;
                const __nv_bfloat16* Vu = V + ((size_t)ul * H + h) * P.N * 128 + qc * 8;
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    const bool valid = rows[p] >= 0;
                    const size_t ro = valid ? (size_t)rows[p] * 128 : 0;
                    const uint32_t nb = valid ? 16u : 0u;
                    rtc::cp_async16(vdst + p * 4096, Vu + ro, nb);
                    rtc::cp_async16(vdst + BOX_BYTES + p * 4096, Vu + ro + 64, nb);
                }
                ++v_loads;
            }
            rtc::cp_async_commit();
            // this step's copies are published once they have landed: wait for them here (the next step's
            // stage wait would come first anyway) -- a step is short next to the fetch of its 64 KB
            rtc::cp_async_wait<0>();
            rtc::fence_async_proxy();
            tma::mbar_arrive(&sy.full[s]);
            if (with_v) tma::mbar_arrive(&sy.v_full);
        }
    } else if (warp == LOADER_WARPS) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            const uint32_t idesc = tc::instr_desc(128, 128);
            uint32_t heads_done = 0;                                // output heads started so far, over all tiles
            for (long long i = 0; i < n_steps; ++i) {
                const int s = (int)(i % STAGES);
                const uint32_t round = (uint32_t)(i / STAGES);
                const int rem = (int)(i % H2), hp = rem % H;
                if (hp == 0) {
                    // a new output head: its accumulator was last used two heads ago
                    const uint32_t buf = heads_done & 1, use = heads_done >> 1;
                    if (use > 0 && !tma::mbar_wait(&sy.acc_empty[buf], (use - 1) & 1, fault, 83)) break;
                }
                if (!tma::mbar_wait(&sy.full[s], round & 1, fault, 84)) break;
                if (!tma::mbar_wait(&sy.w_full[s], round & 1, fault, 85)) break;
                tc::fence_after_sync();
                const uint32_t buf = heads_done & 1;
                const uint32_t k_addr = tma::smem_u32(stage0 + s * STAGE_BYTES), w_addr = k_addr + OPERAND_BYTES;
                const uint32_t d = sy.tmem_base + buf * 128;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t o = (ks >> 2) * BOX_BYTES + (ks & 3) * 32;
                    tc::mma_bf16(d, tc::smem_desc(k_addr + o), tc::smem_desc(w_addr + o), idesc, (hp > 0 || ks > 0) ? 1u : 0u);
                }
                tc::mma_commit(&sy.empty[s]);                       // the stage is free once these products have read it
                if (hp == H - 1) { tc::mma_commit(&sy.acc_full[buf]); ++heads_done; }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp & 3;                       // TMEM lanes this warp may read: 32 (warp % 4) ..
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = sy.tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint32_t v_addr = tma::smem_u32(Vs) + (uint32_t)r * 128u;
        asm volatile("griddepcontrol.wait;\n" ::: "memory");
        const long long n_heads = (gt_hi - gt_lo) * H;
        float e_tok = 0.f;
        for (long long j = 0; j < n_heads; ++j) {
            const uint32_t buf = (uint32_t)(j & 1), use = (uint32_t)(j >> 1);
            if (!tma::mbar_wait_warp(&sy.v_full, (uint32_t)j & 1, fault, 86)) break;
            if (!tma::mbar_wait_warp(&sy.acc_full[buf], use & 1, fault, 87)) break;
            tc::fence_after_sync();
            uint32_t ra[32], rb[32];
            const uint32_t taddr = lane_addr + buf * 128;
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
                for (int k = 0; k < 32; k += 4) {
                    const float a = __uint_as_float(cur[k]) - __uint_as_float(vv[k >> 1] << 16);
                    const float b = __uint_as_float(cur[k + 1]) - __uint_as_float(vv[k >> 1] & 0xffff0000u);
                    const float c2 = __uint_as_float(cur[k + 2]) - __uint_as_float(vv[(k >> 1) + 1] << 16);
                    const float d2 = __uint_as_float(cur[k + 3]) - __uint_as_float(vv[(k >> 1) + 1] & 0xffff0000u);
                    e0 = fmaf(a, a, e0); e1 = fmaf(b, b, e1); e2 = fmaf(c2, c2, e2); e3 = fmaf(d2, d2, e3);
                }
            }
            tc::fence_before_sync();
            __syncwarp();
            if (lane == 0) { tma::mbar_arrive(&sy.acc_empty[buf]); tma::mbar_arrive(&sy.v_empty); }
            e_tok += (e0 + e1) + (e2 + e3);
            if ((int)(j % H) == H - 1) {                   // the last output head of the tile: the token's residual is complete
                const long long gt = gt_lo + j / H;
                const int ul = (int)(gt / P.tpu), t = (int)(gt - (long long)ul * P.tpu);
                const int row = t * TILE + r;
                if (row < P.n_idx) eps[(size_t)ul * P.n_idx + row] = e_tok;
                e_tok = 0.f;
            }
        }
    }
    tc::fence_before_sync();
    __syncthreads();
    if (warp == LOADER_WARPS) {
        __syncwarp();
        tc::fence_after_sync();
        tc::tmem_dealloc(sy.tmem_base, TMEM_COLS);
    }
}

}  // namespace rlt
}  // namespace vec
#endif
