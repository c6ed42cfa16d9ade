// Decode attention with one map per layer on warp-level MMAs (bf16, head_dim 128, 8 KV heads, at most
// 32 query heads per layer): the split and merge kernels of the factored form
//   o_a = sum_R p_i v_{i,h} + sum_h' W[h][h'] (sum_A p_i k_{i,h'})          (paper Sections 3.2 and 5.1)
// in which a block owns a slice of the tokens of one (sequence, layer) and ALL its heads, so that every
// approximated key is read once for the key sums of all query heads of the layer.
//
// Split kernel: 8 warps, warp w = KV head w.  The slice is walked in tiles that fill one 64 KB stage (two
// stages, cp.async, the next tile in flight while this one is worked on; a third stage would leave the
// first-level cache, where the spilled registers live, a few KB): 16 retained tokens (keys and
// values of the 8 heads) or 32 approximated tokens (keys of the 8 heads).  Per tile
//   phase 1  warp h: logits of its g query heads against head h's keys (M = the heads padded to 16 rows),
//            online softmax; for an approximated tile the probabilities go to shared memory as bf16
//            hi + lo, P[32 query heads][32 tokens], with the rescaling factor of each query head;
//   phase 2  warp h': its accumulator acc_k[32 query heads][128] (key sums over head h') is rescaled and
//            takes P K_h' (both halves of P); for a retained tile warp h adds P V_h for its own heads.
// Records have the layout of the CUDA-core split kernel: per (unit, split, head) m, l, acc_v[128],
// acc_k[8][128].
#ifndef VECTOR_DECODE_LAYER_MMA_CUH_
#define VECTOR_DECODE_LAYER_MMA_CUH_

#include "common.cuh"
#include "decode_bf16.cuh"
#include "residual_tc.cuh"

namespace vec {
namespace dlm {

constexpr int HKV = 8, THREADS = 32 * HKV, MQ = 32;        // query heads per layer the accumulators hold
constexpr int RT = 16, AT = 32;                            // tokens per retained / approximated tile
constexpr int STAGE_BYTES = 65536, HEAD_RET = RT * 256, HEAD_APX = AT * 256;
constexpr int PS_ROW = 80;                                 // bytes per row of P: 32 tokens + padding (conflict-free ldmatrix)
constexpr int STAGES = 2;
constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + 2 * MQ * PS_ROW + MQ * 4 + 128;
constexpr int REC = 2 + 128 + HKV * 128;

// grid (n_splits, U / 8), THREADS threads, SMEM_BYTES dynamic shared memory.
__global__ void __launch_bounds__(THREADS, 1)
decode_layer_mma(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ ret_k,
                 const __nv_bfloat16* __restrict__ ret_v, const __nv_bfloat16* __restrict__ apx_k, long long cap_ret,
                 long long cap_apx, int n_ret, int n_apx, int g, float scale_log2e, float* __restrict__ partial) {
    extern __shared__ __align__(128) unsigned char lsm[];
    unsigned char* stage0 = lsm;
    unsigned char* ps_hi = lsm + STAGES * STAGE_BYTES;
    unsigned char* ps_lo = ps_hi + MQ * PS_ROW;
    float* alpha_s = reinterpret_cast<float*>(ps_lo + MQ * PS_ROW);
    const int split = blockIdx.x, n_splits = gridDim.x, ul = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, h = tid >> 5;
    const int gid = lane >> 2, tig = lane & 3, mat = lane >> 3, r8 = lane & 7;
    const int n_rt = (n_ret + RT - 1) / RT, n_at = (n_apx + AT - 1) / AT, n_tiles = n_rt + n_at;
    const int per = (n_tiles + n_splits - 1) / n_splits;
    const int t_lo = min(n_tiles, split * per), t_hi = min(n_tiles, t_lo + per);
    const size_t u = (size_t)ul * HKV + h;

    for (int i = tid; i < 2 * MQ * PS_ROW / 4 + MQ; i += THREADS) reinterpret_cast<uint32_t*>(ps_hi)[i] = 0u;   // P and the factors
    // the g query rows of this head as A fragments (rows g .. 15 zero)
    uint32_t qa[8][2];
    {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + (u * g + min(gid, g - 1)) * 128);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = gid < g ? qrow[ks * 8 + tig] : 0u;
            qa[ks][1] = gid < g ? qrow[ks * 8 + 4 + tig] : 0u;
        }
    }
    float acc_k[2][16][4], acc_v[16][2];
#pragma unroll
    for (int n = 0; n < 16; ++n) {
        acc_v[n][0] = acc_v[n][1] = 0.f;
#pragma unroll
        for (int mt = 0; mt < 2; ++mt) acc_k[mt][n][0] = acc_k[mt][n][1] = acc_k[mt][n][2] = acc_k[mt][n][3] = 0.f;
    }
    float m = -INFINITY, l = 0.f;

    // 4096 16-byte pieces per tile, 16 per thread; rows past the pool's end are filled with zeros.  A thread's
    // pieces share the 16-byte column (tid & 15) and the token row (tid >> 4, + 16 for every other piece of an
    // approximated tile); they differ in the head (and, retained, in keys or values): fixed strides from one address.
    const int p_tok = tid >> 4, p_ch = tid & 15;
    const uint32_t p_dst = (uint32_t)(p_tok * 256 + ((p_ch ^ (p_tok & 7)) << 4));
    const size_t ret_head = (size_t)cap_ret * 128, apx_head = (size_t)cap_apx * 128;      // elements from one head's pool to the next
    auto load_tile = [&](int t, unsigned char* st) {
        const uint32_t dst = tma::smem_u32(st) + p_dst;
        if (t < n_rt) {
            const int tok = t * RT + p_tok;
            const bool in = tok < n_ret;
            const size_t off = ((size_t)ul * HKV * cap_ret + (in ? tok : 0)) * 128 + p_ch * 8;
            const __nv_bfloat16* ks = ret_k + off;
            const __nv_bfloat16* vs = ret_v + off;
#pragma unroll
            for (int hh = 0; hh < HKV; ++hh) {
                rtc::cp_async16(dst + hh * HEAD_RET, ks + hh * ret_head, in ? 16u : 0u);
                rtc::cp_async16(dst + 32768 + hh * HEAD_RET, vs + hh * ret_head, in ? 16u : 0u);
            }
        } else {
            const int tok = (t - n_rt) * AT + p_tok;
            const bool in0 = tok < n_apx, in1 = tok + 16 < n_apx;
            const __nv_bfloat16* k0 = apx_k + ((size_t)ul * HKV * cap_apx + (in0 ? tok : 0)) * 128 + p_ch * 8;
            const __nv_bfloat16* k1 = apx_k + ((size_t)ul * HKV * cap_apx + (in1 ? tok + 16 : 0)) * 128 + p_ch * 8;
#pragma unroll
            for (int hh = 0; hh < HKV; ++hh) {
                rtc::cp_async16(dst + hh * HEAD_APX, k0 + hh * apx_head, in0 ? 16u : 0u);
                rtc::cp_async16(dst + hh * HEAD_APX + 16 * 256, k1 + hh * apx_head, in1 ? 16u : 0u);
            }
        }
    };
    auto prefetch = [&](int t) {
        if (t < t_hi) load_tile(t, stage0 + ((t - t_lo) % STAGES) * STAGE_BYTES);
        rtc::cp_async_commit();
    };

    prefetch(t_lo);
    for (int t = t_lo; t < t_hi; ++t) {
        unsigned char* st = stage0 + ((t - t_lo) % STAGES) * STAGE_BYTES;
        rtc::cp_async_wait<0>();
        __syncthreads();                       // the tile has landed; everyone is done with the stage of tile t - 1, P and the factors
        prefetch(t + 1);                       // into the stage of tile t - 1
        const bool retained = t < n_rt;
        const int ntok = retained ? min(RT, n_ret - t * RT) : min(AT, n_apx - (t - n_rt) * AT);
        const uint32_t kbase = tma::smem_u32(st) + h * (retained ? HEAD_RET : HEAD_APX);
        // ---- phase 1: logits of this head's query rows, 16 tokens per ldmatrix
        float sc[4][2], zz[2];
#pragma unroll
        for (int n = 0; n < 4; ++n) sc[n][0] = sc[n][1] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (j == 0 || !retained) {
                    uint32_t b0, b1, b2, b3;
                    dbf::ldsm_x4(kbase + (j * 16 + r8 + (mat >> 1) * 8) * 256 + (((2 * ks + (mat & 1)) ^ r8) << 4), b0, b1, b2, b3);
                    dbf::mma_lo8(sc[2 * j][0], sc[2 * j][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b0, b1);
                    dbf::mma_lo8(sc[2 * j + 1][0], sc[2 * j + 1][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b2, b3);
                }
            }
        }
        float mx = -INFINITY;
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            const int kc = n * 8 + 2 * tig;
            sc[n][0] = kc < ntok ? sc[n][0] * scale_log2e : -INFINITY;
            sc[n][1] = kc + 1 < ntok ? sc[n][1] * scale_log2e : -INFINITY;
            mx = fmaxf(mx, fmaxf(sc[n][0], sc[n][1]));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m, mx);              // finite: a tile holds at least one token
        const float alpha = exp2f(m - m_new);
        float ls = 0.f;
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            sc[n][0] = exp2f(sc[n][0] - m_new);
            sc[n][1] = exp2f(sc[n][1] - m_new);
            ls += sc[n][0] + sc[n][1];
        }
        l = l * alpha + ls;
        m = m_new;
        if (gid < g) {
            if (tig == 0) alpha_s[h * g + gid] = alpha;
            if (!retained) {
#pragma unroll
                for (int n = 0; n < 4; ++n) {
                    const uint32_t hi = dbf::pack_bf16(sc[n][0], sc[n][1]);
                    const uint32_t lo = dbf::pack_bf16(sc[n][0] - __uint_as_float(hi << 16), sc[n][1] - __uint_as_float(hi & 0xffff0000u));
                    *reinterpret_cast<uint32_t*>(ps_hi + (h * g + gid) * PS_ROW + (n * 8 + 2 * tig) * 2) = hi;
                    *reinterpret_cast<uint32_t*>(ps_lo + (h * g + gid) * PS_ROW + (n * 8 + 2 * tig) * 2) = lo;
                }
            }
        }
        const int changed = __syncthreads_or(gid < g && alpha != 1.f);
        // ---- phase 2: rescale, then the tile's contribution
        if (changed) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const float f0 = alpha_s[16 * mt + gid], f1 = alpha_s[16 * mt + 8 + gid];
#pragma unroll
                for (int n = 0; n < 16; ++n) { acc_k[mt][n][0] *= f0; acc_k[mt][n][1] *= f0; acc_k[mt][n][2] *= f1; acc_k[mt][n][3] *= f1; }
            }
#pragma unroll
            for (int n = 0; n < 16; ++n) { acc_v[n][0] *= alpha; acc_v[n][1] *= alpha; }
        }
        if (retained) {
            // sum p v for this head's own query rows: P from the registers, hi then lo
            const uint32_t vbase = tma::smem_u32(st) + 32768 + h * HEAD_RET;
            const uint32_t a0 = dbf::pack_bf16(sc[0][0], sc[0][1]), a2 = dbf::pack_bf16(sc[1][0], sc[1][1]);
            const uint32_t l0 = dbf::pack_bf16(sc[0][0] - __uint_as_float(a0 << 16), sc[0][1] - __uint_as_float(a0 & 0xffff0000u));
            const uint32_t l2 = dbf::pack_bf16(sc[1][0] - __uint_as_float(a2 << 16), sc[1][1] - __uint_as_float(a2 & 0xffff0000u));
            // the hi and the lo product of an accumulator are kept a whole sweep apart: back to back the second
            // would wait for the first
#pragma unroll
            for (int part = 0; part < 2; ++part) {
                const uint32_t x0 = part ? l0 : a0, x2 = part ? l2 : a2;
#pragma unroll
                for (int np = 0; np < 8; ++np) {
                    uint32_t b0, b1, b2, b3;
                    dbf::ldsm_x4_t(vbase + (r8 + (mat & 1) * 8) * 256 + (((2 * np + (mat >> 1)) ^ r8) << 4), b0, b1, b2, b3);
                    dbf::mma_lo8(acc_v[2 * np][0], acc_v[2 * np][1], zz[0], zz[1], x0, x2, b0, b1);
                    dbf::mma_lo8(acc_v[2 * np + 1][0], acc_v[2 * np + 1][1], zz[0], zz[1], x0, x2, b2, b3);
                }
            }
        } else {
            // key sums over head h (= this warp) for all query heads of the layer: P[32 x 32] K_h[32 x 128]
            const uint32_t pa = (uint32_t)(((lane & 7) + ((lane >> 3) & 1) * 8) * PS_ROW + (lane >> 4) * 16);
            const uint32_t ph = tma::smem_u32(ps_hi) + pa, pl = tma::smem_u32(ps_lo) + pa;
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
                uint32_t ah[2][4], al[2][4];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    dbf::ldsm_x4(ph + mt * 16 * PS_ROW + kk * 32, ah[mt][0], ah[mt][1], ah[mt][2], ah[mt][3]);
                    dbf::ldsm_x4(pl + mt * 16 * PS_ROW + kk * 32, al[mt][0], al[mt][1], al[mt][2], al[mt][3]);
                }
#pragma unroll
                for (int part = 0; part < 2; ++part) {             // hi sweep, then lo sweep (see above)
#pragma unroll
                    for (int np = 0; np < 8; ++np) {
                        uint32_t b0, b1, b2, b3;
                        dbf::ldsm_x4_t(kbase + (kk * 16 + r8 + (mat & 1) * 8) * 256 + (((2 * np + (mat >> 1)) ^ r8) << 4), b0, b1, b2, b3);
#pragma unroll
                        for (int mt = 0; mt < 2; ++mt) {
                            const uint32_t* a = part ? al[mt] : ah[mt];
                            dbf::mma_16(acc_k[mt][2 * np], a[0], a[1], a[2], a[3], b0, b1);
                            dbf::mma_16(acc_k[mt][2 * np + 1], a[0], a[1], a[2], a[3], b2, b3);
                        }
                    }
                }
            }
        }
    }
    // ---- records.  Warp h: m, l and sum p v of its own query rows; every warp: its head's key sums for all rows
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (gid < g) {
        float* rec = partial + ((u * n_splits + split) * g + gid) * REC;
        if (tig == 0) { rec[0] = m * 0.69314718055994531f; rec[1] = l; }
#pragma unroll
        for (int n = 0; n < 16; ++n) *reinterpret_cast<float2*>(rec + 2 + n * 8 + 2 * tig) = make_float2(acc_v[n][0], acc_v[n][1]);
    }
    const int n_q = HKV * g;
#pragma unroll
    for (int mt = 0; mt < 2; ++mt) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int a = 16 * mt + 8 * half + gid;                 // query head of the layer
            if (a < n_q) {
                float* rec = partial + ((((size_t)ul * HKV + a / g) * n_splits + split) * g + a % g) * REC + 2 + 128 + h * 128;
#pragma unroll
                for (int n = 0; n < 16; ++n)
                    *reinterpret_cast<float2*>(rec + n * 8 + 2 * tig) = make_float2(acc_k[mt][n][2 * half], acc_k[mt][n][2 * half + 1]);
            }
        }
    }
}

// Merge for the same shapes: combines the splits' records of a unit, applies row block h of the layer's map
// to the merged key sums of all heads and normalises,
//   o_a = (sum_s f_s acc_v_s + W[h rows] sum_s f_s acc_k_s) / sum_s f_s l_s,   f_s = exp(m_s - max m).
// grid (U), 256 threads.  The product runs on warp-level MMAs: M = the head's 128 output channels (warp w:
// rows 16 w ..), N = the unit's g query heads (padded to 8), K = 8 x 128; A fragments straight from the map
// (16-byte loads: thread (row r, quarter t) holds columns 8 (t + 4 jj) .. + 7 of rows r and r + 8 of a
// 128-column block, the k slots of an MMA step follow that order in both operands), the key sums as bf16
// hi + lo in shared memory.
template <typename TO>
__global__ void __launch_bounds__(256)
decode_layer_merge_mma(const float* __restrict__ partial, const __nv_bfloat16* __restrict__ W, int L, int g, int n_splits,
                       TO* __restrict__ out) {
    constexpr int KD = HKV * 128;
    __shared__ __align__(16) __nv_bfloat16 akh[8][KD], akl[8][KD];          // 32 KB
    __shared__ float accv[8][128], pw[8][128], fs[8][32], Ls[8];
    const int u = blockIdx.x, tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const int h = u % HKV, layer = (u / HKV) % L;
    const int row = lane >> 2, quarter = lane & 3;
    const float* rec0 = partial + (size_t)u * n_splits * g * REC;
    // factors of the splits: warp a < g takes head a
    if (wid < g) {
        const float mj = lane < n_splits ? rec0[((size_t)lane * g + wid) * REC] : -INFINITY;
        const float lj = lane < n_splits ? rec0[((size_t)lane * g + wid) * REC + 1] : 0.f;
        const float M = warp_max(mj);
        const float f = mj > -INFINITY ? __expf(mj - M) : 0.f;
        fs[wid][lane] = f;
        const float Lsum = warp_sum(f * lj);
        if (lane == 0) Ls[wid] = Lsum;
    }
    for (int i = tid; i < (8 - g) * KD; i += 256) {            // columns of B beyond the unit's heads
        akh[g + i / KD][i % KD] = __float2bfloat16_rn(0.f);
        akl[g + i / KD][i % KD] = __float2bfloat16_rn(0.f);
    }
    __syncthreads();
    // merged sums: element e of a record's 128 + 1024 values, coalesced over the threads; eight splits' loads
    // in flight at a time
    for (int a = 0; a < g; ++a) {
        for (int e = tid; e < 128 + KD; e += 256) {
            const float* src = rec0 + (size_t)a * REC + 2 + e;
            float v = 0.f;
            for (int s0 = 0; s0 < n_splits; s0 += 8) {
                float x[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) x[k] = src[(size_t)min(s0 + k, n_splits - 1) * g * REC];      // always a valid record
#pragma unroll
                for (int k = 0; k < 8; ++k) v = fmaf(s0 + k < n_splits ? fs[a][s0 + k] : 0.f, x[k], v);
            }
            if (e < 128) accv[a][e] = v;
            else {
                const __nv_bfloat16 hi = __float2bfloat16_rn(v);
                akh[a][e - 128] = hi;
                akl[a][e - 128] = __float2bfloat16_rn(v - __bfloat162float(hi));
            }
        }
    }
    __syncthreads();
    // rows 16 wid .. of the head's block of the map times the key sums
    {
        const uint4* Wr0 = reinterpret_cast<const uint4*>(W + ((size_t)layer * KD + (size_t)h * 128 + 16 * wid + row) * KD);
        const uint4* Wr1 = Wr0 + 8 * (KD / 8);                 // row + 8
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 2
        for (int kc = 0; kc < HKV; ++kc) {                     // 128 columns a time: 16 pieces of 16 bytes per row
            uint4 A[8];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                A[2 * jj + 0] = Wr0[kc * 16 + quarter + 4 * jj];
                A[2 * jj + 1] = Wr1[kc * 16 + quarter + 4 * jj];
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const uint4 r0 = A[2 * jj], r1 = A[2 * jj + 1];
                const int col = kc * 128 + 8 * (quarter + 4 * jj);
                const uint4 bh = *reinterpret_cast<const uint4*>(&akh[row][col]);      // B column = head `row`
                const uint4 bl = *reinterpret_cast<const uint4*>(&akl[row][col]);
                dbf::mma_16(d, r0.x, r1.x, r0.y, r1.y, bh.x, bh.y);
                dbf::mma_16(d, r0.x, r1.x, r0.y, r1.y, bl.x, bl.y);
                dbf::mma_16(d, r0.z, r1.z, r0.w, r1.w, bh.z, bh.w);
                dbf::mma_16(d, r0.z, r1.z, r0.w, r1.w, bl.z, bl.w);
            }
        }
        // d[0], d[1]: row `row`, heads 2 quarter and 2 quarter + 1; d[2], d[3]: row `row` + 8
        if (2 * quarter < g) { pw[2 * quarter][16 * wid + row] = d[0]; pw[2 * quarter][16 * wid + row + 8] = d[2]; }
        if (2 * quarter + 1 < g) { pw[2 * quarter + 1][16 * wid + row] = d[1]; pw[2 * quarter + 1][16 * wid + row + 8] = d[3]; }
    }
    __syncthreads();
    for (int i = tid; i < g * 128; i += 256) {
        const int a = i >> 7, c = i & 127;
        store_out(out + ((size_t)u * g + a) * 128 + c, (accv[a][c] + pw[a][c]) / Ls[a]);
    }
}

}  // namespace dlm
}  // namespace vec
#endif
