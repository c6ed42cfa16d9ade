// Generation-time attention over the mixed cache with ONE map per layer (paper Section 5.1: the
// map is calibrated layer-wise; Section 3.2, Step 3: approximated values are rebuilt as W k).
// A token's tier holds for all KV heads of its layer, so the pools of the Hkv heads of a layer list
// the same tokens, and the value of an approximated token for head h is row block h of W applied to
// the token's keys of ALL heads.  Factored form, per query head a of KV head h:
//   o_a = sum_R p_i v_{i,h} + sum_h' W[h][h'] (sum_A p_i k_{i,h'}),   p = softmax over head h's keys,
// so besides its own head's keys (logits) and values a unit needs the p-weighted sum of the
// approximated keys of every head of the layer.
//
//   split  grid (n_splits, U, ceil(Hkv / 4)): online softmax over a slice of the logical key range
//          [0, n_ret + n_apx) of head h; block z accumulates the key sums of heads 4 z .. 4 z + 3
//          (block 0 also sum p v); emits (m, l, acc_v[d], acc_k[Hkv][d]) per head
//   merge  grid (U): combines the splits, applies the blocks W[h][h'] to the key sums, normalises
// CUDA-core kernels (any supported dtype and head size): a first device path of this variant, bound
// by the re-reading of the approximated keys (each of them enters the sums of all Hkv units of its layer).
#include "common.cuh"
#include "decode_layer_mma.cuh"
#include "internal.h"

namespace vec {

template <typename T, int EPL> struct LRow;
template <> struct LRow<float, 4> {
    static __device__ __forceinline__ void load(const float* p, int lane, float (&o)[4]) {
        const float4 v = reinterpret_cast<const float4*>(p)[lane];
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct LRow<float, 2> {
    static __device__ __forceinline__ void load(const float* p, int lane, float (&o)[2]) {
        const float2 v = reinterpret_cast<const float2*>(p)[lane];
        o[0] = v.x; o[1] = v.y;
    }
};
template <> struct LRow<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, int lane, float (&o)[4]) {
        const uint2 v = reinterpret_cast<const uint2*>(p)[lane];
        o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
        o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    }
};
template <> struct LRow<__nv_bfloat16, 2> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, int lane, float (&o)[2]) {
        const uint32_t v = reinterpret_cast<const uint32_t*>(p)[lane];
        o[0] = __uint_as_float(v << 16); o[1] = __uint_as_float(v & 0xffff0000u);
    }
};

constexpr int LAYER_HZ = 4;          // key-sum heads per block

// Record per (unit, split, head): [m, l, acc_v[D], acc_k[Hkv][D]].
__host__ __device__ inline int layer_rec_floats(int D, int Hkv) { return 2 + D + Hkv * D; }

template <typename T, int D, int G>
__global__ void __launch_bounds__(128)
decode_layer_split(const T* __restrict__ q, const T* __restrict__ ret_k, const T* __restrict__ ret_v,
                   const T* __restrict__ apx_k, int64_t cap_ret, int64_t cap_apx, int n_ret, int n_apx, int g,
                   int Hkv, float scale, float* __restrict__ partial) {
    constexpr int EPL = D / 32;
    const int REC = layer_rec_floats(D, Hkv);
    extern __shared__ float sm[];                    // [4 warps][G][2 + D + LAYER_HZ * D]
    constexpr int WREC = 2 + D + LAYER_HZ * D;
    const int u = blockIdx.y, split = blockIdx.x, n_splits = gridDim.x, z = blockIdx.z;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int h = u % Hkv, ul = u / Hkv;             // this unit's head and its (sequence, layer)
    const int h0 = z * LAYER_HZ, nh = min(LAYER_HZ, Hkv - h0);
    const int total = n_ret + n_apx;
    const int per = (total + n_splits - 1) / n_splits;
    const int lo = split * per, hi = min(total, lo + per);

    float qr[G][EPL], av[G][EPL], ak[G][LAYER_HZ][EPL], m[G], l[G];
#pragma unroll
    for (int a = 0; a < G; ++a) {
        m[a] = -INFINITY;
        l[a] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            av[a][e] = 0.f; qr[a][e] = 0.f;
#pragma unroll
            for (int k = 0; k < LAYER_HZ; ++k) ak[a][k][e] = 0.f;
        }
        if (a < g) {
            LRow<T, EPL>::load(q + ((size_t)u * g + a) * D, lane, qr[a]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) qr[a][e] *= scale;
        }
    }
    for (int i = lo + wid; i < hi; i += 4) {
        const bool retained = i < n_ret;
        const T* kp = retained ? ret_k + ((size_t)u * cap_ret + i) * D : apx_k + ((size_t)u * cap_apx + (i - n_ret)) * D;
        float kx[EPL], vx[EPL], ko[LAYER_HZ][EPL];
        LRow<T, EPL>::load(kp, lane, kx);
        if (retained) {
            if (z == 0) LRow<T, EPL>::load(ret_v + ((size_t)u * cap_ret + i) * D, lane, vx);
        } else {
#pragma unroll
            for (int k = 0; k < LAYER_HZ; ++k)
                if (k < nh) LRow<T, EPL>::load(apx_k + (((size_t)ul * Hkv + h0 + k) * cap_apx + (i - n_ret)) * D, lane, ko[k]);
        }
#pragma unroll
        for (int a = 0; a < G; ++a) {
            if (a < g) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(qr[a][e], kx[e], s);
                s = warp_sum(s);
                const float mn = fmaxf(m[a], s);
                const float corr = __expf(m[a] - mn);     // first row: exp(-inf) = 0
                const float p = __expf(s - mn);
                m[a] = mn;
                l[a] = l[a] * corr + p;
#pragma unroll
                for (int e = 0; e < EPL; ++e) {
                    av[a][e] *= corr;
                    if (retained && z == 0) av[a][e] = fmaf(p, vx[e], av[a][e]);
#pragma unroll
                    for (int k = 0; k < LAYER_HZ; ++k) {
                        ak[a][k][e] *= corr;
                        if (!retained && k < nh) ak[a][k][e] = fmaf(p, ko[k][e], ak[a][k][e]);
                    }
                }
            }
        }
    }
    float* mine = sm + (size_t)wid * G * WREC;
#pragma unroll
    for (int a = 0; a < G; ++a) {
        if (a < g) {
            float* r = mine + a * WREC;
            if (lane == 0) { r[0] = m[a]; r[1] = l[a]; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                r[2 + lane * EPL + e] = av[a][e];
#pragma unroll
                for (int k = 0; k < LAYER_HZ; ++k) r[2 + D + k * D + lane * EPL + e] = ak[a][k][e];
            }
        }
    }
    __syncthreads();
    float* out = partial + ((size_t)u * n_splits + split) * g * REC;
    for (int a = 0; a < g; ++a) {
        const float* r0 = sm + a * WREC;
        const size_t ws = (size_t)G * WREC;          // stride between the four warps' copies
        const float M = fmaxf(fmaxf(r0[0], r0[ws]), fmaxf(r0[2 * ws], r0[3 * ws]));
        float f[4];
#pragma unroll
        for (int wv = 0; wv < 4; ++wv) f[wv] = r0[wv * ws] > -INFINITY ? __expf(r0[wv * ws] - M) : 0.f;
        for (int c = threadIdx.x; c < WREC; c += 128) {
            float v;
            if (c == 0) v = M;
            else v = f[0] * r0[c] + f[1] * r0[ws + c] + f[2] * r0[2 * ws + c] + f[3] * r0[3 * ws + c];
            if (c < 2 + D) {
                if (z == 0) out[(size_t)a * REC + c] = v;                 // m, l and sum p v: block 0 writes them (all z agree on m, l)
            } else {
                const int k = (c - 2 - D) / D, cc = (c - 2 - D) % D;
                if (k < nh) out[(size_t)a * REC + 2 + D + (size_t)(h0 + k) * D + cc] = v;
            }
        }
    }
}

// grid (U), D threads.  W: [L][Hkv D][Hkv D] of type T (y = W x over the whole-layer vectors).
template <typename T, typename TO, int D>
__global__ void __launch_bounds__(D)
decode_layer_merge(const float* __restrict__ partial, const T* __restrict__ W, int L, int Hkv, int g, int n_splits,
                   TO* __restrict__ out) {
    extern __shared__ float aks[];                   // [Hkv][D]: the merged key sums of the head at hand
    const int REC = layer_rec_floats(D, Hkv);
    const int u = blockIdx.x, c = threadIdx.x;
    const int h = u % Hkv, ul = u / Hkv, layer = ul % L;
    const size_t DL = (size_t)Hkv * D;
    const T* Wrow = W + (size_t)layer * DL * DL + ((size_t)h * D + c) * DL;      // row h D + c of the layer's map
    for (int a = 0; a < g; ++a) {
        const float* rec = partial + ((size_t)u * n_splits * g + a) * REC;
        const size_t stride = (size_t)g * REC;
        float M = -INFINITY;
        for (int s = 0; s < n_splits; ++s) M = fmaxf(M, rec[s * stride]);
        float Lsum = 0.f, accv = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float* r = rec + s * stride;
            const float f = r[0] > -INFINITY ? __expf(r[0] - M) : 0.f;
            Lsum += f * r[1];
            accv += f * r[2 + c];
        }
        __syncthreads();
        for (int k = 0; k < Hkv; ++k) {
            float acck = 0.f;
            for (int s = 0; s < n_splits; ++s) {
                const float* r = rec + s * stride;
                const float f = r[0] > -INFINITY ? __expf(r[0] - M) : 0.f;
                acck += f * r[2 + D + (size_t)k * D + c];
            }
            aks[k * D + c] = acck;
        }
        __syncthreads();
        float proj = 0.f;
        for (int c2 = 0; c2 < Hkv * D; ++c2) proj = fmaf(to_f32(Wrow[c2]), aks[c2], proj);
        store_out(out + ((size_t)u * g + a) * D + c, (accv + proj) / Lsum);
    }
}

int layer_decode_splits(int U, int64_t rows) {
    int64_t want = (4 * (int64_t)sm_count() + U - 1) / U;
    const int64_t max_by_rows = (rows + 255) / 256;   // at least 256 rows per split
    if (want > max_by_rows) want = max_by_rows;
    if (want > 32) want = 32;
    if (want < 1) want = 1;
    return (int)want;
}

template <typename T, int D, int G>
static vector_status launch_layer(const Dims& dm, int Hkv, int L, const void* q, const vector_cache* ch, const void* W, void* out,
                                  int out_dtype, float* partial, cudaStream_t st) {
    const int n_splits = layer_decode_splits(dm.U, ch->n_ret + ch->n_apx);
    const dim3 grid(n_splits, dm.U, (Hkv + LAYER_HZ - 1) / LAYER_HZ);
    const size_t smem = (size_t)4 * G * (2 + D + LAYER_HZ * D) * sizeof(float);
    auto kern = decode_layer_split<T, D, G>;
    VEC_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    kern<<<grid, 128, smem, st>>>((const T*)q, (const T*)ch->ret_k, (const T*)ch->ret_v, (const T*)ch->apx_k, ch->cap_ret,
                                  ch->cap_apx, (int)ch->n_ret, (int)ch->n_apx, dm.g, Hkv, dm.scale, partial);
    VEC_LAUNCH_CHECK();
    const size_t msmem = (size_t)Hkv * D * sizeof(float);
    if (out_dtype == VECTOR_F32)
        decode_layer_merge<T, float, D><<<dm.U, D, msmem, st>>>(partial, (const T*)W, L, Hkv, dm.g, n_splits, (float*)out);
    else
        decode_layer_merge<T, __nv_bfloat16, D><<<dm.U, D, msmem, st>>>(partial, (const T*)W, L, Hkv, dm.g, n_splits,
                                                                        (__nv_bfloat16*)out);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

// bf16, head_dim 128, 8 KV heads, at most 32 query heads per layer: the split kernel on warp-level MMAs,
// a block per (slice of the tokens, sequence, layer), and a merge kernel that applies the map the same way.
static vector_status launch_layer_mma(const Dims& dm, int L, const void* q, const vector_cache* ch, const void* W, void* out,
                                      int out_dtype, float* partial, cudaStream_t st) {
    using T = __nv_bfloat16;
    static PerDeviceOnce once;
    if (once.first()) {
        const cudaError_t e = cudaFuncSetAttribute(dlm::decode_layer_mma, cudaFuncAttributeMaxDynamicSharedMemorySize, dlm::SMEM_BYTES);
        if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    }
    const int UL = dm.U / dlm::HKV;
    const int64_t tiles = (ch->n_ret + dlm::RT - 1) / dlm::RT + (ch->n_apx + dlm::AT - 1) / dlm::AT;
    int64_t n_splits = (2 * (int64_t)sm_count() + UL - 1) / UL;       // two rounds of blocks
    if (n_splits > tiles) n_splits = tiles;
    if (n_splits > 32) n_splits = 32;
    if (n_splits < 1) n_splits = 1;
    dlm::decode_layer_mma<<<dim3((unsigned)n_splits, UL), dlm::THREADS, dlm::SMEM_BYTES, st>>>(
        (const T*)q, (const T*)ch->ret_k, (const T*)ch->ret_v, (const T*)ch->apx_k, (long long)ch->cap_ret, (long long)ch->cap_apx,
        (int)ch->n_ret, (int)ch->n_apx, dm.g, dm.scale * 1.4426950408889634f, partial);
    VEC_LAUNCH_CHECK();
    if (out_dtype == VECTOR_F32)
        dlm::decode_layer_merge_mma<float><<<dm.U, 256, 0, st>>>(partial, (const T*)W, L, dm.g, (int)n_splits, (float*)out);
    else
        dlm::decode_layer_merge_mma<T><<<dm.U, 256, 0, st>>>(partial, (const T*)W, L, dm.g, (int)n_splits, (T*)out);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

template <typename T, int D>
static vector_status launch_layer_g(const Dims& dm, int Hkv, int L, const void* q, const vector_cache* ch, const void* W,
                                    void* out, int out_dtype, float* partial, cudaStream_t st) {
    if (dm.g <= 2) return launch_layer<T, D, 2>(dm, Hkv, L, q, ch, W, out, out_dtype, partial, st);
    if (dm.g <= 4) return launch_layer<T, D, 4>(dm, Hkv, L, q, ch, W, out, out_dtype, partial, st);
    return launch_layer<T, D, 8>(dm, Hkv, L, q, ch, W, out, out_dtype, partial, st);
}

}  // namespace vec

using namespace vec;

extern "C" size_t vector_layer_workspace_bytes(const vector_shape* shape, const vector_budget* budget) {
    Dims dm;
    if (check_shape(shape, &dm) != VECTOR_OK || !budget) return 0;
    const int Hkv = shape->n_kv_heads;
    const int UL = dm.U / Hkv;
    // decode: split records; route: pool list and residuals per (sequence, layer)
    const size_t dec = (size_t)dm.U * 32 * dm.g * layer_rec_floats(dm.d, Hkv) * sizeof(float);
    const size_t rt = align256((size_t)UL * (size_t)budget->n_pool * sizeof(int32_t)) +
                      align256((size_t)UL * (size_t)budget->n_pool * sizeof(float));
    return align256(dec > rt ? dec : rt) + 256;
}

extern "C" vector_status vector_decode_attn_layer(const vector_shape* shape, const void* q, const vector_cache* cache,
                                                  const void* W_layer, void* out, int32_t out_dtype, void* ws,
                                                  size_t ws_bytes, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!q || !cache || !W_layer || !out) return VECTOR_ERR_NULL;
    if (out_dtype != VECTOR_F32 && out_dtype != VECTOR_BF16) return VECTOR_ERR_DTYPE;
    if (dm.rope) return VECTOR_ERR_UNSUPPORTED;
    if (cache->n_ret < 0 || cache->n_apx < 0 || cache->n_ret + cache->n_apx <= 0 ||
        cache->n_ret + cache->n_apx > (int64_t(1) << 30) || cache->cap_ret < cache->n_ret || cache->cap_apx < cache->n_apx)
        return VECTOR_ERR_SHAPE;
    if (cache->n_ret > 0 && (!cache->ret_k || !cache->ret_v)) return VECTOR_ERR_NULL;
    if (cache->n_apx > 0 && !cache->apx_k) return VECTOR_ERR_NULL;
    const int Hkv = shape->n_kv_heads, L = shape->n_layers;
    const bool mma = dm.dtype == VECTOR_BF16 && dm.d == 128 && Hkv == dlm::HKV && Hkv * dm.g <= dlm::MQ;
    const int n_splits = mma ? 32 : layer_decode_splits(dm.U, cache->n_ret + cache->n_apx);      // the MMA path takes up to 32
    const size_t need = (size_t)dm.U * n_splits * dm.g * layer_rec_floats(dm.d, Hkv) * sizeof(float);
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need) return VECTOR_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float* partial = (float*)ws;
    if (mma) return launch_layer_mma(dm, L, q, cache, W_layer, out, out_dtype, partial, st);
    if (dm.dtype == VECTOR_F32)
        return dm.d == 64 ? launch_layer_g<float, 64>(dm, Hkv, L, q, cache, W_layer, out, out_dtype, partial, st)
                          : launch_layer_g<float, 128>(dm, Hkv, L, q, cache, W_layer, out, out_dtype, partial, st);
    return dm.d == 64 ? launch_layer_g<__nv_bfloat16, 64>(dm, Hkv, L, q, cache, W_layer, out, out_dtype, partial, st)
                      : launch_layer_g<__nv_bfloat16, 128>(dm, Hkv, L, q, cache, W_layer, out, out_dtype, partial, st);
}
