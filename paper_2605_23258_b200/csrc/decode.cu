// Generation-time attention over the mixed cache (paper Section 3.2, Step 3):
// one softmax over the exact keys of the retained and the key-only pool; a
// retained token contributes its stored value, an approximated token W k.
// Factored form: o = sum_R p_i v_i + W (sum_A p_i k_i), so the kernel streams
// both pools once, accumulating p-weighted values and p-weighted keys, and the
// d x d map is applied once per query head in the merge step.
//
//   split  grid (n_splits, U): online softmax over a slice of the logical key
//          range [0, n_ret + n_apx); emits (m, l, acc_v[d], acc_k[d]) per head
//   merge  grid (U): combines the splits, applies W to acc_k, normalises
#include <cmath>
#include <mutex>

#include "common.cuh"
#include "decode_bf16.cuh"
#include "decode_pertile_tc.cuh"
#include "internal.h"

namespace vec {

template <typename T, int EPL> struct RowLoad;
template <> struct RowLoad<float, 4> {
    static __device__ __forceinline__ void load(const float* p, int lane, float (&o)[4]) {
        float4 v = reinterpret_cast<const float4*>(p)[lane];
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
template <> struct RowLoad<float, 2> {
    static __device__ __forceinline__ void load(const float* p, int lane, float (&o)[2]) {
        float2 v = reinterpret_cast<const float2*>(p)[lane];
        o[0] = v.x; o[1] = v.y;
    }
};
template <> struct RowLoad<__nv_bfloat16, 4> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, int lane, float (&o)[4]) {
        uint2 v = reinterpret_cast<const uint2*>(p)[lane];
        o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
        o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
    }
};
template <> struct RowLoad<__nv_bfloat16, 2> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, int lane, float (&o)[2]) {
        uint32_t v = reinterpret_cast<const uint32_t*>(p)[lane];
        o[0] = __uint_as_float(v << 16); o[1] = __uint_as_float(v & 0xffff0000u);
    }
};

// Partial record per (unit, split, head): [m, l, acc_v[D], acc_k[D]]
template <int D> struct Rec { static constexpr int floats = 2 + 2 * D; };

// With ROPE the approximated value is W applied to the key turned back by its original position
// (apx_pos): the logit still uses the stored key, only the p-weighted key sum takes the turned one.
// A lane holds EPL consecutive channels; the partner channel c +- D/2 sits in lane ^ 16.
template <typename T, int D, int G, bool ROPE>
__global__ void __launch_bounds__(128)
decode_split_generic(const T* __restrict__ q, const T* __restrict__ ret_k, const T* __restrict__ ret_v,
                     const T* __restrict__ apx_k, const int32_t* __restrict__ apx_pos, int64_t cap_ret,
                     int64_t cap_apx, int n_ret, int n_apx, int g, float scale, float theta,
                     float* __restrict__ partial) {
    constexpr int EPL = D / 32;
    constexpr int REC = Rec<D>::floats;
    __shared__ float sm[4][G][REC];
    __shared__ double inv_freq[D / 2];
    if (ROPE) { rope_fill_inv_freq(inv_freq, D, theta); __syncthreads(); }
    const int u = blockIdx.y, split = blockIdx.x, n_splits = gridDim.x;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int total = n_ret + n_apx;
    const int per = (total + n_splits - 1) / n_splits;
    const int lo = split * per, hi = min(total, lo + per);

    float qr[G][EPL], av[G][EPL], ak[G][EPL], m[G], l[G];
#pragma unroll
    for (int a = 0; a < G; ++a) {
        m[a] = -INFINITY;
        l[a] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) { av[a][e] = 0.f; ak[a][e] = 0.f; qr[a][e] = 0.f; }
        if (a < g) {
            RowLoad<T, EPL>::load(q + ((size_t)u * g + a) * D, lane, qr[a]);
#pragma unroll
            for (int e = 0; e < EPL; ++e) qr[a][e] *= scale;
        }
    }
    for (int i = lo + wid; i < hi; i += 4) {
        const bool retained = i < n_ret;
        const T* kp = retained ? ret_k + ((size_t)u * cap_ret + i) * D
                               : apx_k + ((size_t)u * cap_apx + (i - n_ret)) * D;
        float kx[EPL], vx[EPL];
        RowLoad<T, EPL>::load(kp, lane, kx);
        if (retained) RowLoad<T, EPL>::load(ret_v + ((size_t)u * cap_ret + i) * D, lane, vx);
        float kt[EPL];                       // what an approximated token contributes: the key, or the key turned back
#pragma unroll
        for (int e = 0; e < EPL; ++e) kt[e] = kx[e];
        if (ROPE && !retained) {
            const double pos = (double)apx_pos[(size_t)u * cap_apx + (i - n_ret)];
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                float cs, sn;
                rope_cos_sin(pos, inv_freq[(lane * EPL + e) % (D / 2)], cs, sn);
                const float other = __shfl_xor_sync(0xffffffffu, kx[e], 16);
                kt[e] = lane < 16 ? fmaf(kx[e], cs, other * sn) : fmaf(kx[e], cs, -other * sn);
            }
        }
#pragma unroll
        for (int a = 0; a < G; ++a) {
            if (a < g) {
                float s = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) s = fmaf(qr[a][e], kx[e], s);
                s = warp_sum(s);
                float mn = fmaxf(m[a], s);
                float corr = __expf(m[a] - mn);     // first row: exp(-inf) = 0
                float p = __expf(s - mn);
                m[a] = mn;
                l[a] = l[a] * corr + p;
#pragma unroll
                for (int e = 0; e < EPL; ++e) {
                    av[a][e] *= corr;
                    ak[a][e] *= corr;
                    if (retained) av[a][e] = fmaf(p, vx[e], av[a][e]);
                    else          ak[a][e] = fmaf(p, kt[e], ak[a][e]);
                }
            }
        }
    }
#pragma unroll
    for (int a = 0; a < G; ++a) {
        if (a < g) {
            if (lane == 0) { sm[wid][a][0] = m[a]; sm[wid][a][1] = l[a]; }
#pragma unroll
            for (int e = 0; e < EPL; ++e) {
                sm[wid][a][2 + lane * EPL + e] = av[a][e];
                sm[wid][a][2 + D + lane * EPL + e] = ak[a][e];
            }
        }
    }
    __syncthreads();
    float* out = partial + ((size_t)u * n_splits + split) * g * REC;
    for (int a = 0; a < g; ++a) {
        float M = fmaxf(fmaxf(sm[0][a][0], sm[1][a][0]), fmaxf(sm[2][a][0], sm[3][a][0]));
        float f[4];
#pragma unroll
        for (int wv = 0; wv < 4; ++wv) f[wv] = sm[wv][a][0] > -INFINITY ? __expf(sm[wv][a][0] - M) : 0.f;
        for (int c = threadIdx.x; c < REC; c += 128) {
            float v;
            if (c == 0) v = M;
            else v = f[0] * sm[0][a][c] + f[1] * sm[1][a][c] + f[2] * sm[2][a][c] + f[3] * sm[3][a][c];
            out[a * REC + c] = v;
        }
    }
}

// grid (U), D threads.
template <typename T, typename TO, int D>
__global__ void __launch_bounds__(D)
decode_merge_generic(const float* __restrict__ partial, const T* __restrict__ W, int LH, int g, int n_splits,
                     TO* __restrict__ out) {
    constexpr int REC = Rec<D>::floats;
    __shared__ float aks[D];
    const int u = blockIdx.x, c = threadIdx.x;
    const T* Wu = W + (size_t)(u % LH) * D * D;
    for (int a = 0; a < g; ++a) {
        const float* rec = partial + ((size_t)u * n_splits * g + a) * REC;
        const size_t stride = (size_t)g * REC;
        float M = -INFINITY;
        for (int s = 0; s < n_splits; ++s) M = fmaxf(M, rec[s * stride]);
        float L = 0.f, accv = 0.f, acck = 0.f;
        for (int s = 0; s < n_splits; ++s) {
            const float* r = rec + s * stride;
            float f = r[0] > -INFINITY ? __expf(r[0] - M) : 0.f;
            L += f * r[1];
            accv += f * r[2 + c];
            acck += f * r[2 + D + c];
        }
        __syncthreads();
        aks[c] = acck;
        __syncthreads();
        float proj = 0.f;
#pragma unroll 8
        for (int c2 = 0; c2 < D; ++c2) proj = fmaf(to_f32(Wu[(size_t)c * D + c2]), aks[c2], proj);
        store_out(out + ((size_t)u * g + a) * D + c, (accv + proj) / L);
    }
}

template <typename T, int D, int G>
static vector_status launch_decode(const Dims& dm, const void* q, const vector_cache* ch, const void* W, void* out,
                                   int out_dtype, float* partial, cudaStream_t st) {
    const int n_splits = decode_num_splits(dm.U, ch->n_ret + ch->n_apx);
    dim3 grid(n_splits, dm.U);
    auto kern = dm.rope ? decode_split_generic<T, D, G, true> : decode_split_generic<T, D, G, false>;
    kern<<<grid, 128, 0, st>>>((const T*)q, (const T*)ch->ret_k, (const T*)ch->ret_v, (const T*)ch->apx_k,
                               ch->apx_pos, ch->cap_ret, ch->cap_apx, (int)ch->n_ret, (int)ch->n_apx, dm.g,
                               dm.scale, dm.theta, partial);
    VEC_LAUNCH_CHECK();
    if (out_dtype == VECTOR_F32)
        decode_merge_generic<T, float, D><<<dm.U, D, 0, st>>>(partial, (const T*)W, dm.LH, dm.g, n_splits,
                                                             (float*)out);
    else
        decode_merge_generic<T, __nv_bfloat16, D><<<dm.U, D, 0, st>>>(partial, (const T*)W, dm.LH, dm.g, n_splits,
                                                                     (__nv_bfloat16*)out);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

// Fault word that bounded waits inside kernels write to (0 = none).
static __device__ int g_kernel_fault;
int* kernel_fault_address() {
    static int* addr[PerDeviceOnce::kMax] = {};      // per device, looked up with that device current
    static std::mutex mu;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PerDeviceOnce::kMax) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_kernel_fault) == cudaSuccess) addr[dev] = (int*)p;
    }
    return addr[dev];
}

// bf16, head_dim 128: persistent TMA + tensor-core streaming kernel and the record merge.
static vector_status launch_decode_bf16_d128(const Dims& dm, const void* q, const vector_cache* ch, const void* W,
                                             void* out, int out_dtype, int mode, float* partial, cudaStream_t st) {
    using T = __nv_bfloat16;
    static PerDeviceOnce once;
    if (once.first()) {
        cudaError_t e = cudaFuncSetAttribute(dbf::decode_stream_bf16_d128<false>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, dbf::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(dbf::decode_stream_bf16_d128<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     dbf::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(dpt::decode_stream_pertile_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, dpt::SMEM_BYTES);
        if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    }
    int* fault = kernel_fault_address();
    if (!fault) return VECTOR_ERR_CUDA;
    const dbf::Plan pl = dbf::make_plan(dm.U, ch->n_ret, ch->n_apx, sm_count());
    if (pl.s_max > decode_stream_slots(dm.U)) return VECTOR_ERR_WORKSPACE;
    dbf::Maps maps;
    const uint64_t row_b = 256;
    bool ok = true;
    if (ch->n_ret > 0) {
        ok = ok && tma::encode_bf16_3d(&maps.ret_k, ch->ret_k, 128, (uint64_t)ch->n_ret, (uint64_t)dm.U, row_b,
                                       (uint64_t)ch->cap_ret * row_b, 64, 64);
        ok = ok && tma::encode_bf16_3d(&maps.ret_v, ch->ret_v, 128, (uint64_t)ch->n_ret, (uint64_t)dm.U, row_b,
                                       (uint64_t)ch->cap_ret * row_b, 64, 64);
    }
    if (ch->n_apx > 0)
        ok = ok && tma::encode_bf16_3d(&maps.apx_k, ch->apx_k, 128, (uint64_t)ch->n_apx, (uint64_t)dm.U, row_b,
                                       (uint64_t)ch->cap_apx * row_b, 64, 64);
    if (!ok) return VECTOR_ERR_CUDA;
    if (ch->n_ret == 0) { maps.ret_k = maps.apx_k; maps.ret_v = maps.apx_k; }   // never dereferenced: no such tiles
    if (ch->n_apx == 0) maps.apx_k = maps.ret_k;
    const float c2 = dm.scale * 1.4426950408889634f;
    RopePhases ph = {};
    if (dm.rope) rope_phases(dm.theta, 128, &ph);
    if (mode == 1) {
        // reconstruction tile by tile on the tensor cores: its own streaming kernel, two consumer warps
        dpt::Maps pm;
        pm.ret_k = maps.ret_k; pm.ret_v = maps.ret_v; pm.apx_k = maps.apx_k;
        if (!tma::encode_bf16_3d(&pm.w, W, 128, 128, (uint64_t)dm.LH, row_b, 128 * row_b, 64, 128)) return VECTOR_ERR_CUDA;
        if (ch->n_apx > 0 && !tma::encode_bf16_3d(&pm.apx_k, ch->apx_k, 128, (uint64_t)ch->n_apx, (uint64_t)dm.U, row_b,
                                                  (uint64_t)ch->cap_apx * row_b, 64, 128))
            return VECTOR_ERR_CUDA;
        dpt::decode_stream_pertile_tc<<<pl.B, dpt::THREADS, dpt::SMEM_BYTES, st>>>(
            (const T*)q, pm, pl, (int)ch->n_ret, (int)ch->n_apx, dm.g, dm.LH, c2, partial, fault);
    } else if (dm.rope)
        dbf::decode_stream_bf16_d128<true><<<pl.B, dbf::ROPE_THREADS, dbf::SMEM_BYTES, st>>>(
            (const T*)q, maps, pl, (int)ch->n_ret, (int)ch->n_apx, dm.g, dm.LH, c2, partial, fault, ch->apx_pos,
            (long long)ch->cap_apx, ph);
    else
        dbf::decode_stream_bf16_d128<false><<<pl.B, dbf::THREADS, dbf::SMEM_BYTES, st>>>(
            (const T*)q, maps, pl, (int)ch->n_ret, (int)ch->n_apx, dm.g, dm.LH, c2, partial, fault, nullptr, 0, ph);
    VEC_LAUNCH_CHECK();
    // programmatic dependent launch: the merge blocks start while the streaming kernel drains
    const float* rec = partial;
    const int apply_w = mode == 1 ? 0 : 1;
    const int cw = mode == 1 ? dpt::CONSUMERS : dbf::CONSUMER_WARPS;      // records a block leaves per unit
    const T* Wp = (const T*)W;
    // blocks of 128 g threads; up to four heads leave the merge 128 registers a thread
#define VEC_MERGE(TO, MAXT)                                                                                                  \
    VEC_CUDA_CHECK(launch_maybe_dependent(true, dbf::decode_merge_bf16_d128<TO, MAXT>, dim3(dm.U), dim3(128 * dm.g), 0, st, rec, \
                                          Wp, dm.LH, dm.g, pl, apply_w, cw, (TO*)out))
    if (out_dtype == VECTOR_F32) { if (dm.g <= 4) VEC_MERGE(float, 512); else VEC_MERGE(float, 1024); }
    else { if (dm.g <= 4) VEC_MERGE(T, 512); else VEC_MERGE(T, 1024); }
#undef VEC_MERGE
    return VECTOR_OK;
}

template <typename T, int D>
static vector_status launch_decode_g(const Dims& dm, const void* q, const vector_cache* ch, const void* W,
                                     void* out, int out_dtype, float* partial, cudaStream_t st) {
    if (dm.g <= 2) return launch_decode<T, D, 2>(dm, q, ch, W, out, out_dtype, partial, st);
    if (dm.g <= 4) return launch_decode<T, D, 4>(dm, q, ch, W, out, out_dtype, partial, st);
    return launch_decode<T, D, 8>(dm, q, ch, W, out, out_dtype, partial, st);
}

}  // namespace vec

using namespace vec;

extern "C" vector_status vector_decode_attn(const vector_shape* shape, const void* q, const vector_cache* cache,
                                            const void* W, void* out, int32_t out_dtype, int32_t mode, void* ws,
                                            size_t ws_bytes, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!q || !cache || !W || !out) return VECTOR_ERR_NULL;
    if (out_dtype != VECTOR_F32 && out_dtype != VECTOR_BF16) return VECTOR_ERR_DTYPE;
    if (mode != 0 && mode != 1) return VECTOR_ERR_SHAPE;
    if (cache->n_ret < 0 || cache->n_apx < 0 || cache->n_ret + cache->n_apx <= 0 ||
        cache->n_ret + cache->n_apx > (int64_t(1) << 30) || cache->cap_ret < cache->n_ret ||
        cache->cap_apx < cache->n_apx)
        return VECTOR_ERR_SHAPE;
    if (cache->n_ret > 0 && (!cache->ret_k || !cache->ret_v)) return VECTOR_ERR_NULL;
    if (cache->n_apx > 0 && !cache->apx_k) return VECTOR_ERR_NULL;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < decode_ws_bytes(dm)) return VECTOR_ERR_WORKSPACE;
    // per-tile reconstruction exists for bf16 with head_dim 128 and stored (not rotated-back) keys
    if (mode == 1 && (dm.rope || dm.dtype != VECTOR_BF16 || dm.d != 128)) return VECTOR_ERR_UNSUPPORTED;
    if (dm.rope && cache->n_apx > 0 && !cache->apx_pos) return VECTOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    float* partial = (float*)ws;
    if (dm.dtype == VECTOR_F32)
        return dm.d == 64 ? launch_decode_g<float, 64>(dm, q, cache, W, out, out_dtype, partial, st)
                          : launch_decode_g<float, 128>(dm, q, cache, W, out, out_dtype, partial, st);
    if (dm.d == 64) return launch_decode_g<__nv_bfloat16, 64>(dm, q, cache, W, out, out_dtype, partial, st);
    return launch_decode_bf16_d128(dm, q, cache, W, out, out_dtype, mode, partial, st);
}

// ---------------------------------------------------------------------------
// Allocation-free variant: the split-KV partial records live in a fixed array
// of the library's device image instead of a caller-provided workspace.
namespace vec {

static __device__ __align__(256) unsigned char g_decode_scratch[VECTOR_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mu;
static void* g_scratch_addr[kMaxDevices] = {};

// In host code `g_decode_scratch` is only a handle; the address a kernel can use
// comes from cudaGetSymbolAddress, once per device, with that device current.
static vector_status static_scratch_address(void** out) {
    int dev = -1;
    VEC_CUDA_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return VECTOR_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        VEC_CUDA_CHECK(cudaGetSymbolAddress(&p, g_decode_scratch));
        if (!p) return VECTOR_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return VECTOR_OK;
}

}  // namespace vec

extern "C" size_t vector_decode_scratch_bytes(const vector_shape* shape) {
    Dims dm;
    if (check_shape(shape, &dm) != VECTOR_OK) return 0;
    return decode_ws_bytes(dm);
}

extern "C" vector_status vector_decode_attn_static(const vector_shape* shape, const void* q,
                                                   const vector_cache* cache, const void* W, void* out,
                                                   int32_t out_dtype, int32_t mode, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (decode_ws_bytes(dm) > (size_t)VECTOR_STATIC_SCRATCH_BYTES) return VECTOR_ERR_WORKSPACE;
    void* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != VECTOR_OK) return rc;
    return vector_decode_attn(shape, q, cache, W, out, out_dtype, mode, scratch,
                              (size_t)VECTOR_STATIC_SCRATCH_BYTES, stream);
}

extern "C" int vector_device_fault(void) {
    int* addr = vec::kernel_fault_address();
    if (!addr) return -1;
    int v = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpy(&v, addr, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return -1;
    if (v != 0) cudaMemcpy(addr, &zero, sizeof(int), cudaMemcpyHostToDevice);
    return v;
}
