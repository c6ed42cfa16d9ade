// Three-way routing (paper Section 3.2): Step 1 pool selection by base score,
// Step 2 reconstruction residual on the pool, Step 3 truncation by residual.
//
// Both selections are exact top-k with the lower index winning ties, done as a
// most-significant-digit radix select on an order-preserving 32-bit image of
// the fp32 value (4 histogram passes of 8 bits find the k-th key and how many
// ties of it are taken), followed by one ordered pass whose block-wide prefix
// sums place the chosen indices in ascending order.  One thread block per unit.
#include "common.cuh"
#include "internal.h"
#include "residual_tc.cuh"

namespace vec {

constexpr int SEL_THREADS = 1024;

struct SelectResult {
    uint32_t kth_key;   // image of the k-th best value
    int take_ties;      // how many elements equal to it are taken (lowest indices first)
};

// Best = largest image.  For "k smallest" the caller passes inverted images.
template <bool SMALLEST>
__device__ __forceinline__ uint32_t select_image(float v) {
    uint32_t k = ordered_key(v);
    return SMALLEST ? ~k : k;
}

// hist[bin] += 1 for every lane with `valid`.  When the whole warp hits one bin (common in the later
// passes, where the surviving keys share their leading bits) a single lane adds the count.
// Every lane of the warp must call it.
__device__ __forceinline__ void hist_add(int* hist, int bin, bool valid) {
    const unsigned active = __ballot_sync(0xffffffffu, valid);
    if (active == 0) return;
    const int first = __shfl_sync(0xffffffffu, bin, __ffs(active) - 1);
    if (__ballot_sync(0xffffffffu, valid && bin != first) == 0) {
        if ((int)(threadIdx.x & 31) == __ffs(active) - 1) atomicAdd(&hist[first], __popc(active));
    } else if (valid) {
        atomicAdd(&hist[bin], 1);
    }
}

// Finds the k-th largest image among vals[0..n) (1 <= k <= n).  All threads of the
// block call it and all get the result.  hist: 256 ints of shared memory; bc: 2 ints.
template <bool SMALLEST>
__device__ SelectResult radix_select(const float* __restrict__ vals, int n, int k, int* hist, int* bc) {
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int b = threadIdx.x; b < 256; b += blockDim.x) hist[b] = 0;
        __syncthreads();
        // eight independent loads in flight per thread: the pass is bound by memory latency otherwise
        for (int base = 0; base < n; base += 8 * blockDim.x) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = base + j * blockDim.x + threadIdx.x;
                v[j] = i < n ? vals[i] : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int i = base + j * blockDim.x + threadIdx.x;
                const uint32_t key = select_image<SMALLEST>(v[j]);
                hist_add(hist, (key >> shift) & 255, i < n && (key & mask) == prefix);
            }
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            // warp 0: the bin, counted from the top, in which the cumulative count reaches `remaining`
            int c[8], tot = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = hist[255 - (threadIdx.x * 8 + j)]; tot += c[j]; }
            int inc = tot;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, o);
                if ((int)threadIdx.x >= o) inc += t;
            }
            int cum = inc - tot;                            // count in the bins above this lane's eight
            if (cum < remaining && inc >= remaining) {      // exactly one lane
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (cum + c[j] >= remaining) { bc[0] = 255 - (threadIdx.x * 8 + j); bc[1] = remaining - cum; break; }
                    cum += c[j];
                }
            }
        }
        __syncthreads();
        prefix |= (uint32_t)bc[0] << shift;
        mask |= 255u << shift;
        remaining = bc[1];              // rank wanted inside the chosen bin (1-based)
        __syncthreads();
    }
    SelectResult r;
    r.kth_key = prefix;
    r.take_ties = remaining;   // all strictly better elements precede; `remaining` ties complete k
    return r;
}

// The ordered pass both selections end with.  Every warp owns a contiguous piece of the input and
// walks it 32 elements at a time (coalesced); positions inside a warp come from ballots, the
// offsets of the warps from one small scan by warp 0.  `emit(i, chosen, pos)` is called for every
// element i: pos is its rank among the chosen ones if chosen, else among the others.
struct OrderedScratch { int gt[32], tie[32], out[32], quota[32]; };

template <bool SMALLEST, typename Emit>
__device__ __forceinline__ void ordered_pass(const float* __restrict__ vals, int n, const SelectResult& sel, bool any,
                                             OrderedScratch& sc, Emit emit) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    const int per_w = (((n + nw - 1) / nw) + 31) & ~31;
    const int w0 = min(n, wid * per_w), w1 = min(n, w0 + per_w);
    int n_gt = 0, n_tie = 0;
    if (any) {
        for (int base = w0; base < w1; base += 128) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = base + 32 * j + lane < w1 ? vals[base + 32 * j + lane] : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = base + 32 * j + lane < w1;
                const uint32_t key = select_image<SMALLEST>(v[j]);
                n_gt += __popc(__ballot_sync(0xffffffffu, in && key > sel.kth_key));
                n_tie += __popc(__ballot_sync(0xffffffffu, in && key == sel.kth_key));
            }
        }
    }
    if (lane == 0) { sc.gt[wid] = n_gt; sc.tie[wid] = n_tie; }
    __syncthreads();
    if (wid == 0) {
        const int t = lane < nw ? sc.tie[lane] : 0;
        int inc = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += x; }
        const int quota = max(0, min(t, sel.take_ties - (inc - t)));       // ties go to the lowest indices
        const int c = (lane < nw ? sc.gt[lane] : 0) + quota;
        int ci = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, ci, o); if (lane >= o) ci += x; }
        sc.out[lane] = ci - c;
        sc.quota[lane] = quota;
    }
    __syncthreads();
    int pos = sc.out[wid], ties_left = sc.quota[wid];
    for (int base = w0; base < w1; base += 128) {
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) v[j] = base + 32 * j + lane < w1 ? vals[base + 32 * j + lane] : 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int i = base + 32 * j + lane;
            const bool in = i < w1;
            const uint32_t key = select_image<SMALLEST>(v[j]);
            const bool tie = any && in && key == sel.kth_key;
            const unsigned tb = __ballot_sync(0xffffffffu, tie);
            const bool chosen = any && in && (key > sel.kth_key || (tie && __popc(tb & lt) < ties_left));
            const unsigned cb = __ballot_sync(0xffffffffu, chosen);
            const int before = pos + __popc(cb & lt);               // chosen elements before this one in the unit
            if (in) emit(i, chosen, chosen ? before : i - before);
            pos += __popc(cb);
            ties_left -= min(ties_left, __popc(tb));
        }
    }
}

// Step 1.  grid (U), SEL_THREADS threads.
__global__ void __launch_bounds__(SEL_THREADS, 2)
pool_select_kernel(const float* __restrict__ scores, int64_t N, int n_pool, int32_t* __restrict__ pool_idx) {
    __shared__ int hist[256];
    __shared__ int bc[2];
    __shared__ OrderedScratch sc;
    const int u = blockIdx.x, n = (int)N;
    const float* s = scores + (size_t)u * N;
    int32_t* out = pool_idx + (size_t)u * n_pool;
    if (n_pool <= 0) return;
    const SelectResult sel = radix_select<false>(s, n, n_pool, hist, bc);
    ordered_pass<false>(s, n, sel, true, sc, [&](int i, bool chosen, int pos) { if (chosen) out[pos] = i; });
}

// Step 3.  grid (U), SEL_THREADS threads.
__global__ void __launch_bounds__(SEL_THREADS, 2)
truncate_kernel(const float* __restrict__ eps, const int32_t* __restrict__ pool_idx, int64_t N, int n_pool,
                int n_apx, uint8_t* __restrict__ tier, int32_t* __restrict__ ret_idx,
                int32_t* __restrict__ apx_idx) {
    __shared__ int hist[256];
    __shared__ int bc[2];
    __shared__ OrderedScratch sc;
    const int u = blockIdx.x;
    const float* e = eps + (size_t)u * n_pool;
    const int32_t* pool = pool_idx + (size_t)u * n_pool;
    uint8_t* tr = tier + (size_t)u * N;
    const int n_ret = n_pool - n_apx;
    int32_t* ro = ret_idx + (size_t)u * n_ret;
    int32_t* ao = apx_idx + (size_t)u * n_apx;
    if ((N & 15) == 0) {
        for (int64_t i = threadIdx.x; i < N / 16; i += SEL_THREADS) reinterpret_cast<uint4*>(tr)[i] = make_uint4(0, 0, 0, 0);
    } else {
        for (int64_t i = threadIdx.x; i < N; i += SEL_THREADS) tr[i] = 0;
    }
    __syncthreads();
    SelectResult sel;
    sel.kth_key = 0xffffffffu;
    sel.take_ties = 0;
    if (n_apx > 0) sel = radix_select<true>(e, n_pool, n_apx, hist, bc);
    ordered_pass<true>(e, n_pool, sel, n_apx > 0, sc, [&](int p, bool is_apx, int pos) {
        const int32_t token = pool[p];
        if (is_apx) { ao[pos] = token; tr[token] = 1; }
        else        { ro[pos] = token; tr[token] = 2; }
    });
}

// Step 2 on CUDA cores.  grid (ceil(n_idx / 64), U), 256 threads; W^T staged in
// dynamic shared memory as fp32 (D * (D+1) floats) plus one key row per warp.
// With ROPE the regressor sees the key turned back by its position (the token index): channel c
// pairs with c + D/2, angle -pos * theta^(-2c/D).
template <typename T, int D, bool ROPE>
__global__ void __launch_bounds__(256)
residual_generic(const T* __restrict__ K, const T* __restrict__ V, const T* __restrict__ W, int64_t N,
                 int LH, const int32_t* __restrict__ idx, int n_idx, float theta, float* __restrict__ eps) {
    extern __shared__ float smem[];
    __shared__ double inv_freq[D / 2];
    float* Wt = smem;                       // Wt[c_in * (D+1) + c_out]
    float* ks = smem + D * (D + 1);         // [8][D]
    if (ROPE) rope_fill_inv_freq(inv_freq, D, theta);
    const int u = blockIdx.y, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const T* Wu = W + (size_t)(u % LH) * D * D;
    for (int e = threadIdx.x; e < D * D; e += 256) {
        int co = e / D, ci = e % D;
        Wt[ci * (D + 1) + co] = to_f32(Wu[e]);
    }
    __syncthreads();
    const int p_begin = blockIdx.x * 64;
    const int p_end = min(n_idx, p_begin + 64);
    float* kw = ks + wid * D;
    for (int p = p_begin + wid; p < p_end; p += 8) {
        const int64_t tok = idx[(size_t)u * n_idx + p];
        const T* kr = K + ((size_t)u * N + tok) * D;
        const T* vr = V + ((size_t)u * N + tok) * D;
        __syncwarp();
#pragma unroll
        for (int c = lane; c < D; c += 32) kw[c] = to_f32(kr[c]);
        __syncwarp();
        if (ROPE) {
#pragma unroll
            for (int c = lane; c < D / 2; c += 32) {
                float cs, sn;
                rope_cos_sin((double)tok, inv_freq[c], cs, sn);
                const float x = kw[c], y = kw[c + D / 2];
                kw[c] = fmaf(x, cs, y * sn);
                kw[c + D / 2] = fmaf(y, cs, -x * sn);
            }
            __syncwarp();
        }
        float e = 0.f;
#pragma unroll
        for (int m = 0; m < D / 32; ++m) {
            int co = lane + 32 * m;
            float pred = 0.f;
#pragma unroll 8
            for (int ci = 0; ci < D; ++ci) pred = fmaf(Wt[ci * (D + 1) + co], kw[ci], pred);
            float r = to_f32(vr[co]) - pred;
            e = fmaf(r, r, e);
        }
        e = warp_sum(e);
        if (lane == 0) eps[(size_t)u * n_idx + p] = e;
    }
}

template <typename T, int D>
static vector_status launch_residual(const Dims& dm, const void* K, const void* V, const void* W, int64_t N,
                                     const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st) {
    if (n_idx == 0) return VECTOR_OK;
    size_t smem = (size_t)(D * (D + 1) + 8 * D) * sizeof(float);
    auto kern = dm.rope ? residual_generic<T, D, true> : residual_generic<T, D, false>;
    VEC_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    dim3 grid((unsigned)((n_idx + 63) / 64), dm.U);
    kern<<<grid, 256, smem, st>>>((const T*)K, (const T*)V, (const T*)W, N, dm.LH, idx, (int)n_idx, dm.theta, eps);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

// bf16, head_dim 128: gather + tcgen05 residual kernel.
static vector_status launch_residual_tc(const Dims& dm, const void* K, const void* V, const void* W, int64_t N,
                                        const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st) {
    if (n_idx == 0) return VECTOR_OK;
    static PerDeviceOnce once;
    if (once.first()) {
        cudaError_t e = cudaFuncSetAttribute(rtc::residual_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, rtc::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(rtc::residual_tc_rope, cudaFuncAttributeMaxDynamicSharedMemorySize, rtc::R_SMEM_BYTES);
        if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    }
    int* fault = kernel_fault_address();
    if (!fault) return VECTOR_ERR_CUDA;
    CUtensorMap mapW;
    if (!tma::encode_bf16_3d(&mapW, W, 128, 128, (uint64_t)dm.LH, 256, 128 * 256, 64, 128)) return VECTOR_ERR_CUDA;
    rtc::Params P;
    P.U = dm.U; P.LH = dm.LH; P.n_idx = (int)n_idx; P.N = N;
    P.tpu = (int)((n_idx + rtc::TILE - 1) / rtc::TILE);
    P.n_tiles = (long long)dm.U * P.tpu;
    const int blocks = (int)(P.n_tiles < 148 ? P.n_tiles : 148);
    if (dm.rope) {
        RopePhases ph;
        rope_phases(dm.theta, 128, &ph);
        rtc::residual_tc_rope<<<blocks, rtc::R_THREADS, rtc::R_SMEM_BYTES, st>>>((const __nv_bfloat16*)K, (const __nv_bfloat16*)V,
                                                                                 mapW, idx, P, ph, eps, fault);
    } else {
        rtc::residual_tc<<<blocks, rtc::THREADS, rtc::SMEM_BYTES, st>>>((const __nv_bfloat16*)K, (const __nv_bfloat16*)V, mapW,
                                                                        idx, P, eps, fault);
    }
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

static vector_status residual_dispatch(const Dims& dm, const void* K, const void* V, const void* W, int64_t N,
                                       const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st) {
    if (dm.dtype == VECTOR_BF16 && dm.d == 128) return launch_residual_tc(dm, K, V, W, N, idx, n_idx, eps, st);
    if (dm.dtype == VECTOR_F32)
        return dm.d == 64 ? launch_residual<float, 64>(dm, K, V, W, N, idx, n_idx, eps, st)
                          : launch_residual<float, 128>(dm, K, V, W, N, idx, n_idx, eps, st);
    return dm.d == 64 ? launch_residual<__nv_bfloat16, 64>(dm, K, V, W, N, idx, n_idx, eps, st)
                      : launch_residual<__nv_bfloat16, 128>(dm, K, V, W, N, idx, n_idx, eps, st);
}

}  // namespace vec

using namespace vec;

extern "C" vector_status vector_pool_select(const vector_shape* shape, const vector_budget* budget,
                                            const float* scores, int32_t* pool_idx, void* ws, size_t ws_bytes,
                                            void* stream) {
    (void)ws; (void)ws_bytes;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!scores || !pool_idx) return VECTOR_ERR_NULL;
    pool_select_kernel<<<dm.U, SEL_THREADS, 0, (cudaStream_t)stream>>>(scores, budget->n_tokens,
                                                                       (int)budget->n_pool, pool_idx);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" vector_status vector_residual(const vector_shape* shape, const void* K, const void* V, const void* W,
                                         int64_t N, const int32_t* idx, int64_t n_idx, float* eps, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!K || !V || !W || !idx || !eps) return VECTOR_ERR_NULL;
    if (N <= 0 || N > (int64_t(1) << 30) || n_idx < 0 || n_idx > N) return VECTOR_ERR_SHAPE;
    return residual_dispatch(dm, K, V, W, N, idx, n_idx, eps, (cudaStream_t)stream);
}

extern "C" vector_status vector_truncate(const vector_shape* shape, const vector_budget* budget, const float* eps,
                                         const int32_t* pool_idx, uint8_t* tier, int32_t* ret_idx,
                                         int32_t* apx_idx, void* ws, size_t ws_bytes, void* stream) {
    (void)ws; (void)ws_bytes;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!eps || !pool_idx || !tier) return VECTOR_ERR_NULL;
    if ((budget->n_ret > 0 && !ret_idx) || (budget->n_apx > 0 && !apx_idx)) return VECTOR_ERR_NULL;
    truncate_kernel<<<dm.U, SEL_THREADS, 0, (cudaStream_t)stream>>>(
        eps, pool_idx, budget->n_tokens, (int)budget->n_pool, (int)budget->n_apx, tier, ret_idx, apx_idx);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" vector_status vector_route(const vector_shape* shape, const vector_budget* budget, const float* scores,
                                      const void* K, const void* V, const void* W, uint8_t* tier,
                                      int32_t* ret_idx, int32_t* apx_idx, float* eps_out, int32_t* pool_idx_out,
                                      void* ws, size_t ws_bytes, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!scores || !K || !V || !W || !tier) return VECTOR_ERR_NULL;
    if ((budget->n_ret > 0 && !ret_idx) || (budget->n_apx > 0 && !apx_idx)) return VECTOR_ERR_NULL;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < select_ws_bytes(dm, *budget)) return VECTOR_ERR_WORKSPACE;
    char* p = (char*)ws;
    int32_t* pool = pool_idx_out ? pool_idx_out : (int32_t*)p;
    p += align256((size_t)dm.U * (size_t)budget->n_pool * sizeof(int32_t));
    float* eps = eps_out ? eps_out : (float*)p;
    cudaStream_t st = (cudaStream_t)stream;
    pool_select_kernel<<<dm.U, SEL_THREADS, 0, st>>>(scores, budget->n_tokens, (int)budget->n_pool, pool);
    VEC_LAUNCH_CHECK();
    rc = residual_dispatch(dm, K, V, W, budget->n_tokens, pool, budget->n_pool, eps, st);
    if (rc != VECTOR_OK) return rc;
    truncate_kernel<<<dm.U, SEL_THREADS, 0, st>>>(eps, pool, budget->n_tokens, (int)budget->n_pool,
                                                  (int)budget->n_apx, tier, ret_idx, apx_idx);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}
