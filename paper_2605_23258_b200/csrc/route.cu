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

// Finds the k-th largest image among vals[0..n) (1 <= k <= n).  All threads of the
// block call it and all get the result.  hist: 256 ints of shared memory; bc: 2 ints.
template <bool SMALLEST>
__device__ SelectResult radix_select(const float* __restrict__ vals, int n, int k, int* hist, int* bc) {
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int b = threadIdx.x; b < 256; b += blockDim.x) hist[b] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += blockDim.x) {
            uint32_t key = select_image<SMALLEST>(vals[i]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            int cum = 0, b = 255;
            for (; b > 0; --b) {
                if (cum + hist[b] >= remaining) break;
                cum += hist[b];
            }
            bc[0] = b;
            bc[1] = remaining - cum;    // rank wanted inside bin b (1-based)
        }
        __syncthreads();
        prefix |= (uint32_t)bc[0] << shift;
        mask |= 255u << shift;
        remaining = bc[1];
        __syncthreads();
    }
    SelectResult r;
    r.kth_key = prefix;
    r.take_ties = remaining;   // all strictly better elements precede; `remaining` ties complete k
    return r;
}

// Block-wide exclusive prefix sum of one int per thread; returns the exclusive
// prefix and writes the block total to *total.  warp_tot: 32 ints of shared memory.
__device__ __forceinline__ int block_exclusive_scan(int v, int* warp_tot, int* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    __syncthreads();            // protects warp_tot against the previous call's readers
    if (lane == 31) warp_tot[wid] = inc;
    __syncthreads();
    if (wid == 0) {
        int t = lane < nw ? warp_tot[lane] : 0;
        int ti = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int s = __shfl_up_sync(0xffffffffu, ti, o);
            if (lane >= o) ti += s;
        }
        warp_tot[lane] = ti - t;   // exclusive warp offsets; lane 31 holds total - last
        if (lane == 31) *total = ti;
    }
    __syncthreads();
    return warp_tot[wid] + inc - v;
}

// Step 1.  grid (U), SEL_THREADS threads.
__global__ void __launch_bounds__(SEL_THREADS)
pool_select_kernel(const float* __restrict__ scores, int64_t N, int n_pool, int32_t* __restrict__ pool_idx) {
    __shared__ int hist[256];
    __shared__ int bc[2];
    __shared__ int warp_tot[32];
    __shared__ int tot;
    const int u = blockIdx.x, n = (int)N;
    const float* s = scores + (size_t)u * N;
    int32_t* out = pool_idx + (size_t)u * n_pool;
    if (n_pool <= 0) return;
    SelectResult sel = radix_select<false>(s, n, n_pool, hist, bc);
    int ties_seen = 0, written = 0;
    for (int base = 0; base < n; base += SEL_THREADS) {
        int i = base + threadIdx.x;
        uint32_t key = i < n ? select_image<false>(s[i]) : 0u;
        int is_tie = (i < n && key == sel.kth_key) ? 1 : 0;
        int tie_rank = ties_seen + block_exclusive_scan(is_tie, warp_tot, &tot);
        ties_seen += tot;
        int chosen = (i < n && (key > sel.kth_key || (is_tie && tie_rank < sel.take_ties))) ? 1 : 0;
        int pos = written + block_exclusive_scan(chosen, warp_tot, &tot);
        written += tot;
        if (chosen) out[pos] = i;
    }
}

// Step 3.  grid (U), SEL_THREADS threads.
__global__ void __launch_bounds__(SEL_THREADS)
truncate_kernel(const float* __restrict__ eps, const int32_t* __restrict__ pool_idx, int64_t N, int n_pool,
                int n_apx, uint8_t* __restrict__ tier, int32_t* __restrict__ ret_idx,
                int32_t* __restrict__ apx_idx) {
    __shared__ int hist[256];
    __shared__ int bc[2];
    __shared__ int warp_tot[32];
    __shared__ int tot;
    const int u = blockIdx.x;
    const float* e = eps + (size_t)u * n_pool;
    const int32_t* pool = pool_idx + (size_t)u * n_pool;
    uint8_t* tr = tier + (size_t)u * N;
    const int n_ret = n_pool - n_apx;
    int32_t* ro = ret_idx + (size_t)u * n_ret;
    int32_t* ao = apx_idx + (size_t)u * n_apx;
    for (int64_t i = threadIdx.x; i < N; i += SEL_THREADS) tr[i] = 0;
    __syncthreads();
    SelectResult sel;
    sel.kth_key = 0xffffffffu;
    sel.take_ties = 0;
    if (n_apx > 0) sel = radix_select<true>(e, n_pool, n_apx, hist, bc);
    int ties_seen = 0, n_a_written = 0, n_r_written = 0;
    for (int base = 0; base < n_pool; base += SEL_THREADS) {
        int p = base + threadIdx.x;
        bool in = p < n_pool;
        uint32_t key = in ? select_image<true>(e[p]) : 0u;
        int is_tie = (in && n_apx > 0 && key == sel.kth_key) ? 1 : 0;
        int tie_rank = ties_seen + block_exclusive_scan(is_tie, warp_tot, &tot);
        ties_seen += tot;
        int is_apx = (in && n_apx > 0 && (key > sel.kth_key || (is_tie && tie_rank < sel.take_ties))) ? 1 : 0;
        int a_pos = n_a_written + block_exclusive_scan(is_apx, warp_tot, &tot);
        n_a_written += tot;
        int is_ret = (in && !is_apx) ? 1 : 0;
        int r_pos = n_r_written + block_exclusive_scan(is_ret, warp_tot, &tot);
        n_r_written += tot;
        if (in) {
            int32_t token = pool[p];
            if (is_apx) { ao[a_pos] = token; tr[token] = 1; }
            else        { ro[r_pos] = token; tr[token] = 2; }
        }
    }
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
    static bool configured = false;
    if (!configured) {
        VEC_CUDA_CHECK(cudaFuncSetAttribute(rtc::residual_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, rtc::SMEM_BYTES));
        configured = true;
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
    rtc::residual_tc<<<blocks, rtc::THREADS, rtc::SMEM_BYTES, st>>>((const __nv_bfloat16*)K, (const __nv_bfloat16*)V, mapW,
                                                                    idx, P, eps, fault);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

static vector_status residual_dispatch(const Dims& dm, const void* K, const void* V, const void* W, int64_t N,
                                       const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st) {
    // the de-rotating variant exists on the CUDA-core path only
    if (!dm.rope && dm.dtype == VECTOR_BF16 && dm.d == 128) return launch_residual_tc(dm, K, V, W, N, idx, n_idx, eps, st);
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
