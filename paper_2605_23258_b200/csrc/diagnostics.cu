// Diagnostics of a routed cache (paper Section 4): the importance-weighted distortion E, the mean
// relative reconstruction error over the approximated set (1 - R^2_approx) and the threshold of
// Proposition 1.  One block per unit; sums are carried in fp64 and reduced in a fixed order.
#include "common.cuh"
#include "internal.h"

namespace vec {

constexpr int DG_THREADS = 256;

__device__ __forceinline__ double block_sum(double v, double* sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    double t = 0.0;
    for (int w = 0; w < DG_THREADS / 32; ++w) t += sh[w];
    return t;
}
__device__ __forceinline__ float block_max(float v, float* sh) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    v = warp_max(v);
    __syncthreads();
    if (lane == 0) sh[wid] = v;
    __syncthreads();
    float t = sh[0];
    for (int w = 1; w < DG_THREADS / 32; ++w) t = fmaxf(t, sh[w]);
    return t;
}

// grid (U), DG_THREADS threads.  out[u][8] = E, R2_approx, mu_A, sum_evicted_w, sum_approximated_w,
// w_bar, w_star, threshold.
template <typename T, int D>
__global__ void __launch_bounds__(DG_THREADS)
diagnostics_kernel(const float* __restrict__ importance, const uint8_t* __restrict__ tier,
                   const int32_t* __restrict__ pool_idx, const float* __restrict__ eps, const T* __restrict__ V,
                   int64_t N, int n_pool, float* __restrict__ out) {
    __shared__ double shd[DG_THREADS / 32];
    __shared__ float shf[DG_THREADS / 32];
    const int u = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const float* w = importance + (size_t)u * N;
    const uint8_t* tr = tier + (size_t)u * N;
    double total = 0.0, sum_e = 0.0;
    float w_star = 0.f;
    for (int64_t i = threadIdx.x; i < N; i += DG_THREADS) {
        const float wi = w[i];
        total += wi;
        if (tr[i] == 0) { sum_e += wi; w_star = fmaxf(w_star, wi); }
    }
    total = block_sum(total, shd);
    sum_e = block_sum(sum_e, shd);
    w_star = block_max(w_star, shf);
    // approximated tokens: a warp per pool entry, relative error = eps / ||v||^2
    double sum_a = 0.0, sum_a_rel = 0.0, mu = 0.0, n_a = 0.0;
    const T* Vu = V + (size_t)u * N * D;
    for (int p = wid; p < n_pool; p += DG_THREADS / 32) {
        const int32_t tok = pool_idx[(size_t)u * n_pool + p];
        if (tr[tok] != 1) continue;                       // uniform across the warp
        float v2 = 0.f;
#pragma unroll
        for (int c = lane; c < D; c += 32) { const float x = to_f32(Vu[(size_t)tok * D + c]); v2 = fmaf(x, x, v2); }
        v2 = warp_sum(v2);
        if (lane == 0) {
            const float e = eps[(size_t)u * n_pool + p];
            const double rel = v2 > 0.f ? (double)e / (double)v2 : (e > 0.f ? 1.0 : 0.0);
            sum_a += w[tok];
            sum_a_rel += (double)w[tok] * rel;
            mu += rel;
            n_a += 1.0;
        }
    }
    sum_a = block_sum(sum_a, shd);
    sum_a_rel = block_sum(sum_a_rel, shd);
    mu = block_sum(mu, shd);
    n_a = block_sum(n_a, shd);
    if (threadIdx.x == 0) {
        float* o = out + (size_t)u * 8;
        const double inv = total > 0.0 ? 1.0 / total : 0.0;
        const double se = sum_e * inv, sa = sum_a * inv, sar = sum_a_rel * inv, ws = (double)w_star * inv;
        const double m = n_a > 0.0 ? mu / n_a : 0.0;
        const double wb = n_pool > 0 ? (1.0 - se) / (double)n_pool : 0.0;
        o[0] = (float)(se + sar);
        o[1] = (float)(1.0 - m);
        o[2] = (float)m;
        o[3] = (float)se;
        o[4] = (float)sa;
        o[5] = (float)wb;
        o[6] = (float)ws;
        o[7] = (float)((ws + wb) > 0.0 ? wb / (ws + wb) : 0.0);
    }
}

// ---- R^2 of the map over a whole context (the statistic of the paper's predictability table) ----
__global__ void iota_rows_kernel(int32_t* __restrict__ idx, int64_t N) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < N) idx[(size_t)blockIdx.y * N + i] = (int32_t)i;
}

constexpr int R2_ROWS = 2048;   // tokens per block of the reduction

// grid (ceil(N / R2_ROWS), U), DG_THREADS threads.  acc[u][D + 2] (fp64, zeroed by the caller) receives the
// per-channel sums of v, then sum ||v||^2 and sum eps.  Thread t owns channel t % D of rows t / D, t / D + rpp, ...
template <typename T, int D>
__global__ void __launch_bounds__(DG_THREADS)
r2_partial_kernel(const T* __restrict__ V, const float* __restrict__ eps, int64_t N, double* __restrict__ acc) {
    __shared__ double shd[DG_THREADS / 32];
    __shared__ double chan[DG_THREADS];
    const int u = blockIdx.y;
    const int64_t r0 = (int64_t)blockIdx.x * R2_ROWS, r1 = min(N, r0 + (int64_t)R2_ROWS);
    constexpr int RPP = DG_THREADS / D;            // rows per pass
    const int c = threadIdx.x % D, rr = threadIdx.x / D;
    const T* Vu = V + (size_t)u * N * D;
    double s = 0.0, s2 = 0.0;
    for (int64_t r = r0 + rr; r < r1; r += RPP) {
        const double x = (double)to_f32(Vu[(size_t)r * D + c]);
        s += x;
        s2 = fma(x, x, s2);
    }
    double e = 0.0;
    for (int64_t r = r0 + threadIdx.x; r < r1; r += DG_THREADS) e += (double)eps[(size_t)u * N + r];
    chan[threadIdx.x] = s;
    s2 = block_sum(s2, shd);
    e = block_sum(e, shd);
    double* a = acc + (size_t)u * (D + 2);
    if (threadIdx.x < D) {
        double t = 0.0;
#pragma unroll
        for (int k = 0; k < RPP; ++k) t += chan[threadIdx.x + k * D];
        atomicAdd(a + threadIdx.x, t);
    }
    if (threadIdx.x == 0) { atomicAdd(a + D, s2); atomicAdd(a + D + 1, e); }
}

// out[u][4] = { R^2, SS_res, SS_tot, N }
__global__ void r2_finish_kernel(const double* __restrict__ acc, int D, int64_t N, int U, float* __restrict__ out) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    const double* a = acc + (size_t)u * (D + 2);
    double m2 = 0.0;
    for (int c = 0; c < D; ++c) m2 += a[c] * a[c];
    const double ss_tot = a[D] - m2 / (double)N, ss_res = a[D + 1];
    float* o = out + (size_t)u * 4;
    o[0] = (float)(ss_tot > 0.0 ? 1.0 - ss_res / ss_tot : (ss_res > 0.0 ? -INFINITY : 1.0));
    o[1] = (float)ss_res;
    o[2] = (float)ss_tot;
    o[3] = (float)N;
}

static size_t r2_ws_bytes(const Dims& dm, int64_t N) {
    return align256((size_t)dm.U * (size_t)N * sizeof(int32_t)) + align256((size_t)dm.U * (size_t)N * sizeof(float)) +
           align256((size_t)dm.U * (size_t)(dm.d + 2) * sizeof(double));
}

}  // namespace vec

extern "C" vector_status vector_diagnostics(const vector_shape* shape, const vector_budget* budget,
                                            const float* importance, const uint8_t* tier, const int32_t* pool_idx,
                                            const float* eps, const void* V, float* out, void* stream) {
    using namespace vec;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!importance || !tier || !pool_idx || !eps || !V || !out) return VECTOR_ERR_NULL;
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t N = budget->n_tokens;
    const int np = (int)budget->n_pool;
#define VEC_DIAG(T, D) diagnostics_kernel<T, D><<<dm.U, DG_THREADS, 0, st>>>(importance, tier, pool_idx, eps, (const T*)V, N, np, out)
    if (dm.dtype == VECTOR_F32) { if (dm.d == 64) VEC_DIAG(float, 64); else VEC_DIAG(float, 128); }
    else { if (dm.d == 64) VEC_DIAG(__nv_bfloat16, 64); else VEC_DIAG(__nv_bfloat16, 128); }
#undef VEC_DIAG
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" size_t vector_r2_global_workspace_bytes(const vector_shape* shape, int64_t N) {
    using namespace vec;
    Dims dm;
    if (check_shape(shape, &dm) != VECTOR_OK || N <= 0) return 0;
    return r2_ws_bytes(dm, N);
}

extern "C" vector_status vector_r2_global(const vector_shape* shape, const void* K, const void* V, const void* W,
                                          int64_t N, float* out, void* ws, size_t ws_bytes, void* stream) {
    using namespace vec;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!K || !V || !W || !out) return VECTOR_ERR_NULL;
    if (N <= 0 || N > (int64_t(1) << 30)) return VECTOR_ERR_SHAPE;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < r2_ws_bytes(dm, N)) return VECTOR_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* p = (char*)ws;
    int32_t* idx = (int32_t*)p;  p += align256((size_t)dm.U * (size_t)N * sizeof(int32_t));
    float* eps = (float*)p;      p += align256((size_t)dm.U * (size_t)N * sizeof(float));
    double* acc = (double*)p;
    if (cudaMemsetAsync(acc, 0, (size_t)dm.U * (size_t)(dm.d + 2) * sizeof(double), st) != cudaSuccess) return VECTOR_ERR_CUDA;
    iota_rows_kernel<<<dim3((unsigned)((N + 255) / 256), dm.U), 256, 0, st>>>(idx, N);
    VEC_LAUNCH_CHECK();
    if ((rc = vector_residual(shape, K, V, W, N, idx, N, eps, stream)) != VECTOR_OK) return rc;
    const dim3 grid((unsigned)((N + R2_ROWS - 1) / R2_ROWS), dm.U);
#define VEC_R2(T, D) r2_partial_kernel<T, D><<<grid, DG_THREADS, 0, st>>>((const T*)V, eps, N, acc)
    if (dm.dtype == VECTOR_F32) { if (dm.d == 64) VEC_R2(float, 64); else VEC_R2(float, 128); }
    else { if (dm.d == 64) VEC_R2(__nv_bfloat16, 64); else VEC_R2(__nv_bfloat16, 128); }
#undef VEC_R2
    VEC_LAUNCH_CHECK();
    r2_finish_kernel<<<(dm.U + 127) / 128, 128, 0, st>>>(acc, dm.d, N, dm.U, out);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" vector_status vector_sync_check(void* stream) {
    int* addr = vec::kernel_fault_address();
    if (!addr) return VECTOR_ERR_CUDA;
    cudaStream_t st = (cudaStream_t)stream;
    int v = 0;
    if (cudaMemcpyAsync(&v, addr, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return VECTOR_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return VECTOR_ERR_CUDA;
    if (v == 0) return VECTOR_OK;
    if (cudaMemsetAsync(addr, 0, sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        return VECTOR_ERR_CUDA;
    return VECTOR_ERR_TIMEOUT;
}
