// Base importance score (the scorer that Step 1 of the pipeline calls): causal
// observation-window attention mass per key, summed over window rows and the
// query heads of a KV head, then max-pooled along the sequence.
//
// The softmax normaliser of every window row is needed before the per-key sum
// over rows can be formed, so the logits are computed twice:
//   pass 1  per (unit, row tile, key chunk): running (max, sum exp) per row
//   combine per unit: lse[row] from the chunk partials
//   pass 2  per (unit, key tile): raw[key] = sum_rows exp(logit - lse[row])
//   pool    score[i] = max raw over the centred window (prefix only); +inf in the window
#include "common.cuh"
#include "internal.h"
#include "score_tc.cuh"

namespace vec {

constexpr int ST = 64;    // tile edge (rows and keys) of the CUDA-core score kernels
constexpr int SK = 32;    // head-dim slice staged per step

// acc[i][j] += sum_c Q[row0 + ty + 16 i][c] * K[key0 + tx + 16 j][c]
template <typename T, int D>
__device__ __forceinline__ void tile_qk(const T* __restrict__ Qu, const T* __restrict__ Ku, int R,
                                        int64_t N, int row0, int64_t key0, float (*Qs)[SK + 1],
                                        float (*Ks)[SK + 1], float acc[4][4]) {
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int dc = 0; dc < D; dc += SK) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < (ST * SK) / 256; ++e) {
            int idx = tid + 256 * e, r = idx / SK, c = idx % SK;
            int row = row0 + r;
            int64_t key = key0 + r;
            Qs[r][c] = row < R ? to_f32(Qu[(size_t)row * D + dc + c]) : 0.f;
            Ks[r][c] = key < N ? to_f32(Ku[(size_t)key * D + dc + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < SK; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = Qs[ty + 16 * i][kk];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Ks[tx + 16 * j][kk];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
}

// grid (n_chunks, row_tiles, U), 256 threads
template <typename T, int D>
__global__ void __launch_bounds__(256)
score_pass1_generic(const T* __restrict__ Q, const T* __restrict__ K, int64_t N, int R, int w,
                    float scale, int64_t chunk_len, float2* __restrict__ partial) {
    __shared__ float Qs[ST][SK + 1];
    __shared__ float Ks[ST][SK + 1];
    const int u = blockIdx.z, row0 = blockIdx.y * ST, chunk = blockIdx.x, n_chunks = gridDim.x;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const T* Qu = Q + (size_t)u * R * D;
    const T* Ku = K + (size_t)u * N * D;
    const int64_t k_begin = (int64_t)chunk * chunk_len;
    const int64_t k_end = min(N, k_begin + chunk_len);
    float m[4], l[4];
    int64_t last_visible[4];   // row j of the window sits at position N - w + j
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m[i] = -INFINITY;
        l[i] = 0.f;
        int row = row0 + ty + 16 * i;
        last_visible[i] = row < R ? N - w + (row % w) : -1;
    }
    for (int64_t key0 = k_begin; key0 < k_end; key0 += ST) {
        float acc[4][4];
        tile_qk<T, D>(Qu, Ku, R, N, row0, key0, Qs, Ks, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s[4], mx = m[i];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int64_t key = key0 + tx + 16 * j;
                s[j] = (key < k_end && key <= last_visible[i]) ? acc[i][j] * scale : -INFINITY;
                mx = fmaxf(mx, s[j]);
            }
            if (mx > -INFINITY) {
                float sum = l[i] * __expf(m[i] - mx);   // m = -inf -> factor 0
#pragma unroll
                for (int j = 0; j < 4; ++j) sum += expf(s[j] - mx);
                m[i] = mx;
                l[i] = sum;
            }
        }
    }
    // combine the 16 threads (one half-warp) that share a row
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float M = m[i];
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        float v = (m[i] > -INFINITY) ? l[i] * expf(m[i] - M) : 0.f;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        int row = row0 + ty + 16 * i;
        if (tx == 0 && row < R) partial[((size_t)u * n_chunks + chunk) * R + row] = make_float2(M, v);
    }
}

// grid (U), block 256: lse[u][row] from the chunk partials
__global__ void score_lse_combine(const float2* __restrict__ partial, int R, int n_chunks,
                                  float* __restrict__ lse) {
    const int u = blockIdx.x;
    for (int row = threadIdx.x; row < R; row += blockDim.x) {
        float M = -INFINITY;
        for (int c = 0; c < n_chunks; ++c) M = fmaxf(M, partial[((size_t)u * n_chunks + c) * R + row].x);
        float L = 0.f;
        for (int c = 0; c < n_chunks; ++c) {
            float2 p = partial[((size_t)u * n_chunks + c) * R + row];
            if (p.x > -INFINITY) L += p.y * expf(p.x - M);
        }
        lse[(size_t)u * R + row] = M + logf(L);
    }
}

// grid (key_tiles, U), 256 threads
template <typename T, int D>
__global__ void __launch_bounds__(256)
score_pass2_generic(const T* __restrict__ Q, const T* __restrict__ K, int64_t N, int R, int w,
                    float scale, const float* __restrict__ lse, float* __restrict__ raw) {
    __shared__ float Qs[ST][SK + 1];
    __shared__ float Ks[ST][SK + 1];
    __shared__ float red[16][ST];
    const int u = blockIdx.y;
    const int64_t key0 = (int64_t)blockIdx.x * ST;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const T* Qu = Q + (size_t)u * R * D;
    const T* Ku = K + (size_t)u * N * D;
    const float* lse_u = lse + (size_t)u * R;
    float col[4] = {0.f, 0.f, 0.f, 0.f};
    for (int row0 = 0; row0 < R; row0 += ST) {
        float acc[4][4];
        tile_qk<T, D>(Qu, Ku, R, N, row0, key0, Qs, Ks, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            int row = row0 + ty + 16 * i;
            if (row < R) {
                float ls = lse_u[row];
                int64_t last_visible = N - w + (row % w);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    int64_t key = key0 + tx + 16 * j;
                    if (key <= last_visible) col[j] += expf(acc[i][j] * scale - ls);
                }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty][tx + 16 * j] = col[j];
    __syncthreads();
    if (tid < ST) {
        float s = 0.f;
#pragma unroll
        for (int t = 0; t < 16; ++t) s += red[t][tid];
        int64_t key = key0 + tid;
        if (key < N) raw[(size_t)u * N + key] = s;
    }
}

// score[i] = max_{|j-i| <= r, 0 <= j < N-w} raw[j] for i < N-w ; +inf for the window tokens
__global__ void score_pool_kernel(const float* __restrict__ raw, int64_t N, int w, int r, int64_t total,
                                  float* __restrict__ score) {
    int64_t gi = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (gi >= total) return;
    int64_t u = gi / N, i = gi - u * N;
    int64_t P = N - w;
    float best = INFINITY;
    if (i < P) {
        best = -INFINITY;
        int64_t lo = max((int64_t)0, i - r), hi = min(P - 1, i + r);
        for (int64_t j = lo; j <= hi; ++j) best = fmaxf(best, raw[u * N + j]);
    }
    score[gi] = best;
}

template <typename T, int D>
static vector_status launch_score(const Dims& dm, const void* Q, const void* K, int64_t N, float* scores,
                                  float* raw, float2* partial, float* lse, cudaStream_t st) {
    const int n_chunks = score_num_chunks(dm.U, dm.R, N);
    int64_t chunk_len = (N + n_chunks - 1) / n_chunks;
    chunk_len = (chunk_len + 127) / 128 * 128;
    const int row_tiles = (dm.R + ST - 1) / ST;
    dim3 g1(n_chunks, row_tiles, dm.U);
    score_pass1_generic<T, D><<<g1, 256, 0, st>>>((const T*)Q, (const T*)K, N, dm.R, dm.w, dm.scale,
                                                  chunk_len, partial);
    VEC_LAUNCH_CHECK();
    score_lse_combine<<<dm.U, 256, 0, st>>>(partial, dm.R, n_chunks, lse);
    VEC_LAUNCH_CHECK();
    dim3 g2((unsigned)((N + ST - 1) / ST), dm.U);
    score_pass2_generic<T, D><<<g2, 256, 0, st>>>((const T*)Q, (const T*)K, N, dm.R, dm.w, dm.scale, lse, raw);
    VEC_LAUNCH_CHECK();
    int64_t total = (int64_t)dm.U * N;
    score_pool_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(raw, N, dm.w, dm.pool_kernel / 2,
                                                                       total, scores);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

// bf16, head_dim 128: tcgen05 passes.  Workspace: chunk partials | lse | per-row-block key sums.
static vector_status launch_score_tc(const Dims& dm, const void* Q, const void* K, int64_t N, float* scores,
                                     float* raw_out, char* ws, cudaStream_t st) {
    const ScoreTcPlan pl = score_tc_plan(dm.U, dm.R, N);
    float2* partial = (float2*)ws;
    ws += align256((size_t)dm.U * 2 * pl.n_chunks * dm.R * 2 * sizeof(float));
    float* lse2 = (float*)ws;
    ws += align256((size_t)dm.U * dm.R * sizeof(float));
    float* raw_part = (float*)ws;
    static PerDeviceOnce once;
    if (once.first()) {
        cudaError_t e = cudaFuncSetAttribute(stc::score_pass1_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, stc::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(stc::score_pass2_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, stc::SMEM_BYTES);
        if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    }
    int* fault = kernel_fault_address();
    if (!fault) return VECTOR_ERR_CUDA;
    CUtensorMap mapQ, mapK;
    if (!tma::encode_bf16_3d(&mapQ, Q, 128, (uint64_t)dm.R, (uint64_t)dm.U, 256, (uint64_t)dm.R * 256, 64, 128) ||
        !tma::encode_bf16_3d(&mapK, K, 128, (uint64_t)N, (uint64_t)dm.U, 256, (uint64_t)N * 256, 64, 128))
        return VECTOR_ERR_CUDA;
    stc::Params P;
    P.U = dm.U; P.R = dm.R; P.RG = pl.RG; P.w = dm.w; P.N = N;
    P.nt = pl.nt; P.tpc = pl.tpc; P.n_chunks = pl.n_chunks; P.n_items = pl.n_items;
    P.c = dm.scale * 1.4426950408889634f;
    const int sms = sm_count();
    const int blocks = pl.n_items < sms ? pl.n_items : sms;
    stc::score_pass1_tc<<<blocks, stc::THREADS, stc::SMEM_BYTES, st>>>(mapQ, mapK, P, partial, fault);
    VEC_LAUNCH_CHECK();
    stc::score_lse2_combine<<<dm.U, 256, 0, st>>>(partial, dm.R, 2 * pl.n_chunks, lse2);
    VEC_LAUNCH_CHECK();
    stc::score_pass2_tc<<<blocks, stc::THREADS, stc::SMEM_BYTES, st>>>(mapQ, mapK, P, lse2, raw_part, fault);
    VEC_LAUNCH_CHECK();
    dim3 gp((unsigned)((N + stc::POOL_TILE - 1) / stc::POOL_TILE), dm.U);
    if ((N & 3) == 0)
        stc::score_pool_parts_v4<<<gp, 256, 0, st>>>(raw_part, 2 * pl.RG, N, dm.w, dm.pool_kernel / 2, raw_out, scores);
    else
        stc::score_pool_parts<<<gp, 256, 0, st>>>(raw_part, 2 * pl.RG, N, dm.w, dm.pool_kernel / 2, raw_out, scores);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

}  // namespace vec

extern "C" float vector_score_exp2_fma_share(void) { return (float)vec::stc::POLY16 / 16.0f; }

extern "C" vector_status vector_score(const vector_shape* shape, const void* Q_obs, const void* K, int64_t N,
                                      float* scores, float* raw_out, void* ws, size_t ws_bytes, void* stream) {
    using namespace vec;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!Q_obs || !K || !scores) return VECTOR_ERR_NULL;
    if (N < dm.w || N > (int64_t(1) << 30)) return VECTOR_ERR_SHAPE;
    if ((int64_t)((N + ST - 1) / ST) > 0x7fffffff) return VECTOR_ERR_SHAPE;
    const bool need_raw = raw_out == nullptr;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < score_ws_bytes(dm, N, need_raw)) return VECTOR_ERR_WORKSPACE;
    char* p = (char*)ws;
    if (score_uses_tc(dm)) return launch_score_tc(dm, Q_obs, K, N, scores, raw_out, p, (cudaStream_t)stream);
    float2* partial = (float2*)p;
    p += align256((size_t)dm.U * score_num_chunks(dm.U, dm.R, N) * dm.R * 2 * sizeof(float));
    float* lse = (float*)p;
    p += align256((size_t)dm.U * dm.R * sizeof(float));
    float* raw = need_raw ? (float*)p : raw_out;
    cudaStream_t st = (cudaStream_t)stream;
    if (dm.dtype == VECTOR_F32) {
        return dm.d == 64 ? launch_score<float, 64>(dm, Q_obs, K, N, scores, raw, partial, lse, st)
                          : launch_score<float, 128>(dm, Q_obs, K, N, scores, raw, partial, lse, st);
    }
    return dm.d == 64 ? launch_score<__nv_bfloat16, 64>(dm, Q_obs, K, N, scores, raw, partial, lse, st)
                      : launch_score<__nv_bfloat16, 128>(dm, Q_obs, K, N, scores, raw, partial, lse, st);
}
