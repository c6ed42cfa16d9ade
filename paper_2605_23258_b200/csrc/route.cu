// Three-way routing (paper Section 3.2): Step 1 pool selection by base score,
// Step 2 reconstruction residual on the pool, Step 3 truncation by residual.
//
// Both selections are exact top-k with the lower index winning ties (select.cuh): a
// most-significant-digit radix select on an order-preserving 32-bit image of the fp32
// value, followed by one ordered walk whose block-wide prefix sums place the chosen
// indices in ascending order.  One thread block per unit.
#include "common.cuh"
#include "internal.h"
#include "residual_layer_tc.cuh"
#include "residual_tc.cuh"
#include "select.cuh"

namespace vec {

using sel::Layout;

// Blocks of 32 warps (one resident per multiprocessor, masks and list in up to 200 KB) for inputs beyond a
// quarter of a million elements, of 16 warps (two resident) for medium ones and of 8 warps (four resident)
// for short ones, where what a block costs is its fixed sequence of barriers rather than its passes.
constexpr int SEL_SHORT = 8192, SEL_MANY = 32768, SEL_LONG = 262144;
constexpr size_t SEL_SMEM_LONG = 200 * 1024, SEL_SMEM_MID = 92 * 1024, SEL_SMEM_SHORT = 36 * 1024;
#define VEC_SEL_BOUNDS(NW) __launch_bounds__(32 * NW, NW == 32 ? 1 : NW == 16 ? 2 : 4)

// The general selection (select_emit) as functions of their own: the kernels run the lean path inline and
// come here only when it gives up, so its registers are not theirs to carry.
template <int NW>
__device__ __noinline__ void pool_select_general(const float* __restrict__ s, int n, int n_pool, int32_t* __restrict__ out,
                                                 sel::Scratch& S, const Layout& L, uint32_t* dyn) {
    sel::select_emit<false, NW, true>(s, n, n_pool, true, S, L, dyn, [&](int i, bool chosen, int pos) { if (chosen) out[pos] = i; });
}

struct PoolOut {
    int32_t* out;
    __device__ __forceinline__ int32_t* list() const { return out; }
};

struct TruncateOut {
    const int32_t* pool;
    uint8_t* tr;
    int32_t* ro;
    int32_t* ao;
    int64_t N;
    __device__ __forceinline__ int fetch(int p) const { return pool[p]; }
    __device__ __forceinline__ void put(int, int token, bool is_apx, int pos) const {
        if ((uint64_t)(int64_t)token >= (uint64_t)N) return;          // a pool entry outside the unit is dropped
        if (is_apx) { ao[pos] = token; tr[token] = 1; }
        else        { ro[pos] = token; tr[token] = 2; }
    }
    __device__ __forceinline__ void operator()(int p, bool is_apx, int pos) const { put(p, pool[p], is_apx, pos); }
};

template <int NW>
__device__ __noinline__ void truncate_general(const float* __restrict__ e, int n_pool, int n_apx, const TruncateOut& emit,
                                              sel::Scratch& S, const Layout& L, uint32_t* dyn) {
    sel::select_emit<true, NW, false>(e, n_pool, n_apx, n_apx > 0, S, L, dyn, emit);
}

// Step 1.  grid (U), 32 NW threads, L.bytes() of dynamic shared memory.
template <int NW>
__global__ void VEC_SEL_BOUNDS(NW)
pool_select_kernel(const float* __restrict__ scores, int64_t N, int n_pool, int32_t* __restrict__ pool_idx, const Layout L) {
    __shared__ sel::Scratch S;
    extern __shared__ __align__(16) uint32_t sel_dyn[];
    // inside vector_route the residual kernel is launched as a programmatic dependent: its blocks may
    // take SMs as this grid's blocks leave them; it reads the index lists only after its own wait
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int u = blockIdx.x, n = (int)N;
    const float* s = scores + (size_t)u * N;
    int32_t* out = pool_idx + (size_t)u * n_pool;
    if (n_pool <= 0) return;
    if (L.keyed && sel::select_lean<false, NW, true>(s, n, n_pool, S, L, sel_dyn, PoolOut{out})) return;
    pool_select_general<NW>(s, n, n_pool, out, S, L, sel_dyn);
}

// Step 3.  grid (U), 32 NW threads, L.bytes() of dynamic shared memory (the residuals' images are
// staged there when the lean path cannot run and they fit).
template <int NW>
__global__ void VEC_SEL_BOUNDS(NW)
truncate_kernel(const float* __restrict__ eps, const int32_t* __restrict__ pool_idx, int64_t N, int n_pool,
                int n_apx, uint8_t* __restrict__ tier, int32_t* __restrict__ ret_idx,
                int32_t* __restrict__ apx_idx, const Layout L) {
    __shared__ sel::Scratch S;
    extern __shared__ __align__(16) uint32_t sel_dyn[];
    const int u = blockIdx.x;
    const float* e = eps + (size_t)u * n_pool;
    uint8_t* tr = tier + (size_t)u * N;
    if ((N & 15) == 0) {
        for (int64_t i = threadIdx.x; i < N / 16; i += 32 * NW) reinterpret_cast<uint4*>(tr)[i] = make_uint4(0, 0, 0, 0);
    } else {
        for (int64_t i = threadIdx.x; i < N; i += 32 * NW) tr[i] = 0;
    }
    // everything above touches only the tier map; the residuals and the pool list belong to the
    // kernels before this one (a no-op unless launched as a programmatic dependent)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    __syncthreads();
    const int n_ret = n_pool - n_apx;
    const TruncateOut emit = {pool_idx + (size_t)u * n_pool, tr, ret_idx + (size_t)u * n_ret, apx_idx + (size_t)u * n_apx, N};
    if (L.keyed && n_apx > 0 && sel::select_lean<true, NW, false>(e, n_pool, n_apx, S, L, sel_dyn, emit)) return;
    truncate_general<NW>(e, n_pool, n_apx, emit, S, L, sel_dyn);
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
        if ((uint64_t)tok >= (uint64_t)N) {          // an index outside the unit reads as a row of zeros
            if (lane == 0) eps[(size_t)u * n_idx + p] = 0.f;
            continue;
        }
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
                                        const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st, bool dependent) {
    if (n_idx == 0) return VECTOR_OK;
    static PerDeviceOnce once;
    if (once.first()) {
        cudaError_t e = cudaFuncSetAttribute(rtc::residual_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             rtc::RCfg<false>::SMEM_BYTES);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(rtc::residual_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     rtc::RCfg<true>::SMEM_BYTES);
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
    const int sms = sm_count();
    const int blocks = (int)(P.n_tiles < sms ? P.n_tiles : sms);
    RopePhases ph = {};
    if (dm.rope) rope_phases(dm.theta, 128, &ph);
    // dependent: blocks may take SMs while the kernel that writes idx drains; the loaders wait for it
    const __nv_bfloat16* Kp = (const __nv_bfloat16*)K;
    const __nv_bfloat16* Vp = (const __nv_bfloat16*)V;
    if (dm.rope)
        VEC_CUDA_CHECK(launch_maybe_dependent(dependent, rtc::residual_tc<true>, dim3(blocks), dim3(rtc::R_THREADS),
                                              rtc::RCfg<true>::SMEM_BYTES, st, Kp, Vp, mapW, idx, P, ph, eps, fault));
    else
        VEC_CUDA_CHECK(launch_maybe_dependent(dependent, rtc::residual_tc<false>, dim3(blocks), dim3(rtc::R_THREADS),
                                              rtc::RCfg<false>::SMEM_BYTES, st, Kp, Vp, mapW, idx, P, ph, eps, fault));
    return VECTOR_OK;
}

static vector_status residual_dispatch(const Dims& dm, const void* K, const void* V, const void* W, int64_t N,
                                       const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st,
                                       bool dependent = false) {
    if (dm.dtype == VECTOR_BF16 && dm.d == 128) return launch_residual_tc(dm, K, V, W, N, idx, n_idx, eps, st, dependent);
    if (dm.dtype == VECTOR_F32)
        return dm.d == 64 ? launch_residual<float, 64>(dm, K, V, W, N, idx, n_idx, eps, st)
                          : launch_residual<float, 128>(dm, K, V, W, N, idx, n_idx, eps, st);
    return dm.d == 64 ? launch_residual<__nv_bfloat16, 64>(dm, K, V, W, N, idx, n_idx, eps, st)
                      : launch_residual<__nv_bfloat16, 128>(dm, K, V, W, N, idx, n_idx, eps, st);
}

// One-time opt-in to the dynamic shared memory of the selection kernels.
static vector_status select_kernels_setup() {
    static PerDeviceOnce once;
    if (!once.first()) return VECTOR_OK;
    cudaError_t e = cudaFuncSetAttribute(pool_select_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_LONG);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(pool_select_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_MID);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(pool_select_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_SHORT);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(truncate_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_LONG);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(truncate_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_MID);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(truncate_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SEL_SMEM_SHORT);
    if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    return VECTOR_OK;
}

// Block size, shared-memory budget and smallest useful list of U selections over n elements each.  Short
// inputs take the small blocks; so do medium ones when there are units enough to fill the small blocks'
// slots twice over (the phases after the two passes are latency, which more resident blocks hide).
struct SelPlan { int nw; Layout L; };
static SelPlan plan_selection(int64_t n, int U) {
    SelPlan p;
    const bool small = n < SEL_SHORT || (n < SEL_MANY && U >= 2 * 4 * sm_count());
    const size_t budget = small ? SEL_SMEM_SHORT : n < SEL_LONG ? SEL_SMEM_MID : SEL_SMEM_LONG;
    const int min_cand = small ? 1024 : 2048;
    p.nw = small ? 8 : n < SEL_LONG ? 16 : 32;
    p.L = sel::plan_layout(n, false, budget, min_cand, p.nw);
    if (!p.L.keyed) p.L = sel::plan_layout(n, true, budget, min_cand, p.nw);       // the general path stages the images
    return p;
}

static vector_status launch_pool_select(const Dims& dm, const vector_budget* budget, const float* scores, int32_t* pool,
                                        cudaStream_t st) {
    vector_status rc = select_kernels_setup();
    if (rc != VECTOR_OK) return rc;
    const int64_t n = budget->n_tokens;
    const SelPlan p = plan_selection(n, dm.U);
    const Layout L = p.L;
    if (p.nw == 8) pool_select_kernel<8><<<dm.U, 256, L.bytes(), st>>>(scores, n, (int)budget->n_pool, pool, L);
    else if (p.nw == 16) pool_select_kernel<16><<<dm.U, 512, L.bytes(), st>>>(scores, n, (int)budget->n_pool, pool, L);
    else pool_select_kernel<32><<<dm.U, 1024, L.bytes(), st>>>(scores, n, (int)budget->n_pool, pool, L);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

static vector_status launch_truncate(const Dims& dm, const vector_budget* budget, const float* eps, const int32_t* pool,
                                     uint8_t* tier, int32_t* ret_idx, int32_t* apx_idx, cudaStream_t st,
                                     bool dependent = false) {
    vector_status rc = select_kernels_setup();
    if (rc != VECTOR_OK) return rc;
    const SelPlan p = plan_selection(budget->n_pool, dm.U);
    const Layout L = p.L;
    // dependent: may start (and clear the tier map) while the kernel before it in the stream drains
#define VEC_TRUNC(NW)                                                                                                   \
    VEC_CUDA_CHECK(launch_maybe_dependent(dependent, truncate_kernel<NW>, dim3(dm.U), dim3(32 * NW), L.bytes(), st, eps, \
                                          pool, (int64_t)budget->n_tokens, (int)budget->n_pool, (int)budget->n_apx, tier, \
                                          ret_idx, apx_idx, L))
    if (p.nw == 8) VEC_TRUNC(8);
    else if (p.nw == 16) VEC_TRUNC(16);
    else VEC_TRUNC(32);
#undef VEC_TRUNC
    return VECTOR_OK;
}

// ---- one map per layer: a token's tier holds for all KV heads of its layer -----------------------
// Layer score of a token = the sum of its per-head base scores (window tokens stay +inf), summed in
// head order.  grid (ceil(N / 256), B L), 256 threads.
__global__ void __launch_bounds__(256)
layer_scores_kernel(const float* __restrict__ scores, int64_t N, int Hkv, float* __restrict__ layer_scores) {
    const int ul = blockIdx.y;
    const int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (i >= N) return;
    float s = 0.f;
    for (int h = 0; h < Hkv; ++h) s += scores[((size_t)ul * Hkv + h) * N + i];
    layer_scores[(size_t)ul * N + i] = s;
}

// Step 2 with one map per layer on CUDA cores (any dtype and head size): a warp per listed token,
// the token's keys of all heads in shared memory, lane = output channels lane, lane + 32, ...
// grid (ceil(n_idx / 8), B L), 256 threads, dynamic shared memory 8 * Hkv * D floats.
template <typename T, int D>
__global__ void __launch_bounds__(256)
residual_layer_generic(const T* __restrict__ K, const T* __restrict__ V, const T* __restrict__ W, int64_t N, int L,
                       int Hkv, const int32_t* __restrict__ idx, int n_idx, float* __restrict__ eps) {
    extern __shared__ float ksm[];
    const int ul = blockIdx.y, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int DL = Hkv * D;
    const int p = blockIdx.x * 8 + wid;
    if (p >= n_idx) return;
    const int64_t tok = idx[(size_t)ul * n_idx + p];
    if ((uint64_t)tok >= (uint64_t)N) {              // an index outside the unit reads as rows of zeros
        if (lane == 0) eps[(size_t)ul * n_idx + p] = 0.f;
        return;
    }
    float* kw = ksm + (size_t)wid * DL;
    for (int c = lane; c < DL; c += 32) kw[c] = to_f32(K[(((size_t)ul * Hkv + c / D) * N + tok) * D + c % D]);
    __syncwarp();
    const T* Wl = W + (size_t)(ul % L) * DL * DL;
    float e = 0.f;
    for (int co = lane; co < DL; co += 32) {
        const T* row = Wl + (size_t)co * DL;
        float pred = 0.f;
        for (int ci = 0; ci < DL; ++ci) pred = fmaf(to_f32(row[ci]), kw[ci], pred);
        const float r = to_f32(V[(((size_t)ul * Hkv + co / D) * N + tok) * D + co % D]) - pred;
        e = fmaf(r, r, e);
    }
    e = warp_sum(e);
    if (lane == 0) eps[(size_t)ul * n_idx + p] = e;
}

static vector_status residual_layer_dispatch(const Dims& dm, int Hkv, int L, const void* K, const void* V, const void* W,
                                             int64_t N, const int32_t* idx, int64_t n_idx, float* eps, cudaStream_t st,
                                             bool dependent) {
    if (n_idx == 0) return VECTOR_OK;
    const int UL = dm.U / Hkv;
    if (dm.dtype == VECTOR_BF16 && dm.d == 128) {
        static PerDeviceOnce once;
        if (once.first()) {
            const cudaError_t e = cudaFuncSetAttribute(rlt::residual_layer_tc, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                       rlt::SMEM_BYTES);
            if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
        }
        int* fault = kernel_fault_address();
        if (!fault) return VECTOR_ERR_CUDA;
        const uint64_t DL = (uint64_t)Hkv * 128;
        CUtensorMap mapW;
        if (!tma::encode_bf16_3d(&mapW, W, DL, DL, (uint64_t)L, DL * 2, DL * DL * 2, 64, 128)) return VECTOR_ERR_CUDA;
        rlt::Params P;
        P.UL = UL; P.L = L; P.Hkv = Hkv; P.n_idx = (int)n_idx; P.N = N;
        P.tpu = (int)((n_idx + rlt::TILE - 1) / rlt::TILE);
        P.n_tiles = (long long)UL * P.tpu;
        const int sms = sm_count();
        const int blocks = (int)(P.n_tiles < sms ? P.n_tiles : sms);
        VEC_CUDA_CHECK(launch_maybe_dependent(dependent, rlt::residual_layer_tc, dim3(blocks), dim3(rlt::THREADS), rlt::SMEM_BYTES,
                                              st, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, mapW, idx, P, eps, fault));
        return VECTOR_OK;
    }
    const dim3 grid((unsigned)((n_idx + 7) / 8), UL);
    const size_t smem = (size_t)8 * Hkv * dm.d * sizeof(float);
#define VEC_RL(T, D)                                                                                                   \
    do {                                                                                                               \
        VEC_CUDA_CHECK(cudaFuncSetAttribute(residual_layer_generic<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                            (int)smem));                                                               \
        residual_layer_generic<T, D><<<grid, 256, smem, st>>>((const T*)K, (const T*)V, (const T*)W, N, L, Hkv, idx,   \
                                                              (int)n_idx, eps);                                        \
    } while (0)
    if (dm.dtype == VECTOR_F32) { if (dm.d == 64) VEC_RL(float, 64); else VEC_RL(float, 128); }
    else { if (dm.d == 64) VEC_RL(__nv_bfloat16, 64); else VEC_RL(__nv_bfloat16, 128); }
#undef VEC_RL
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
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
    return launch_pool_select(dm, budget, scores, pool_idx, (cudaStream_t)stream);
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
    return launch_truncate(dm, budget, eps, pool_idx, tier, ret_idx, apx_idx, (cudaStream_t)stream);
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
    if ((rc = launch_pool_select(dm, budget, scores, pool, st)) != VECTOR_OK) return rc;
    rc = residual_dispatch(dm, K, V, W, budget->n_tokens, pool, budget->n_pool, eps, st, true);
    if (rc != VECTOR_OK) return rc;
    return launch_truncate(dm, budget, eps, pool, tier, ret_idx, apx_idx, st, true);
}

extern "C" vector_status vector_layer_scores(const vector_shape* shape, const float* scores, int64_t N,
                                             float* layer_scores, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!scores || !layer_scores) return VECTOR_ERR_NULL;
    if (N <= 0 || N > (int64_t(1) << 30)) return VECTOR_ERR_SHAPE;
    const int Hkv = shape->n_kv_heads;
    const dim3 grid((unsigned)((N + 255) / 256), dm.U / Hkv);
    layer_scores_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(scores, N, Hkv, layer_scores);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" vector_status vector_residual_layer(const vector_shape* shape, const void* K, const void* V, const void* W_layer,
                                               int64_t N, const int32_t* idx, int64_t n_idx, float* eps, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!K || !V || !W_layer || !idx || !eps) return VECTOR_ERR_NULL;
    if (N <= 0 || N > (int64_t(1) << 30) || n_idx < 0 || n_idx > N) return VECTOR_ERR_SHAPE;
    if (dm.rope) return VECTOR_ERR_UNSUPPORTED;
    return residual_layer_dispatch(dm, shape->n_kv_heads, shape->n_layers, K, V, W_layer, N, idx, n_idx, eps,
                                   (cudaStream_t)stream, false);
}

extern "C" vector_status vector_route_layer(const vector_shape* shape, const vector_budget* budget, const float* layer_scores,
                                            const void* K, const void* V, const void* W_layer, uint8_t* tier,
                                            int32_t* ret_idx, int32_t* apx_idx, float* eps_out, int32_t* pool_idx_out,
                                            void* ws, size_t ws_bytes, void* stream) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!layer_scores || !K || !V || !W_layer || !tier) return VECTOR_ERR_NULL;
    if ((budget->n_ret > 0 && !ret_idx) || (budget->n_apx > 0 && !apx_idx)) return VECTOR_ERR_NULL;
    if (dm.rope) return VECTOR_ERR_UNSUPPORTED;
    const int Hkv = shape->n_kv_heads;
    Dims dl = dm;                       // the selections run per (sequence, layer)
    dl.U = dm.U / Hkv;
    const size_t need = align256((size_t)dl.U * (size_t)budget->n_pool * sizeof(int32_t)) +
                        align256((size_t)dl.U * (size_t)budget->n_pool * sizeof(float));
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < need) return VECTOR_ERR_WORKSPACE;
    char* p = (char*)ws;
    int32_t* pool = pool_idx_out ? pool_idx_out : (int32_t*)p;
    p += align256((size_t)dl.U * (size_t)budget->n_pool * sizeof(int32_t));
    float* eps = eps_out ? eps_out : (float*)p;
    cudaStream_t st = (cudaStream_t)stream;
    if ((rc = launch_pool_select(dl, budget, layer_scores, pool, st)) != VECTOR_OK) return rc;
    rc = residual_layer_dispatch(dm, Hkv, shape->n_layers, K, V, W_layer, budget->n_tokens, pool, budget->n_pool, eps, st, true);
    if (rc != VECTOR_OK) return rc;
    return launch_truncate(dl, budget, eps, pool, tier, ret_idx, apx_idx, st, true);
}
