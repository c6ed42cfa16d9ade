// Three-way routing (paper Section 3.2): Step 1 pool selection by base score,
// Step 2 reconstruction residual on the pool, Step 3 truncation by residual.
//
// Both selections are exact top-k with the lower index winning ties, done as a
// most-significant-digit radix select on an order-preserving 32-bit image of
// the fp32 value (3 histogram passes of 11, 11 and 10 bits find the k-th key and
// how many ties of it are taken; the third runs over a short list of
// candidates), followed by one ordered walk whose block-wide prefix sums place
// the chosen indices in ascending order.  One thread block per unit.
#include "common.cuh"
#include "internal.h"
#include "residual_tc.cuh"

namespace vec {

constexpr int SEL_THREADS = 1024;

// Best = largest image.  For "k smallest" the caller passes inverted images.
template <bool SMALLEST>
__device__ __forceinline__ uint32_t select_image(float v) {
    uint32_t k = ordered_key(v);
    return SMALLEST ? ~k : k;
}

// hist[bin] += 1 if `valid`.  With 11-bit digits the lanes of a warp rarely share a bin, so a plain
// shared-memory atomic per element is cheaper than aggregating equal bins across the warp first;
// equal bins (many equal values) serialise inside the atomic unit and cost time, not correctness.
__device__ __forceinline__ void hist_add(int* hist, int bin, bool valid) {
    if (valid) atomicAdd(&hist[bin], 1);
}

// Scratch of one selection (static shared memory of the block).
constexpr int CAND_CAP = 6144;
constexpr int MASK_GROUPS = 1024;   // groups of 32 elements whose selection is kept as bit masks
struct OrderedScratch { int gt[32], tie[32], out[32], quota[32]; };
constexpr int SEL_BINS = 2048;      // digits of 11, 11 and 10 bits
struct SelectScratch {
    int hist[SEL_BINS];
    int bc[2];
    int part[32];                 // per-warp bin sums of pick_bin
    int n_cand, overflow;
    int32_t cand[CAND_CAP];       // indices of the elements that share the k-th key's leading 11 bits
    uint32_t sel_mask[MASK_GROUPS];   // per group of 32 elements: those above the k-th key
    uint32_t tie_mask[MASK_GROUPS];   // ... and those equal to it
    OrderedScratch os;
};

// The bin of hist[0..SEL_BINS), counted from the top, in which the cumulative count reaches
// `remaining` (-> bc[0]) and the rank wanted inside that bin, 1-based (-> bc[1]).  Every thread of
// the block calls it (one block barrier inside; the caller synchronises before and after): warp w
// sums the 64 bins below SEL_BINS - 64 w, every warp scans the 32 sums, and the one warp whose
// range holds the answer finds the bin with two lane scans.
static_assert(SEL_THREADS == 1024 && SEL_BINS == 2048, "one warp per 64 bins");
__device__ __forceinline__ int lane_scan_incl(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += t;
    }
    return v;
}
__device__ __forceinline__ void pick_bin(const int* hist, int remaining, int* bc, int* part) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int top = SEL_BINS - 1 - wid * 64;                // this warp's bins: top, top - 1, .., top - 63
    const int c0 = hist[top - lane], c1 = hist[top - 32 - lane];
    const int tot = __reduce_add_sync(0xffffffffu, c0 + c1);
    if (lane == 0) part[wid] = tot;
    __syncthreads();
    const int p = part[lane];
    const int above = __shfl_sync(0xffffffffu, lane_scan_incl(p, lane) - p, wid);      // count in the warps above this one
    if (above < remaining && above + tot >= remaining) {     // exactly one warp
        const int r = remaining - above;
        const int s0 = lane_scan_incl(c0, lane), tot0 = __shfl_sync(0xffffffffu, s0, 31);
        const int s1 = tot0 + lane_scan_incl(c1, lane);
        if (s0 - c0 < r && s0 >= r) { bc[0] = top - lane; bc[1] = r - (s0 - c0); }
        if (s1 - c1 < r && s1 >= r) { bc[0] = top - 32 - lane; bc[1] = r - (s1 - c1); }
    }
}

// One histogram pass over all of vals on the digit at `shift`, among the elements whose image
// matches prefix under mask.  Eight independent loads in flight per thread: the pass is bound by
// memory latency otherwise.
template <bool SMALLEST>
__device__ __forceinline__ void hist_pass_all(const float* __restrict__ vals, int n, int shift, uint32_t digit_mask,
                                              uint32_t prefix, uint32_t mask, int* hist, uint32_t* stage = nullptr) {
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
            if (stage && i < n) stage[i] = key;          // keep the image for the later passes
            hist_add(hist, (key >> shift) & digit_mask, i < n && (key & mask) == prefix);
        }
    }
}

// Piece of the input that warp `wid` owns in the ordered passes: [w0, w1), a multiple of 32 long.
__device__ __forceinline__ int ordered_chunk(int n, int nw) { return (((n + nw - 1) / nw) + 31) & ~31; }

// Exact top-k of vals[0..n) (largest images; for "k smallest" the images are inverted) with the
// lower index winning ties, emitted in index order: emit(i, chosen, pos) is called for every element
// i, pos being its rank among the chosen ones if chosen, else among the others.  1 <= k <= n
// unless !any (nothing is chosen then).  All threads of the block call it.
//
// The k-th key is found by a most-significant-digit radix select with digits of 11, 11 and 10 bits.
// Pass 1 reads the whole input.  Pass 2 reads it once more, warp by contiguous piece, and on the
// way (a) notes per group of 32 elements, as a bit mask, those whose leading 11 bits already beat
// the k-th key's and (b) lists the indices of those that share them (the candidates: a quarter of
// a binade of values, a few thousand at most).  Pass 3 runs over the list; so does the final
// classification, which adds the candidates above the k-th key to the masks and marks its ties in
// a second mask.  The per-piece counts and the emission in index order then need the masks only,
// not the values.  Two fallbacks read the input again instead: more than CAND_CAP candidates
// (pass 3 and the classification walk the input), more than 32 MASK_GROUPS elements (the masks are
// not kept).  With `stage` (n words of shared memory) pass 1 also keeps the images there and the
// later passes never go back to global memory.
template <bool SMALLEST, typename Emit>
__device__ __forceinline__ void select_emit(const float* __restrict__ vals, int n, int k, bool any, SelectScratch& S, Emit emit,
                                            uint32_t* stage = nullptr) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    const int per_w = ordered_chunk(n, nw);
    const int w0 = min(n, wid * per_w), w1 = min(n, w0 + per_w);
    const bool masked = n <= 32 * MASK_GROUPS;
    uint32_t kth = 0xffffffffu;
    int take_ties = 0;
    if (threadIdx.x < 32) { S.os.gt[threadIdx.x] = 0; S.os.tie[threadIdx.x] = 0; }
    if (masked)
        for (int g = threadIdx.x; g < MASK_GROUPS; g += blockDim.x) { S.sel_mask[g] = 0u; S.tie_mask[g] = 0u; }
    if (any) {
        // ---- pass 1: leading 11 bits
        for (int b = threadIdx.x; b < SEL_BINS; b += blockDim.x) S.hist[b] = 0;
        if (threadIdx.x == 0) { S.n_cand = 0; S.overflow = 0; }
        __syncthreads();
        hist_pass_all<SMALLEST>(vals, n, 21, 2047u, 0u, 0u, S.hist, stage);
        __syncthreads();
        pick_bin(S.hist, k, S.bc, S.part);
        __syncthreads();
        const uint32_t bin1 = (uint32_t)S.bc[0];
        int remaining = S.bc[1];
        __syncthreads();
        // ---- pass 2: next 11 bits among the candidates; masks of the sure ones; candidate list
        for (int b = threadIdx.x; b < SEL_BINS; b += blockDim.x) S.hist[b] = 0;
        __syncthreads();
        for (int base = w0; base < w1; base += 128) {
            uint32_t kv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + 32 * j + lane;
                kv[j] = i >= w1 ? 0u : stage ? stage[i] : select_image<SMALLEST>(vals[i]);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + 32 * j + lane;
                const bool in = i < w1;
                const uint32_t key = kv[j];
                const uint32_t d1 = key >> 21;
                if (masked) {
                    const unsigned gb = __ballot_sync(0xffffffffu, in && d1 > bin1);
                    if (lane == 0 && base + 32 * j < w1) S.sel_mask[(base >> 5) + j] = gb;
                }
                if (in && d1 == bin1) {
                    atomicAdd(&S.hist[(key >> 10) & 2047], 1);
                    const int at = atomicAdd(&S.n_cand, 1);
                    if (at < CAND_CAP) S.cand[at] = i;
                    else S.overflow = 1;
                }
            }
        }
        __syncthreads();
        pick_bin(S.hist, remaining, S.bc, S.part);
        __syncthreads();
        uint32_t prefix = (bin1 << 21) | ((uint32_t)S.bc[0] << 10);
        const uint32_t mask = 0xfffffc00u;
        remaining = S.bc[1];
        const bool listed = S.overflow == 0;
        const int n_cand = S.n_cand;
        __syncthreads();
        // ---- pass 3: the last 10 bits
        for (int b = threadIdx.x; b < SEL_BINS; b += blockDim.x) S.hist[b] = 0;
        __syncthreads();
        if (listed) {
            for (int j = threadIdx.x; j < n_cand; j += blockDim.x) {
                const uint32_t key = stage ? stage[S.cand[j]] : select_image<SMALLEST>(vals[S.cand[j]]);
                hist_add(S.hist, key & 1023, (key & mask) == prefix);
            }
        } else {
            hist_pass_all<SMALLEST>(vals, n, 0, 1023u, prefix, mask, S.hist);
        }
        __syncthreads();
        pick_bin(S.hist, remaining, S.bc, S.part);
        __syncthreads();
        prefix |= (uint32_t)S.bc[0];
        remaining = S.bc[1];
        __syncthreads();
        kth = prefix;
        take_ties = remaining;          // all strictly better elements precede; `remaining` ties complete k
        // ---- the candidates against the k-th key
        if (masked && listed) {
            for (int j = threadIdx.x; j < n_cand; j += blockDim.x) {
                const int i = S.cand[j];
                const uint32_t key = stage ? stage[i] : select_image<SMALLEST>(vals[i]);
                if (key > kth) atomicOr(&S.sel_mask[i >> 5], 1u << (i & 31));
                else if (key == kth) atomicOr(&S.tie_mask[i >> 5], 1u << (i & 31));
            }
        } else if (masked) {
            for (int base = w0; base < w1; base += 128) {
                float v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) v[j] = base + 32 * j + lane < w1 ? vals[base + 32 * j + lane] : 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool in = base + 32 * j + lane < w1;
                    const uint32_t key = select_image<SMALLEST>(v[j]);
                    const unsigned gb = __ballot_sync(0xffffffffu, in && key > kth);
                    const unsigned tb = __ballot_sync(0xffffffffu, in && key == kth);
                    if (lane == 0 && base + 32 * j < w1) { S.sel_mask[(base >> 5) + j] = gb; S.tie_mask[(base >> 5) + j] = tb; }
                }
            }
        }
    }
    __syncthreads();
    // ---- per piece: how many better elements, how many ties
    if (masked) {
        int g2 = 0, t2 = 0;
        for (int g = (w0 >> 5) + lane; g < ((w1 + 31) >> 5); g += 32) { g2 += __popc(S.sel_mask[g]); t2 += __popc(S.tie_mask[g]); }
        g2 = __reduce_add_sync(0xffffffffu, g2);
        t2 = __reduce_add_sync(0xffffffffu, t2);
        if (lane == 0) { S.os.gt[wid] = g2; S.os.tie[wid] = t2; }
    } else if (any) {
        int g2 = 0, t2 = 0;
        for (int base = w0; base < w1; base += 128) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = base + 32 * j + lane < w1 ? vals[base + 32 * j + lane] : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = base + 32 * j + lane < w1;
                const uint32_t key = select_image<SMALLEST>(v[j]);
                g2 += __popc(__ballot_sync(0xffffffffu, in && key > kth));
                t2 += __popc(__ballot_sync(0xffffffffu, in && key == kth));
            }
        }
        if (lane == 0) { S.os.gt[wid] = g2; S.os.tie[wid] = t2; }
    }
    __syncthreads();
    // ---- offsets of the pieces; ties go to the lowest indices
    if (wid == 0) {
        const int t = lane < nw ? S.os.tie[lane] : 0;
        int inc = t;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, inc, o); if (lane >= o) inc += x; }
        const int quota = max(0, min(t, take_ties - (inc - t)));
        const int c = (lane < nw ? S.os.gt[lane] : 0) + quota;
        int ci = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(0xffffffffu, ci, o); if (lane >= o) ci += x; }
        S.os.out[lane] = ci - c;
        S.os.quota[lane] = quota;
    }
    __syncthreads();
    // ---- emission in index order
    int pos = S.os.out[wid], ties_left = S.os.quota[wid];
    if (masked) {
        for (int base = w0; base < w1; base += 32) {
            const int i = base + lane;
            const unsigned gb = S.sel_mask[base >> 5], tb = S.tie_mask[base >> 5];
            const int take = min(ties_left, __popc(tb));
            const bool chosen = ((gb >> lane) & 1u) || (((tb >> lane) & 1u) && __popc(tb & lt) < take);
            const unsigned cb = __ballot_sync(0xffffffffu, chosen);
            const int before = pos + __popc(cb & lt);               // chosen elements before this one in the unit
            if (i < w1) emit(i, chosen, chosen ? before : i - before);
            pos += __popc(cb);
            ties_left -= take;
        }
    } else {
        for (int base = w0; base < w1; base += 128) {
            float v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = base + 32 * j + lane < w1 ? vals[base + 32 * j + lane] : 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + 32 * j + lane;
                const bool in = i < w1;
                const uint32_t key = select_image<SMALLEST>(v[j]);
                const bool tie = any && in && key == kth;
                const unsigned tb = __ballot_sync(0xffffffffu, tie);
                const bool chosen = any && in && (key > kth || (tie && __popc(tb & lt) < ties_left));
                const unsigned cb = __ballot_sync(0xffffffffu, chosen);
                const int before = pos + __popc(cb & lt);
                if (in) emit(i, chosen, chosen ? before : i - before);
                pos += __popc(cb);
                ties_left -= min(ties_left, __popc(tb));
            }
        }
    }
}

// Step 1.  grid (U), SEL_THREADS threads.
__global__ void __launch_bounds__(SEL_THREADS, 2)
pool_select_kernel(const float* __restrict__ scores, int64_t N, int n_pool, int32_t* __restrict__ pool_idx) {
    __shared__ SelectScratch S;
    // inside vector_route the residual kernel is launched as a programmatic dependent: its blocks may
    // take SMs as this grid's blocks leave them; it reads the index lists only after its own wait
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    const int u = blockIdx.x, n = (int)N;
    const float* s = scores + (size_t)u * N;
    int32_t* out = pool_idx + (size_t)u * n_pool;
    if (n_pool <= 0) return;
    select_emit<false>(s, n, n_pool, true, S, [&](int i, bool chosen, int pos) { if (chosen) out[pos] = i; });
}

// Step 3.  grid (U), SEL_THREADS threads; dynamic shared memory: n_pool words (stage = 1) or none.
__global__ void __launch_bounds__(SEL_THREADS, 2)
truncate_kernel(const float* __restrict__ eps, const int32_t* __restrict__ pool_idx, int64_t N, int n_pool,
                int n_apx, uint8_t* __restrict__ tier, int32_t* __restrict__ ret_idx,
                int32_t* __restrict__ apx_idx, int stage) {
    __shared__ SelectScratch S;
    extern __shared__ uint32_t staged_keys[];        // n_pool words when the launch gave them, else none
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
    // everything above touches only the tier map; the residuals and the pool list belong to the
    // kernels before this one (a no-op unless launched as a programmatic dependent)
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    __syncthreads();
    select_emit<true>(e, n_pool, n_apx, n_apx > 0, S, [&](int p, bool is_apx, int pos) {
        const int32_t token = pool[p];
        if (is_apx) { ao[pos] = token; tr[token] = 1; }
        else        { ro[pos] = token; tr[token] = 2; }
    }, stage ? staged_keys : nullptr);
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

// Residual lists up to this length are kept in shared memory by the truncation kernel (two blocks
// per SM stay resident).
constexpr int TRUNC_STAGE_MAX = 16384;
static vector_status launch_truncate(const Dims& dm, const vector_budget* budget, const float* eps, const int32_t* pool,
                                     uint8_t* tier, int32_t* ret_idx, int32_t* apx_idx, cudaStream_t st,
                                     bool dependent = false) {
    const int stage = budget->n_pool <= TRUNC_STAGE_MAX ? 1 : 0;
    const size_t smem = stage ? (size_t)budget->n_pool * sizeof(uint32_t) : 0;
    static PerDeviceOnce once;
    if (once.first()) {
        const cudaError_t e = cudaFuncSetAttribute(truncate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   TRUNC_STAGE_MAX * (int)sizeof(uint32_t));
        if (e != cudaSuccess) { once.undo(); VEC_CUDA_CHECK(e); }
    }
    // dependent: may start (and clear the tier map) while the kernel before it in the stream drains
    VEC_CUDA_CHECK(launch_maybe_dependent(dependent, truncate_kernel, dim3(dm.U), dim3(SEL_THREADS), smem, st, eps, pool,
                                          (int64_t)budget->n_tokens, (int)budget->n_pool, (int)budget->n_apx, tier, ret_idx,
                                          apx_idx, stage));
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
    pool_select_kernel<<<dm.U, SEL_THREADS, 0, st>>>(scores, budget->n_tokens, (int)budget->n_pool, pool);
    VEC_LAUNCH_CHECK();
    rc = residual_dispatch(dm, K, V, W, budget->n_tokens, pool, budget->n_pool, eps, st, true);
    if (rc != VECTOR_OK) return rc;
    return launch_truncate(dm, budget, eps, pool, tier, ret_idx, apx_idx, st, true);
}
