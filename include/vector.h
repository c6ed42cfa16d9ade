/*
 * libvector -- C ABI of the VECTOR hot path on one NVIDIA B200 (sm_100a).
 *
 * VECTOR (paper Section 3) extends an eviction-based KV-cache compressor with a
 * third token state.  Per (sequence, layer, KV head) -- a "unit" -- a base
 * importance scorer picks an expanded pool of tokens, the reconstruction
 * residual eps_i = ||v_i - W k_i||^2 of a fixed, offline-fitted linear map W is
 * evaluated on the pool, the pool tokens with the smallest residual keep only
 * their key ("approximated"), the rest keep key and value ("retained"), and
 * everything outside the pool is evicted.  At generation time attention runs
 * over both pools with one softmax; an approximated value is rebuilt as W k.
 *
 * General rules of this interface
 *  - Every entry point returns a vector_status; nothing throws, aborts or prints.
 *  - The caller owns every buffer.  The library allocates no device memory; the
 *    device calls take a caller-provided workspace of at least
 *    vector_workspace_bytes() bytes (256-byte aligned).
 *  - "device" pointers must be device memory of the current CUDA device;
 *    "host" pointers plain host memory.  Structs are passed by host pointer.
 *  - Device calls are asynchronous on the cudaStream_t passed as `stream`
 *    (a void* here; NULL = the default stream) and never synchronise.
 *  - Inputs are const; outputs are fully overwritten.
 *  - Layout: unit index u = (b * n_layers + l) * n_kv_heads + h.  All per-unit
 *    arrays are contiguous in u; token rows are contiguous (head_dim elements).
 *    The g = n_q_heads / n_kv_heads query heads of KV head h are a = h*g .. h*g+g-1,
 *    so [B][L][Hq][...] query tensors are [U][g][...] in memory.
 *  - Linear maps follow the paper's column convention y = W x: W[c_out][c_in],
 *    row-major, one d x d map per (layer, KV head): index l * n_kv_heads + h.
 *  - Supported: head_dim 64 or 128; dtype fp32 or bf16; n_q_heads % n_kv_heads == 0,
 *    g <= 8; window * g <= 1024; pool_kernel odd, 1..15; at most 65535 units per call;
 *    every device pointer 16-byte aligned.  The tensor-core kernels (tcgen05 score passes and residual,
 *    TMA-fed decode) serve bf16 with head_dim 128; fp32 and head_dim 64 run on CUDA-core kernels of the
 *    same interface, written for parity rather than speed.
 */
#ifndef VECTOR_H_
#define VECTOR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define VECTOR_API __attribute__((visibility("default")))
#else
#define VECTOR_API
#endif

typedef enum {
    VECTOR_OK = 0,
    VECTOR_ERR_NULL = -1,        /* a required pointer is NULL                      */
    VECTOR_ERR_SHAPE = -2,       /* inconsistent or unsupported shape               */
    VECTOR_ERR_DTYPE = -3,       /* unknown dtype                                   */
    VECTOR_ERR_BUDGET = -4,      /* tier sizes impossible for this N / window       */
    VECTOR_ERR_WORKSPACE = -5,   /* workspace NULL, misaligned or too small         */
    VECTOR_ERR_SINGULAR = -6,    /* Gram matrix not positive definite               */
    VECTOR_ERR_CUDA = -7,        /* a CUDA runtime call failed (see last_cuda_error) */
    VECTOR_ERR_TIMEOUT = -8,     /* a bounded wait inside a kernel gave up (vector_sync_check) */
    VECTOR_ERR_UNSUPPORTED = -9  /* valid request this build does not implement     */
} vector_status;

typedef enum { VECTOR_F32 = 0, VECTOR_BF16 = 1 } vector_dtype;

/* Geometry of one call.  dtype is the element type of Q, K, V, W and the cache. */
typedef struct {
    int32_t batch, n_layers, n_q_heads, n_kv_heads, head_dim;
    int32_t dtype;          /* vector_dtype                                         */
    int32_t window;         /* w: observation-window length of the base scorer      */
    int32_t pool_kernel;    /* max-pool width along the sequence (odd)              */
    float   sm_scale;       /* logit scale; <= 0 means 1/sqrt(head_dim)             */
    int32_t rope_enabled;   /* != 0: the regressor sees the inverse-rotated key     */
    float   rope_theta;     /* rotary base (e.g. 10000)                             */
} vector_shape;

/* Integer tier sizes of one unit (paper Section 3.2; all units share them). */
typedef struct {
    int64_t n_tokens;        /* N                                                   */
    int64_t n_budget_pairs;  /* Bp: full K/V pairs the memory budget pays for       */
    int64_t n_a;             /* p_a * N                                             */
    int64_t n_pool;          /* Bp + n_a   keys kept                                */
    int64_t n_apx;           /* 2 n_a      key-only tokens                          */
    int64_t n_ret;           /* Bp - n_a   tokens with key and value                */
    int64_t n_evict;         /* N - n_pool                                          */
} vector_budget;

/*
 * The mixed cache (paper Section 3.2, Step 3 and Figure 2): a retained K/V pool
 * and a key-only pool, rows in ascending original position.  All device memory,
 * caller-owned.  cap_* are row capacities per unit; n_* the rows in use (equal
 * for all units).  A decoded token is appended by writing its K/V row at
 * ret_*[u][n_ret] and bumping n_ret (<= cap_ret): no library call is needed.
 */
typedef struct {
    void*    ret_k;     /* [U][cap_ret][d]                                          */
    void*    ret_v;     /* [U][cap_ret][d]                                          */
    void*    apx_k;     /* [U][cap_apx][d]                                          */
    int32_t* ret_pos;   /* [U][cap_ret] original token index of each retained row   */
    int32_t* apx_pos;   /* [U][cap_apx]                                             */
    int64_t  cap_ret, cap_apx, n_ret, n_apx;
} vector_cache;

/* Text for a status code (static storage). */
VECTOR_API const char* vector_status_string(vector_status s);
/* The raw cudaError_t of the last VECTOR_ERR_CUDA on this thread (0 if none). */
VECTOR_API int vector_last_cuda_error(void);
/* Kernels this library has launched so far in this process (all threads, all devices): a
 * monotone counter for accounting; the difference across a region is the number of launches
 * the calls inside it made. */
VECTOR_API uint64_t vector_kernel_launches(void);

/*
 * Tier sizes, host only (paper Section 3.2 proportions and Eq. (1)).
 * n_budget_pairs = (1 - p_c) N.  n_a < 0 selects Eq. (1) with its small constant
 * taken as 0: n_a = min(floor((N - Bp)/2), floor(Bp/2)); otherwise n_a is used
 * as given.  Derived: n_pool = Bp + n_a, n_apx = 2 n_a, n_ret = Bp - n_a, so
 * n_pool keys + n_ret values cost exactly Bp pairs.  Errors: VECTOR_ERR_BUDGET
 * if Bp > N, n_a > Bp, n_pool > N, window > N or n_pool < window (the base
 * scorer always keeps its observation window).
 */
VECTOR_API vector_status vector_plan_budget(int64_t n_tokens, int64_t n_budget_pairs, int64_t n_a,
                                 int32_t window, vector_budget* out /* host */);

/*
 * Offline calibration, host only (paper Section 3.1, the OLS objective):
 * W = argmin_W sum_t ||W k_t - v_t||^2 + lambda ||W||_F^2, no intercept, fp64
 * normal equations.  K: host [n][d_k], V: host [n][d_v] of dtype dt; W_out: host
 * fp32 [d_v][d_k]; r2_out (nullable): the global R^2 of the fit on these samples,
 * 1 - sum||v - W k||^2 / sum||v - mean(v)||^2.  VECTOR_ERR_SINGULAR if the
 * regularised Gram matrix is not positive definite.
 */
VECTOR_API vector_status vector_calibrate(const void* K, const void* V, int64_t n, int32_t d_k, int32_t d_v,
                               int32_t dt, double lambda, float* W_out, double* r2_out);

/*
 * Waits inside the kernels are bounded.  This call synchronises the current device and returns
 * the code recorded by a wait that gave up since the last call (0 = none, -1 = CUDA error),
 * clearing it.  Results of the call that recorded a fault are invalid.
 */
VECTOR_API int vector_device_fault(void);

/*
 * The same check as a status and on one stream: waits until the work queued on `stream` has finished,
 * then returns VECTOR_OK, VECTOR_ERR_TIMEOUT if a bounded wait inside a kernel gave up since the last
 * check (the record is cleared; outputs written since then are invalid), or VECTOR_ERR_CUDA.
 */
VECTOR_API vector_status vector_sync_check(void* stream);

/* Bytes of device workspace that suffice for every device call with this shape and budget. */
VECTOR_API size_t vector_workspace_bytes(const vector_shape* shape, const vector_budget* budget);

/*
 * Base importance score (Step 1's scorer, SnapKV-style).  For each unit the last
 * w queries of its g query heads attend causally to all N keys (query j of the
 * window sits at position N-w+j); softmax over the visible keys; the mass each
 * key receives is summed over the window and the g heads; the sums are
 * max-pooled along the sequence with a centred window of pool_kernel over the
 * prefix positions i < N-w; window tokens score +inf.
 * Q_obs: device [U][g][w][d]; K: device [U][N][d]; scores: device fp32 [U][N];
 * raw_out (nullable): device fp32 [U][N], the un-pooled sums.
 */
VECTOR_API vector_status vector_score(const vector_shape* shape, const void* Q_obs, const void* K, int64_t N,
                           float* scores, float* raw_out, void* ws, size_t ws_bytes, void* stream);

/* Build constant of the tensor-core score passes (bf16, head_dim 128): the share of the softmax
 * exponentials that is evaluated by a polynomial on the FMA pipe instead of the special-function
 * unit (the unit that bounds the passes).  For reading the pipe counters of vector_score. */
VECTOR_API float vector_score_exp2_fma_share(void);

/*
 * Query-agnostic base scorer by key geometry, an alternative to vector_score for Step 1 (the
 * paper names KeyDiff among the base scorers, Sections 3.2 and 5.1, "key geometric diversity",
 * without a formula; this is the published idea): with the anchor a = sum_j k_j / ||k_j||,
 * score_i = - <k_i, a> / (||k_i|| ||a||), in [-1, 1]; higher = less like the average key.  No
 * observation window and no pooling (shape->window and pool_kernel are not used by this call, but
 * vector_route still keeps shape->window <= n_pool).  A zero key scores 0.
 * K: device [U][N][d]; scores: device fp32 [U][N].
 */
VECTOR_API vector_status vector_score_keydiff(const vector_shape* shape, const void* K, int64_t N,
                                   float* scores, void* ws, size_t ws_bytes, void* stream);

/*
 * Step 1, budget relaxation: per unit the n_pool largest scores, ties to the
 * lower index.  scores: device fp32 [U][N]; pool_idx: device [U][n_pool] ascending.
 */
VECTOR_API vector_status vector_pool_select(const vector_shape* shape, const vector_budget* budget,
                                 const float* scores, int32_t* pool_idx,
                                 void* ws, size_t ws_bytes, void* stream);

/*
 * Step 2, residual evaluation: eps[u][p] = || v_i - W k~_i ||_2^2, i = idx[u][p],
 * k~ the key or (rope_enabled) its inverse rotation by position i.
 * K, V: device [U][N][d]; W: device [L*Hkv][d][d] of shape->dtype;
 * idx: device [U][n_idx]; eps: device fp32 [U][n_idx].
 */
VECTOR_API vector_status vector_residual(const vector_shape* shape, const void* K, const void* V, const void* W,
                              int64_t N, const int32_t* idx, int64_t n_idx, float* eps, void* stream);

/*
 * Step 3, asymmetric truncation: per unit the n_apx pool tokens with the
 * smallest eps (ties to the lower index) become key-only.  eps: device fp32
 * [U][n_pool] in pool order; pool_idx: device [U][n_pool] ascending;
 * tier: device [U][N], 0 evicted / 1 approximated / 2 retained;
 * ret_idx: device [U][n_ret], apx_idx: device [U][n_apx], both ascending.
 */
VECTOR_API vector_status vector_truncate(const vector_shape* shape, const vector_budget* budget,
                              const float* eps, const int32_t* pool_idx,
                              uint8_t* tier, int32_t* ret_idx, int32_t* apx_idx,
                              void* ws, size_t ws_bytes, void* stream);

/*
 * Steps 1-3 chained on the device with no host round trip (paper Section 3.2).
 * Arguments as in the three calls above; eps_out (nullable): device fp32
 * [U][n_pool]; pool_idx_out (nullable): device [U][n_pool].
 */
VECTOR_API vector_status vector_route(const vector_shape* shape, const vector_budget* budget,
                           const float* scores, const void* K, const void* V, const void* W,
                           uint8_t* tier, int32_t* ret_idx, int32_t* apx_idx,
                           float* eps_out, int32_t* pool_idx_out,
                           void* ws, size_t ws_bytes, void* stream);

/*
 * Compaction into the mixed cache (Step 3's three bullets): rows ret_idx of K
 * and V go to cache->ret_k / ret_v, rows apx_idx of K to cache->apx_k, original
 * indices to ret_pos / apx_pos.  Requires cache->n_ret == budget->n_ret,
 * cache->n_apx == budget->n_apx, capacities >= counts (VECTOR_ERR_SHAPE).
 */
VECTOR_API vector_status vector_compact(const vector_shape* shape, const vector_budget* budget,
                             const void* K, const void* V,
                             const int32_t* ret_idx, const int32_t* apx_idx,
                             const vector_cache* cache, void* stream);

/*
 * Generation-time attention over the mixed cache (Step 3: values of approximated
 * tokens are rebuilt as W k).  Per query head: p = softmax over the keys of both
 * pools jointly (logit = sm_scale * q.k), then
 *   mode 0 (factored):  o = sum_R p_i v_i + W (sum_A p_i k~_i)
 *   mode 1 (per tile):  o = sum_R p_i v_i + sum_A p_i (W k~_i), W k formed tile by tile on the tensor
 *                       cores; bf16, head_dim 128, rope off only (else VECTOR_ERR_UNSUPPORTED); about
 *                       three times slower than mode 0, which gives the same sum by linearity
 * With shape->rope_enabled, k~_i is the stored key turned back by cache->apx_pos (required then);
 * the logit always uses the stored key.
 * q: device [U][g][d] of shape->dtype; out: device [U][g][d] of out_dtype.
 */
VECTOR_API vector_status vector_decode_attn(const vector_shape* shape, const void* q, const vector_cache* cache,
                                 const void* W, void* out, int32_t out_dtype, int32_t mode,
                                 void* ws, size_t ws_bytes, void* stream);

/*
 * Diagnostics of a routed cache (paper Section 4: the distortion measure E, R^2_approx and the
 * condition of Proposition 1).  importance: device fp32 [U][N], non-negative finite weights w_i,
 * normalised per unit to sum 1 by the call (pass the un-pooled sums raw_out of vector_score; the
 * pooled scores carry +inf for the window).  tier, pool_idx, eps: as written by vector_route
 * (eps_out and pool_idx_out are needed).  V: device [U][N][d].  out: device fp32 [U][8] =
 *   { E = sum_evicted w + sum_approx w ||v - W k||^2 / ||v||^2,  R2_approx = 1 - mu_A,
 *     mu_A = mean relative reconstruction error over the approximated tokens,
 *     sum of evicted w, sum of approximated w,  w_bar = (1 - sum evicted w) / n_pool,
 *     w_star = largest evicted w,  threshold = w_bar / (w_star + w_bar) }.
 * Approximation reduces the distortion when R2_approx > threshold (Proposition 1).
 */
VECTOR_API vector_status vector_diagnostics(const vector_shape* shape, const vector_budget* budget,
                                 const float* importance, const uint8_t* tier, const int32_t* pool_idx,
                                 const float* eps, const void* V, float* out /* [U][8] */, void* stream);

/*
 * K -> V predictability of a map over a whole context (the R^2_global of the paper's Section 3.1,
 * "Empirical Evidence", and its cross-model table): per unit, over ALL N tokens,
 *   R^2 = 1 - sum_i ||v_i - W k_i||^2 / sum_i ||v_i - mean(v)||^2.
 * K, V: device [U][N][d]; W: device [L][Hkv][d][d]; out: device fp32 [U][4] = { R^2, SS_res, SS_tot, N }
 * (R^2 = 1 when both sums are 0, -inf when only SS_tot is).  The residuals come from the kernel of
 * vector_residual, the sums are carried in fp64.  ws: at least vector_r2_global_workspace_bytes().
 */
VECTOR_API size_t vector_r2_global_workspace_bytes(const vector_shape* shape, int64_t N);
VECTOR_API vector_status vector_r2_global(const vector_shape* shape, const void* K, const void* V, const void* W,
                                          int64_t N, float* out /* [U][4] */, void* ws, size_t ws_bytes, void* stream);

/*
 * ---- One map per layer --------------------------------------------------------------------------
 * The paper calibrates its map layer-wise (Section 5.1, "Implementation Details"; the Remark of
 * Section 3.1 writes K and V as whole-layer projections): a token's key and value are then the
 * concatenations over the layer's Hkv KV heads, W_layer has shape [Hkv d][Hkv d] (row-major,
 * y = W x, one per layer: device [L][Hkv d][Hkv d] of shape->dtype), and because the reconstruction
 * of one head's value reads every head's key of the token, a token's tier holds for the whole layer:
 * scores, tier maps and index lists are per (sequence, layer), [B][L][...], while K, V, the cache
 * pools, q and out keep the per-head layouts of the calls above (the Hkv pools of a layer list the
 * same tokens).  Calibrate with vector_calibrate on host rows of Hkv d elements (d_k = d_v = Hkv d).
 * RoPE decoupling is not implemented for this variant (VECTOR_ERR_UNSUPPORTED).
 */
/* Bytes of device workspace that suffice for vector_route_layer and vector_decode_attn_layer. */
VECTOR_API size_t vector_layer_workspace_bytes(const vector_shape* shape, const vector_budget* budget);

/* Layer score of a token = the sum over the layer's KV heads of its per-head base scores (window
 * tokens stay +inf).  scores: device fp32 [B][L][Hkv][N]; layer_scores: device fp32 [B][L][N]. */
VECTOR_API vector_status vector_layer_scores(const vector_shape* shape, const float* scores, int64_t N,
                                             float* layer_scores, void* stream);

/* Step 2 with the layer's map: eps[ul][p] = sum_h || v_{i,h} - (W_layer k_i)[h] ||^2, i = idx[ul][p],
 * k_i the token's keys of all heads.  idx: device [B L][n_idx]; eps: device fp32 [B L][n_idx]. */
VECTOR_API vector_status vector_residual_layer(const vector_shape* shape, const void* K, const void* V,
                                               const void* W_layer, int64_t N, const int32_t* idx, int64_t n_idx,
                                               float* eps, void* stream);

/* Steps 1-3 per (sequence, layer) (Section 3.2 with the layer-wise map of Section 5.1).
 * layer_scores: device fp32 [B L][N]; tier: device [B L][N]; ret_idx: device [B L][n_ret]; apx_idx:
 * device [B L][n_apx]; eps_out, pool_idx_out (nullable): device [B L][n_pool]. */
VECTOR_API vector_status vector_route_layer(const vector_shape* shape, const vector_budget* budget,
                                            const float* layer_scores, const void* K, const void* V,
                                            const void* W_layer, uint8_t* tier, int32_t* ret_idx, int32_t* apx_idx,
                                            float* eps_out, int32_t* pool_idx_out, void* ws, size_t ws_bytes,
                                            void* stream);

/* vector_compact with one pair of index lists per (sequence, layer), shared by the layer's heads. */
VECTOR_API vector_status vector_compact_layer(const vector_shape* shape, const vector_budget* budget,
                                              const void* K, const void* V, const int32_t* ret_idx,
                                              const int32_t* apx_idx, const vector_cache* cache, void* stream);

/* Generation-time attention with the layer's map, factored form: per query head a of KV head h,
 *   o_a = sum_R p_i v_{i,h} + sum_h' W_layer[h][h'] (sum_A p_i k_{i,h'}),  p = softmax over head h's keys
 * (W_layer[h][h'] = the d x d block of output head h, input head h').  Arguments as vector_decode_attn. */
VECTOR_API vector_status vector_decode_attn_layer(const vector_shape* shape, const void* q, const vector_cache* cache,
                                                  const void* W_layer, void* out, int32_t out_dtype, void* ws,
                                                  size_t ws_bytes, void* stream);

/*
 * Allocation-free variant of vector_decode_attn (the paper has no counterpart:
 * this entry point exists for the integration, not for the method).
 *
 * Meant for callers that cannot obtain device memory at the time of the call:
 * a serving process whose own pool already owns the whole device so that a
 * later cudaMalloc fails, or a latency-critical decode loop in which the
 * device-wide stall of a cudaMalloc/cudaFree is not acceptable and no spare
 * workspace buffer was planned.  The split-KV partial results, which
 * vector_decode_attn keeps in the caller's workspace, live here in a fixed
 * array of VECTOR_STATIC_SCRATCH_BYTES inside the library's device image; every
 * GPU on which the library is loaded holds that much memory until the process
 * exits.  The call itself performs no cudaMalloc, cudaFree or other allocating
 * routine.  Inputs and outputs are passed exactly as for vector_decode_attn.
 *
 *  - Limit: shapes whose partial results need more than VECTOR_STATIC_SCRATCH_BYTES
 *    (vector_decode_scratch_bytes(shape) reports the need) are rejected with
 *    VECTOR_ERR_WORKSPACE; use vector_decode_attn with your own workspace then.
 *  - The first call on each device looks up the array's device address (with
 *    that device current).  Make that first call during start-up, before any
 *    stream capture begins.
 *  - All calls on a device share the one array, and it keeps whatever the last
 *    call left there.  Nothing in it has to start at zero: each call overwrites
 *    every partial record before reading it.  Two calls that overlap on the GPU
 *    (different streams, no ordering between them) race on the array and give
 *    undefined results; order them on one stream or with events.
 */
#define VECTOR_STATIC_SCRATCH_BYTES (16u << 20)
VECTOR_API size_t vector_decode_scratch_bytes(const vector_shape* shape);
VECTOR_API vector_status vector_decode_attn_static(const vector_shape* shape, const void* q,
                                                   const vector_cache* cache, const void* W, void* out,
                                                   int32_t out_dtype, int32_t mode, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VECTOR_H_ */
