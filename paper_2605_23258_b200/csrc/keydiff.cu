// Query-agnostic base scorer by key geometry (a KeyDiff-style scorer; the paper names it among the
// base scorers of Step 1 as "key geometric diversity" and gives no formula):
//   anchor a = sum_j k_j / ||k_j||,   score_i = - <k_i, a> / (||k_i|| ||a||).
// Two passes over K, both bound by HBM: pass 1 forms per-chunk partial anchors and keeps 1 / ||k_i||,
// pass 2 reduces the partials in a fixed order (so the result does not depend on scheduling) and
// takes the cosines.
#include "common.cuh"
#include "internal.h"

namespace vec {

// Eight lanes share a key row, so a warp reduces four rows with three shuffles.  A row is cut into
// 16-byte pieces; lane segment s (0..7) takes pieces s, s + 8, ...: each load instruction of the warp
// covers whole 128-byte lines.
template <typename T> struct Piece;
template <> struct Piece<__nv_bfloat16> {
    static constexpr int EPP = 8;
    static __device__ __forceinline__ uint4 load_raw(const __nv_bfloat16* p) { return *reinterpret_cast<const uint4*>(p); }
    static __device__ __forceinline__ void expand(const uint4 v, float (&o)[8]) {
        o[0] = __uint_as_float(v.x << 16); o[1] = __uint_as_float(v.x & 0xffff0000u);
        o[2] = __uint_as_float(v.y << 16); o[3] = __uint_as_float(v.y & 0xffff0000u);
        o[4] = __uint_as_float(v.z << 16); o[5] = __uint_as_float(v.z & 0xffff0000u);
        o[6] = __uint_as_float(v.w << 16); o[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};
template <> struct Piece<float> {
    static constexpr int EPP = 4;
    static __device__ __forceinline__ uint4 load_raw(const float* p) { return *reinterpret_cast<const uint4*>(p); }
    static __device__ __forceinline__ void expand(const uint4 r, float (&o)[4]) {
        const float4 v = make_float4(__uint_as_float(r.x), __uint_as_float(r.y), __uint_as_float(r.z), __uint_as_float(r.w));
        o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
    }
};
__device__ __forceinline__ float sum8(float v) {        // over the eight lanes of a row
    v += __shfl_xor_sync(0xffffffffu, v, 1);
    v += __shfl_xor_sync(0xffffffffu, v, 2);
    v += __shfl_xor_sync(0xffffffffu, v, 4);
    return v;
}

constexpr int KD_WARPS = 8;
constexpr int KD_ROWS = 4;        // rows per warp and load
constexpr int KD_BATCH = 8;       // row groups a warp has in flight (kept as raw 16-byte pieces until used)

// grid (chunks, U), 256 threads.  partial[(u * chunks + chunk) * D + c], rinv[u * N + i].
template <typename T, int D>
__global__ void __launch_bounds__(32 * KD_WARPS)
keydiff_anchor_partial(const T* __restrict__ K, int64_t N, int64_t chunk_len, float* __restrict__ partial,
                       float* __restrict__ rinv) {
    constexpr int EPP = Piece<T>::EPP, PPL = D / EPP / 8;      // elements per piece, pieces per lane
    __shared__ float red[KD_WARPS * KD_ROWS][D];
    const int u = blockIdx.y, chunk = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int seg = lane & 7, rsub = lane >> 3;
    const T* Ku = K + (size_t)u * N * D;
    const int64_t r0 = (int64_t)chunk * chunk_len, r1 = min(N, r0 + chunk_len);
    float acc[PPL][EPP];
#pragma unroll
    for (int p = 0; p < PPL; ++p)
#pragma unroll
        for (int e = 0; e < EPP; ++e) acc[p][e] = 0.f;
    for (int64_t base = r0 + wid * KD_ROWS * KD_BATCH; base < r1; base += KD_WARPS * KD_ROWS * KD_BATCH) {
        uint4 raw[KD_BATCH][PPL];
#pragma unroll
        for (int b = 0; b < KD_BATCH; ++b) {
            const int64_t row = base + b * KD_ROWS + rsub;
#pragma unroll
            for (int p = 0; p < PPL; ++p)
                raw[b][p] = row < r1 ? Piece<T>::load_raw(Ku + (size_t)row * D + (p * 8 + seg) * EPP) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int b = 0; b < KD_BATCH; ++b) {
            const int64_t row = base + b * KD_ROWS + rsub;
            float x[PPL][EPP];
#pragma unroll
            for (int p = 0; p < PPL; ++p) Piece<T>::expand(raw[b][p], x[p]);
            float s = 0.f;
#pragma unroll
            for (int p = 0; p < PPL; ++p)
#pragma unroll
                for (int e = 0; e < EPP; ++e) s = fmaf(x[p][e], x[p][e], s);
            s = sum8(s);
            const float ri = s > 0.f ? 1.0f / sqrtf(s) : 0.f;        // a zero key adds nothing
#pragma unroll
            for (int p = 0; p < PPL; ++p)
#pragma unroll
                for (int e = 0; e < EPP; ++e) acc[p][e] = fmaf(x[p][e], ri, acc[p][e]);
            if (seg == 0 && row < r1) rinv[(size_t)u * N + row] = ri;
        }
    }
#pragma unroll
    for (int p = 0; p < PPL; ++p)
#pragma unroll
        for (int e = 0; e < EPP; ++e) red[wid * KD_ROWS + rsub][(p * 8 + seg) * EPP + e] = acc[p][e];
    __syncthreads();
    for (int c = threadIdx.x; c < D; c += 32 * KD_WARPS) {
        float s = 0.f;
#pragma unroll
        for (int wv = 0; wv < KD_WARPS * KD_ROWS; ++wv) s += red[wv][c];
        partial[((size_t)u * gridDim.x + chunk) * D + c] = s;
    }
}

// grid (chunks, U), 256 threads.
template <typename T, int D>
__global__ void __launch_bounds__(32 * KD_WARPS)
keydiff_cosine(const T* __restrict__ K, int64_t N, int64_t chunk_len, const float* __restrict__ partial,
               const float* __restrict__ rinv, float* __restrict__ scores) {
    constexpr int EPP = Piece<T>::EPP, PPL = D / EPP / 8;
    __shared__ float a_s[D];
    __shared__ float wsum[KD_WARPS];
    const int u = blockIdx.y, chunk = blockIdx.x, lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int seg = lane & 7, rsub = lane >> 3;
    const int n_chunks = gridDim.x;
    float sq = 0.f;
    for (int c = threadIdx.x; c < D; c += 32 * KD_WARPS) {
        float s = 0.f;
        for (int j = 0; j < n_chunks; ++j) s += partial[((size_t)u * n_chunks + j) * D + c];
        a_s[c] = s;
        sq += s * s;
    }
    sq = warp_sum(sq);
    if (lane == 0) wsum[wid] = sq;
    __syncthreads();
    float an2 = 0.f;
#pragma unroll
    for (int wv = 0; wv < KD_WARPS; ++wv) an2 += wsum[wv];
    const float inv_an = an2 > 0.f ? 1.0f / sqrtf(an2) : 0.f;              // zero anchor: every score is 0
    float a[PPL][EPP];
#pragma unroll
    for (int p = 0; p < PPL; ++p)
#pragma unroll
        for (int e = 0; e < EPP; ++e) a[p][e] = a_s[(p * 8 + seg) * EPP + e];
    const T* Ku = K + (size_t)u * N * D;
    const int64_t r0 = (int64_t)chunk * chunk_len, r1 = min(N, r0 + chunk_len);
    for (int64_t base = r0 + wid * KD_ROWS * KD_BATCH; base < r1; base += KD_WARPS * KD_ROWS * KD_BATCH) {
        uint4 raw[KD_BATCH][PPL];
        float ri[KD_BATCH];
#pragma unroll
        for (int b = 0; b < KD_BATCH; ++b) {
            const int64_t row = base + b * KD_ROWS + rsub;
#pragma unroll
            for (int p = 0; p < PPL; ++p)
                raw[b][p] = row < r1 ? Piece<T>::load_raw(Ku + (size_t)row * D + (p * 8 + seg) * EPP) : make_uint4(0, 0, 0, 0);
            ri[b] = (seg == 0 && row < r1) ? rinv[(size_t)u * N + row] : 0.f;
        }
#pragma unroll
        for (int b = 0; b < KD_BATCH; ++b) {
            const int64_t row = base + b * KD_ROWS + rsub;
            float x[PPL][EPP];
#pragma unroll
            for (int p = 0; p < PPL; ++p) Piece<T>::expand(raw[b][p], x[p]);
            float s = 0.f;
#pragma unroll
            for (int p = 0; p < PPL; ++p)
#pragma unroll
                for (int e = 0; e < EPP; ++e) s = fmaf(x[p][e], a[p][e], s);
            s = sum8(s);
            if (seg == 0 && row < r1) scores[(size_t)u * N + row] = -s * ri[b] * inv_an;
        }
    }
}

static int keydiff_chunks(int U, int64_t N) {
    int64_t want = (8 * sm_count() + U - 1) / U;
    const int64_t max_by_rows = (N + 255) / 256;
    if (want > max_by_rows) want = max_by_rows;
    if (want > 64) want = 64;
    if (want < 1) want = 1;
    return (int)want;
}

size_t keydiff_ws_bytes(const Dims& D, int64_t N) {
    return align256((size_t)D.U * keydiff_chunks(D.U, N) * D.d * sizeof(float)) + align256((size_t)D.U * (size_t)N * sizeof(float));
}

template <typename T, int D>
static vector_status launch_keydiff(const Dims& dm, const void* K, int64_t N, float* scores, char* ws, cudaStream_t st) {
    const int chunks = keydiff_chunks(dm.U, N);
    int64_t chunk_len = (N + chunks - 1) / chunks;
    chunk_len = (chunk_len + 127) / 128 * 128;
    float* partial = (float*)ws;
    float* rinv = (float*)(ws + align256((size_t)dm.U * chunks * dm.d * sizeof(float)));
    dim3 grid(chunks, dm.U);
    keydiff_anchor_partial<T, D><<<grid, 32 * KD_WARPS, 0, st>>>((const T*)K, N, chunk_len, partial, rinv);
    VEC_LAUNCH_CHECK();
    keydiff_cosine<T, D><<<grid, 32 * KD_WARPS, 0, st>>>((const T*)K, N, chunk_len, partial, rinv, scores);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

}  // namespace vec

extern "C" vector_status vector_score_keydiff(const vector_shape* shape, const void* K, int64_t N, float* scores,
                                              void* ws, size_t ws_bytes, void* stream) {
    using namespace vec;
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if (!K || !scores) return VECTOR_ERR_NULL;
    if (N <= 0 || N > (int64_t(1) << 30)) return VECTOR_ERR_SHAPE;
    if (!ws || ((uintptr_t)ws & 255) || ws_bytes < keydiff_ws_bytes(dm, N)) return VECTOR_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* p = (char*)ws;
    if (dm.dtype == VECTOR_F32)
        return dm.d == 64 ? launch_keydiff<float, 64>(dm, K, N, scores, p, st) : launch_keydiff<float, 128>(dm, K, N, scores, p, st);
    return dm.d == 64 ? launch_keydiff<__nv_bfloat16, 64>(dm, K, N, scores, p, st)
                      : launch_keydiff<__nv_bfloat16, 128>(dm, K, N, scores, p, st);
}
