// Compaction into the mixed cache (paper Section 3.2, Step 3): retained tokens
// keep key and value, approximated tokens keep the key only.  Pure data
// movement: a thread moves one 16-byte piece of each of four rows, the four
// loads in flight together.
#include "common.cuh"
#include "internal.h"

namespace vec {

constexpr int COMPACT_THREADS = 64;      // small blocks: many independent gathers in flight per SM, even tail
constexpr int COMPACT_PASSES = 4;

// Logical row r of a unit: [0, n_ret) K -> ret_k ; [n_ret, 2 n_ret) V -> ret_v ;
// [2 n_ret, 2 n_ret + n_apx) K -> apx_k.  A row is `pieces` = 2^lp pieces of 16 bytes; a block owns
// COMPACT_PASSES * (COMPACT_THREADS >> lp) consecutive rows of one unit.  grid: U * chunks blocks.
// idx_div = 1: one pair of index lists per unit; idx_div = Hkv: one pair per (sequence, layer), shared
// by the layer's KV heads (routing with one map per layer).
__global__ void __launch_bounds__(COMPACT_THREADS)
compact_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, int64_t N, int lp,
               const int32_t* __restrict__ ret_idx, const int32_t* __restrict__ apx_idx, int n_ret, int n_apx,
               uint4* __restrict__ ret_k, uint4* __restrict__ ret_v, uint4* __restrict__ apx_k,
               int32_t* __restrict__ ret_pos, int32_t* __restrict__ apx_pos, int64_t cap_ret, int64_t cap_apx,
               int chunks, int idx_div) {
    const int rows = 2 * n_ret + n_apx, pieces = 1 << lp;
    const int u = blockIdx.x / chunks, chunk = blockIdx.x - u * chunks;
    const int ui = u / idx_div;                      // owner of the index lists: the unit, or its (sequence, layer)
    const int piece = threadIdx.x & (pieces - 1), rsub = threadIdx.x >> lp, per_pass = COMPACT_THREADS >> lp;
    const uint4* src[COMPACT_PASSES];
    uint4* dst[COMPACT_PASSES];
    int32_t* pos[COMPACT_PASSES];
    int32_t tok[COMPACT_PASSES];
#pragma unroll
    for (int p = 0; p < COMPACT_PASSES; ++p) {
        const int r = (chunk * COMPACT_PASSES + p) * per_pass + rsub;
        src[p] = nullptr; dst[p] = nullptr; pos[p] = nullptr; tok[p] = 0;
        if (r >= rows) continue;
        if (r < n_ret) {
            tok[p] = ret_idx[(size_t)ui * n_ret + r];
            src[p] = K; dst[p] = ret_k + (((size_t)u * cap_ret + r) << lp) + piece;
            pos[p] = ret_pos + (size_t)u * cap_ret + r;
        } else if (r < 2 * n_ret) {
            const int q = r - n_ret;
            tok[p] = ret_idx[(size_t)ui * n_ret + q];
            src[p] = V; dst[p] = ret_v + (((size_t)u * cap_ret + q) << lp) + piece;
        } else {
            const int q = r - 2 * n_ret;
            tok[p] = apx_idx[(size_t)ui * n_apx + q];
            src[p] = K; dst[p] = apx_k + (((size_t)u * cap_apx + q) << lp) + piece;
            pos[p] = apx_pos + (size_t)u * cap_apx + q;
        }
        if ((unsigned long long)(long long)tok[p] >= (unsigned long long)N) src[p] = nullptr;   // an index outside the unit: row skipped
    }
    uint4 v[COMPACT_PASSES];
#pragma unroll
    for (int p = 0; p < COMPACT_PASSES; ++p)
        if (src[p]) v[p] = src[p][(((size_t)u * N + tok[p]) << lp) + piece];
#pragma unroll
    for (int p = 0; p < COMPACT_PASSES; ++p) {
        if (!src[p]) continue;
        *dst[p] = v[p];
        if (piece == 0 && pos[p]) *pos[p] = tok[p];
    }
}

}  // namespace vec

using namespace vec;

static vector_status compact_launch(const vector_shape* shape, const vector_budget* budget, const void* K,
                                    const void* V, const int32_t* ret_idx, const int32_t* apx_idx,
                                    const vector_cache* cache, void* stream, bool per_layer) {
    Dims dm;
    vector_status rc = check_shape(shape, &dm);
    if (rc != VECTOR_OK) return rc;
    if ((rc = check_budget(budget, dm.w)) != VECTOR_OK) return rc;
    if (!K || !V || !cache) return VECTOR_ERR_NULL;
    if (cache->n_ret != budget->n_ret || cache->n_apx != budget->n_apx || cache->cap_ret < cache->n_ret ||
        cache->cap_apx < cache->n_apx)
        return VECTOR_ERR_SHAPE;
    if (budget->n_ret > 0 && (!ret_idx || !cache->ret_k || !cache->ret_v || !cache->ret_pos)) return VECTOR_ERR_NULL;
    if (budget->n_apx > 0 && (!apx_idx || !cache->apx_k || !cache->apx_pos)) return VECTOR_ERR_NULL;
    const int pieces = dm.d * dm.esize / 16;
    const int64_t rows = 2 * budget->n_ret + budget->n_apx;
    if (rows == 0) return VECTOR_OK;
    int lp = 0;
    while ((1 << lp) < pieces) ++lp;                  // pieces is 8, 16 or 32 for the supported shapes
    const int rows_per_block = COMPACT_PASSES * (COMPACT_THREADS >> lp);
    const int64_t chunks = (rows + rows_per_block - 1) / rows_per_block;
    const int64_t blocks = (int64_t)dm.U * chunks;
    if (blocks > 0x7fffffffLL) return VECTOR_ERR_SHAPE;
    compact_kernel<<<(unsigned)blocks, COMPACT_THREADS, 0, (cudaStream_t)stream>>>(
        (const uint4*)K, (const uint4*)V, budget->n_tokens, lp, ret_idx, apx_idx, (int)budget->n_ret,
        (int)budget->n_apx, (uint4*)cache->ret_k, (uint4*)cache->ret_v, (uint4*)cache->apx_k, cache->ret_pos,
        cache->apx_pos, cache->cap_ret, cache->cap_apx, (int)chunks, per_layer ? shape->n_kv_heads : 1);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}

extern "C" vector_status vector_compact(const vector_shape* shape, const vector_budget* budget, const void* K,
                                        const void* V, const int32_t* ret_idx, const int32_t* apx_idx,
                                        const vector_cache* cache, void* stream) {
    return compact_launch(shape, budget, K, V, ret_idx, apx_idx, cache, stream, false);
}

extern "C" vector_status vector_compact_layer(const vector_shape* shape, const vector_budget* budget, const void* K,
                                              const void* V, const int32_t* ret_idx, const int32_t* apx_idx,
                                              const vector_cache* cache, void* stream) {
    return compact_launch(shape, budget, K, V, ret_idx, apx_idx, cache, stream, true);
}
