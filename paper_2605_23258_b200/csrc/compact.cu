// Compaction into the mixed cache (paper Section 3.2, Step 3): retained tokens
// keep key and value, approximated tokens keep the key only.  Pure data
// movement: every thread moves one 16-byte piece of one row.
#include "common.cuh"
#include "internal.h"

namespace vec {

// Logical row r of a unit: [0, n_ret) K -> ret_k ; [n_ret, 2 n_ret) V -> ret_v ;
// [2 n_ret, 2 n_ret + n_apx) K -> apx_k.   grid-stride over U * rows * pieces.
__global__ void __launch_bounds__(256)
compact_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V, int64_t N, int pieces,
               const int32_t* __restrict__ ret_idx, const int32_t* __restrict__ apx_idx, int n_ret, int n_apx,
               uint4* __restrict__ ret_k, uint4* __restrict__ ret_v, uint4* __restrict__ apx_k,
               int32_t* __restrict__ ret_pos, int32_t* __restrict__ apx_pos, int64_t cap_ret, int64_t cap_apx,
               int64_t total) {
    const int rows = 2 * n_ret + n_apx;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total;
         t += (int64_t)gridDim.x * blockDim.x) {
        int piece = (int)(t % pieces);
        int64_t rr = t / pieces;
        int r = (int)(rr % rows);
        int64_t u = rr / rows;
        if (r < n_ret) {
            int32_t tok = ret_idx[u * n_ret + r];
            ret_k[(u * cap_ret + r) * pieces + piece] = K[(u * N + tok) * pieces + piece];
            if (piece == 0) ret_pos[u * cap_ret + r] = tok;
        } else if (r < 2 * n_ret) {
            int q = r - n_ret;
            int32_t tok = ret_idx[u * n_ret + q];
            ret_v[(u * cap_ret + q) * pieces + piece] = V[(u * N + tok) * pieces + piece];
        } else {
            int q = r - 2 * n_ret;
            int32_t tok = apx_idx[u * n_apx + q];
            apx_k[(u * cap_apx + q) * pieces + piece] = K[(u * N + tok) * pieces + piece];
            if (piece == 0) apx_pos[u * cap_apx + q] = tok;
        }
    }
}

}  // namespace vec

using namespace vec;

extern "C" vector_status vector_compact(const vector_shape* shape, const vector_budget* budget, const void* K,
                                        const void* V, const int32_t* ret_idx, const int32_t* apx_idx,
                                        const vector_cache* cache, void* stream) {
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
    const int64_t total = (int64_t)dm.U * rows * pieces;
    if (total == 0) return VECTOR_OK;
    int64_t blocks = (total + 255) / 256;
    if (blocks > 148 * 32) blocks = 148 * 32;
    compact_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
        (const uint4*)K, (const uint4*)V, budget->n_tokens, pieces, ret_idx, apx_idx, (int)budget->n_ret,
        (int)budget->n_apx, (uint4*)cache->ret_k, (uint4*)cache->ret_v, (uint4*)cache->apx_k, cache->ret_pos,
        cache->apx_pos, cache->cap_ret, cache->cap_apx, total);
    VEC_LAUNCH_CHECK();
    return VECTOR_OK;
}
