// Exact top-k selection with the lower index winning ties, emitted in index order: the
// building block of Step 1 (the n_pool largest scores) and Step 3 (the n_apx smallest
// residuals) of the routing (paper Section 3.2).  One thread block per unit.
//
// The k-th key is found by a most-significant-digit radix select on an order-preserving
// 32-bit image of the fp32 value, digits of 11, 11 and 10 bits:
//   pass 1  reads the whole input and counts the leading digit;
//   pass 2  reads it once more, warp by contiguous piece, and on the way (a) notes per group
//           of 32 elements, as a bit mask, those whose leading digit already beats the k-th
//           key's and (b) lists the indices of those that share it (the candidates: a quarter
//           of a binade of values) while counting their second digit;
//   pass 3  and the classification of the candidates against the k-th key run over the list;
//   the per-piece counts and the emission in index order (block-wide prefix sums) then need
//           the masks only, not the values.
// The masks, the candidate list and (for the residuals) the images kept by pass 1 live in
// dynamic shared memory sized to the input, so a context of 131072 tokens keeps its masks.
// Fallbacks that read the input again: more candidates than the list holds (pass 3 and the
// classification walk the input), no room for the masks (inputs beyond a few hundred
// thousand elements).
#ifndef VECTOR_SELECT_CUH_
#define VECTOR_SELECT_CUH_

#include "common.cuh"

namespace vec {
namespace sel {

constexpr int SEL_BINS = 2048;                 // digits of 11, 11 and 10 bits
constexpr unsigned FULL = 0xffffffffu;

// Best = largest image.  For "k smallest" the images are inverted.
template <bool SMALLEST>
__device__ __forceinline__ uint32_t select_image(float v) {
    const uint32_t k = ordered_key(v);
    return SMALLEST ? ~k : k;
}

struct OrderedScratch { int gt[32], tie[32], out[32], quota[32]; };
// Static shared memory of one selection.
struct Scratch {
    int hist[SEL_BINS];
    int bc[2];
    int part[32];                 // per-warp bin sums of pick_bin
    int n_cand, overflow;
    OrderedScratch os;
};
// Dynamic shared memory of one selection: cand[cand_cap] | sel_mask[groups] | tie_mask[groups] | stage[stage_words].
struct Layout {
    int cand_cap;                 // candidates the list holds
    int groups;                   // mask words (one per 32 elements), 0 = masks not kept
    int stage_words;              // images kept by pass 1 (0 or n)
    __host__ __device__ size_t bytes() const { return ((size_t)cand_cap + 2 * (size_t)groups + (size_t)stage_words) * 4; }
};

__device__ __forceinline__ int lane_scan_incl(int v, int lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += t;
    }
    return v;
}

// hist[bin] += 1 if `valid`.  A plain shared-memory atomic per element: equal bins inside a warp (many
// equal values) serialise in the atomic unit, which costs less than sorting them out with ballots first.
__device__ __forceinline__ void hist_add(int* hist, int bin, bool valid) {
    if (valid) atomicAdd(&hist[bin], 1);
}

// The bin of hist[0..SEL_BINS), counted from the top, in which the cumulative count reaches
// `remaining` (-> bc[0]) and the rank wanted inside that bin, 1-based (-> bc[1]).  Every thread of
// the block calls it (one block barrier inside; the caller synchronises before and after): warp w
// sums the SEL_BINS / NW bins of its range, every warp scans the NW sums, and the one warp whose
// range holds the answer finds the lane, the lane its bin.
template <int NW>
__device__ __forceinline__ void pick_bin(const int* hist, int remaining, int* bc, int* part) {
    constexpr int BW = SEL_BINS / NW, BPL = BW / 32;
    static_assert(BPL >= 1 && BPL * 32 * NW == SEL_BINS, "bins must divide among the lanes");
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int r0 = wid * BW + lane * BPL;                   // rank from the top of this lane's first bin
    int c[BPL], tot_l = 0;
#pragma unroll
    for (int j = 0; j < BPL; ++j) { c[j] = hist[SEL_BINS - 1 - (r0 + j)]; tot_l += c[j]; }
    const int tot = __reduce_add_sync(FULL, tot_l);
    if (lane == 0) part[wid] = tot;
    __syncthreads();
    const int p = lane < NW ? part[lane] : 0;
    const int above = __shfl_sync(FULL, lane_scan_incl(p, lane) - p, wid);      // count in the warps above this one
    if (above < remaining && above + tot >= remaining) {     // exactly one warp
        const int r = remaining - above;
        const int s = lane_scan_incl(tot_l, lane);
        if (s - tot_l < r && s >= r) {                       // exactly one lane
            int acc = s - tot_l;
#pragma unroll
            for (int j = 0; j < BPL; ++j) {
                if (acc < r && acc + c[j] >= r) { bc[0] = SEL_BINS - 1 - (r0 + j); bc[1] = r - acc; }
                acc += c[j];
            }
        }
    }
}

// One histogram pass over all of vals on the digit at `shift`, among the elements whose image
// matches prefix under mask.  Eight independent loads in flight per thread: the pass is bound by
// memory latency otherwise.
template <bool SMALLEST>
__device__ __forceinline__ void hist_pass_all(const float* __restrict__ vals, int n, int shift, uint32_t digit_mask,
                                              uint32_t prefix, uint32_t mask, int* hist, uint32_t* stage_out) {
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
            if (stage_out && i < n) stage_out[i] = key;          // keep the image for the later passes
            hist_add(hist, (key >> shift) & digit_mask, i < n && (key & mask) == prefix);
        }
    }
}

// Piece of the input that warp `wid` owns in the ordered passes: [w0, w1), a multiple of 32 long.
__device__ __forceinline__ int ordered_chunk(int n, int nw) { return (((n + nw - 1) / nw) + 31) & ~31; }

// Exact top-k of vals[0..n) (largest images; for "k smallest" the images are inverted) with the
// lower index winning ties, emitted in index order: emit(i, chosen, pos) is called for every element
// i, pos being its rank among the chosen ones if chosen, else among the others.  1 <= k <= n
// unless !any (nothing is chosen then).  With CHOSEN_ONLY the caller has no use for the elements that
// are not chosen, and groups of 32 without a chosen one are passed over.  All threads of the block
// (32 NW of them) call it; dyn is the block's dynamic shared memory laid out as L describes.
template <bool SMALLEST, int NW, bool CHOSEN_ONLY, typename Emit>
__device__ __forceinline__ void select_emit(const float* __restrict__ vals, int n, int k, bool any, Scratch& S, const Layout L,
                                            uint32_t* dyn, Emit emit) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const unsigned lt = (1u << lane) - 1u;
    int32_t* cand = reinterpret_cast<int32_t*>(dyn);
    uint32_t* sel_mask = dyn + L.cand_cap;
    uint32_t* tie_mask = sel_mask + L.groups;
    uint32_t* stage = L.stage_words ? tie_mask + L.groups : nullptr;
    const bool masked = L.groups > 0;
    const int per_w = ordered_chunk(n, NW);
    const int w0 = min(n, wid * per_w), w1 = min(n, w0 + per_w);
    uint32_t kth = 0xffffffffu;
    int take_ties = 0;
    if (threadIdx.x < 32) { S.os.gt[threadIdx.x] = 0; S.os.tie[threadIdx.x] = 0; }
    if (masked)
        for (int g = threadIdx.x; g < L.groups; g += blockDim.x) { sel_mask[g] = 0u; tie_mask[g] = 0u; }
    if (any) {
        // ---- pass 1: leading 11 bits
        for (int b = threadIdx.x; b < SEL_BINS; b += blockDim.x) S.hist[b] = 0;
        if (threadIdx.x == 0) { S.n_cand = 0; S.overflow = 0; }
        __syncthreads();
        hist_pass_all<SMALLEST>(vals, n, 21, 2047u, 0u, 0u, S.hist, stage);
        __syncthreads();
        pick_bin<NW>(S.hist, k, S.bc, S.part);
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
                    const unsigned gb = __ballot_sync(FULL, in && d1 > bin1);
                    if (lane == 0 && base + 32 * j < w1) sel_mask[(base >> 5) + j] = gb;
                }
                if (in && d1 == bin1) {
                    atomicAdd(&S.hist[(key >> 10) & 2047], 1);
                    const int at = atomicAdd(&S.n_cand, 1);
                    if (at < L.cand_cap) cand[at] = i;
                    else S.overflow = 1;
                }
            }
        }
        __syncthreads();
        pick_bin<NW>(S.hist, remaining, S.bc, S.part);
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
                const uint32_t key = stage ? stage[cand[j]] : select_image<SMALLEST>(vals[cand[j]]);
                hist_add(S.hist, key & 1023, (key & mask) == prefix);
            }
        } else {
            hist_pass_all<SMALLEST>(vals, n, 0, 1023u, prefix, mask, S.hist, nullptr);
        }
        __syncthreads();
        pick_bin<NW>(S.hist, remaining, S.bc, S.part);
        __syncthreads();
        prefix |= (uint32_t)S.bc[0];
        remaining = S.bc[1];
        __syncthreads();
        kth = prefix;
        take_ties = remaining;          // all strictly better elements precede; `remaining` ties complete k
        // ---- the candidates against the k-th key
        if (masked && listed) {
            for (int j = threadIdx.x; j < n_cand; j += blockDim.x) {
                const int i = cand[j];
                const uint32_t key = stage ? stage[i] : select_image<SMALLEST>(vals[i]);
                if (key > kth) atomicOr(&sel_mask[i >> 5], 1u << (i & 31));
                else if (key == kth) atomicOr(&tie_mask[i >> 5], 1u << (i & 31));
            }
        } else if (masked) {
            for (int base = w0; base < w1; base += 128) {
                uint32_t kv[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int i = base + 32 * j + lane;
                    kv[j] = i >= w1 ? 0u : stage ? stage[i] : select_image<SMALLEST>(vals[i]);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool in = base + 32 * j + lane < w1;
                    const unsigned gb = __ballot_sync(FULL, in && kv[j] > kth);
                    const unsigned tb = __ballot_sync(FULL, in && kv[j] == kth);
                    if (lane == 0 && base + 32 * j < w1) { sel_mask[(base >> 5) + j] = gb; tie_mask[(base >> 5) + j] = tb; }
                }
            }
        }
    }
    __syncthreads();
    // ---- per piece: how many better elements, how many ties
    if (masked) {
        int g2 = 0, t2 = 0;
        for (int g = (w0 >> 5) + lane; g < ((w1 + 31) >> 5); g += 32) { g2 += __popc(sel_mask[g]); t2 += __popc(tie_mask[g]); }
        g2 = __reduce_add_sync(FULL, g2);
        t2 = __reduce_add_sync(FULL, t2);
        if (lane == 0) { S.os.gt[wid] = g2; S.os.tie[wid] = t2; }
    } else if (any) {
        int g2 = 0, t2 = 0;
        for (int base = w0; base < w1; base += 128) {
            uint32_t kv[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int i = base + 32 * j + lane;
                kv[j] = i >= w1 ? 0u : stage ? stage[i] : select_image<SMALLEST>(vals[i]);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = base + 32 * j + lane < w1;
                g2 += __popc(__ballot_sync(FULL, in && kv[j] > kth));
                t2 += __popc(__ballot_sync(FULL, in && kv[j] == kth));
            }
        }
        if (lane == 0) { S.os.gt[wid] = g2; S.os.tie[wid] = t2; }
    }
    __syncthreads();
    // ---- offsets of the pieces; ties go to the lowest indices
    if (wid == 0) {
        const int t = lane < NW ? S.os.tie[lane] : 0;
        const int inc = lane_scan_incl(t, lane);
        const int quota = max(0, min(t, take_ties - (inc - t)));
        const int c = (lane < NW ? S.os.gt[lane] : 0) + quota;
        const int ci = lane_scan_incl(c, lane);
        S.os.out[lane] = ci - c;
        S.os.quota[lane] = quota;
    }
    __syncthreads();
    // ---- emission in index order
    int pos = S.os.out[wid], ties_left = S.os.quota[wid];
    if (masked) {
        for (int base = w0; base < w1; base += 32) {
            const int i = base + lane;
            const unsigned gb = sel_mask[base >> 5], tb = tie_mask[base >> 5];
            if (CHOSEN_ONLY && gb == 0u && (tb == 0u || ties_left == 0)) continue;
            const int take = min(ties_left, __popc(tb));
            const bool chosen = ((gb >> lane) & 1u) || (((tb >> lane) & 1u) && __popc(tb & lt) < take);
            const unsigned cb = __ballot_sync(FULL, chosen);
            const int before = pos + __popc(cb & lt);               // chosen elements before this one in the unit
            if (i < w1) emit(i, chosen, chosen ? before : i - before);
            pos += __popc(cb);
            ties_left -= take;
        }
    } else {
        for (int base = w0; base < w1; base += 32) {
            const int i = base + lane;
            const bool in = i < w1;
            const uint32_t key = in ? (stage ? stage[i] : select_image<SMALLEST>(vals[i])) : 0u;
            const bool tie = any && in && key == kth;
            const unsigned tb = __ballot_sync(FULL, tie);
            const bool chosen = any && in && (key > kth || (tie && __popc(tb & lt) < ties_left));
            const unsigned cb = __ballot_sync(FULL, chosen);
            const int before = pos + __popc(cb & lt);
            if (in) emit(i, chosen, chosen ? before : i - before);
            pos += __popc(cb);
            ties_left -= min(ties_left, __popc(tb));
        }
    }
}

// Shared-memory plan of one selection over n elements within `budget_bytes`: a candidate list of
// at least `min_cand` entries, the masks when they fit, the staged images when asked for and they
// fit, and whatever is left goes to a longer candidate list (up to 16384 entries: a quarter binade
// rarely holds more).
inline Layout plan_layout(int64_t n, bool want_stage, size_t budget_bytes, int min_cand) {
    Layout L;
    L.groups = 0; L.stage_words = 0;
    size_t used = (size_t)min_cand * 4;
    const size_t groups = (size_t)((n + 31) / 32);
    if (used + 2 * groups * 4 <= budget_bytes) { L.groups = (int)groups; used += 2 * groups * 4; }
    if (want_stage && used + (size_t)n * 4 <= budget_bytes) { L.stage_words = (int)n; used += (size_t)n * 4; }
    size_t cap = (budget_bytes - used) / 4 + (size_t)min_cand;
    const size_t want = (size_t)(n < 16384 ? n : 16384);
    if (cap > want) cap = want;
    if (cap < (size_t)min_cand) cap = (size_t)min_cand;
    L.cand_cap = (int)cap;
    return L;
}

}  // namespace sel
}  // namespace vec
#endif
