// Exact top-k selection with the lower index winning ties, emitted in index order: the
// building block of Step 1 (the n_pool largest scores) and Step 3 (the n_apx smallest
// residuals) of the routing (paper Section 3.2).  One thread block per unit.
//
// The k-th key is found on an order-preserving 32-bit image of the fp32 value.  Two paths:
//
// select_lean (the one that normally runs): a histogram of the leading 11 bits over the whole input;
//   one more pass that writes, per 32 elements, a bit mask of the elements whose leading bits beat the
//   k-th key's (chosen) and one of those that share them (candidates: a quarter of a binade of
//   values); each warp lists its own candidates, their next 11 bits are counted, and the few that
//   share those as well are ranked against each other directly; the emission in index order then
//   needs the masks only.  It gives up when a warp's share of the candidate list overflows or many
//   values are equal, and then
// select_emit (the general one) runs: a most-significant-digit radix select with digits of 11, 11 and
//   10 bits whose passes fall back to re-reading the input when the list or the masks do not fit.
//
// The masks, the candidate list, the warps' transposition tiles and (general path, residuals) the
// images kept by pass 1 live in dynamic shared memory sized to the input.
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
struct __align__(16) Scratch {
    int hist[SEL_BINS];
    int hist2[SEL_BINS];          // second digit of the lean path (the first histogram is still being read)
    int bc[6];                    // (bin, rank inside it) of up to three digits
    int part[32];                 // per-warp bin sums of pick_bin
    int n_cand, overflow, n_above, n_small;
    uint32_t small[256];          // offsets of the candidates that share the k-th key's leading bits (lean path)
    OrderedScratch os;
};
// Dynamic shared memory of one selection: cand[cand_cap] | sel_mask[groups] | tie_mask[groups] | stage[stage_words]
// or, for the lean path, ... | tie_mask[groups] | tiles[tile_words].
// With `keyed` the list is read as cand_cap / 2 indices followed by their cand_cap / 2 images (the lean path).
struct Layout {
    int cand_cap;                 // candidates the list holds (words)
    int groups;                   // mask words (one per 32 elements), 0 = masks not kept
    int stage_words;              // images kept by pass 1 (0 or n)
    int keyed;                    // 1: the lean path may run (masks kept, cand_cap a multiple of 8)
    int tile_words;               // the lean path's per-warp transposition tiles, behind the masks
    __host__ __device__ size_t bytes() const {
        return ((size_t)cand_cap + 2 * (size_t)groups + (size_t)stage_words + (size_t)tile_words) * 4;
    }
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


// ---- the lean path ------------------------------------------------------------------------------
// The same selection written for few instructions per element; it needs the masks and a keyed
// candidate list (Layout::keyed) and gives up, before it has emitted anything, when more candidates
// turn up than the list holds -- the caller then runs select_emit.

// The bin search of pick_bin done by the first four warps only (16 bins a lane): a fortieth of the
// instructions, the other warps wait at the barrier.  Results go to bc[0] (bin) and bc[1] (rank inside it).
__device__ __forceinline__ void pick_bin_few(const int* hist, int remaining, int* bc, int* part) {
    constexpr int NWP = 4, BW = SEL_BINS / NWP, BPL = BW / 32;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int r0 = wid * BW + lane * BPL;                    // rank from the top of this lane's first bin
    int tot_l = 0, tot = 0;
    if (wid < NWP) {
        const int4* h4 = reinterpret_cast<const int4*>(hist + (SEL_BINS - r0 - BPL));     // this lane's bins, ascending address
#pragma unroll
        for (int q = 0; q < BPL / 4; ++q) { const int4 x = h4[q]; tot_l += (x.x + x.y) + (x.z + x.w); }
        tot = __reduce_add_sync(FULL, tot_l);
        if (lane == 0) part[wid] = tot;
    }
    __syncthreads();
    if (wid < NWP) {
        int above = 0;
#pragma unroll
        for (int w = 0; w < NWP; ++w) above += w < wid ? part[w] : 0;
        if (above < remaining && above + tot >= remaining) {     // exactly one warp
            const int r = remaining - above;
            const int s = lane_scan_incl(tot_l, lane);
            if (s - tot_l < r && s >= r) {                       // exactly one lane: walks its bins from the top
                int acc = s - tot_l;
                for (int j = 0; j < BPL; ++j) {
                    const int c = hist[SEL_BINS - 1 - (r0 + j)];
                    if (acc < r && acc + c >= r) { bc[0] = SEL_BINS - 1 - (r0 + j); bc[1] = r - acc; }
                    acc += c;
                }
            }
        }
    }
}

template <bool SMALLEST>
__device__ __forceinline__ uint32_t image_of_bits(uint32_t u) {
    const uint32_t k = u ^ (uint32_t)(((int32_t)u >> 31) | (int32_t)0x80000000);
    return SMALLEST ? ~k : k;
}

// Histogram of the leading 11 bits of every element: 16-byte loads, DEPTH of them in flight per thread all the
// time (a slot's next load is issued as soon as its value has been taken).
template <bool SMALLEST, int DEPTH>
__device__ __forceinline__ void hist_pass_lean(const float* __restrict__ vals, int n, int* hist) {
    const int nt = blockDim.x;
    if ((reinterpret_cast<uintptr_t>(vals) & 15) == 0) {
        const uint4* p = reinterpret_cast<const uint4*>(vals);
        const int n4 = n >> 2;
        uint4 nx[DEPTH];
#pragma unroll
        for (int j = 0; j < DEPTH; ++j) if ((int)threadIdx.x + j * nt < n4) nx[j] = __ldg(p + threadIdx.x + j * nt);
        for (int base = threadIdx.x; base < n4; base += DEPTH * nt) {
#pragma unroll
            for (int j = 0; j < DEPTH; ++j) {
                if (base + j * nt < n4) {
                    const uint4 x = nx[j];
                    if (base + (DEPTH + j) * nt < n4) nx[j] = __ldg(p + base + (DEPTH + j) * nt);     // the slot's next load
                    atomicAdd(&hist[image_of_bits<SMALLEST>(x.x) >> 21], 1);
                    atomicAdd(&hist[image_of_bits<SMALLEST>(x.y) >> 21], 1);
                    atomicAdd(&hist[image_of_bits<SMALLEST>(x.z) >> 21], 1);
                    atomicAdd(&hist[image_of_bits<SMALLEST>(x.w) >> 21], 1);
                }
            }
        }
        const int i = (n4 << 2) + threadIdx.x;
        if (i < n) atomicAdd(&hist[image_of_bits<SMALLEST>(__float_as_uint(vals[i])) >> 21], 1);
    } else {
        for (int i = threadIdx.x; i < n; i += nt) atomicAdd(&hist[image_of_bits<SMALLEST>(__float_as_uint(vals[i])) >> 21], 1);
    }
}

// Requires L.keyed, L.groups > 0 and 1 <= k <= n.  Returns false (block-uniform, nothing handed out) when it
// gives up: a warp's share of the candidate list overflowed, or more than SMALL_MAX candidates share the
// leading 11 bits of the k-th key's offset (many equal values).  What is handed out goes through `sink`:
//   CHOSEN_ONLY:  sink.list() is the global array that receives the k chosen indices in ascending order;
//   otherwise:    sink.fetch(i) loads what element i's emission needs (called four groups ahead, so that the
//                 load is under way while the ranks are worked out) and sink.put(i, fetched, chosen, pos)
//                 is called for every element, pos being its rank among the chosen or among the others.
//
// The leading 11 bits of the k-th key come from a histogram over the whole input (16-byte loads, a handful
// of instructions per 32 elements).  ONE more pass then writes, per 32 elements, the mask of those with larger
// leading bits (they are chosen) and the mask of those with the same (the candidates, a quarter binade of
// values): two comparisons and two ballots per 32 elements.  Each warp then lists its own candidates (a lane
// per mask word, then a gather of their values), the next 11 bits of the k-th key come from one histogram of
// the list, and the few candidates that share those too are ranked against each other directly.
constexpr int SMALL_MAX = 256;
// 16-byte loads a lane keeps in flight in the pass: blocks of 32 warps run one to a multiprocessor and have to
// cover the memory latency alone.
__host__ __device__ constexpr int lean_loads_per_lane(int nw) { return nw == 32 ? 4 : 2; }

template <bool SMALLEST, int NW, bool CHOSEN_ONLY, typename Sink>
__device__ __forceinline__ bool select_lean(const float* __restrict__ vals, int n, int k, Scratch& S, const Layout L,
                                            uint32_t* dyn, Sink sink) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    constexpr int NT = 32 * NW;
    const unsigned lt = (1u << lane) - 1u;
    const int cap = L.cand_cap >> 1;
    const int seg = (cap / NW) & ~3;                          // a warp's share of the list
    int32_t* cand = reinterpret_cast<int32_t*>(dyn) + wid * seg;
    uint32_t* ckey = dyn + cap + wid * seg;
    uint32_t* sel_mask = dyn + L.cand_cap;
    uint32_t* tie_mask = sel_mask + L.groups;                 // during the pass: the candidates' mask
    // pieces of whole chunks (CH elements: TPL 16-byte loads per lane), so that a warp's loads, its
    // transposition tile and its mask words (four at a time) line up
    constexpr int TPL = lean_loads_per_lane(NW), CH = TPL * 128;
    uint32_t* tile = tie_mask + L.groups + wid * CH;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(vals) & 15) == 0;
    const int per_w = (((n + NW - 1) / NW) + CH - 1) / CH * CH;
    const int w0 = min(n, wid * per_w), w1 = min(n, w0 + per_w);
    const int gw0 = w0 >> 5, gw1 = w0 < w1 ? (w1 + 31) >> 5 : gw0;     // the piece's mask words (an empty piece owns none)
    int my_c = 0;
    constexpr int sh_a = 10;                                 // the candidates' offsets inside their bin have 21 bits
    for (int b = threadIdx.x; b < SEL_BINS; b += NT) { S.hist[b] = 0; S.hist2[b] = 0; }
    if (threadIdx.x == 0) { S.n_cand = 0; S.n_above = 0; S.overflow = 0; S.n_small = 0; }
    __syncthreads();
    // ---- the leading digit of the k-th key
    hist_pass_lean<SMALLEST, (NW == 32 ? 8 : 4)>(vals, n, S.hist);
    __syncthreads();
    pick_bin_few(S.hist, k, S.bc, S.part);
    __syncthreads();
    const uint32_t bin1 = (uint32_t)S.bc[0];
    {
        // ---- the pass.  A warp takes its piece chunk by chunk: 16-byte loads into registers (the next chunk's
        // are issued before this chunk is worked on), from there through its tile in shared memory, out of
        // which lane l reads element 32 g + l, so that a ballot is the mask word of 32 consecutive elements.
        const uint32_t key0 = bin1 << 21, hi_max = key0 | 0x1fffffu;        // the smallest and largest image with that digit
        uint4 r[TPL];
        auto issue = [&](int base) {
            if (vec_ok && base + CH <= w1) {
#pragma unroll
                for (int q = 0; q < TPL; ++q) r[q] = __ldg(reinterpret_cast<const uint4*>(vals + base + 128 * q + 4 * lane));
            } else {
#pragma unroll
                for (int q = 0; q < TPL; ++q) {
                    const int i = base + 128 * q + 4 * lane;
                    r[q].x = i + 0 < w1 ? __float_as_uint(vals[i + 0]) : 0u;
                    r[q].y = i + 1 < w1 ? __float_as_uint(vals[i + 1]) : 0u;
                    r[q].z = i + 2 < w1 ? __float_as_uint(vals[i + 2]) : 0u;
                    r[q].w = i + 3 < w1 ? __float_as_uint(vals[i + 3]) : 0u;
                }
            }
        };
        if (w0 < w1) issue(w0);
        for (int base = w0; base < w1; base += CH) {
#pragma unroll
            for (int q = 0; q < TPL; ++q) reinterpret_cast<uint4*>(tile)[32 * q + lane] = r[q];
            __syncwarp();
            if (base + CH < w1) issue(base + CH);
            const bool whole = base + CH <= w1;
#pragma unroll
            for (int q = 0; q < TPL; ++q) {
                unsigned gb[4], cb[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t key = image_of_bits<SMALLEST>(tile[128 * q + 32 * j + lane]);
                    gb[j] = __ballot_sync(FULL, key > hi_max);
                    cb[j] = __ballot_sync(FULL, key >= key0) & ~gb[j];
                }
                const int c0 = base + 128 * q;
                if (!whole) {                                        // the piece ends inside this chunk
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int left = w1 - (c0 + 32 * j);
                        const unsigned valid = left >= 32 ? FULL : left > 0 ? (1u << left) - 1u : 0u;
                        gb[j] &= valid;
                        cb[j] &= valid;
                    }
                }
                if (lane == 0 && c0 < w1) {                          // whole groups of four words: the arrays are padded to that
                    *reinterpret_cast<uint4*>(sel_mask + (c0 >> 5)) = make_uint4(gb[0], gb[1], gb[2], gb[3]);
                    *reinterpret_cast<uint4*>(tie_mask + (c0 >> 5)) = make_uint4(cb[0], cb[1], cb[2], cb[3]);
                }
            }
            __syncwarp();                                    // the tile is read before the next chunk lands in it
        }
        // ---- the warp's candidates: a lane per mask word lists their indices in its share of the list (and
        // clears the word, which becomes the ties' mask), then their values are gathered, four loads in flight
        int above = 0;
        my_c = 0;
        for (int gbase = gw0; gbase < gw1; gbase += 32) {
            const int g = gbase + lane;
            uint32_t cm = 0u;
            if (g < gw1) { above += __popc(sel_mask[g]); cm = tie_mask[g]; tie_mask[g] = 0u; }
            const int c = __popc(cm);
            const int inc = lane_scan_incl(c, lane);
            int at = my_c + inc - c;
            while (cm) {
                const int b = __ffs((int)cm) - 1;
                cm &= cm - 1u;
                if (at < seg) cand[at] = (g << 5) + b;
                ++at;
            }
            my_c += __shfl_sync(FULL, inc, 31);
        }
        above = __reduce_add_sync(FULL, above);
        __syncwarp();
        const int listed = min(my_c, seg);
        for (int j0 = lane; j0 < listed; j0 += 128) {
            uint32_t x[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) x[t] = j0 + 32 * t < listed ? __float_as_uint(vals[cand[j0 + 32 * t]]) : 0u;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                if (j0 + 32 * t < listed) {
                    const uint32_t rel = image_of_bits<SMALLEST>(x[t]) - key0;
                    ckey[j0 + 32 * t] = rel;
                    atomicAdd(&S.hist2[rel >> sh_a], 1);
                }
            }
        }
        if (lane == 0) {
            if (above) atomicAdd(&S.n_above, above);
            if (my_c > seg) S.overflow = 1;
        }
    }
    __syncthreads();
    const int n_above = S.n_above;
    if (S.overflow) { __syncthreads(); return false; }       // everyone has read the flag before the caller resets it
    // ---- the k-th key's offset inside its bin: its leading 11 bits from the list's histogram ...
    pick_bin_few(S.hist2, k - n_above, S.bc, S.part);
    __syncthreads();
    const uint32_t prefix = (uint32_t)S.bc[0];
    const int rank = S.bc[1];                                // of the k-th key among the candidates that share them
    if (S.hist2[prefix] > SMALL_MAX) { __syncthreads(); return false; }      // many equal values: the general path's job
    // ... and the rest by ranking those few against each other
    for (int j = lane; j < my_c; j += 32) {
        const uint32_t rel = ckey[j];
        if ((rel >> sh_a) == prefix) S.small[atomicAdd(&S.n_small, 1)] = rel;
    }
    __syncthreads();
    {
        const int ns = S.n_small;
        if (threadIdx.x < ns) {
            const uint32_t v = S.small[threadIdx.x];
            int greater = 0, equal = 0;
            for (int j = 0; j < ns; ++j) { const uint32_t x = S.small[j]; greater += x > v; equal += x == v; }
            if (greater < rank && rank <= greater + equal) { S.bc[4] = (int)v; S.bc[5] = rank - greater; }   // ties write the same
        }
    }
    __syncthreads();
    const uint32_t kth = (uint32_t)S.bc[4];
    const int take_ties = S.bc[5];          // all strictly better elements are chosen; `take_ties` ties complete k
    // ---- the candidates against the k-th key (a warp's candidates lie in its own piece, so do its mask words)
    for (int j = lane; j < my_c; j += 32) {
        const uint32_t rel = ckey[j];
        const int i = cand[j];
        if (rel > kth) atomicOr(&sel_mask[i >> 5], 1u << (i & 31));
        else if (rel == kth) atomicOr(&tie_mask[i >> 5], 1u << (i & 31));
    }
    __syncwarp();
    // ---- per piece: how many better elements, how many ties
    {
        int g2 = 0, t2 = 0;
        for (int g = gw0 + lane; g < gw1; g += 32) { g2 += __popc(sel_mask[g]); t2 += __popc(tie_mask[g]); }
        g2 = __reduce_add_sync(FULL, g2);
        t2 = __reduce_add_sync(FULL, t2);
        if (lane == 0) { S.os.gt[wid] = g2; S.os.tie[wid] = t2; }
    }
    __syncthreads();                                         // also: every read of the list is behind us
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
    // ---- handing out in index order
    int pos = S.os.out[wid], ties_left = S.os.quota[wid];
    if constexpr (CHOSEN_ONLY) {
        // A lane per mask word: ranks by a warp scan of the words' counts, then each lane walks its set bits.
        // The indices go to the list's place in shared memory first when they fit (the lanes' stores are
        // scattered), and from there to the global list in one coalesced sweep.
        int32_t* const out = sink.list();
        int32_t* const stage = reinterpret_cast<int32_t*>(dyn);
        const bool staged = k <= L.cand_cap;
        int32_t* const dst = staged ? stage : out;
        for (int gbase = gw0; gbase < gw1; gbase += 32) {
            const int g = gbase + lane;
            uint32_t sm = g < gw1 ? sel_mask[g] : 0u;
            const uint32_t tm = g < gw1 ? tie_mask[g] : 0u;
            if (ties_left > 0 && __any_sync(FULL, tm != 0u)) {          // warp-uniform
                const int t = __popc(tm);
                const int inc = lane_scan_incl(t, lane);
                int take = max(0, min(t, ties_left - (inc - t)));       // the lowest `take` ties of this word
                uint32_t x = tm;
                while (take-- > 0) { const uint32_t low = x & (0u - x); sm |= low; x ^= low; }
                ties_left -= min(ties_left, __shfl_sync(FULL, inc, 31));
            }
            const int c = __popc(sm);
            const int inc = lane_scan_incl(c, lane);
            int at = pos + inc - c;
            const int ibase = g << 5;
            while (sm) {
                const int b = __ffs((int)sm) - 1;
                sm &= sm - 1u;
                dst[at++] = ibase + b;
            }
            pos += __shfl_sync(FULL, inc, 31);
        }
        if (staged) {
            __syncthreads();
            for (int j = threadIdx.x; j < k; j += NT) out[j] = stage[j];
        }
    } else {
        int nx[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) nx[j] = w0 + 32 * j + lane < w1 ? sink.fetch(w0 + 32 * j + lane) : 0;
        for (int base = w0; base < w1; base += 128) {
            int fetched[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) fetched[j] = nx[j];
#pragma unroll
            for (int j = 0; j < 4; ++j) nx[j] = base + 128 + 32 * j + lane < w1 ? sink.fetch(base + 128 + 32 * j + lane) : 0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                if (base + 32 * j < w1) {                            // warp-uniform
                    const int i = base + 32 * j + lane;
                    const unsigned gbits = sel_mask[(base >> 5) + j], tb = tie_mask[(base >> 5) + j];
                    const int take = min(ties_left, __popc(tb));
                    const bool chosen = ((gbits >> lane) & 1u) || (((tb >> lane) & 1u) && __popc(tb & lt) < take);
                    const unsigned cb = __ballot_sync(FULL, chosen);
                    const int before = pos + __popc(cb & lt);       // chosen elements before this one in the unit
                    if (i < w1) sink.put(i, fetched[j], chosen, chosen ? before : i - before);
                    pos += __popc(cb);
                    ties_left -= take;
                }
            }
        }
    }
    return true;
}

// Shared-memory plan of one selection over n elements within `budget_bytes`: a candidate list of
// at least `min_cand` entries, the masks when they fit, the staged images when asked for and they
// fit, and whatever is left goes to a longer candidate list (up to 16384 entries: a quarter binade
// rarely holds more).
inline Layout plan_layout(int64_t n, bool want_stage, size_t budget_bytes, int min_cand, int nw) {
    Layout L;
    L.groups = 0; L.stage_words = 0; L.keyed = 0; L.tile_words = 0;
    size_t used = (size_t)min_cand * 4;
    const size_t groups = ((size_t)((n + 31) / 32) + 3) & ~size_t(3);       // whole 16-byte groups: what follows stays aligned
    if (used + 2 * groups * 4 <= budget_bytes) { L.groups = (int)groups; used += 2 * groups * 4; }
    if (want_stage && used + (size_t)n * 4 <= budget_bytes) { L.stage_words = (int)n; used += (size_t)n * 4; }
    size_t cap = (budget_bytes - used) / 4 + (size_t)min_cand;
    const size_t want = (size_t)(n < 16384 ? n : 16384);
    if (cap > want) cap = want;
    if (cap < (size_t)min_cand) cap = (size_t)min_cand;
    L.cand_cap = (int)cap;
    L.keyed = 0;
    if (L.groups > 0 && L.stage_words == 0) {
        // the lean path: indices and images side by side, twice the words when they fit
        const size_t tiles = (size_t)nw * lean_loads_per_lane(nw) * 128;
        const size_t fixed = 2 * groups + tiles;
        if (budget_bytes / 4 > fixed) {
            // words: index and image of every candidate, in shares of whole 4-entry groups for up to 32 warps
            size_t keyed = (2 * (size_t)(n < 32768 ? n : 32768) + 255) & ~size_t(255);
            const size_t room = (budget_bytes / 4 - fixed) & ~size_t(255);
            if (keyed > room) keyed = room;
            if (keyed >= 512) { L.cand_cap = (int)keyed; L.keyed = 1; L.tile_words = (int)tiles; }
        }
    }
    return L;
}

}  // namespace sel
}  // namespace vec
#endif
