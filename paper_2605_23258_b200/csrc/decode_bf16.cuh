// Decode attention over the mixed cache for bf16, head_dim 128 (HBM-bound).
//
// Every K/V row is read once.  Each unit's rows are cut into 32 KB tiles -- a
// retained tile = 64 keys + their 64 values, a key-only tile = 128 keys -- and
// the global tile sequence is dealt out in equal contiguous ranges to one
// persistent block per SM: the load is balanced by bytes and there is no wave tail.
//
// Inside a block one producer thread streams the tiles with TMA
// (cp.async.bulk.tensor, 128-byte swizzle, zero fill past the end of a pool)
// into six 32 KB slots guarded by full/empty mbarriers.  Tiles go round-robin
// to three consumer warps, each with two slots of its own (tile i: warp i % 3,
// slot i % 6), so a warp sees every phase of the barriers it waits on -- with a
// parity wait, a waiter that skipped a phase could take an old completion for
// the one it wants, since TMA copies land out of order.  A warp works through a
// whole tile on its own, 64 keys at a time, and never synchronises with the others:
//   S = Q K^T      64 m16n8k16 bf16 MMAs (eight independent accumulators), the g
//                  query heads padded to the MMA rows
//   online softmax in fp32 registers, one rescale per 64 keys (exp2, scale folded in)
//   O += P V  (retained tile)  or  A += P K  (key-only tile: the p-weighted key
//             sum that the merge step multiplies by W); P enters as bf16 hi in
//             MMA rows 0-7 and bf16 lo in rows 8-15, one MMA for both parts
// RoPE decoupling (ROPE): the value of a key-only token is W applied to the key turned back by its
// original position.  The logits use the stored keys; before the P K product the warp rotates its 64
// keys in shared memory, channel c with c + 64 by the angle -pos * theta^(-2c/128).  The angle is
// taken exactly modulo one turn in 64-bit fixed point (pos * phase[c] wraps by itself), its sine and
// cosine by the fast units.
// A warp keeps one running state (m, l, O or A) per unit and writes it as its
// partial record when it leaves the unit; a warp that met no tile of a unit the
// block touches writes an empty record.  The merge kernel combines a unit's
// records, applies W and normalises.
#ifndef VECTOR_DECODE_BF16_CUH_
#define VECTOR_DECODE_BF16_CUH_

#include "common.cuh"
#include "internal.h"
#include "tcgen05.cuh"
#include "tma.cuh"

namespace vec {
namespace dbf {

constexpr int KEYS = 64;                     // keys per softmax step (and per TMA box)
constexpr int SLOTS = 6;                     // a multiple of CONSUMER_WARPS: a slot always serves the same warp
constexpr int SLOT_BYTES = 32768;            // retained: K 16 KB | V 16 KB; key-only: keys 0-63 | keys 64-127
constexpr int HALF_BYTES = 16384;            // 64 rows of 256 B as two swizzled 64 x 128 B boxes
constexpr int BOX_BYTES = 8192;              // 64 rows x 128 bytes
constexpr int CONSUMER_WARPS = 3;
constexpr int THREADS = 32 * (CONSUMER_WARPS + 1);
// With RoPE decoupling the block carries helper warps that turn a tile's keys back for the warp
// that owns the tile: a team is that warp plus four helpers (warps 4 + 4 team .. 7 + 4 team), one
// per warp scheduler (scheduler = warp index modulo 4), since the sine / cosine unit is per scheduler.
constexpr int ROPE_HELPERS = 4;
constexpr int ROPE_THREADS = 32 * (CONSUMER_WARPS + 1 + ROPE_HELPERS * CONSUMER_WARPS);
constexpr int ROPE_TEAM_THREADS = 32 * (1 + ROPE_HELPERS);
static_assert(CONSUMER_WARPS + 1 == 4 && ROPE_HELPERS == 4, "register hand-over is per warpgroup: owners + producer, then helpers");
constexpr int REC = 4 + 2 * 128;             // m, l, value-scale, pad, acc_v[128], acc_k[128]
constexpr int SMEM_BYTES = SLOTS * SLOT_BYTES + 1024;   // + alignment slack; barriers live in static smem

// How the tile sequence is dealt to blocks; the same arithmetic runs on host and device.
struct Plan {
    int n_rt, n_at, n_tiles;   // retained / key-only / all tiles per unit
    long long T;               // tiles of all units
    int B;                     // blocks
    int s_max;                 // record slots per unit
};
__host__ __device__ inline Plan make_plan(int U, long long n_ret, long long n_apx, int max_blocks) {
    Plan p;
    p.n_rt = (int)((n_ret + KEYS - 1) / KEYS);
    p.n_at = (int)((n_apx + 2 * KEYS - 1) / (2 * KEYS));
    p.n_tiles = p.n_rt + p.n_at;
    p.T = (long long)U * p.n_tiles;
    long long b = p.T / 2;                       // at least two tiles per block
    if (b > max_blocks) b = max_blocks;               // one persistent block per multiprocessor
    if (b > 11LL * U) b = 11LL * U;              // at most 12 record slots per unit (merge kernel limit)
    p.B = (int)(b < 1 ? 1 : b);
    p.s_max = (p.B + U - 1) / U + 1;
    return p;
}
// Block b owns the tiles [b T / B, (b+1) T / B).
__host__ __device__ inline long long tile_begin(int b, const Plan& p) { return (long long)b * p.T / p.B; }
__host__ __device__ inline int block_of_tile(long long x, const Plan& p) { return (int)(((x + 1) * p.B - 1) / p.T); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8) += A(16x16) B(16x8) with A rows 8..15 zero: the upper accumulator half is fed zeros and
// its (zero) result parked in a scratch pair.
__device__ __forceinline__ void mma_lo8(float& c0, float& c1, float& z0, float& z1, uint32_t a0, uint32_t a2,
                                        uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%10,%10};\n"
        : "+f"(c0), "+f"(c1), "=f"(z0), "=f"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ void mma_16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// The same product with fp16 operands (the keys turned back under RoPE decoupling are held in fp16).
__device__ __forceinline__ void mma_16_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                           uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// Two floats to an fp16 pair, low half first; values beyond the fp16 range go to its largest finite number.
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;\n" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float f16_lo(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v & 0xffffu))); }
__device__ __forceinline__ float f16_hi(uint32_t v) { return __half2float(__ushort_as_half((unsigned short)(v >> 16))); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// RoPE decoupling: rows 16 member .. 16 member + 15 of the 64 keys at kbase (two swizzled boxes:
// channels 0-63 | 64-127) are turned back by their positions, in place, and left there as fp16 (a
// turned key is not a bf16 number; eleven bits keep the key sum within the tolerance of the output,
// eight do not; |k| beyond 65504 saturates).  Channel c pairs with
// c + 64; the angle is position * theta^(-2c/128), taken as the 32-bit product of the position and
// the per-channel phase (turns per position as a fraction of 2^32), which is the angle modulo one turn.  pos16: lane l
// holds the position of row 16 member + (l & 15).
__device__ __forceinline__ void derotate_rows(uint32_t kbase, int nrows, int member, uint32_t pos16,
                                              const uint32_t* phase_s, int lane) {
    const int qc = lane & 7;                                        // 16-byte chunk: channel pairs 8 qc .. 8 qc + 7
    uint32_t phase[8];                                              // this lane's eight channel pairs
#pragma unroll
    for (int c = 0; c < 8; ++c) phase[c] = phase_s[qc * 8 + c];
#pragma unroll 1
    for (int j = 0; j < 4; j += 2) {
        // two rows per round, the loads of both ahead of the stores
        uint32_t off[2], pos[2], xs[2][4], ys[2][4];
        bool live[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int rl = 4 * (j + u) + (lane >> 3), r = 16 * member + rl;
            pos[u] = __shfl_sync(0xffffffffu, pos16, rl);
            live[u] = r < nrows;
            off[u] = (uint32_t)r * 128u + (uint32_t)((qc ^ (r & 7)) << 4);
            if (live[u]) {
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(xs[u][0]), "=r"(xs[u][1]), "=r"(xs[u][2]), "=r"(xs[u][3]) : "r"(kbase + off[u]));
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(ys[u][0]), "=r"(ys[u][1]), "=r"(ys[u][2]), "=r"(ys[u][3]) : "r"(kbase + BOX_BYTES + off[u]));
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) { xs[u][e] = 0u; ys[u][e] = 0u; }
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float x[2], y[2], cs[2], sn[2], xo[2], yo[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    x[h] = __uint_as_float(h ? (xs[u][e] & 0xffff0000u) : (xs[u][e] << 16));
                    y[h] = __uint_as_float(h ? (ys[u][e] & 0xffff0000u) : (ys[u][e] << 16));
                    rope_phase32_cos_sin(pos[u], phase[2 * e + h], cs[h], sn[h]);
                }
                // both pairs of the word at once on the packed FMA path
                const uint64_t x2 = tc::pack2(x[0], x[1]), y2 = tc::pack2(y[0], y[1]);
                const uint64_t c2 = tc::pack2(cs[0], cs[1]), s2 = tc::pack2(sn[0], sn[1]);
                tc::unpack2(tc::fma2(x2, c2, tc::mul2(y2, s2)), xo[0], xo[1]);
                tc::unpack2(tc::fma2(y2, c2, tc::mul2(x2, tc::pack2(-sn[0], -sn[1]))), yo[0], yo[1]);
                xs[u][e] = pack_f16(xo[0], xo[1]);
                ys[u][e] = pack_f16(yo[0], yo[1]);
            }
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (live[u]) {
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(kbase + off[u]), "r"(xs[u][0]), "r"(xs[u][1]), "r"(xs[u][2]), "r"(xs[u][3]) : "memory");
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n" ::"r"(kbase + BOX_BYTES + off[u]), "r"(ys[u][0]), "r"(ys[u][1]), "r"(ys[u][2]), "r"(ys[u][3]) : "memory");
            }
        }
    }
    // the slot is refilled by a bulk copy once released: order these stores ahead of it
    asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
}
// All threads of team `team` (its owner warp and the helpers).
__device__ __forceinline__ void team_sync(int team) {
    asm volatile("bar.sync %0, %1;\n" ::"r"(2 + team), "n"(ROPE_TEAM_THREADS) : "memory");
}

static_assert(SLOTS % CONSUMER_WARPS == 0, "a slot must always be consumed by the same warp");

struct Maps {
    CUtensorMap ret_k, ret_v, apx_k;     // rank 3: (128 dims, pool rows, U units), box 64 x 64 x 1, 128B swizzle
};

// grid (plan.B), THREADS threads, SMEM_BYTES dynamic shared memory.
// partial: [U][s_max][CONSUMER_WARPS][g][REC]; slot of (unit u, block b) = b - block_of_tile(first tile of u).
template <bool ROPE>
__global__ void __launch_bounds__(ROPE ? ROPE_THREADS : THREADS, 1)
decode_stream_bf16_d128(const __nv_bfloat16* __restrict__ q, const __grid_constant__ Maps maps, Plan pl, int n_ret,
                        int n_apx, int g, int LH, float scale_log2e, float* __restrict__ partial,
                        int* __restrict__ fault, const int32_t* __restrict__ apx_pos, long long cap_apx,
                        const __grid_constant__ RopePhases rope) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ uint32_t phase_s[ROPE ? 64 : 1];          // the phases rounded to 32 bits
    if (ROPE && threadIdx.x < 64) phase_s[threadIdx.x] = (uint32_t)((rope.phase[threadIdx.x] + 0x80000000ull) >> 32);
    __shared__ volatile int team_ok[CONSUMER_WARPS];     // RoPE: the owner's go / no-go for the tile at hand
    __shared__ __align__(8) uint64_t full_bar[SLOTS];
    __shared__ __align__(8) uint64_t empty_bar[SLOTS];
    // 128B-swizzled TMA boxes want 1024-byte aligned destinations
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int b = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wq = tid >> 5;
    const long long gt_lo = tile_begin(b, pl), gt_hi = tile_begin(b + 1, pl);
    if (gt_lo >= gt_hi) return;
    const int n_my = (int)(gt_hi - gt_lo);
    const int u0 = (int)(gt_lo / pl.n_tiles), t0 = (int)(gt_lo - (long long)u0 * pl.n_tiles);
    const int u_last = (int)((gt_hi - 1) / pl.n_tiles);

    // The merge kernel is launched as a programmatic dependent of this one: its blocks may be
    // scheduled (and fetch W) as soon as SMs free up; it reads the records only after its own
    // griddepcontrol.wait, which returns once this whole grid has finished and flushed.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) { tma::mbar_init(&full_bar[s], 1); tma::mbar_init(&empty_bar[s], 1); }
        tma::mbar_fence_init();
    }
    __syncthreads();

    if (ROPE && wq > CONSUMER_WARPS) {
        // ------------------------------------------------------------------ helpers (RoPE only)
        // A helper walks its owner's key-only tiles and turns back its quarter of each 64 keys
        // between the owner's two team barriers.  It waits on nothing but those barriers, which the
        // owner reaches for every key-only tile whether or not its own (bounded) waits succeeded.
        // The block is compiled for 128 registers a thread (512 threads): the three helper
        // warpgroups hand registers over to the first one (the three owners and the producer).
        asm volatile("setmaxnreg.dec.sync.aligned.u32 96;\n");
        const int team = (wq - CONSUMER_WARPS - 1) / ROPE_HELPERS, member = (wq - CONSUMER_WARPS - 1) % ROPE_HELPERS;
        int i = team;
        for (int u = u0; u <= u_last; ++u) {
            const long long unit_end = (long long)(u + 1) * pl.n_tiles - gt_lo;
            for (; i < n_my && i < unit_end; i += CONSUMER_WARPS) {
                const int t = (int)(gt_lo + i - (long long)u * pl.n_tiles);
                if (t < pl.n_rt) continue;
                const int r0 = (t - pl.n_rt) * 2 * KEYS;
                const int32_t* pr = apx_pos + (size_t)u * cap_apx + r0 + 16 * member + (lane & 15);
                const int n0 = min(KEYS, n_apx - r0), n1 = min(KEYS, n_apx - r0 - KEYS);      // n1 <= 0: no second half
                const uint32_t p0 = 16 * member + (lane & 15) < n0 ? (uint32_t)__ldg(pr) : 0u;
                const uint32_t p1 = 16 * member + (lane & 15) < n1 ? (uint32_t)__ldg(pr + KEYS) : 0u;
                team_sync(team);                                   // the owner has published its verdict
                if (!team_ok[team]) continue;
                const uint32_t base = tma::smem_u32(smem + (i % SLOTS) * SLOT_BYTES);
                team_sync(team);                                   // the owner has its scores of half 0
                derotate_rows(base, n0, member, p0, phase_s, lane);
                team_sync(team);                                   // ... and of half 1, if there is one
                if (n1 > 0) {
                    derotate_rows(base + HALF_BYTES, n1, member, p1, phase_s, lane);
                    team_sync(team);
                }
            }
        }
        return;
    }

    if (ROPE) asm volatile("setmaxnreg.inc.sync.aligned.u32 216;\n");
    if (wq == CONSUMER_WARPS) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            tma::prefetch_map(&maps.ret_k); tma::prefetch_map(&maps.ret_v); tma::prefetch_map(&maps.apx_k);
            const uint64_t pol = tma::policy_evict_first();      // the cache is read once per step
            int u = u0, t = t0;
            for (int i = 0; i < n_my; ++i) {
                const int s = i % SLOTS, round = i / SLOTS;
                if (round > 0 && !tma::mbar_wait(&empty_bar[s], (round - 1) & 1, fault, 1)) break;
                unsigned char* st = smem + s * SLOT_BYTES;
                tma::mbar_expect_tx(&full_bar[s], SLOT_BYTES);
                if (t < pl.n_rt) {
                    const int row0 = t * KEYS;
                    tma::load_3d_hint(st, &maps.ret_k, 0, row0, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + BOX_BYTES, &maps.ret_k, 64, row0, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES, &maps.ret_v, 0, row0, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES + BOX_BYTES, &maps.ret_v, 64, row0, u, &full_bar[s], pol);
                } else {
                    const int row0 = (t - pl.n_rt) * 2 * KEYS;
                    tma::load_3d_hint(st, &maps.apx_k, 0, row0, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + BOX_BYTES, &maps.apx_k, 64, row0, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES, &maps.apx_k, 0, row0 + KEYS, u, &full_bar[s], pol);
                    tma::load_3d_hint(st + HALF_BYTES + BOX_BYTES, &maps.apx_k, 64, row0 + KEYS, u, &full_bar[s], pol);
                }
                if (++t == pl.n_tiles) { t = 0; ++u; }
            }
        }
        return;      // the consumers wait on every tile's full barrier, so no copy outlives the block
    }
    // ---------------------------------------------------------------------- consumers
    const int gid = lane >> 2, tig = lane & 3;
    // per-lane ldmatrix geometry (swizzle: 16-byte chunk index XOR (row & 7), rows are 128 bytes)
    const int mat = lane >> 3, r8 = lane & 7;
    const uint32_t qk_row = (uint32_t)(r8 + (mat >> 1) * 8) * 128u;      // QK: matrices = (keys 0-7|8-15) x (chunk lo|hi)
    const uint32_t qk_x = (uint32_t)(((mat & 1) ^ r8) << 4);
    const uint32_t pv_row = (uint32_t)(r8 + (mat & 1) * 8) * 128u;       // PV: matrices = (chunk lo|hi) x (keys 0-7|8-15)
    const uint32_t pv_x = (uint32_t)(((mat >> 1) ^ r8) << 4);

    uint32_t qa[8][2];
    float acc[16][4];                  // [dim tile][c0,c1: P_hi rows | c2,c3: P_lo rows]
    float m = -INFINITY, l = 0.f, stash_scale = 1.f;
    bool stashed = false;

    auto record_of = [&](int unit) -> float* {
        int slot = b - block_of_tile((long long)unit * pl.n_tiles, pl);
        if (slot < 0 || slot >= pl.s_max) { atomicCAS(fault, 0, 5); slot = 0; }     // cannot happen; never write out of bounds
        return partial + ((((size_t)unit * pl.s_max + slot) * CONSUMER_WARPS + wq) * g + gid) * REC;
    };
    auto load_q = [&](int unit) {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)unit * g + min(gid, g - 1)) * 128);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = gid < g ? qrow[ks * 8 + tig] : 0u;
            qa[ks][1] = gid < g ? qrow[ks * 8 + 4 + tig] : 0u;
        }
    };
    auto store_acc = [&](float* dst) {       // dims n*8 + 2 tig + {0,1} of head row gid
#pragma unroll
        for (int n = 0; n < 16; ++n)
            *reinterpret_cast<float2*>(dst + n * 8 + 2 * tig) = make_float2(acc[n][0] + acc[n][2], acc[n][1] + acc[n][3]);
    };
    auto zero_acc = [&]() {
#pragma unroll
        for (int n = 0; n < 16; ++n) { acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f; }
    };
    // Writes this warp's record of `unit` (an all-zero one with m = -inf if it met none of its tiles).
    auto flush = [&](int unit) {
        float lt = l;
        lt += __shfl_xor_sync(0xffffffffu, lt, 1);
        lt += __shfl_xor_sync(0xffffffffu, lt, 2);
        if (gid < g) {
            float* rec = record_of(unit);
            if (tig == 0) *reinterpret_cast<float4*>(rec) = make_float4(m * 0.69314718055994531f, lt, stashed ? stash_scale : 1.f, 0.f);
            if (stashed) store_acc(rec + 4 + 128);      // value part was written at the pool switch
            else {
                store_acc(rec + 4);
#pragma unroll
                for (int n = 0; n < 16; ++n) *reinterpret_cast<float2*>(rec + 4 + 128 + n * 8 + 2 * tig) = make_float2(0.f, 0.f);
            }
        }
        zero_acc();
        m = -INFINITY; l = 0.f; stash_scale = 1.f; stashed = false;
    };
    // One softmax step over the 64 keys at kbase (two swizzled boxes), in two parts.  The first
    // leaves the step's weights p in sc (this thread: head gid, keys 8 n + 2 tig, + 1), brings m, l
    // and the accumulators to the new running maximum and returns the factor it applied to them.
    auto scores64 = [&](uint32_t kbase, int nrows, bool retained, int unit, float (&sc)[8][2]) -> float {
        // ---- S = Q K^T: eight 8-key column tiles, each its own accumulator chain over the 8 k-steps
        float zz[2];
#pragma unroll
        for (int n = 0; n < 8; ++n) { sc[n][0] = 0.f; sc[n][1] = 0.f; }
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {          // 16 keys per ldmatrix
                uint32_t b0, b1, b2, b3;
                // k-step ks covers 16-byte chunks 2ks, 2ks+1 of the 256-byte row: box ks/4, chunk (2ks)%8 (+1)
                ldsm_x4(kbase + (ks >> 2) * BOX_BYTES + j * 16 * 128 + qk_row + ((((2 * ks) & 7) << 4) ^ qk_x), b0, b1, b2, b3);
                mma_lo8(sc[2 * j][0], sc[2 * j][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b0, b1);
                mma_lo8(sc[2 * j + 1][0], sc[2 * j + 1][1], zz[0], zz[1], qa[ks][0], qa[ks][1], b2, b3);
            }
        }
        // ---- online softmax over these 64 keys (row = head gid, shared by the 4 threads of a quad)
        float mx = -INFINITY;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            const int kc = n * 8 + 2 * tig;
            sc[n][0] = kc < nrows ? sc[n][0] * scale_log2e : -INFINITY;
            sc[n][1] = kc + 1 < nrows ? sc[n][1] * scale_log2e : -INFINITY;
            mx = fmaxf(mx, fmaxf(sc[n][0], sc[n][1]));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        if (!retained && !stashed) {           // first key-only keys of this unit for this warp: park sum p v
            if (gid < g) store_acc(record_of(unit) + 4);
            zero_acc();
            stashed = true;
            stash_scale = 1.f;
        }
        const float m_new = fmaxf(m, mx);      // finite: key 0 of the step is valid for every row
        const float alpha = exp2f(m - m_new);  // 0 on the first step
        float ls = 0.f;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            sc[n][0] = exp2f(sc[n][0] - m_new);
            sc[n][1] = exp2f(sc[n][1] - m_new);
            ls += sc[n][0] + sc[n][1];
        }
        l = l * alpha + ls;
        m = m_new;
        stash_scale *= alpha;
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
            {
#pragma unroll
                for (int n = 0; n < 16; ++n) { acc[n][0] *= alpha; acc[n][1] *= alpha; acc[n][2] *= alpha; acc[n][3] *= alpha; }
            }
        }
        return alpha;
    };
    // The second part adds p x (the 64 rows at vbase: values, or the keys themselves for a key-only tile).
    auto accumulate64 = [&](uint32_t vbase, bool retained, float (&sc)[8][2]) {
        // ---- accumulate P x (V rows | K rows): four k-steps of 16 keys x 16 column tiles of 8 dims
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {
            // P as bf16 hi (MMA rows 0-7) + lo (rows 8-15)
            const float p00 = sc[2 * kk][0], p01 = sc[2 * kk][1], p10 = sc[2 * kk + 1][0], p11 = sc[2 * kk + 1][1];
            if (ROPE && !retained) {
                // the turned keys are fp16: so are the weights, again as hi + lo
                const uint32_t a0 = pack_f16(p00, p01), a2 = pack_f16(p10, p11);
                const uint32_t a1 = pack_f16(p00 - f16_lo(a0), p01 - f16_hi(a0)), a3 = pack_f16(p10 - f16_lo(a2), p11 - f16_hi(a2));
#pragma unroll
                for (int np = 0; np < 8; ++np) {
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(vbase + (np >> 2) * BOX_BYTES + kk * 16 * 128 + pv_row + ((((2 * np) & 7) << 4) ^ pv_x), b0, b1, b2, b3);
                    mma_16_f16(acc[2 * np], a0, a1, a2, a3, b0, b1);
                    mma_16_f16(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
                }
                continue;
            }
            const __nv_bfloat16 h00 = __float2bfloat16_rn(p00), h01 = __float2bfloat16_rn(p01);
            const __nv_bfloat16 h10 = __float2bfloat16_rn(p10), h11 = __float2bfloat16_rn(p11);
            const uint32_t a0 = pack_bf16(__bfloat162float(h00), __bfloat162float(h01));
            const uint32_t a2 = pack_bf16(__bfloat162float(h10), __bfloat162float(h11));
            const uint32_t a1 = pack_bf16(p00 - __bfloat162float(h00), p01 - __bfloat162float(h01));
            const uint32_t a3 = pack_bf16(p10 - __bfloat162float(h10), p11 - __bfloat162float(h11));
#pragma unroll
            for (int np = 0; np < 8; ++np) {
                uint32_t b0, b1, b2, b3;
                ldsm_x4_t(vbase + (np >> 2) * BOX_BYTES + kk * 16 * 128 + pv_row + ((((2 * np) & 7) << 4) ^ pv_x), b0, b1, b2, b3);
                mma_16(acc[2 * np], a0, a1, a2, a3, b0, b1);
                mma_16(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
            }
        }
    };

    auto step64 = [&](uint32_t kbase, uint32_t vbase, int nrows, bool retained, int unit) {
        float sc[8][2];
        scores64(kbase, nrows, retained, unit, sc);
        accumulate64(vbase, retained, sc);
    };
    // A key-only tile under RoPE decoupling.  The scores come from the keys as stored, the key sum
    // wants them without the rotation: the helpers turn each half back between the two uses, and
    // the owner forms the second half's scores (then the first half's sum) in the meantime.
    auto rope_tile = [&](uint32_t base, int n0, int n1, int unit) {
        float sc0[8][2], sc1[8][2];
        scores64(base, n0, false, unit, sc0);
        team_sync(wq);                         // every lane is past its last read of half 0 as stored
        if (n1 > 0) {
            const float alpha = scores64(base + HALF_BYTES, n1, false, unit, sc1);
#pragma unroll
            for (int n = 0; n < 8; ++n) { sc0[n][0] *= alpha; sc0[n][1] *= alpha; }     // the sums moved to the new maximum
        }
        team_sync(wq);                         // half 0 is turned back (and half 1 is free to be)
        accumulate64(base, false, sc0);
        if (n1 > 0) {
            team_sync(wq);                     // half 1 is turned back
            accumulate64(base + HALF_BYTES, false, sc1);
        }
    };

    zero_acc();
    // Walk the units the block touches; this warp owns the block's tiles i with i % CONSUMER_WARPS == wq.
    int i = wq;                                        // index into the block's tile sequence
    bool ok = true;                                    // false once a wait gave up: keep walking, touch nothing
    for (int u = u0; u <= u_last; ++u) {
        const long long unit_end = (long long)(u + 1) * pl.n_tiles - gt_lo;     // first sequence index past the unit
        bool loaded = false;
        for (; i < n_my && i < unit_end; i += CONSUMER_WARPS) {
            const int s = i % SLOTS, round = i / SLOTS;
            const int t = (int)(gt_lo + i - (long long)u * pl.n_tiles);
            if (ok) {
                if (!loaded) { load_q(u); loaded = true; }
                ok = tma::mbar_wait_warp(&full_bar[s], round & 1, fault, 2);
            }
            if (ROPE && t >= pl.n_rt) {        // tell the helpers whether this key-only tile is worked on
                if (lane == 0) team_ok[wq] = ok ? 1 : 0;
                team_sync(wq);
            }
            if (!ok) continue;
            const uint32_t base = tma::smem_u32(smem + s * SLOT_BYTES);
            if (t < pl.n_rt) {
                step64(base, base + HALF_BYTES, min(KEYS, n_ret - t * KEYS), true, u);
            } else {
                const int r0 = (t - pl.n_rt) * 2 * KEYS;
                if (ROPE) {
                    rope_tile(base, min(KEYS, n_apx - r0), min(KEYS, n_apx - r0 - KEYS), u);
                } else {
                    step64(base, base, min(KEYS, n_apx - r0), false, u);
                    if (n_apx - r0 > KEYS)
                        step64(base + HALF_BYTES, base + HALF_BYTES, min(KEYS, n_apx - r0 - KEYS), false, u);
                }
            }
            __syncwarp();
            if (lane == 0) tma::mbar_arrive(&empty_bar[s]);
        }
        flush(u);
    }
}

// Merge for head_dim 128: grid (U), 128 g threads -- thread (a, c) owns output dim c of head a.
// Combines the records of a unit, applies the unit's map to the p-weighted key sum and normalises:
//   o = (sum_j f_j s_j acc_v_j + W sum_j f_j acc_k_j) / sum_j f_j l_j,   f_j = exp(m_j - max m).
// Every load of a phase is independent of the others, so a phase costs one memory latency.
// The product W (sum f acc_k) runs on warp-level MMAs, M = 128 output channels (warp w takes rows 16 w ..),
// N = the unit's g query heads (padded to 8), K = 128: the A fragments are read straight from the map in
// global memory, 16 bytes a load -- thread (row r, quarter t) of a warp holds columns 8 (t + 4 jj) .. + 7 of
// rows r and r + 8, and the k slots of MMA step 2 jj + h stand for columns 8 (t + 4 jj) + 4 h .. + 3, which the
// B fragments follow; the key sum enters as bf16 hi + lo (sixteen mantissa bits), the map's elements are bf16
// as stored.
template <typename TO, int MAXT>
__global__ void __launch_bounds__(MAXT, MAXT == 512 ? 3 : 1)
decode_merge_bf16_d128(const float* __restrict__ partial, const __nv_bfloat16* __restrict__ W, int LH, int g,
                       Plan pl, int apply_w, int cw, TO* __restrict__ out) {
    __shared__ __align__(16) __nv_bfloat16 akh[8][128], akl[8][128];      // key sums per head, hi and lo halves
    __shared__ float pw[8][128];               // W times the key sum
    __shared__ float fv[8][48], fk[8][48];     // per head, per record: factor for the value part / the key part
    __shared__ float Ls[8];
    const int u = blockIdx.x, tid = threadIdx.x, a = tid >> 7, c = tid & 127, lane = tid & 31;
    const int wid = tid >> 5, nwarps = blockDim.x >> 5, row = lane >> 2, quarter = lane & 3;
    // A fragments of 16 rows of W (the maps of a layer stay in L2: every sequence of the batch reads them)
    const uint4* Wu = reinterpret_cast<const uint4*>(W + (size_t)(u % LH) * 128 * 128);       // 16 pieces per 256-byte row
    uint4 A[8];
    auto load_rows = [&](int mt) {
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            A[2 * jj + 0] = Wu[(16 * mt + row) * 16 + quarter + 4 * jj];
            A[2 * jj + 1] = Wu[(16 * mt + row + 8) * 16 + quarter + 4 * jj];
        }
    };
    for (int i = tid; i < (8 - g) * 128; i += blockDim.x) {       // columns of B beyond the unit's heads
        akh[g + i / 128][i % 128] = __float2bfloat16_rn(0.f);
        akl[g + i / 128][i % 128] = __float2bfloat16_rn(0.f);
    }
    // everything above reads only W, which the streaming kernel does not write; its records from here on
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    const int first = block_of_tile((long long)u * pl.n_tiles, pl);
    const int n_rec = (block_of_tile((long long)(u + 1) * pl.n_tiles - 1, pl) - first + 1) * cw;   // <= 36; cw records per block
    const float* base = partial + (size_t)u * pl.s_max * cw * g * REC;
    // The first six records' sums are requested before the headers are looked at, so that the two loads
    // share one memory latency (a unit lies in one or two blocks of the streaming kernel, three records
    // each, unless it is very long).
    constexpr int NPRE = 6;
    float rv[NPRE], rk[NPRE];
#pragma unroll
    for (int k = 0; k < NPRE; ++k) {
        const int j = min(k, n_rec - 1);
        const float* r = base + ((size_t)j * g + a) * REC + 4;
        rv[k] = r[c];
        rk[k] = r[128 + c];
    }
    if (c < 32) {
        // first warp of head a: headers of records lane and lane + 32
        float mj[2], lj[2], sj[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int j = lane + 32 * k;
            mj[k] = -INFINITY; lj[k] = 0.f; sj[k] = 0.f;
            if (j < n_rec) {
                const float4 h = *reinterpret_cast<const float4*>(base + ((size_t)j * g + a) * REC);
                mj[k] = h.x; lj[k] = h.y; sj[k] = h.z;
            }
        }
        const float M = warp_max(fmaxf(mj[0], mj[1]));
        float Lsum = 0.f;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int j = lane + 32 * k;
            const float f = mj[k] > -INFINITY ? __expf(mj[k] - M) : 0.f;
            if (j < 48) { fk[a][j] = f; fv[a][j] = f * sj[k]; }
            Lsum += f * lj[k];
        }
        Lsum = warp_sum(Lsum);
        if (lane == 0) Ls[a] = Lsum;
    }
    __syncthreads();
    float av = 0.f, ak = 0.f;
    for (int j0 = 0; j0 < n_rec; j0 += NPRE) {
        if (j0 > 0) {
#pragma unroll
            for (int k = 0; k < NPRE; ++k) {
                const int j = min(j0 + k, n_rec - 1);
                const float* r = base + ((size_t)j * g + a) * REC + 4;
                rv[k] = r[c];
                rk[k] = r[128 + c];
            }
        }
#pragma unroll
        for (int k = 0; k < NPRE; ++k) {
            if (j0 + k < n_rec) {
                av = fmaf(fv[a][j0 + k], rv[k], av);
                ak = fmaf(fk[a][j0 + k], rk[k], ak);
            }
        }
    }
    if (!apply_w) {           // per-tile form: the second part of a record is already sum p (W k)
        store_out(out + ((size_t)u * g + a) * 128 + c, (av + ak) / Ls[a]);
        return;
    }
    {
        const __nv_bfloat16 hi = __float2bfloat16_rn(ak);
        akh[a][c] = hi;
        akl[a][c] = __float2bfloat16_rn(ak - __bfloat162float(hi));
    }
    __syncthreads();
    for (int mt = wid; mt < 8; mt += nwarps) {
        load_rows(mt);
        float d[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int jj = 0; jj < 4; ++jj) {
            const uint4 r0 = A[2 * jj], r1 = A[2 * jj + 1];
            const int col = 8 * (quarter + 4 * jj);
            const uint4 bh = *reinterpret_cast<const uint4*>(&akh[row][col]);      // B column = head `row`
            const uint4 bl = *reinterpret_cast<const uint4*>(&akl[row][col]);
            mma_16(d, r0.x, r1.x, r0.y, r1.y, bh.x, bh.y);
            mma_16(d, r0.x, r1.x, r0.y, r1.y, bl.x, bl.y);
            mma_16(d, r0.z, r1.z, r0.w, r1.w, bh.z, bh.w);
            mma_16(d, r0.z, r1.z, r0.w, r1.w, bl.z, bl.w);
        }
        // d[0], d[1]: row `row`, heads 2 quarter and 2 quarter + 1; d[2], d[3]: row `row` + 8
        if (2 * quarter < g) { pw[2 * quarter][16 * mt + row] = d[0]; pw[2 * quarter][16 * mt + row + 8] = d[2]; }
        if (2 * quarter + 1 < g) { pw[2 * quarter + 1][16 * mt + row] = d[1]; pw[2 * quarter + 1][16 * mt + row + 8] = d[3]; }
    }
    __syncthreads();
    store_out(out + ((size_t)u * g + a) * 128 + c, (av + pw[a][c]) / Ls[a]);
}

}  // namespace dbf
}  // namespace vec
#endif
