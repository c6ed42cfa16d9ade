// Internal declarations shared by the translation units of libvector (host side).
#ifndef VECTOR_INTERNAL_H_
#define VECTOR_INTERNAL_H_

#include <cstddef>
#include <cstdint>

#include "vector.h"

namespace vec {

// Geometry derived from a validated vector_shape.
struct Dims {
    int U;        // units = batch * n_layers * n_kv_heads
    int LH;       // maps  = n_layers * n_kv_heads
    int g;        // query heads per KV head
    int d;        // head_dim
    int w;        // observation window
    int R;        // score rows per unit = g * w
    int pool_kernel;
    int dtype;
    int esize;    // bytes per element
    float scale;
    int rope;
    float theta;
};

// phase[c] = frac(theta^(-2c/d) / (2 pi)) * 2^64, c < d/2 <= 64: the turns channel pair c makes per
// position, as a 64-bit fraction.  The top 32 bits of position * phase (modulo 2^64) are then the
// rotary angle of that pair, in turns modulo one, to 2^-32 of a turn for any 32-bit position.
struct RopePhases { unsigned long long phase[64]; };
void rope_phases(float theta, int d, RopePhases* out);

// Checks a shape against what the kernels support and fills Dims.
vector_status check_shape(const vector_shape* s, Dims* out);
// Checks internal consistency of tier sizes (the identities of the planner).
vector_status check_budget(const vector_budget* b, int window);

void set_last_cuda_error(int e);
// Adds one to the process-wide count of kernels launched by the library (vector_kernel_launches).
void count_launch();

// Multiprocessors of the current device (read once per device); the B200's 148 when no device
// can be queried, so that the host-only sizing calls still answer.
int sm_count();

// ---- workspace layout (bytes, each region 256-byte aligned) ----
// Number of key chunks the first score pass splits a unit's keys into.
int score_num_chunks(int U, int R, int64_t N);
size_t score_ws_bytes(const Dims& D, int64_t N, bool need_raw);
// Work split of the tensor-core score kernels (bf16, head_dim 128): row groups of up to 256 window
// rows, 128-key tiles, and per unit `n_chunks` chunks of `tpc` tiles; an item is (unit, chunk, row group).
struct ScoreTcPlan { int RG, nt, tpc, n_chunks, n_items; };
ScoreTcPlan score_tc_plan(int U, int R, int64_t N);
inline bool score_uses_tc(const Dims& D) { return D.dtype == VECTOR_BF16 && D.d == 128; }
// Device address (on the current device) of the word in which bounded waits inside kernels record
// that they gave up; NULL if it cannot be resolved.
int* kernel_fault_address();

// One-time set-up that has to happen once per device (kernel attributes are per device): returns true
// the first time it is called with the current device for this flag set, false afterwards (and false,
// doing nothing, if the device index is out of range).  Thread-safe.
struct PerDeviceOnce {
    static constexpr int kMax = 64;
    unsigned char done[kMax] = {};
    bool first();          // defined in host.cpp
    void undo();           // the set-up failed: try again on the next call
};
size_t select_ws_bytes(const Dims& D, const vector_budget& b);
// Number of key splits of one unit in decode attention for `rows` logical keys.
int decode_num_splits(int U, int64_t rows);
// Record slots per unit that the persistent bf16 decode kernel may use (two blocks per SM).
int decode_stream_slots(int U);
size_t decode_ws_bytes(const Dims& D);
size_t keydiff_ws_bytes(const Dims& D, int64_t N);

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

}  // namespace vec

#define VEC_CUDA_CHECK(expr)                                  \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) {                             \
            vec::set_last_cuda_error((int)e__);               \
            return VECTOR_ERR_CUDA;                           \
        }                                                     \
    } while (0)

#define VEC_LAUNCH_CHECK()                    \
    do {                                      \
        vec::count_launch();                  \
        VEC_CUDA_CHECK(cudaPeekAtLastError()); \
    } while (0)

#endif  // VECTOR_INTERNAL_H_
