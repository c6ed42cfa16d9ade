// Host-only entry points of libvector: status text, the tier planner and the
// offline least-squares calibration, plus the argument checks the device entry
// points share.  The only CUDA calls in this file are cudaGetDevice and the query of the
// multiprocessor count.
#include <atomic>
#include <cmath>
#include <mutex>
#include <cuda_runtime_api.h>
#include <cstring>
#include <vector>

#include "internal.h"

namespace vec {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

static std::atomic<unsigned long long> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

void rope_phases(float theta, int d, RopePhases* out) {
    for (int c = 0; c < 64; ++c) {
        if (c >= d / 2) { out->phase[c] = 0ull; continue; }
        const long double f = powl((long double)theta, -2.0L * c / (long double)d) / 6.283185307179586476925286766559L;
        out->phase[c] = (unsigned long long)ldexpl(f - floorl(f), 64);
    }
}

static std::mutex g_once_mu;
int sm_count() {
    static int cached[PerDeviceOnce::kMax] = {};
    constexpr int kDefault = 148;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= PerDeviceOnce::kMax) {
        (void)cudaGetLastError();
        return kDefault;
    }
    std::lock_guard<std::mutex> lock(g_once_mu);
    if (cached[dev] <= 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = kDefault;
        cached[dev] = n;
    }
    return cached[dev];
}
bool PerDeviceOnce::first() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMax) return false;
    std::lock_guard<std::mutex> lock(g_once_mu);
    if (done[dev]) return false;
    done[dev] = 1;
    return true;
}
void PerDeviceOnce::undo() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMax) return;
    std::lock_guard<std::mutex> lock(g_once_mu);
    done[dev] = 0;
}

vector_status check_shape(const vector_shape* s, Dims* out) {
    if (!s || !out) return VECTOR_ERR_NULL;
    if (s->dtype != VECTOR_F32 && s->dtype != VECTOR_BF16) return VECTOR_ERR_DTYPE;
    if (s->batch <= 0 || s->n_layers <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0)
        return VECTOR_ERR_SHAPE;
    if (s->n_q_heads % s->n_kv_heads != 0) return VECTOR_ERR_SHAPE;
    if (s->head_dim != 64 && s->head_dim != 128) return VECTOR_ERR_SHAPE;
    int g = s->n_q_heads / s->n_kv_heads;
    if (g > 8) return VECTOR_ERR_SHAPE;
    if (s->window <= 0 || (int64_t)s->window * g > 1024) return VECTOR_ERR_SHAPE;
    if (s->pool_kernel < 1 || s->pool_kernel > 15 || (s->pool_kernel % 2) == 0) return VECTOR_ERR_SHAPE;
    int64_t U = (int64_t)s->batch * s->n_layers * s->n_kv_heads;
    if (U > 65535) return VECTOR_ERR_SHAPE;
    if (s->rope_enabled && !(s->rope_theta > 1.0f)) return VECTOR_ERR_SHAPE;
    out->U = (int)U;
    out->LH = s->n_layers * s->n_kv_heads;
    out->g = g;
    out->d = s->head_dim;
    out->w = s->window;
    out->R = g * s->window;
    out->pool_kernel = s->pool_kernel;
    out->dtype = s->dtype;
    out->esize = s->dtype == VECTOR_BF16 ? 2 : 4;
    out->scale = s->sm_scale > 0.f ? s->sm_scale : 1.0f / std::sqrt((float)s->head_dim);
    out->rope = s->rope_enabled ? 1 : 0;
    out->theta = s->rope_theta;
    return VECTOR_OK;
}

vector_status check_budget(const vector_budget* b, int window) {
    if (!b) return VECTOR_ERR_NULL;
    if (b->n_tokens <= 0 || b->n_tokens > (int64_t(1) << 30)) return VECTOR_ERR_BUDGET;
    if (b->n_a < 0 || b->n_budget_pairs < 0) return VECTOR_ERR_BUDGET;
    if (b->n_pool != b->n_budget_pairs + b->n_a || b->n_apx != 2 * b->n_a ||
        b->n_ret != b->n_budget_pairs - b->n_a || b->n_evict != b->n_tokens - b->n_pool)
        return VECTOR_ERR_BUDGET;
    if (b->n_ret < 0 || b->n_evict < 0) return VECTOR_ERR_BUDGET;
    if (window > b->n_tokens || b->n_pool < window) return VECTOR_ERR_BUDGET;
    return VECTOR_OK;
}

int score_num_chunks(int U, int R, int64_t N) {
    int64_t tiles = (N + 127) / 128;
    int64_t row_tiles = (R + 63) / 64;
    int64_t want = (8 * sm_count() + (int64_t)U * row_tiles - 1) / ((int64_t)U * row_tiles);
    if (want < 1) want = 1;
    if (want > 64) want = 64;
    if (want > tiles) want = tiles;
    return (int)want;
}

ScoreTcPlan score_tc_plan(int U, int R, int64_t N) {
    ScoreTcPlan p;
    p.RG = (R + 255) / 256;
    p.nt = (int)((N + 127) / 128);
    // chunks per unit: fill whole rounds of one block per SM, but keep chunks long enough that the
    // per-item cost (Q load, pipeline fill) stays small
    const int blocks = sm_count();
    double best = -1.0;
    int best_n = 1;
    const int max_n = p.nt < 64 ? p.nt : 64;
    for (int n = 1; n <= max_n; ++n) {
        const int tpc = (p.nt + n - 1) / n;
        const int n_eff = (p.nt + tpc - 1) / tpc;
        if (n_eff != n) continue;
        const long long items = (long long)U * p.RG * n;
        const long long rounds = (items + blocks - 1) / blocks;
        const double fill = (double)items / (double)(rounds * blocks);
        const double merit = fill * tpc / (tpc + 2.0);
        if (merit > best + 1e-9) { best = merit; best_n = n; }
    }
    p.n_chunks = best_n;
    p.tpc = (p.nt + best_n - 1) / best_n;
    p.n_items = U * p.RG * p.n_chunks;
    return p;
}

size_t score_ws_bytes(const Dims& D, int64_t N, bool need_raw) {
    if (score_uses_tc(D)) {
        const ScoreTcPlan p = score_tc_plan(D.U, D.R, N);
        return align256((size_t)D.U * 2 * p.n_chunks * D.R * 2 * sizeof(float)) + // (reference, sum) partials, two per chunk
               align256((size_t)D.U * D.R * sizeof(float)) +                        // lse
               align256((size_t)D.U * 2 * p.RG * (size_t)N * sizeof(float));        // per-row-block key sums
    }
    size_t b = 0;
    b += align256((size_t)D.U * score_num_chunks(D.U, D.R, N) * D.R * 2 * sizeof(float));  // (max, sum) partials
    b += align256((size_t)D.U * D.R * sizeof(float));                                       // lse
    if (need_raw) b += align256((size_t)D.U * (size_t)N * sizeof(float));
    return b;
}

size_t select_ws_bytes(const Dims& D, const vector_budget& b) {
    // vector_route keeps pool_idx and eps here when the caller does not ask for them
    return align256((size_t)D.U * (size_t)b.n_pool * sizeof(int32_t)) +
           align256((size_t)D.U * (size_t)b.n_pool * sizeof(float));
}

int decode_num_splits(int U, int64_t rows) {
    int64_t want = (4 * sm_count() + U - 1) / U;
    int64_t max_by_rows = (rows + 255) / 256;   // at least 256 rows per split
    if (want > max_by_rows) want = max_by_rows;
    if (want > 64) want = 64;
    if (want < 1) want = 1;
    return (int)want;
}

int decode_stream_slots(int U) {
    int s = (2 * sm_count() + U - 1) / U + 1;
    return s < 12 ? s : 12;
}

size_t decode_ws_bytes(const Dims& D) {
    // the split count never exceeds what decode_num_splits returns for an unbounded row count,
    // nor the record slots per unit of the persistent kernel
    int s = decode_num_splits(D.U, int64_t(1) << 40);
    // split kernel: per (unit, split, head) m, l, acc_v[d], acc_k[d]
    size_t a = (size_t)D.U * s * D.g * (2 + 2 * (size_t)D.d) * sizeof(float);
    // persistent kernel: per (unit, slot, consumer warp, head) a 4-float header, acc_v[128], acc_k[128]
    size_t b = (size_t)D.U * decode_stream_slots(D.U) * 4 * D.g * (4 + 256) * sizeof(float);
    return align256(a > b ? a : b);
}

}  // namespace vec

extern "C" {

const char* vector_status_string(vector_status s) {
    switch (s) {
        case VECTOR_OK: return "ok";
        case VECTOR_ERR_NULL: return "null pointer";
        case VECTOR_ERR_SHAPE: return "bad or unsupported shape";
        case VECTOR_ERR_DTYPE: return "unknown dtype";
        case VECTOR_ERR_BUDGET: return "impossible tier sizes";
        case VECTOR_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case VECTOR_ERR_SINGULAR: return "Gram matrix not positive definite";
        case VECTOR_ERR_CUDA: return "CUDA runtime error";
        case VECTOR_ERR_TIMEOUT: return "timeout";
        case VECTOR_ERR_UNSUPPORTED: return "not implemented in this build";
    }
    return "unknown status";
}

int vector_last_cuda_error(void) { return vec::g_last_cuda_error; }

uint64_t vector_kernel_launches(void) { return (uint64_t)vec::g_launches.load(std::memory_order_relaxed); }

vector_status vector_plan_budget(int64_t n_tokens, int64_t n_budget_pairs, int64_t n_a,
                                 int32_t window, vector_budget* out) {
    if (!out) return VECTOR_ERR_NULL;
    if (n_tokens <= 0 || window < 0) return VECTOR_ERR_SHAPE;
    if (n_budget_pairs < 0 || n_budget_pairs > n_tokens) return VECTOR_ERR_BUDGET;
    if (n_a < 0) {
        // Eq. (1), small constant taken as zero, in token counts
        const int64_t half_compressed = (n_tokens - n_budget_pairs) / 2;
        const int64_t half_budget = n_budget_pairs / 2;
        n_a = half_compressed < half_budget ? half_compressed : half_budget;
    }
    vector_budget b;
    b.n_tokens = n_tokens;
    b.n_budget_pairs = n_budget_pairs;
    b.n_a = n_a;
    b.n_pool = n_budget_pairs + n_a;
    b.n_apx = 2 * n_a;
    b.n_ret = n_budget_pairs - n_a;
    b.n_evict = n_tokens - b.n_pool;
    // the retention tier may be empty but not negative; the pool is at most the context
    if (b.n_ret < 0 || b.n_evict < 0) return VECTOR_ERR_BUDGET;
    if (window > n_tokens || b.n_pool < window) return VECTOR_ERR_BUDGET;
    *out = b;
    return VECTOR_OK;
}

static inline double widen(const void* p, int64_t i, int32_t dt) {
    if (dt == VECTOR_F32) return (double)((const float*)p)[i];
    uint32_t bits = (uint32_t)((const uint16_t*)p)[i] << 16;
    float f;
    std::memcpy(&f, &bits, 4);
    return (double)f;
}

vector_status vector_calibrate(const void* K, const void* V, int64_t n, int32_t d_k, int32_t d_v,
                               int32_t dt, double lambda, float* W_out, double* r2_out) {
    if (!K || !V || !W_out) return VECTOR_ERR_NULL;
    if (dt != VECTOR_F32 && dt != VECTOR_BF16) return VECTOR_ERR_DTYPE;
    if (n <= 0 || d_k <= 0 || d_v <= 0 || d_k > 1024 || d_v > 1024) return VECTOR_ERR_SHAPE;
    if (!(lambda >= 0.0)) return VECTOR_ERR_SHAPE;
    const int m = d_k + d_v;
    // M[a][0..d_k) = sum k_a k_b   (Gram);  M[a][d_k..m) = sum k_a v_c  (cross moments)
    std::vector<double> M((size_t)d_k * m, 0.0), x(m), vsum(d_v, 0.0), vsq(d_v, 0.0);
    for (int64_t t = 0; t < n; ++t) {
        for (int a = 0; a < d_k; ++a) x[a] = widen(K, t * d_k + a, dt);
        for (int c = 0; c < d_v; ++c) {
            double v = widen(V, t * d_v + c, dt);
            x[d_k + c] = v;
            vsum[c] += v;
            vsq[c] += v * v;
        }
        for (int a = 0; a < d_k; ++a) {
            const double ka = x[a];
            double* row = &M[(size_t)a * m];
            for (int j = 0; j < m; ++j) row[j] += ka * x[j];
        }
    }
    // keep the un-regularised moments for the R^2 report
    std::vector<double> G0, C0;
    if (r2_out) {
        G0.resize((size_t)d_k * d_k);
        C0.resize((size_t)d_k * d_v);
        for (int a = 0; a < d_k; ++a) {
            for (int b = 0; b < d_k; ++b) G0[(size_t)a * d_k + b] = M[(size_t)a * m + b];
            for (int c = 0; c < d_v; ++c) C0[(size_t)a * d_v + c] = M[(size_t)a * m + d_k + c];
        }
    }
    for (int a = 0; a < d_k; ++a) M[(size_t)a * m + a] += lambda;
    // Gaussian elimination without pivoting on the SPD system [G + lambda I | C^T]
    // (an outer-product Cholesky in disguise: pivots must stay positive).
    for (int p = 0; p < d_k; ++p) {
        double piv = M[(size_t)p * m + p];
        if (!(piv > 0.0) || !std::isfinite(piv)) return VECTOR_ERR_SINGULAR;
        for (int i = p + 1; i < d_k; ++i) {
            double f = M[(size_t)i * m + p] / piv;
            if (f == 0.0) continue;
            double* ri = &M[(size_t)i * m];
            const double* rp = &M[(size_t)p * m];
            for (int j = p; j < m; ++j) ri[j] -= f * rp[j];
        }
    }
    // back substitution: X = (G + lambda I)^{-1} C^T, [d_k][d_v];  W = X^T
    std::vector<double> X((size_t)d_k * d_v);
    for (int i = d_k - 1; i >= 0; --i) {
        const double* ri = &M[(size_t)i * m];
        for (int c = 0; c < d_v; ++c) {
            double r = ri[d_k + c];
            for (int j = i + 1; j < d_k; ++j) r -= ri[j] * X[(size_t)j * d_v + c];
            X[(size_t)i * d_v + c] = r / ri[i];
        }
    }
    for (int c = 0; c < d_v; ++c)
        for (int a = 0; a < d_k; ++a) W_out[(size_t)c * d_k + a] = (float)X[(size_t)a * d_v + c];
    if (r2_out) {
        // SSE = sum|v|^2 - 2 tr(W C0) + tr(W G0 W^T), with W = X^T in fp64
        double sse = 0.0, sst = 0.0;
        for (int c = 0; c < d_v; ++c) {
            double wc = 0.0, wgw = 0.0;
            for (int a = 0; a < d_k; ++a) {
                double xa = X[(size_t)a * d_v + c];
                wc += xa * C0[(size_t)a * d_v + c];
                double t = 0.0;
                for (int b = 0; b < d_k; ++b) t += G0[(size_t)a * d_k + b] * X[(size_t)b * d_v + c];
                wgw += xa * t;
            }
            sse += vsq[c] - 2.0 * wc + wgw;
            sst += vsq[c] - vsum[c] * vsum[c] / (double)n;
        }
        *r2_out = sst > 0.0 ? 1.0 - sse / sst : 0.0;
    }
    return VECTOR_OK;
}

size_t vector_workspace_bytes(const vector_shape* shape, const vector_budget* budget) {
    vec::Dims D;
    if (vec::check_shape(shape, &D) != VECTOR_OK || !budget) return 0;
    size_t a = vec::score_ws_bytes(D, budget->n_tokens, true);
    size_t b = vec::select_ws_bytes(D, *budget);
    size_t c = vec::decode_ws_bytes(D);
    size_t k = vec::keydiff_ws_bytes(D, budget->n_tokens);
    size_t r = a > b ? a : b;
    r = r > c ? r : c;
    return (r > k ? r : k) + 256;
}

}  // extern "C"
