/*
 * VECTOR oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded fp64 restatement of what the VECTOR hot path
 * computes (offline calibration, observation-window scoring, three-way routing,
 * compaction, attention over the mixed cache).  It exists so that the CUDA
 * library can be checked against something written directly from the paper's
 * definitions.  It shares no code, header, table or helper with the CUDA path;
 * only tests, the smoke check and the CPU-baseline leg of the benchmark may
 * call it.  The product must never route through it.
 *
 * Conventions (paper, Section 3.1 remark footnote): vectors are columns and a
 * linear map acts as y = W x, so W is stored row-major as W[c_out][c_in].
 * All arrays are dense row-major doubles unless noted; scores enter the routing
 * step as IEEE fp32 because that is the precision in which the kernels take the
 * top-k decisions.  Every function works on ONE unit = one (sequence, layer,
 * KV head); units are independent in every step.
 *
 * Every function is pinned by the CPU tests (closed forms, brute force,
 * invariants, special cases); none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_BUDGET -2
#define ORACLE_ERR_SINGULAR -3

typedef struct {
    int64_t n_tokens;       /* N                                   */
    int64_t n_budget_pairs; /* Bp  = (1-p_c) N full K/V pairs      */
    int64_t n_a;            /* p_a N                               */
    int64_t n_pool;         /* (1-p_c+p_a) N  = Bp + n_a           */
    int64_t n_apx;          /* 2 p_a N        = 2 n_a              */
    int64_t n_ret;          /* (1-p_c-p_a) N  = Bp - n_a           */
    int64_t n_evict;        /* (p_c-p_a) N    = N - n_pool         */
} oracle_budget;

/* Eq. (1): p_a = min(p_c/2, (1 - p_c - eps)/2), in real numbers. */
double oracle_p_a_deploy(double p_c, double eps) {
    double a = p_c / 2.0, b = (1.0 - p_c - eps) / 2.0;
    return a < b ? a : b;
}

/*
 * Section 3.2 tier sizes in integers.  Bp is the number of full pairs the
 * memory budget pays for ((1-p_c) N).  n_a < 0 asks for Eq. (1) with eps -> 0:
 * p_c N / 2 = (N-Bp)/2 and (1-p_c) N / 2 = Bp/2, each rounded down.  Everything
 * else is derived so that the memory identity of Section 3.2 (pool keys plus
 * retained values cost exactly Bp pairs: n_pool + n_ret = 2 Bp) holds exactly.
 */
int oracle_plan_budget(int64_t n_tokens, int64_t n_budget_pairs, int64_t n_a,
                       int32_t window, oracle_budget* out) {
    if (!out || n_tokens <= 0 || window < 0) return ORACLE_ERR_ARG;
    if (n_budget_pairs < 0 || n_budget_pairs > n_tokens) return ORACLE_ERR_BUDGET;
    if (n_a < 0) {
        int64_t a = (n_tokens - n_budget_pairs) / 2;
        int64_t b = n_budget_pairs / 2;
        n_a = a < b ? a : b;
    }
    /* an explicit n_a may empty the retention tier (the sensitivity sweep of Section 5.3
       reaches p_a = 0.5 at p_c = 0.5) but not make it negative, nor outgrow the context */
    if (n_a > n_budget_pairs) return ORACLE_ERR_BUDGET;
    if (n_budget_pairs + n_a > n_tokens) return ORACLE_ERR_BUDGET;
    out->n_tokens = n_tokens;
    out->n_budget_pairs = n_budget_pairs;
    out->n_a = n_a;
    out->n_pool = n_budget_pairs + n_a;
    out->n_apx = 2 * n_a;
    out->n_ret = n_budget_pairs - n_a;
    out->n_evict = n_tokens - out->n_pool;
    /* the observation window is always kept by the base scorer */
    if (window > n_tokens || out->n_pool < window) return ORACLE_ERR_BUDGET;
    return ORACLE_OK;
}

/*
 * Section 3.1, the OLS objective: W = argmin_W sum_t || W k_t - v_t ||^2, no
 * intercept, plus the ridge term lambda ||W||_F^2 the configurations ask for.
 * Normal equations: W (G + lambda I) = C with G = sum k k^T (d_k x d_k) and
 * C = sum v k^T (d_v x d_k).  Solved by Cholesky of the symmetric matrix.
 * K: [n][d_k], V: [n][d_v], W_out: [d_v][d_k].
 */
int oracle_calibrate(const double* K, const double* V, int64_t n, int32_t d_k,
                     int32_t d_v, double lambda, double* W_out) {
    if (!K || !V || !W_out || n <= 0 || d_k <= 0 || d_v <= 0) return ORACLE_ERR_ARG;
    double* G = (double*)calloc((size_t)d_k * d_k, sizeof(double));
    double* C = (double*)calloc((size_t)d_v * d_k, sizeof(double));
    if (!G || !C) { free(G); free(C); return ORACLE_ERR_ARG; }
    for (int64_t t = 0; t < n; ++t) {
        const double* k = K + t * d_k;
        const double* v = V + t * d_v;
        for (int a = 0; a < d_k; ++a)
            for (int b = 0; b < d_k; ++b) G[a * d_k + b] += k[a] * k[b];
        for (int c = 0; c < d_v; ++c)
            for (int a = 0; a < d_k; ++a) C[c * d_k + a] += v[c] * k[a];
    }
    for (int a = 0; a < d_k; ++a) G[a * d_k + a] += lambda;
    /* Cholesky G = L L^T, L stored in the lower triangle of G */
    for (int j = 0; j < d_k; ++j) {
        double s = G[j * d_k + j];
        for (int p = 0; p < j; ++p) s -= G[j * d_k + p] * G[j * d_k + p];
        if (!(s > 0.0) || !isfinite(s)) { free(G); free(C); return ORACLE_ERR_SINGULAR; }
        double ljj = sqrt(s);
        G[j * d_k + j] = ljj;
        for (int i = j + 1; i < d_k; ++i) {
            double r = G[i * d_k + j];
            for (int p = 0; p < j; ++p) r -= G[i * d_k + p] * G[j * d_k + p];
            G[i * d_k + j] = r / ljj;
        }
    }
    /* each row w of W solves (L L^T) w = c  (the matrix is symmetric) */
    for (int c = 0; c < d_v; ++c) {
        double* w = W_out + (size_t)c * d_k;
        const double* rhs = C + (size_t)c * d_k;
        for (int i = 0; i < d_k; ++i) {           /* L y = rhs */
            double r = rhs[i];
            for (int p = 0; p < i; ++p) r -= G[i * d_k + p] * w[p];
            w[i] = r / G[i * d_k + i];
        }
        for (int i = d_k - 1; i >= 0; --i) {      /* L^T x = y */
            double r = w[i];
            for (int p = i + 1; p < d_k; ++p) r -= G[p * d_k + i] * w[p];
            w[i] = r / G[i * d_k + i];
        }
    }
    free(G); free(C);
    return ORACLE_OK;
}

/*
 * Inverse rotary embedding of one key (Section 3.1, "RoPE Decoupling"): the
 * regressor sees R_m^{-1} k.  Half-split pairing: channel c pairs with c + d/2
 * and the pair is turned by the angle -m * theta^(-2c/d).
 */
void oracle_rope_inverse(const double* k, int32_t d, int64_t pos, double theta, double* out) {
    int h = d / 2;
    for (int c = 0; c < h; ++c) {
        double ang = (double)pos * pow(theta, -2.0 * (double)c / (double)d);
        double cs = cos(ang), sn = sin(ang);
        double x = k[c], y = k[c + h];
        out[c] = x * cs + y * sn;
        out[c + h] = -x * sn + y * cs;
    }
}

/* Forward rotary embedding, used only by tests and input generation checks. */
void oracle_rope_forward(const double* k, int32_t d, int64_t pos, double theta, double* out) {
    int h = d / 2;
    for (int c = 0; c < h; ++c) {
        double ang = (double)pos * pow(theta, -2.0 * (double)c / (double)d);
        double cs = cos(ang), sn = sin(ang);
        double x = k[c], y = k[c + h];
        out[c] = x * cs - y * sn;
        out[c + h] = x * sn + y * cs;
    }
}

/*
 * Base importance score (the SnapKV-style scorer the pipeline's Step 1 calls):
 * the last w queries of each of the g query heads that share this KV head
 * attend causally to all N keys; softmax over the visible keys; the attention
 * mass each key receives is summed over window rows and heads (raw); raw is
 * max-pooled along the sequence over the prefix positions i < N - w with a
 * centred kernel; the window tokens themselves get +inf (always kept).
 * Q: [g][w][d], K: [N][d]; raw_out (nullable) and score_out: [N].
 */
int oracle_score(const double* Q, const double* K, int32_t g, int32_t w, int32_t d,
                 int64_t N, double scale, int32_t pool_kernel,
                 double* raw_out, double* score_out) {
    if (!Q || !K || !score_out || g <= 0 || w <= 0 || d <= 0 || N < w) return ORACLE_ERR_ARG;
    if (pool_kernel < 1 || (pool_kernel % 2) == 0) return ORACLE_ERR_ARG;
    double* raw = (double*)calloc((size_t)N, sizeof(double));
    double* s = (double*)malloc((size_t)N * sizeof(double));
    if (!raw || !s) { free(raw); free(s); return ORACLE_ERR_ARG; }
    for (int a = 0; a < g; ++a) {
        for (int j = 0; j < w; ++j) {
            const double* q = Q + ((size_t)a * w + j) * d;
            int64_t t = N - w + j;           /* absolute position of this query */
            double m = -INFINITY;
            for (int64_t i = 0; i <= t; ++i) {
                double dot = 0.0;
                const double* k = K + i * d;
                for (int c = 0; c < d; ++c) dot += q[c] * k[c];
                s[i] = scale * dot;
                if (s[i] > m) m = s[i];
            }
            double z = 0.0;
            for (int64_t i = 0; i <= t; ++i) { s[i] = exp(s[i] - m); z += s[i]; }
            for (int64_t i = 0; i <= t; ++i) raw[i] += s[i] / z;
        }
    }
    int64_t P = N - w;                        /* prefix length */
    int r = pool_kernel / 2;
    for (int64_t i = 0; i < P; ++i) {
        double best = -INFINITY;
        for (int64_t j = i - r; j <= i + r; ++j)
            if (j >= 0 && j < P && raw[j] > best) best = raw[j];
        score_out[i] = best;
    }
    for (int64_t i = P; i < N; ++i) score_out[i] = INFINITY;
    if (raw_out) memcpy(raw_out, raw, (size_t)N * sizeof(double));
    free(raw); free(s);
    return ORACLE_OK;
}

/*
 * Query-agnostic base scorer by key geometry (the KeyDiff-style scorer the paper names among
 * the base scorers of Step 1 and describes as "key geometric diversity"; it gives no formula, so
 * this follows the published idea): the anchor is the mean of the unit-normalised keys, and a
 * token is the more important the less its key points along the anchor:
 *   a = (1/N) sum_j k_j / ||k_j||,   score_i = - <k_i, a> / (||k_i|| ||a||).
 * No observation window, no pooling.  A zero key has cosine 0 with everything (score 0); if
 * the anchor itself is zero every score is 0.  K: [N][d]; score_out: [N].
 */
int oracle_score_keydiff(const double* K, int32_t d, int64_t N, double* score_out) {
    if (!K || !score_out || d <= 0 || N <= 0) return ORACLE_ERR_ARG;
    double* a = (double*)calloc((size_t)d, sizeof(double));
    double* nrm = (double*)malloc((size_t)N * sizeof(double));
    if (!a || !nrm) { free(a); free(nrm); return ORACLE_ERR_ARG; }
    for (int64_t i = 0; i < N; ++i) {
        const double* k = K + i * d;
        double n2 = 0.0;
        for (int c = 0; c < d; ++c) n2 += k[c] * k[c];
        nrm[i] = sqrt(n2);
        if (nrm[i] > 0.0)
            for (int c = 0; c < d; ++c) a[c] += k[c] / nrm[i];
    }
    double an2 = 0.0;
    for (int c = 0; c < d; ++c) { a[c] /= (double)N; an2 += a[c] * a[c]; }
    double an = sqrt(an2);
    for (int64_t i = 0; i < N; ++i) {
        const double* k = K + i * d;
        double dot = 0.0;
        for (int c = 0; c < d; ++c) dot += k[c] * a[c];
        score_out[i] = (nrm[i] > 0.0 && an > 0.0) ? -dot / (nrm[i] * an) : 0.0;
    }
    free(a); free(nrm);
    return ORACLE_OK;
}

/* ---- routing ---- */
typedef struct { float key; int32_t idx; } f_item;
typedef struct { double key; int32_t idx; } d_item;

static int cmp_score_desc(const void* a, const void* b) {
    const f_item* x = (const f_item*)a; const f_item* y = (const f_item*)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);     /* ties: lower index first */
}
static int cmp_eps_asc(const void* a, const void* b) {
    const f_item* x = (const f_item*)a; const f_item* y = (const f_item*)b;
    if (x->key < y->key) return -1;
    if (x->key > y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}
static int cmp_int(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

/*
 * Step 1 (budget relaxation): the n_pool tokens with the largest base score,
 * ties to the lower index.  pool_idx_out: [n_pool], ascending token order.
 */
int oracle_pool_select(const float* score, int64_t N, int64_t n_pool, int32_t* pool_idx_out) {
    if (!score || !pool_idx_out || n_pool < 0 || n_pool > N) return ORACLE_ERR_ARG;
    f_item* it = (f_item*)malloc((size_t)N * sizeof(f_item));
    if (!it) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < N; ++i) { it[i].key = score[i]; it[i].idx = (int32_t)i; }
    qsort(it, (size_t)N, sizeof(f_item), cmp_score_desc);
    for (int64_t i = 0; i < n_pool; ++i) pool_idx_out[i] = it[i].idx;
    qsort(pool_idx_out, (size_t)n_pool, sizeof(int32_t), cmp_int);
    free(it);
    return ORACLE_OK;
}

/*
 * Step 2 (residual evaluation): eps_i = || v_i - W k~_i ||_2^2 for the listed
 * tokens, k~ the key itself or its inverse rotation.  K,V: [N][d]; W: [d][d]
 * (y = W x); eps_out: [n_idx] doubles in the order of idx.
 */
int oracle_residual(const double* K, const double* V, const double* W, int32_t d,
                    const int32_t* idx, int64_t n_idx, int32_t rope, double theta,
                    double* eps_out) {
    if (!K || !V || !W || !idx || !eps_out || d <= 0) return ORACLE_ERR_ARG;
    double* kt = (double*)malloc((size_t)d * sizeof(double));
    if (!kt) return ORACLE_ERR_ARG;
    for (int64_t p = 0; p < n_idx; ++p) {
        int64_t i = idx[p];
        const double* k = K + i * d;
        const double* v = V + i * d;
        if (rope) oracle_rope_inverse(k, d, i, theta, kt);
        else memcpy(kt, k, (size_t)d * sizeof(double));
        double e = 0.0;
        for (int c = 0; c < d; ++c) {
            double pred = 0.0;
            for (int c2 = 0; c2 < d; ++c2) pred += W[(size_t)c * d + c2] * kt[c2];
            double r = v[c] - pred;
            e += r * r;
        }
        eps_out[p] = e;
    }
    free(kt);
    return ORACLE_OK;
}

/*
 * Step 3 (asymmetric truncation): among the pool, the n_apx tokens with the
 * smallest eps (ties to the lower index) lose their value (tier 1); the other
 * pool tokens keep key and value (tier 2); tokens outside the pool are evicted
 * (tier 0).  eps is fp32, in the order of pool_idx.  ret_idx/apx_idx ascending.
 */
int oracle_truncate(const float* eps, const int32_t* pool_idx, int64_t n_pool, int64_t n_apx,
                    int64_t N, uint8_t* tier_out, int32_t* ret_idx_out, int32_t* apx_idx_out) {
    if (!eps || !pool_idx || !tier_out || n_apx < 0 || n_apx > n_pool) return ORACLE_ERR_ARG;
    f_item* it = (f_item*)malloc((size_t)(n_pool > 0 ? n_pool : 1) * sizeof(f_item));
    if (!it) return ORACLE_ERR_ARG;
    for (int64_t p = 0; p < n_pool; ++p) { it[p].key = eps[p]; it[p].idx = pool_idx[p]; }
    qsort(it, (size_t)n_pool, sizeof(f_item), cmp_eps_asc);
    memset(tier_out, 0, (size_t)N);
    for (int64_t p = 0; p < n_pool; ++p) tier_out[it[p].idx] = (p < n_apx) ? 1 : 2;
    int64_t nr = 0, na = 0;
    for (int64_t i = 0; i < N; ++i) {
        if (tier_out[i] == 1) { if (apx_idx_out) apx_idx_out[na] = (int32_t)i; ++na; }
        else if (tier_out[i] == 2) { if (ret_idx_out) ret_idx_out[nr] = (int32_t)i; ++nr; }
    }
    free(it);
    return (na == n_apx && nr == n_pool - n_apx) ? ORACLE_OK : ORACLE_ERR_ARG;
}

/*
 * Steps 1-3 chained.  eps is rounded to fp32 before Step 3 because that is the
 * precision in which the kernels rank residuals.  eps_out (nullable): [n_pool]
 * doubles in pool order; pool_idx_out (nullable): [n_pool].
 */
int oracle_route(const float* score, const double* K, const double* V, const double* W,
                 int64_t N, int32_t d, int64_t n_pool, int64_t n_apx, int32_t rope, double theta,
                 uint8_t* tier_out, int32_t* ret_idx_out, int32_t* apx_idx_out,
                 double* eps_out, int32_t* pool_idx_out) {
    int32_t* pool = (int32_t*)malloc((size_t)(n_pool > 0 ? n_pool : 1) * sizeof(int32_t));
    double* eps = (double*)malloc((size_t)(n_pool > 0 ? n_pool : 1) * sizeof(double));
    float* epsf = (float*)malloc((size_t)(n_pool > 0 ? n_pool : 1) * sizeof(float));
    int rc = ORACLE_ERR_ARG;
    if (pool && eps && epsf) {
        rc = oracle_pool_select(score, N, n_pool, pool);
        if (rc == ORACLE_OK) rc = oracle_residual(K, V, W, d, pool, n_pool, rope, theta, eps);
        if (rc == ORACLE_OK) {
            for (int64_t p = 0; p < n_pool; ++p) epsf[p] = (float)eps[p];
            rc = oracle_truncate(epsf, pool, n_pool, n_apx, N, tier_out, ret_idx_out, apx_idx_out);
        }
        if (rc == ORACLE_OK) {
            if (eps_out) memcpy(eps_out, eps, (size_t)n_pool * sizeof(double));
            if (pool_idx_out) memcpy(pool_idx_out, pool, (size_t)n_pool * sizeof(int32_t));
        }
    }
    free(pool); free(eps); free(epsf);
    return rc;
}

/*
 * Compaction (Section 3.2, Step 3 bullets): gather the rows named by an index
 * list; positions are the original token indices.  src: [N][d]; dst: [n_idx][d].
 */
int oracle_gather_rows(const double* src, int32_t d, const int32_t* idx, int64_t n_idx,
                       double* dst, int32_t* pos_out) {
    if (!src || !idx || !dst) return ORACLE_ERR_ARG;
    for (int64_t p = 0; p < n_idx; ++p) {
        memcpy(dst + p * d, src + (int64_t)idx[p] * d, (size_t)d * sizeof(double));
        if (pos_out) pos_out[p] = idx[p];
    }
    return ORACLE_OK;
}

/*
 * Generation-time attention over the mixed cache (Section 3.2, Step 3): one
 * softmax over the exact keys of both pools; retained tokens contribute their
 * stored value, approximated tokens the reconstruction W k~.  Two forms:
 *   per-token:  o = sum_R p_i v_i + sum_A p_i (W k~_i)
 *   factored:   o = sum_R p_i v_i + W (sum_A p_i k~_i)
 * q: [g][d]; ret_k, ret_v: [n_ret][d]; apx_k: [n_apx][d]; apx_pos: [n_apx]
 * (used only when rope != 0); out_token / out_factored (either nullable): [g][d].
 */
int oracle_attend(const double* q, int32_t g, int32_t d,
                  const double* ret_k, const double* ret_v, int64_t n_ret,
                  const double* apx_k, const int32_t* apx_pos, int64_t n_apx,
                  const double* W, double scale, int32_t rope, double theta,
                  double* out_token, double* out_factored) {
    if (!q || !W || g <= 0 || d <= 0 || n_ret < 0 || n_apx < 0 || n_ret + n_apx <= 0)
        return ORACLE_ERR_ARG;
    int64_t n = n_ret + n_apx;
    double* p = (double*)malloc((size_t)n * sizeof(double));
    double* kt = (double*)malloc((size_t)d * sizeof(double));
    double* vh = (double*)malloc((size_t)d * sizeof(double));
    double* acc = (double*)malloc((size_t)d * sizeof(double));
    if (!p || !kt || !vh || !acc) { free(p); free(kt); free(vh); free(acc); return ORACLE_ERR_ARG; }
    for (int a = 0; a < g; ++a) {
        const double* qa = q + (size_t)a * d;
        double m = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            const double* k = (i < n_ret) ? ret_k + i * d : apx_k + (i - n_ret) * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qa[c] * k[c];
            p[i] = scale * dot;
            if (p[i] > m) m = p[i];
        }
        double z = 0.0;
        for (int64_t i = 0; i < n; ++i) { p[i] = exp(p[i] - m); z += p[i]; }
        for (int64_t i = 0; i < n; ++i) p[i] /= z;

        if (out_token) {
            double* o = out_token + (size_t)a * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t i = 0; i < n_ret; ++i)
                for (int c = 0; c < d; ++c) o[c] += p[i] * ret_v[i * d + c];
            for (int64_t i = 0; i < n_apx; ++i) {
                const double* k = apx_k + i * d;
                if (rope) oracle_rope_inverse(k, d, apx_pos[i], theta, kt);
                else memcpy(kt, k, (size_t)d * sizeof(double));
                for (int c = 0; c < d; ++c) {
                    double r = 0.0;
                    for (int c2 = 0; c2 < d; ++c2) r += W[(size_t)c * d + c2] * kt[c2];
                    vh[c] = r;
                }
                for (int c = 0; c < d; ++c) o[c] += p[n_ret + i] * vh[c];
            }
        }
        if (out_factored) {
            double* o = out_factored + (size_t)a * d;
            for (int c = 0; c < d; ++c) { o[c] = 0.0; acc[c] = 0.0; }
            for (int64_t i = 0; i < n_ret; ++i)
                for (int c = 0; c < d; ++c) o[c] += p[i] * ret_v[i * d + c];
            for (int64_t i = 0; i < n_apx; ++i) {
                const double* k = apx_k + i * d;
                if (rope) oracle_rope_inverse(k, d, apx_pos[i], theta, kt);
                else memcpy(kt, k, (size_t)d * sizeof(double));
                for (int c = 0; c < d; ++c) acc[c] += p[n_ret + i] * kt[c];
            }
            for (int c = 0; c < d; ++c) {
                double r = 0.0;
                for (int c2 = 0; c2 < d; ++c2) r += W[(size_t)c * d + c2] * acc[c2];
                o[c] += r;
            }
        }
    }
    free(p); free(kt); free(vh); free(acc);
    return ORACLE_OK;
}


/*
 * The same attention with ONE map per layer (Section 5.1 "Implementation Details" calibrates the
 * map layer-wise; the Remark of Section 3.1 writes K and V as whole-layer projections): a token's
 * key and value are the concatenations over the layer's Hkv KV heads, k_i, v_i in R^{Hkv d}, and an
 * approximated token's value is W k_i with W of shape [Hkv d][Hkv d].  The tier of a token holds
 * for all heads of the layer.  Query head a belongs to KV head h = a / (Hq / Hkv); its logits use
 * slice h of the keys, its output slice h of the (stored or reconstructed) values:
 *   per-token:  o_a = sum_R p_i v_i[h] + sum_A p_i (W k_i)[h]
 *   factored:   o_a = sum_R p_i v_i[h] + W[h rows] (sum_A p_i k_i)
 * q: [Hq][d]; ret_k, ret_v: [n_ret][Hkv d]; apx_k: [n_apx][Hkv d]; outputs (either nullable): [Hq][d].
 */
int oracle_attend_layer(const double* q, int32_t Hq, int32_t Hkv, int32_t d,
                        const double* ret_k, const double* ret_v, int64_t n_ret,
                        const double* apx_k, int64_t n_apx, const double* W, double scale,
                        double* out_token, double* out_factored) {
    if (!q || !W || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || d <= 0 || n_ret < 0 || n_apx < 0 || n_ret + n_apx <= 0)
        return ORACLE_ERR_ARG;
    const int64_t n = n_ret + n_apx;
    const int64_t D = (int64_t)Hkv * d;
    const int g = Hq / Hkv;
    double* p = (double*)malloc((size_t)n * sizeof(double));
    double* acc = (double*)malloc((size_t)D * sizeof(double));
    if (!p || !acc) { free(p); free(acc); return ORACLE_ERR_ARG; }
    for (int a = 0; a < Hq; ++a) {
        const int h = a / g;
        const double* qa = q + (size_t)a * d;
        double m = -INFINITY;
        for (int64_t i = 0; i < n; ++i) {
            const double* k = ((i < n_ret) ? ret_k + i * D : apx_k + (i - n_ret) * D) + (size_t)h * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qa[c] * k[c];
            p[i] = scale * dot;
            if (p[i] > m) m = p[i];
        }
        double z = 0.0;
        for (int64_t i = 0; i < n; ++i) { p[i] = exp(p[i] - m); z += p[i]; }
        for (int64_t i = 0; i < n; ++i) p[i] /= z;
        if (out_token) {
            double* o = out_token + (size_t)a * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t i = 0; i < n_ret; ++i)
                for (int c = 0; c < d; ++c) o[c] += p[i] * ret_v[i * D + (size_t)h * d + c];
            for (int64_t i = 0; i < n_apx; ++i) {
                const double* k = apx_k + i * D;
                for (int c = 0; c < d; ++c) {
                    double r = 0.0;                 /* row h d + c of W against the whole concatenated key */
                    for (int64_t c2 = 0; c2 < D; ++c2) r += W[((size_t)h * d + c) * D + c2] * k[c2];
                    o[c] += p[n_ret + i] * r;
                }
            }
        }
        if (out_factored) {
            double* o = out_factored + (size_t)a * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t c2 = 0; c2 < D; ++c2) acc[c2] = 0.0;
            for (int64_t i = 0; i < n_ret; ++i)
                for (int c = 0; c < d; ++c) o[c] += p[i] * ret_v[i * D + (size_t)h * d + c];
            for (int64_t i = 0; i < n_apx; ++i)
                for (int64_t c2 = 0; c2 < D; ++c2) acc[c2] += p[n_ret + i] * apx_k[i * D + c2];
            for (int c = 0; c < d; ++c) {
                double r = 0.0;
                for (int64_t c2 = 0; c2 < D; ++c2) r += W[((size_t)h * d + c) * D + c2] * acc[c2];
                o[c] += r;
            }
        }
    }
    free(p); free(acc);
    return ORACLE_OK;
}

/*
 * Diagnostics of one routed unit (Section 4: the distortion measure E, R^2_approx and the
 * threshold of Proposition 1).  importance: [N] non-negative weights w_i (normalised here to sum 1);
 * tier: [N] 0 evicted / 1 approximated / 2 retained; K, V: [N][d]; W: [d][d] (y = W x).
 *   E            = sum_{evicted} w_i + sum_{approximated} w_i ||v_i - W k_i||^2 / ||v_i||^2
 *   mu_A         = mean over the approximated tokens of ||v_i - W k_i||^2 / ||v_i||^2
 *   R2_approx    = 1 - mu_A
 *   w_bar        = (1 - sum_{evicted} w_i) / (number of tokens kept in the pool)
 *   w_star       = the largest weight among the evicted tokens (the token at the eviction boundary)
 *   threshold    = w_bar / (w_star + w_bar)    (approximation pays off when R2_approx exceeds it)
 * out[8] = { E, R2_approx, mu_A, sum_evicted_w, sum_approximated_w, w_bar, w_star, threshold }.
 * A token with v = 0 counts a relative error of 0 when its residual is 0 too, else 1.
 */
int oracle_diagnostics(const double* importance, const uint8_t* tier, const double* K, const double* V,
                       const double* W, int64_t N, int32_t d, double* out) {
    if (!importance || !tier || !K || !V || !W || !out || N <= 0 || d <= 0) return ORACLE_ERR_ARG;
    double total = 0.0;
    for (int64_t i = 0; i < N; ++i) {
        if (!(importance[i] >= 0.0) || isinf(importance[i])) return ORACLE_ERR_ARG;
        total += importance[i];
    }
    if (!(total > 0.0)) return ORACLE_ERR_ARG;
    double sum_e = 0.0, sum_a = 0.0, sum_a_rel = 0.0, mu = 0.0, w_star = 0.0;
    int64_t n_a = 0, n_kept = 0;
    for (int64_t i = 0; i < N; ++i) {
        const double w = importance[i] / total;
        if (tier[i] == 0) {
            sum_e += w;
            if (w > w_star) w_star = w;
            continue;
        }
        ++n_kept;
        if (tier[i] == 1) {
            const double* k = K + i * d;
            const double* v = V + i * d;
            double r2 = 0.0, v2 = 0.0;
            for (int c = 0; c < d; ++c) {
                double pred = 0.0;
                for (int j = 0; j < d; ++j) pred += W[(size_t)c * d + j] * k[j];
                r2 += (v[c] - pred) * (v[c] - pred);
                v2 += v[c] * v[c];
            }
            const double rel = v2 > 0.0 ? r2 / v2 : (r2 > 0.0 ? 1.0 : 0.0);
            sum_a += w;
            sum_a_rel += w * rel;
            mu += rel;
            ++n_a;
        }
    }
    mu = n_a > 0 ? mu / (double)n_a : 0.0;
    const double w_bar = n_kept > 0 ? (1.0 - sum_e) / (double)n_kept : 0.0;
    out[0] = sum_e + sum_a_rel;
    out[1] = 1.0 - mu;
    out[2] = mu;
    out[3] = sum_e;
    out[4] = sum_a;
    out[5] = w_bar;
    out[6] = w_star;
    out[7] = (w_star + w_bar) > 0.0 ? w_bar / (w_star + w_bar) : 0.0;
    return ORACLE_OK;
}
