"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Each test compares the oracle with something it did not compute itself: numbers
the paper prints, closed forms, brute force built from library routines
(scipy softmax, numpy lstsq, maximum_filter1d, stable argsort), invariants and
special cases.  A plausible slip in the oracle (dropped term, wrong sign or
index, transposed operand, off-by-one in the causal mask or the pooling window)
fails at least one of them.
"""
import os

import numpy as np
import pytest
from scipy.ndimage import maximum_filter1d
from scipy.special import softmax
from scipy.stats import norm

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


# --------------------------------------------------------------------------- plan
def test_p_a_matches_printed_table(oracle):
    # Section 5.1 / Appendix C.1 print the four values that Eq. (1) gives.
    for p_c, p_a in _rows("p_a_table.txt"):
        assert oracle.p_a_deploy(p_c, 0.0) == pytest.approx(p_a, abs=1e-12)
    # the small constant of Eq. (1) only ever lowers the second branch
    assert oracle.p_a_deploy(0.9, 0.01) == pytest.approx(0.045, abs=1e-12)
    assert oracle.p_a_deploy(0.25, 0.01) == pytest.approx(0.125, abs=1e-12)


def test_integer_plan_reproduces_proportions(oracle):
    N = 8000  # every proportion below is an integer at this N
    for p_c, p_a, ev, ap, re, keys, vals in _rows("tier_proportions.txt"):
        Bp = round((1 - p_c) * N)
        b = oracle.plan_budget(N, Bp, -1, 0)
        assert b.n_a == round(p_a * N)
        assert b.n_evict == round(ev * N)
        assert b.n_apx == round(ap * N)
        assert b.n_ret == round(re * N)
        assert b.n_pool == round(keys * N)
        assert b.n_ret == round(vals * N)


@pytest.mark.parametrize("N,pct", [(1024, 25), (8192, 10), (8192, 20), (8192, 40), (32768, 20),
                                   (16384, 10), (131072, 5), (1000, 33), (77, 50), (5, 100)])
def test_memory_identity_and_partition(oracle, N, pct):
    Bp = oracle.budget_pairs(N, pct)
    b = oracle.plan_budget(N, Bp, -1, 0)
    # keys of the pool + values of the retained tokens = 2 Bp vectors = Bp pairs
    assert b.n_pool + b.n_ret == 2 * Bp
    assert 2 * b.n_ret + b.n_apx == 2 * Bp
    assert b.n_evict + b.n_apx + b.n_ret == N
    assert b.n_apx == 2 * b.n_a and b.n_pool == Bp + b.n_a
    assert 2 * b.n_a <= Bp and b.n_pool <= N           # both branches of Eq. (1)
    assert b.n_a == min((N - Bp) // 2, Bp // 2)


def test_plan_sizes_of_benchmark_configs(oracle):
    want = {(1024, 25): (256, 128, 384, 256, 128, 640),
            (8192, 10): (819, 409, 1228, 818, 410, 6964),
            (32768, 20): (6553, 3276, 9829, 6552, 3277, 22939),
            (16384, 10): (1638, 819, 2457, 1638, 819, 13927),
            (131072, 5): (6553, 3276, 9829, 6552, 3277, 121243)}
    for (N, pct), (Bp, na, npool, napx, nret, nev) in want.items():
        b = oracle.plan_budget(N, oracle.budget_pairs(N, pct), -1, 64)
        assert (b.n_budget_pairs, b.n_a, b.n_pool, b.n_apx, b.n_ret, b.n_evict) == \
               (Bp, na, npool, napx, nret, nev)


def test_plan_rejects_impossible_budgets(oracle):
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(100, 101, -1, 0)          # more pairs than tokens
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(100, 10, 11, 0)           # more approximated pairs than the budget holds
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(100, 90, 20, 0)           # pool larger than the context
    with pytest.raises(oracle.OracleError):
        oracle.plan_budget(100, 10, -1, 32)          # pool smaller than the window
    assert oracle.plan_budget(100, 10, 0, 8).n_apx == 0
    # Section 5.3 sweeps p_a up to 0.5 at p_c = 0.5: everything approximated, nothing retained
    b = oracle.plan_budget(100, 50, 50, 0)
    assert (b.n_pool, b.n_apx, b.n_ret, b.n_evict) == (100, 100, 0, 0)


# ---------------------------------------------------------------------- calibrate
def _kv(rng, n, dk, dv, noise):
    K = rng.normal(size=(n, dk)) * np.exp(rng.uniform(np.log(0.5), np.log(4), size=dk))
    Wt = rng.normal(size=(dv, dk)) / np.sqrt(dk)
    V = K @ Wt.T + noise * rng.normal(size=(n, dv))
    return K, V, Wt


def test_calibrate_recovers_noise_free_map(oracle):
    rng = np.random.default_rng(1)
    K, V, Wt = _kv(rng, 4096, 24, 16, 0.0)
    W = oracle.calibrate(K, V, 1e-4)
    assert W.shape == (16, 24)                         # y = W x: [d_v][d_k], not transposed
    assert np.max(np.abs(W - Wt)) < 1e-6


def test_calibrate_matches_lstsq_and_normal_equation_identity(oracle):
    rng = np.random.default_rng(2)
    n, dk, dv, lam = 600, 12, 9, 0.37
    K, V, _ = _kv(rng, n, dk, dv, 0.8)
    V = V + 3.0                                        # a constant offset: no intercept is fitted
    W = oracle.calibrate(K, V, lam)
    # ridge as an augmented least-squares problem, solved by LAPACK's SVD routine
    A = np.vstack([K, np.sqrt(lam) * np.eye(dk)])
    Bm = np.vstack([V, np.zeros((dk, dv))])
    X, *_ = np.linalg.lstsq(A, Bm, rcond=None)         # K X ~ V  ->  W = X^T
    assert np.allclose(W, X.T, rtol=1e-9, atol=1e-10)
    # stationarity: sum (v - W k) k^T = lambda W
    R = V - K @ W.T
    assert np.allclose(R.T @ K, lam * W, rtol=1e-8, atol=1e-8)
    # and it is NOT the centred (with-intercept) solution
    Kc, Vc = K - K.mean(0), V - V.mean(0)
    Xc, *_ = np.linalg.lstsq(np.vstack([Kc, np.sqrt(lam) * np.eye(dk)]),
                             np.vstack([Vc, np.zeros((dk, dv))]), rcond=None)
    assert np.max(np.abs(W - Xc.T)) > 1e-3


def test_calibrate_singular_without_ridge(oracle):
    K = np.random.default_rng(4).normal(size=(50, 4))
    K[:, 2] = 0.0                                      # a dead channel: exact zero pivot
    V = np.ones((50, 3))
    with pytest.raises(oracle.OracleError) as e:
        oracle.calibrate(K, V, 0.0)
    assert e.value.code == oracle.ERR_SINGULAR
    oracle.calibrate(K, V, 1e-3)                       # ridge makes it solvable


def test_calibrate_r2_of_generator(oracle):
    # V = K W^T + sigma z: the fitted map explains Var(KW)/(Var(KW)+sigma^2) of the variance
    rng = np.random.default_rng(3)
    K, V, Wt = _kv(rng, 20000, 16, 16, 1.0)
    W = oracle.calibrate(K, V, 1e-4)
    sse = np.sum((V - K @ W.T) ** 2)
    sst = np.sum((V - V.mean(0)) ** 2)
    sig = np.sum(np.var(K @ Wt.T, axis=0))
    assert 1 - sse / sst == pytest.approx(sig / (sig + 16 * 1.0), abs=0.01)


def test_r2_global_against_library_and_closed_forms(oracle):
    from sklearn.metrics import r2_score
    rng = np.random.default_rng(31)
    K, V, Wt = _kv(rng, 700, 16, 16, 0.7)
    V = V + 3.0                                         # a mean the total sum of squares must remove
    W = rng.standard_normal((16, 16)) * 0.3
    r = oracle.r2_global(K, V, W)
    # the library's variance-weighted multi-output R^2 is the same ratio of sums
    assert r["r2"] == pytest.approx(r2_score(V, K @ W.T, multioutput="variance_weighted"), abs=1e-12)
    assert r["n"] == 700
    # exact map: 1; zero map: 1 - sum||v||^2 / SS_tot, below zero once the mean is not
    assert oracle.r2_global(K, K @ W.T, W)["r2"] == pytest.approx(1.0, abs=1e-12)
    z = oracle.r2_global(K, V, np.zeros((16, 16)))
    assert z["ss_res"] == pytest.approx(np.sum(V * V)) and z["r2"] < 0
    # a transposed map is a different, worse predictor
    assert oracle.r2_global(K, K @ W.T, W.T)["r2"] < 0.9
    # on its own calibration samples the least-squares fit without intercept explains what the generator puts in
    Kc, Vc, Wc = _kv(rng, 20000, 16, 16, 1.0)
    sig = np.sum(np.var(Kc @ Wc.T, axis=0))
    assert oracle.r2_global(Kc, Vc, oracle.calibrate(Kc, Vc, 1e-4))["r2"] == pytest.approx(sig / (sig + 16.0), abs=0.01)
    # constant values: nothing to explain
    assert oracle.r2_global(K, np.ones((700, 16)), np.zeros((16, 16)))["r2"] == -np.inf


# -------------------------------------------------------------------------- score
def _brute_raw(Q, K, scale):
    """Full causal attention over all N positions with a library softmax; only
    the last w rows are real queries, taken from the window."""
    g, w, d = Q.shape
    N = K.shape[0]
    raw = np.zeros(N)
    mask = np.tril(np.ones((N, N), dtype=bool))        # row t sees keys <= t
    for a in range(g):
        Qfull = np.zeros((N, d))
        Qfull[N - w:] = Q[a]
        S = scale * (Qfull @ K.T)
        S[~mask] = -np.inf
        A = softmax(S, axis=1)
        raw += A[N - w:].sum(axis=0)
    return raw


def _pool_ref(raw, N, w, kernel):
    pre = raw[:N - w]
    pooled = maximum_filter1d(pre, size=kernel, mode="constant", cval=-np.inf)
    return np.concatenate([pooled, np.full(w, np.inf)])


@pytest.mark.parametrize("g,w,d,N,kernel", [(2, 4, 8, 37, 7), (1, 3, 5, 16, 3), (3, 8, 16, 64, 5),
                                            (2, 5, 4, 5, 7), (2, 5, 4, 8, 7)])
def test_score_against_brute_force(oracle, g, w, d, N, kernel):
    rng = np.random.default_rng(10 + N)
    Q = rng.normal(size=(g, w, d)) * 1.5
    K = rng.normal(size=(N, d)) * 1.5
    scale = 1 / np.sqrt(d)
    raw, sc = oracle.score(Q, K, scale, kernel)
    ref = _brute_raw(Q, K, scale)
    assert np.allclose(raw, ref, rtol=1e-11, atol=1e-14)
    assert np.sum(raw) == pytest.approx(g * w, rel=1e-12)        # every softmax row sums to one
    want = _pool_ref(ref, N, w, kernel)
    assert np.array_equal(np.isinf(sc), np.isinf(want))
    assert np.allclose(sc[:N - w], want[:N - w], rtol=1e-11, atol=1e-14)
    assert np.all(sc[N - w:] == np.inf)


def test_score_zero_queries_closed_form(oracle):
    # with q = 0 every visible key gets 1/(t+1) from the row at position t
    g, w, d, N = 3, 6, 4, 40
    K = np.random.default_rng(0).normal(size=(N, d))
    raw, _ = oracle.score(np.zeros((g, w, d)), K, 0.5, 1)
    t = np.arange(N - w, N)
    want = np.array([g * np.sum(1.0 / (t[t >= i] + 1)) for i in range(N)])
    assert np.allclose(raw, want, rtol=1e-13)


def test_score_kernel_one_is_identity_and_single_row_is_softmax(oracle):
    rng = np.random.default_rng(5)
    Q = rng.normal(size=(1, 1, 8))
    K = rng.normal(size=(33, 8))
    raw, sc = oracle.score(Q, K, 0.3, 1)
    assert np.allclose(raw, softmax(0.3 * (K @ Q[0, 0])), rtol=1e-12)
    assert np.array_equal(sc[:32], raw[:32]) and sc[32] == np.inf


def test_score_scale_and_causality_matter(oracle):
    # the last window row sees every key, the first window row does not see later window keys
    rng = np.random.default_rng(6)
    g, w, d, N = 1, 4, 8, 12
    Q = rng.normal(size=(g, w, d))
    K = rng.normal(size=(N, d))
    raw, _ = oracle.score(Q, K, 1.0, 1)
    K2 = K.copy()
    K2[N - 1] += 100.0 * Q[0, 0]       # only row w-1 can see the last key
    raw2, _ = oracle.score(Q, K2, 1.0, 1)
    row0 = softmax(K[:N - w + 1] @ Q[0, 0])
    row0_2 = softmax(K2[:N - w + 1] @ Q[0, 0])
    assert np.allclose(row0, row0_2)
    assert raw2[N - 1] != pytest.approx(raw[N - 1])


# -------------------------------------------------------------------------- route
def test_pool_select_is_stable_topk(oracle):
    rng = np.random.default_rng(7)
    s = rng.integers(0, 6, size=200).astype(np.float32)     # many ties
    s[[5, 17]] = np.inf
    for k in (0, 1, 2, 3, 50, 199, 200):
        got = oracle.pool_select(s, k)
        want = np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:k])
        assert np.array_equal(got, want)


def test_residual_against_numpy_and_exact_zero(oracle):
    rng = np.random.default_rng(8)
    N, d = 50, 6
    K = rng.integers(-3, 4, size=(N, d)).astype(np.float64)
    W = rng.integers(-2, 3, size=(d, d)).astype(np.float64)      # not symmetric
    idx = np.array([3, 0, 49, 7, 7], dtype=np.int32)
    V = K @ W.T
    assert np.all(oracle.residual(K, V, W, idx) == 0.0)
    V2 = V + rng.normal(size=V.shape)
    want = np.sum((V2[idx] - np.einsum("ce,ne->nc", W, K[idx])) ** 2, axis=1)
    assert np.allclose(oracle.residual(K, V2, W, idx), want, rtol=1e-13)
    # a transposed map must not pass
    assert not np.allclose(oracle.residual(K, V2, W.T.copy(), idx), want)


def test_truncate_orders_by_residual_with_index_ties(oracle):
    pool = np.array([2, 5, 6, 9, 11, 20], dtype=np.int32)
    eps = np.array([0.5, 0.1, 0.5, 0.1, 0.9, 0.5], dtype=np.float32)
    tier, ret, apx = oracle.truncate(eps, pool, 3, 24)
    # two 0.1's first, then the 0.5 with the lowest token index
    assert apx.tolist() == [2, 5, 9] and ret.tolist() == [6, 11, 20]
    want = np.zeros(24, np.uint8)
    want[[2, 5, 9]] = 1
    want[[6, 11, 20]] = 2
    assert np.array_equal(tier, want)


def _route_case(rng, N, d, noise):
    K = rng.normal(size=(N, d))
    Wt = rng.normal(size=(d, d)) / np.sqrt(d)
    V = K @ Wt.T + noise * rng.normal(size=(N, 1)) * rng.normal(size=(N, d))
    s = rng.random(N).astype(np.float32)
    return K, V, Wt, s


def test_route_invariants_and_full_sort(oracle):
    rng = np.random.default_rng(9)
    N, d = 300, 8
    K, V, W, s = _route_case(rng, N, d, 1.0)
    s[rng.integers(0, N, 60)] = 0.25                      # ties in the base score
    b = oracle.plan_budget(N, 90, -1, 0)
    r = oracle.route(s, K, V, W, b.n_pool, b.n_apx)
    pool, ret, apx = r["pool_idx"], r["ret_idx"], r["apx_idx"]
    assert len(ret) == b.n_ret and len(apx) == b.n_apx
    assert 2 * len(ret) + len(apx) == 2 * b.n_budget_pairs          # budget in K/V vectors
    assert np.array_equal(np.sort(np.concatenate([ret, apx])), pool)
    assert len(np.intersect1d(ret, apx)) == 0
    assert np.all(np.diff(ret) > 0) and np.all(np.diff(apx) > 0)
    # Step 1 by an independent stable sort
    assert np.array_equal(pool, np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:b.n_pool]))
    # Step 2/3 by an independent computation and sort on fp32 residuals
    eps = np.sum((V[pool] - K[pool] @ W.T) ** 2, axis=1)
    assert np.allclose(r["eps"], eps, rtol=1e-12)
    order = np.lexsort((pool, eps.astype(np.float32)))
    assert np.array_equal(apx, np.sort(pool[order[:b.n_apx]]))
    assert eps[np.isin(pool, apx)].max() <= eps[np.isin(pool, ret)].min()
    tier = r["tier"]
    assert np.all(tier[apx] == 1) and np.all(tier[ret] == 2) and tier.sum() == len(apx) + 2 * len(ret)


def test_route_without_approximation_is_plain_eviction(oracle):
    rng = np.random.default_rng(11)
    N, d = 128, 4
    K, V, W, s = _route_case(rng, N, d, 1.0)
    b = oracle.plan_budget(N, 40, 0, 0)
    r = oracle.route(s, K, V, W, b.n_pool, b.n_apx)
    assert len(r["apx_idx"]) == 0
    assert np.array_equal(r["ret_idx"], np.sort(np.argsort(-s.astype(np.float64), kind="stable")[:40]))
    assert set(np.unique(r["tier"])) == {0, 2}


def test_route_gaussian_residuals_match_example_1(oracle):
    # scalar residuals r ~ N(0, sigma^2), eps = r^2 (d = 1, W = 0, v = r): the mean
    # residual inside the approximated set follows Example 1's truncated-normal expression
    rng = np.random.default_rng(42)
    N, sigma = 200000, 1.7
    for p_c, p_a, f, z, factor in _rows("example1_factor.txt"):
        zz = norm.ppf(0.5 + p_a / (1 - p_c + p_a))
        ff = 2 * p_a / (1 - p_c + p_a)
        closed = 1 - 2 * zz * norm.pdf(zz) / ff
        assert closed == pytest.approx(factor, abs=1e-5) and zz == pytest.approx(z, abs=1e-5)
        K = np.zeros((N, 1))
        V = sigma * rng.normal(size=(N, 1))
        s = rng.random(N).astype(np.float32)              # importance independent of residual
        b = oracle.plan_budget(N, round((1 - p_c) * N), round(p_a * N), 0)
        r = oracle.route(s, K, V, np.zeros((1, 1)), b.n_pool, b.n_apx)
        got = np.mean(V[r["apx_idx"], 0] ** 2) / sigma ** 2
        assert got == pytest.approx(closed, abs=4.0 / np.sqrt(b.n_apx))
        # the approximated set is the central part: its largest |r| is about eta = sigma z
        assert np.max(np.abs(V[r["apx_idx"], 0])) / sigma == pytest.approx(zz, abs=0.02)


def test_rope_inverse_properties(oracle):
    rng = np.random.default_rng(12)
    k = rng.normal(size=16)
    assert np.allclose(oracle.rope_inverse(k, 0), k)
    for pos in (1, 17, 4095):
        kr = oracle.rope_forward(k, pos, 10000.0)
        assert np.allclose(oracle.rope_inverse(kr, pos, 10000.0), k, atol=1e-12)
        assert np.linalg.norm(kr) == pytest.approx(np.linalg.norm(k))
    # d = 2: a single pair turned by the angle pos * theta^0 = pos radians
    out = oracle.rope_forward(np.array([1.0, 0.0]), 1, 10000.0)
    assert np.allclose(out, [np.cos(1.0), np.sin(1.0)])
    # channel c uses the angle pos * theta^(-2c/d), pairing c with c + d/2
    d, theta, pos = 8, 100.0, 3
    e = np.zeros(d)
    e[2] = 1.0
    ang = pos * theta ** (-2 * 2 / d)
    want = np.zeros(d)
    want[2], want[2 + d // 2] = np.cos(ang), np.sin(ang)
    assert np.allclose(oracle.rope_forward(e, pos, theta), want)
    # residual with rope: keys rotated by their position, map fitted on unrotated keys
    N, d = 20, 8
    K0 = rng.normal(size=(N, d))
    W = rng.normal(size=(d, d))
    V = K0 @ W.T
    Kr = np.stack([oracle.rope_forward(K0[i], i, 500.0) for i in range(N)])
    idx = np.arange(N, dtype=np.int32)
    assert np.max(oracle.residual(Kr, V, W, idx, rope=True, theta=500.0)) < 1e-20
    assert np.max(oracle.residual(Kr, V, W, idx, rope=False)) > 1e-3


# ------------------------------------------------------------------------- attend
def _attn_ref(q, k, v, scale):
    return softmax(scale * (q @ k.T), axis=1) @ v


def test_attend_without_approximation_is_textbook_attention(oracle):
    rng = np.random.default_rng(13)
    g, d, n = 3, 8, 40
    q, k, v = rng.normal(size=(g, d)), rng.normal(size=(n, d)), rng.normal(size=(n, d))
    W = rng.normal(size=(d, d))
    o1, o2 = oracle.attend(q, k, v, np.zeros((0, d)), W, 0.4)
    ref = _attn_ref(q, k, v, 0.4)
    assert np.allclose(o1, ref, rtol=1e-12, atol=1e-14) and np.allclose(o2, ref, rtol=1e-12, atol=1e-14)


def test_attend_exact_recovery_when_values_are_linear_in_keys(oracle):
    rng = np.random.default_rng(14)
    g, d, n = 2, 8, 60
    q, k = rng.normal(size=(g, d)), rng.normal(size=(n, d))
    W = rng.normal(size=(d, d)) / np.sqrt(d)
    v = k @ W.T
    ref = _attn_ref(q, k, v, 0.35)
    for n_ret in (0, 1, 17, 59, 60):                    # whatever the tier split
        o1, o2 = oracle.attend(q, k[:n_ret], v[:n_ret], k[n_ret:], W, 0.35)
        assert np.allclose(o1, ref, rtol=1e-11, atol=1e-13)
        assert np.allclose(o2, ref, rtol=1e-11, atol=1e-13)


def test_attend_general_case_against_materialised_values(oracle):
    rng = np.random.default_rng(15)
    g, d, nr, na = 4, 16, 33, 21
    q = rng.normal(size=(g, d))
    rk, rv, ak = rng.normal(size=(nr, d)), rng.normal(size=(nr, d)), rng.normal(size=(na, d))
    W = rng.normal(size=(d, d))                          # not symmetric: W vs W^T differ
    ref = _attn_ref(q, np.vstack([rk, ak]), np.vstack([rv, ak @ W.T]), 0.25)
    o1, o2 = oracle.attend(q, rk, rv, ak, W, 0.25)
    assert np.allclose(o1, ref, rtol=1e-11, atol=1e-13)
    assert np.max(np.abs(o1 - o2)) <= 1e-12 * np.max(np.abs(ref))     # factored == per token
    # zero map: approximated tokens only enlarge the softmax denominator
    z1, _ = oracle.attend(q, rk, rv, ak, np.zeros((d, d)), 0.25)
    P = softmax(0.25 * (q @ np.vstack([rk, ak]).T), axis=1)
    assert np.allclose(z1, P[:, :nr] @ rv, rtol=1e-11, atol=1e-13)
    # order inside the pools does not matter
    pr, pa = rng.permutation(nr), rng.permutation(na)
    p1, _ = oracle.attend(q, rk[pr], rv[pr], ak[pa], W, 0.25)
    assert np.allclose(p1, o1, rtol=1e-11, atol=1e-13)
    # one approximated key alone: the output is its reconstructed value
    s1, s2 = oracle.attend(q, np.zeros((0, d)), np.zeros((0, d)), ak[:1], W, 0.25)
    assert np.allclose(s1, np.tile(W @ ak[0], (g, 1))) and np.allclose(s2, s1)


def test_attend_with_rope_uses_unrotated_keys_for_values_only(oracle):
    rng = np.random.default_rng(16)
    g, d, na, theta = 2, 8, 12, 1000.0
    q = rng.normal(size=(g, d))
    k0 = rng.normal(size=(na, d))
    pos = rng.permutation(200)[:na].astype(np.int32)
    kr = np.stack([oracle.rope_forward(k0[i], int(pos[i]), theta) for i in range(na)])
    W = rng.normal(size=(d, d))
    # logits use the stored (rotated) keys, values the map applied to the unrotated ones
    ref = _attn_ref(q, kr, k0 @ W.T, 0.3)
    o1, o2 = oracle.attend(q, np.zeros((0, d)), np.zeros((0, d)), kr, W, 0.3, apx_pos=pos,
                           rope=True, theta=theta)
    assert np.allclose(o1, ref, rtol=1e-10, atol=1e-12) and np.allclose(o2, ref, rtol=1e-10, atol=1e-12)


def test_end_to_end_no_eviction_noise_free_equals_uncompressed(oracle):
    rng = np.random.default_rng(17)
    g, w, d, N = 2, 4, 8, 48
    Q = rng.normal(size=(g, w, d))
    K = rng.normal(size=(N, d))
    Wt = rng.normal(size=(d, d)) / np.sqrt(d)
    V = K @ Wt.T
    W = oracle.calibrate(K, V, 1e-10)
    _, sc = oracle.score(Q, K, 1 / np.sqrt(d), 7)
    # n_pool = N: Bp + n_a = N with n_apx = 2 n_a <= Bp
    b = oracle.plan_budget(N, 32, 16, w)
    assert b.n_pool == N
    r = oracle.route(sc.astype(np.float32), K, V, W, b.n_pool, b.n_apx)
    rk, rpos = oracle.gather_rows(K, r["ret_idx"])
    rv, _ = oracle.gather_rows(V, r["ret_idx"])
    ak, apos = oracle.gather_rows(K, r["apx_idx"])
    assert np.array_equal(rk, K[r["ret_idx"]]) and np.array_equal(rpos, r["ret_idx"])
    assert np.array_equal(ak, K[r["apx_idx"]]) and np.array_equal(apos, r["apx_idx"])
    q = rng.normal(size=(g, d))
    o1, o2 = oracle.attend(q, rk, rv, ak, W, 1 / np.sqrt(d))
    ref = _attn_ref(q, K, V, 1 / np.sqrt(d))
    assert np.allclose(o1, ref, atol=1e-7) and np.allclose(o2, ref, atol=1e-7)


def test_keydiff_scorer_pins(oracle):
    """The key-geometry scorer against what its definition fixes (none of these retypes the formula):
    identical keys all sit on the anchor; two unit keys at angle t are bisected by it; scores do not
    change when keys are rescaled or reordered; an isolated direction scores highest; the range is [-1, 1]."""
    rng = np.random.default_rng(3)
    d = 16
    k = rng.standard_normal(d)
    same = np.tile(k, (9, 1)) * rng.uniform(0.1, 5.0, size=(9, 1))          # same direction, different lengths
    assert np.allclose(oracle.score_keydiff(same), -1.0, atol=1e-12)
    for t in (0.3, 1.0, 2.5):
        two = np.zeros((2, d)); two[0, 0] = 1.0; two[1, 0], two[1, 1] = np.cos(t), np.sin(t)
        assert np.allclose(oracle.score_keydiff(two), -np.cos(t / 2), atol=1e-12)
    K = rng.standard_normal((200, d)) + 2.0 * k                              # a cloud around one direction
    s0 = oracle.score_keydiff(K)
    assert np.all(s0 >= -1 - 1e-12) and np.all(s0 <= 1 + 1e-12)
    scale = rng.uniform(0.01, 100.0, size=(200, 1))
    assert np.allclose(oracle.score_keydiff(K * scale), s0, atol=1e-10)      # lengths do not matter
    perm = rng.permutation(200)
    assert np.allclose(oracle.score_keydiff(K[perm]), s0[perm], atol=1e-12)  # order does not matter
    K2 = K.copy(); K2[17] = -3.0 * k                                         # one key pointing the other way
    s2 = oracle.score_keydiff(K2)
    assert int(np.argmax(s2)) == 17 and s2[17] > 0.9
    # rotating every key by one orthogonal map leaves all cosines unchanged
    Qm, _ = np.linalg.qr(rng.standard_normal((d, d)))
    assert np.allclose(oracle.score_keydiff(K @ Qm.T), s0, atol=1e-10)
    # a zero key is orthogonal to everything; antipodal pairs cancel the anchor
    K3 = K.copy(); K3[5] = 0.0
    assert oracle.score_keydiff(K3)[5] == 0.0
    assert np.all(oracle.score_keydiff(np.stack([k, -k])) == 0.0)


def test_diagnostics_pins(oracle):
    """Distortion measure and Proposition 1's threshold (Section 4) on cases worked by hand."""
    rng = np.random.default_rng(5)
    d = 8
    K = rng.standard_normal((4, d)); Wm = rng.standard_normal((d, d)) / 3
    w = np.array([0.4, 0.3, 0.2, 0.1])
    tier = np.array([2, 1, 1, 0], dtype=np.uint8)          # retained, approximated x2, evicted
    # exact reconstruction: approximated tokens cost nothing
    r = oracle.diagnostics(w, tier, K, K @ Wm.T, Wm)
    assert r["E"] == pytest.approx(0.1) and r["r2_approx"] == pytest.approx(1.0) and r["mu_a"] == pytest.approx(0.0, abs=1e-28)
    assert r["sum_evicted_w"] == pytest.approx(0.1) and r["sum_approximated_w"] == pytest.approx(0.5)
    assert r["w_bar"] == pytest.approx(0.9 / 3) and r["w_star"] == pytest.approx(0.1)
    assert r["threshold"] == pytest.approx(0.3 / 0.4)      # w_bar / (w_star + w_bar) = 0.75
    # a zero map reconstructs nothing: every approximated token counts like an evicted one
    V = rng.standard_normal((4, d))
    r0 = oracle.diagnostics(w, tier, K, V, np.zeros((d, d)))
    assert r0["E"] == pytest.approx(0.1 + 0.5) and r0["r2_approx"] == pytest.approx(0.0) and r0["mu_a"] == pytest.approx(1.0)
    # one approximated token with a residual of known relative size: v = W k + t * u with u orthogonal to W k
    k = K[1]; p = Wm @ k
    u = rng.standard_normal(d); u -= u @ p / (p @ p) * p; u *= np.linalg.norm(p) / np.linalg.norm(u)
    V2 = K @ Wm.T; V2[1] = p + 0.5 * u                       # ||r||^2 / ||v||^2 = 0.25 / 1.25 = 0.2
    r2 = oracle.diagnostics(w, tier, K, V2, Wm)
    assert r2["mu_a"] == pytest.approx(0.1) and r2["E"] == pytest.approx(0.1 + 0.3 * 0.2)
    # importance is normalised; no approximation tier -> E is the evicted mass; no eviction -> w_star = 0, threshold 1
    assert oracle.diagnostics(7.0 * w, tier, K, V2, Wm) == pytest.approx(r2)
    r3 = oracle.diagnostics(w, np.array([2, 2, 0, 0], dtype=np.uint8), K, V, Wm)
    assert r3["E"] == pytest.approx(0.3) and r3["sum_approximated_w"] == 0.0 and r3["r2_approx"] == 1.0
    r4 = oracle.diagnostics(w, np.array([2, 1, 1, 2], dtype=np.uint8), K, V2, Wm)
    assert r4["w_star"] == 0.0 and r4["threshold"] == pytest.approx(1.0) and r4["w_bar"] == pytest.approx(0.25)


# ---- one map per layer (Section 5.1: the map is calibrated layer-wise; Section 3.1 Remark: K and V as
#      whole-layer projections): keys and values concatenated over the layer's KV heads
def _layer_case(rng, Hkv=3, d=8, N=40, g=2):
    K = rng.standard_normal((Hkv, N, d))
    V = rng.standard_normal((Hkv, N, d))
    W = rng.standard_normal((Hkv * d, Hkv * d)) / np.sqrt(Hkv * d)
    q = rng.standard_normal((Hkv * g, d))
    return K, V, W, q


def test_layer_map_block_diagonal_reduces_to_the_per_head_maps(oracle):
    """With no cross-head blocks the whole-layer residual is the sum of the per-head residuals and the
    whole-layer attention is the per-head attention over the shared token sets."""
    rng = np.random.default_rng(11)
    Hkv, d, N, g = 3, 8, 40, 2
    K, V, _, q = _layer_case(rng, Hkv, d, N, g)
    blocks = rng.standard_normal((Hkv, d, d)) / np.sqrt(d)
    W = np.zeros((Hkv * d, Hkv * d))
    for h in range(Hkv):
        W[h * d:(h + 1) * d, h * d:(h + 1) * d] = blocks[h]
    idx = np.array([0, 3, 4, 17, 39], dtype=np.int32)
    want = sum(oracle.residual(K[h], V[h], blocks[h], idx) for h in range(Hkv))
    assert np.allclose(oracle.residual_layer(K, V, W, idx), want, rtol=1e-12)
    ret, apx = np.arange(0, 15), np.arange(20, 40)
    o_tok, o_fac = oracle.attend_layer(q, K[:, ret], V[:, ret], K[:, apx], W, 0.3)
    for h in range(Hkv):
        per_tok, _ = oracle.attend(q[h * g:(h + 1) * g], K[h, ret], V[h, ret], K[h, apx], blocks[h], 0.3)
        assert np.allclose(o_tok[h * g:(h + 1) * g], per_tok, rtol=1e-11, atol=1e-13)
    assert np.allclose(o_tok, o_fac, rtol=1e-11, atol=1e-13)


def test_layer_map_against_numpy_with_cross_head_blocks(oracle):
    """Residual and attention re-derived with einsum / a library softmax; a map whose cross-head blocks were
    dropped, or that was applied transposed, gives something else."""
    rng = np.random.default_rng(12)
    Hkv, d, N, g = 2, 8, 30, 3
    K, V, W, q = _layer_case(rng, Hkv, d, N, g)
    Kc = K.transpose(1, 0, 2).reshape(N, Hkv * d)
    Vc = V.transpose(1, 0, 2).reshape(N, Hkv * d)
    idx = np.arange(N, dtype=np.int32)
    want = ((Vc - np.einsum("oc,nc->no", W, Kc)) ** 2).sum(1)
    got = oracle.residual_layer(K, V, W, idx)
    assert np.allclose(got, want, rtol=1e-12)
    assert not np.allclose(got, ((Vc - np.einsum("co,nc->no", W, Kc)) ** 2).sum(1), rtol=1e-3)      # transposed map
    ret, apx = np.arange(0, 12), np.arange(12, 30)
    o_tok, o_fac = oracle.attend_layer(q, K[:, ret], V[:, ret], K[:, apx], W, 0.25)
    Vhat = np.einsum("oc,nc->no", W, Kc[apx]).reshape(len(apx), Hkv, d)       # reconstructed values, whole layer
    for a in range(Hkv * g):
        h = a // g
        keys = np.concatenate([K[h, ret], K[h, apx]])
        p = softmax(0.25 * keys @ q[a])
        want_o = p[:len(ret)] @ V[h, ret] + p[len(ret):] @ Vhat[:, h]
        assert np.allclose(o_tok[a], want_o, rtol=1e-11, atol=1e-13) and np.allclose(o_fac[a], want_o, rtol=1e-11, atol=1e-13)
    Wd = W.copy(); Wd[:d, d:] = 0.0; Wd[d:, :d] = 0.0
    assert not np.allclose(oracle.attend_layer(q, K[:, ret], V[:, ret], K[:, apx], Wd, 0.25)[0], o_tok, rtol=1e-3)


def test_layer_map_exact_recovery_across_heads(oracle):
    """V = W_true K with a dense whole-layer map and no noise: calibration finds the map (cross-head blocks
    included), every residual is zero, routing order is by index, and attention over any retain / approximate
    split equals plain attention over the pool."""
    rng = np.random.default_rng(13)
    Hkv, d, g, n = 2, 8, 2, 600
    Wt = rng.standard_normal((Hkv * d, Hkv * d)) / np.sqrt(Hkv * d)
    Kc = rng.standard_normal((n, Hkv * d))
    Vc = Kc @ Wt.T
    K = Kc.reshape(n, Hkv, d).transpose(1, 0, 2)
    V = Vc.reshape(n, Hkv, d).transpose(1, 0, 2)
    W = oracle.calibrate_layer(K, V, 1e-9)
    assert W.shape == (Hkv * d, Hkv * d) and np.max(np.abs(W - Wt)) < 1e-7
    N = 50
    assert np.max(oracle.residual_layer(K[:, :N], V[:, :N], Wt, np.arange(N, dtype=np.int32))) < 1e-24
    sc = rng.random(N).astype(np.float32)
    r = oracle.route_layer(sc, K[:, :N], V[:, :N], Wt, 30, 20)
    assert np.array_equal(r["pool_idx"], np.sort(np.argsort(-sc, kind="stable")[:30]))
    assert sorted(np.concatenate([r["ret_idx"], r["apx_idx"]]).tolist()) == r["pool_idx"].tolist()
    q = rng.standard_normal((Hkv * g, d))
    pool = r["pool_idx"]
    full, _ = oracle.attend_layer(q, K[:, pool], V[:, pool], K[:, :0], Wt, 0.35)
    for n_ret in (0, 7, 30):
        o_tok, o_fac = oracle.attend_layer(q, K[:, pool[:n_ret]], V[:, pool[:n_ret]], K[:, pool[n_ret:]], Wt, 0.35)
        # the order of keys inside a softmax does not matter: retained first, approximated after
        assert np.allclose(o_tok, full, rtol=1e-10, atol=1e-12) and np.allclose(o_fac, full, rtol=1e-10, atol=1e-12)


def test_layer_score_is_the_sum_over_heads(oracle):
    s = np.array([[0.5, 0.25, np.inf], [0.125, 1.0, np.inf]])
    assert np.array_equal(oracle.layer_score(s), np.array([0.625, 1.25, np.inf]))
