"""Parity of the CUDA path (through the C-ABI) with the CPU oracle on the same seeded inputs.

Tolerances:
  scores          |g - o| <= 1e-3 * max(|o|, 1e-6 * g*w)     (g*w = total attention mass of a unit)
  selections      bit-exact when both sides are fed identical fp32 scores / residuals
  residual eps    |eps_gpu - eps| <= 2 sqrt(eps) ||delta|| + ||delta||^2 + 2^-21 eps with the per-channel
                  rounding bound delta of fp32 accumulation (helpers.eps_close)
  end-to-end      >= 99.9 % of tokens routed alike; each disagreement sits within 1e-3 (relative)
                  of the oracle's own selection threshold
  decode output   |o_gpu - o_oracle| <= 2e-2 with fp32 output; bf16 output adds 2^-8 |o|
"""
import numpy as np
import pytest
import torch

import paper_2605_23258_b200 as vec
from paper_2605_23258_b200 import synth
from paper_2605_23258_b200.pipeline import Compressor

from helpers import budget_of, calibrated_maps, eps_close, oracle_scores, score_close, shape_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.fixture(scope="module", autouse=True)
def _lib():
    assert torch.cuda.is_available(), "these tests need the B200"
    vec.load_library()          # fails loudly if the CUDA library has not been built


SCORE_CASES = [
    # (base workload, overrides)
    (0, {}),                                                    # config 0 as given: fp32, d=64, N=1024
    (0, {"N": 333, "window": 16, "pool_kernel": 5}),            # ragged tail, fp32
    (1, {"N": 1000, "n_kv_heads": 2, "n_q_heads": 8}),          # bf16 d=128, N not a tile multiple
    (1, {"N": 4096 + 77, "n_kv_heads": 1, "n_q_heads": 4}),
    (4, {"N": 2048 + 5, "n_layers": 1, "n_kv_heads": 1, "n_q_heads": 8, "window": 128}),   # g=8, 1024 rows
    (1, {"N": 64, "n_kv_heads": 1, "n_q_heads": 4}),            # N == window: every token is a window token
    (1, {"N": 70, "n_kv_heads": 1, "n_q_heads": 1, "window": 3, "pool_kernel": 1}),        # g=1, tiny window
    (0, {"N": 640, "head_dim": 128, "dtype": "bf16"}),
    (1, {"N": 900, "head_dim": 64, "n_kv_heads": 1, "n_q_heads": 2}),                      # bf16 d=64
    (2, {"N": 1500, "n_layers": 20}),                           # 160 units: several items per block, ring wraps
    (4, {"N": 3000, "n_layers": 3, "n_kv_heads": 2, "n_q_heads": 16}),    # 6 units x 4 row groups of 256 rows
    (1, {"N": 777, "n_kv_heads": 1, "n_q_heads": 6, "window": 50}),       # 300 rows: second row group of 44 rows
]


@pytest.mark.parametrize("base,over", SCORE_CASES)
def test_score_parity(oracle, base, over):
    wl = synth.shrink(synth.WORKLOADS[base], **over)
    K, V, Q = synth.context(wl, DEV)
    sh = shape_of(wl)
    b = vec.vector_plan_budget(wl.N, wl.N, 0, wl.window)
    ws = vec.alloc_workspace(sh, b)
    scores = torch.empty(wl.units, wl.N, dtype=torch.float32, device=DEV)
    raw = torch.empty_like(scores)
    vec.vector_score(sh, Q, K, wl.N, scores, raw, ws)
    scores2 = torch.empty_like(scores)
    vec.vector_score(sh, Q, K, wl.N, scores2, None, ws)        # raw kept in the workspace
    torch.cuda.synchronize()
    assert torch.equal(scores, scores2)
    raw_o, sc_o = oracle_scores(oracle, wl, Q.cpu(), K.cpu())
    mass = wl.group * wl.window
    ok, worst = score_close(scores.cpu().numpy(), sc_o, mass)
    assert ok, f"score off by {worst:.3g} x tolerance"
    ok, worst = score_close(raw.cpu().numpy(), raw_o, mass)
    assert ok, f"raw off by {worst:.3g} x tolerance"
    # the mass every unit distributes is g*w
    assert np.allclose(raw.double().sum(1).cpu().numpy(), mass, rtol=1e-4)


def test_score_logit_far_above_the_running_reference(oracle):
    """One key whose logit beats every other by about 200 log2 units, placed past the first 32 keys in a
    column whose exponential is evaluated by the polynomial: the first pass must notice that the key ran
    away from its running reference (an exponent field that wrapped would pass as a tiny term)."""
    wl = synth.shrink(synth.WORKLOADS[1], N=700, n_kv_heads=1, n_q_heads=4)
    K, _, Q = synth.context(wl, DEV)
    K = (K.float() * 0.05).to(torch.bfloat16)
    Q = (Q.float() * 0.05).to(torch.bfloat16)
    Q[..., 0] = 8.0
    K[0, 49, 0] = 200.0                     # logit 8 * 200 / sqrt(128) = 141 nats; 49 & 15 = 1, second 32-key chunk
    sh = shape_of(wl)
    ws = vec.alloc_workspace(sh, vec.vector_plan_budget(wl.N, wl.N, 0, wl.window))
    scores = torch.empty(wl.units, wl.N, dtype=torch.float32, device=DEV)
    raw = torch.empty_like(scores)
    vec.vector_score(sh, Q, K, wl.N, scores, raw, ws)
    torch.cuda.synchronize()
    raw_o, sc_o = oracle_scores(oracle, wl, Q.cpu(), K.cpu())
    mass = wl.group * wl.window
    assert raw_o[0, 49] > 0.999 * mass
    ok, worst = score_close(raw.cpu().numpy(), raw_o, mass)
    assert ok, f"raw off by {worst:.3g} x tolerance"
    ok, worst = score_close(scores.cpu().numpy(), sc_o, mass)
    assert ok, f"score off by {worst:.3g} x tolerance"


KEYDIFF_CASES = [(0, {}), (0, {"N": 333}), (1, {"N": 1000, "n_kv_heads": 2, "n_q_heads": 8}),
                 (1, {"N": 4096 + 77, "n_kv_heads": 1, "n_q_heads": 4}), (2, {"N": 1500, "n_layers": 20}),
                 (1, {"N": 900, "head_dim": 64, "n_kv_heads": 1, "n_q_heads": 2}), (1, {"N": 1, "n_kv_heads": 1, "n_q_heads": 4})]


@pytest.mark.parametrize("base,over", KEYDIFF_CASES)
def test_keydiff_score_parity(oracle, base, over):
    """Key-geometry scorer: cosines in [-1, 1] from fp32 sums over N rows against the fp64 oracle;
    |g - o| <= 1e-3 max(|o|, 0.05)."""
    wl = synth.shrink(synth.WORKLOADS[base], **over)
    K, _, _ = synth.context(wl, DEV)
    if wl.N > 10:
        K[0, 7] = 0                                        # a zero key scores 0
    sh = shape_of(wl)
    ws = vec.alloc_workspace(sh, vec.vector_plan_budget(wl.N, wl.N, 0, min(wl.window, wl.N)))
    scores = torch.full((wl.units, wl.N), float("nan"), dtype=torch.float32, device=DEV)
    vec.vector_score_keydiff(sh, K, wl.N, scores, ws)
    again = torch.empty_like(scores)
    vec.vector_score_keydiff(sh, K, wl.N, again, ws)
    torch.cuda.synchronize()
    assert torch.equal(scores, again)                      # fixed reduction order: bitwise repeatable
    got = scores.cpu().double().numpy()
    for u in range(wl.units):
        want = oracle.score_keydiff(K[u].cpu())
        assert np.all(np.abs(got[u] - want) <= 1e-3 * np.maximum(np.abs(want), 0.05)), u
    if wl.N > 10:
        assert got[0, 7] == 0.0


def test_keydiff_scores_drive_the_routing(oracle):
    """The second base scorer feeds the same Steps 1-3: end-to-end agreement with the oracle run on its own scores."""
    wl = synth.shrink(synth.WORKLOADS[1], N=2000, n_kv_heads=2, n_q_heads=8, n_calib=2048, window=8)
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    b = budget_of(wl, 30)
    comp = Compressor(sh, b, keep_eps=True)
    vec.vector_score_keydiff(sh, K, wl.N, comp.scores, comp.ws)
    comp.route(K, V, W)
    torch.cuda.synchronize()
    sc_o = np.stack([oracle.score_keydiff(K[u].cpu()) for u in range(wl.units)])
    _assert_routing_agrees(oracle, wl, b, comp, K, V, W.cpu(), sc_o, list(range(wl.units)))
    assert torch.all((comp.tier == 1).sum(1) == b.n_apx) and torch.all((comp.tier == 2).sum(1) == b.n_ret)


def test_diagnostics_parity(oracle):
    """Distortion E, R^2 over the approximated set and Proposition 1's threshold of a routed cache."""
    wl = synth.shrink(synth.WORKLOADS[1], N=3000, n_kv_heads=2, n_q_heads=8, n_calib=2048)
    K, V, Q = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    b = budget_of(wl, 30)
    comp = Compressor(sh, b, keep_eps=True)
    raw = torch.empty(wl.units, wl.N, dtype=torch.float32, device=DEV)
    vec.vector_score(sh, Q, K, wl.N, comp.scores, raw, comp.ws)
    comp.route(K, V, W)
    out = torch.empty(wl.units, 8, dtype=torch.float32, device=DEV)
    vec.vector_diagnostics(sh, b, raw, comp.tier, comp.pool_idx, comp.eps, V, out)
    torch.cuda.synchronize()
    for u in range(wl.units):
        want = oracle.diagnostics(raw[u].cpu(), comp.tier[u].cpu().numpy(), K[u].cpu(), V[u].cpu(), W[u].cpu())
        got = dict(zip(vec.DIAG_FIELDS, out[u].cpu().double().tolist()))
        for name in vec.DIAG_FIELDS:          # fp64 sums of fp32 residuals: the residual's own rounding dominates
            assert got[name] == pytest.approx(want[name], rel=1e-4, abs=1e-7), (u, name, got[name], want[name])
        assert 0.0 <= got["E"] <= 1.0 and got["mu_a"] < 0.5          # the approximated tokens are the reconstructable ones


@pytest.mark.parametrize("dtype,d,N", [("bf16", 128, 3000), ("fp32", 64, 1111), ("bf16", 128, 2048)])
def test_r2_global_parity(oracle, dtype, d, N):
    """R^2 of the calibrated map over every token of the context, per unit, and the stream check after it."""
    wl = synth.shrink(synth.WORKLOADS[1], N=N, n_kv_heads=2, n_q_heads=8, n_calib=2048, head_dim=d, dtype=dtype)
    K, V, _q = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    ws = torch.empty(vec.vector_r2_global_workspace_bytes(sh, wl.N), dtype=torch.uint8, device=DEV)
    out = torch.full((wl.units, 4), float("nan"), dtype=torch.float32, device=DEV)
    vec.vector_r2_global(sh, K, V, W, wl.N, out, ws)
    vec.vector_sync_check()                               # no bounded wait gave up
    for u in range(wl.units):
        want = oracle.r2_global(K[u].cpu(), V[u].cpu(), W[u].cpu())
        got = dict(zip(vec.R2_FIELDS, out[u].cpu().double().tolist()))
        for name in vec.R2_FIELDS:                        # fp64 sums; the fp32 residuals' rounding is what is left
            assert got[name] == pytest.approx(want[name], rel=1e-4), (u, name, got[name], want[name])
        assert got["r2"] < 1.0
    with pytest.raises(vec.VectorError):                  # too small a workspace is refused before any launch
        vec.vector_r2_global(sh, K, V, W, wl.N, out, ws[:256])


def _selection_inputs(U, N, seed, ties):
    g = torch.Generator().manual_seed(seed)
    s = torch.rand(U, N, generator=g)
    if ties == "narrow":
        s = 1.0 + 0.01 * s                              # all values share their leading 11 bits
    elif ties == "equal":
        s = torch.full_like(s, 0.25)
    elif ties:
        s = torch.round(s * 16) / 16                    # many exact ties
    s[:, -8:] = float("inf")
    s[0, : N // 3] = 0.0
    return s


@pytest.mark.parametrize("N,n_pool,ties", [(1000, 300, False), (1000, 300, True), (5000, 4999, True),
                                           (4096, 8, True), (70000, 20000, True), (2048, 2048, False),
                                           (131072, 9829, False),
                                           # more candidates after the first digit than the list holds, with
                                           # and without the bit masks (N above 32768), and nothing but ties
                                           (20000, 7000, "narrow"), (70000, 20000, "narrow"), (32768, 11000, "equal"),
                                           (40000, 100, "equal"),
                                           # longer than the bit masks kept in shared memory can cover
                                           (400000, 50000, True), (400000, 150001, "narrow"), (4097, 33, True)])
def test_pool_select_bit_exact(oracle, N, n_pool, ties):
    U = 3
    s = _selection_inputs(U, N, N + n_pool, ties)
    wl = synth.shrink(synth.WORKLOADS[0], N=N, window=8, n_kv_heads=U, n_q_heads=U)
    sh = shape_of(wl)
    b = vec.Budget(N, n_pool, 0, n_pool, 0, n_pool, N - n_pool)
    out = torch.empty(U, n_pool, dtype=torch.int32, device=DEV)
    vec.vector_pool_select(sh, b, s.to(DEV), out)
    got = out.cpu().numpy()
    for u in range(U):
        assert np.array_equal(got[u], oracle.pool_select(s[u].numpy(), n_pool)), u


@pytest.mark.parametrize("base,over,n_idx", [(0, {}, 384), (1, {"N": 3000, "n_kv_heads": 2, "n_q_heads": 8}, 1001),
                                             (1, {"N": 500, "head_dim": 64, "n_kv_heads": 1, "n_q_heads": 2}, 77),
                                             (0, {"N": 300, "head_dim": 128}, 300),
                                             # 160 units x 10 tiles: blocks own ranges that cross unit boundaries
                                             (2, {"N": 1500, "n_layers": 20}, 1200)])
def test_residual_parity(oracle, base, over, n_idx):
    wl = synth.shrink(synth.WORKLOADS[base], n_calib=1024, **over)
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    g = torch.Generator().manual_seed(5)
    idx = torch.stack([torch.randperm(wl.N, generator=g)[:n_idx].sort().values for _ in range(wl.units)])
    idx = idx.to(torch.int32).to(DEV)
    eps = torch.empty(wl.units, n_idx, dtype=torch.float32, device=DEV)
    vec.vector_residual(shape_of(wl), K, V, W, wl.N, idx, n_idx, eps)
    got = eps.cpu().numpy()
    for u in range(wl.units):
        want = oracle.residual(K[u].cpu(), V[u].cpu(), W[u % W.shape[0]].cpu(), idx[u].cpu().numpy())
        rows = idx[u].long().cpu()
        ok, worst = eps_close(got[u], want, K[u].cpu()[rows], V[u].cpu()[rows], W[u % W.shape[0]].cpu())
        assert ok, f"unit {u}: eps off by {worst:.3g} x bound"


@pytest.mark.parametrize("N,n_pool,n_apx,ties", [(1024, 384, 256, False), (1024, 384, 256, True),
                                                 (4000, 1501, 0, True), (4000, 1500, 1500, True),
                                                 (131072, 9829, 6552, False), (50, 20, 2, True),
                                                 (32768, 11468, 6552, "narrow"), (131072, 45000, 30000, "narrow"),
                                                 (16384, 2457, 1638, False), (500000, 450000, 200000, True)])
def test_truncate_bit_exact(oracle, N, n_pool, n_apx, ties):
    U = 3
    g = torch.Generator().manual_seed(N + n_apx)
    pool = torch.stack([torch.randperm(N, generator=g)[:n_pool].sort().values for _ in range(U)]).to(torch.int32)
    eps = torch.rand(U, n_pool, generator=g) * 3
    if ties == "narrow":
        eps = 2.0 + eps * 0.01                           # one quarter-binade: the candidate list overflows
    elif ties:
        eps = torch.round(eps * 8) / 8
    wl = synth.shrink(synth.WORKLOADS[0], N=N, window=1, n_kv_heads=U, n_q_heads=U)
    n_a = n_apx // 2
    b = vec.Budget(N, n_pool - n_a, n_a, n_pool, n_apx, n_pool - n_apx, N - n_pool)
    tier = torch.empty(U, N, dtype=torch.uint8, device=DEV)
    ret = torch.empty(U, max(n_pool - n_apx, 1), dtype=torch.int32, device=DEV)
    apx = torch.empty(U, max(n_apx, 1), dtype=torch.int32, device=DEV)
    vec.vector_truncate(shape_of(wl), b, eps.to(DEV), pool.to(DEV), tier, ret, apx)
    for u in range(U):
        t, r, a = oracle.truncate(eps[u].numpy(), pool[u].numpy(), n_apx, N)
        assert np.array_equal(tier[u].cpu().numpy(), t)
        assert np.array_equal(ret[u, : n_pool - n_apx].cpu().numpy(), r)
        assert np.array_equal(apx[u, :n_apx].cpu().numpy(), a)


def _oracle_route_unit(oracle, wl, b, score_f32, K, V, W, theta=None):
    if theta is None:
        return oracle.route(score_f32, K, V, W, b.n_pool, b.n_apx)
    return oracle.route(score_f32, K, V, W, b.n_pool, b.n_apx, rope=True, theta=theta)


def _assert_routing_agrees(oracle, wl, b, comp, K, V, W, sc_oracle, units, theta=None):
    """End-to-end agreement of the device routing (fed by device scores) with the oracle's."""
    tier = comp.tier.cpu().numpy()
    total = mism = 0
    for j, u in enumerate(units):
        s32 = sc_oracle[j].astype(np.float32)
        r = _oracle_route_unit(oracle, wl, b, s32, K[j].cpu(), V[j].cpu(), W[u % W.shape[0]].cpu(), theta)
        bad = np.nonzero(tier[j] != r["tier"])[0]
        total += wl.N
        mism += len(bad)
        if len(bad) == 0:
            continue
        # thresholds of the oracle's own two selections
        pool = r["pool_idx"]
        in_pool = np.zeros(wl.N, bool)
        in_pool[pool] = True
        fin = np.isfinite(sc_oracle[j])
        thr_s = np.min(sc_oracle[j][in_pool & fin]) if b.n_evict > 0 and np.any(in_pool & fin) else None
        eps_all = oracle.residual(K[j].cpu(), V[j].cpu(), W[u % W.shape[0]].cpu(), np.arange(wl.N, dtype=np.int32),
                                  rope=theta is not None, theta=theta or 10000.0)
        is_apx = r["tier"] == 1
        thr_e = np.max(eps_all[is_apx]) if b.n_apx > 0 else None
        for i in bad:
            near_s = thr_s is not None and abs(sc_oracle[j][i] - thr_s) <= 1e-3 * max(abs(thr_s), 1e-6 * wl.group * wl.window)
            near_e = thr_e is not None and abs(eps_all[i] - thr_e) <= 1e-3 * abs(thr_e)
            assert near_s or near_e, f"unit {u} token {i}: routed differently away from any threshold"
    assert mism <= 1e-3 * total, f"{mism} of {total} tokens routed differently"


def _run_pipeline_case(oracle, wl, percent, units=None, decode_steps=2, n_a=-1, theta=None):
    """Device pipeline on the given units, compared step by step with the oracle.  With `theta` the
    stored keys carry rotary position embedding and the regressor sees them turned back."""
    units = list(range(wl.units)) if units is None else units
    K, V, Q = synth.context(wl, DEV, units)
    if theta is not None:
        K = synth.rope_keys(K, theta)
    Wfull = calibrated_maps(wl)
    LH = wl.n_layers * wl.n_kv_heads
    # the device call indexes maps by u % LH; give it one map per listed unit in that layout
    W = torch.stack([Wfull[u % LH] for u in units]).to(DEV)
    sub = synth.shrink(wl, batch=1, n_layers=1, n_kv_heads=len(units), n_q_heads=len(units) * wl.group)
    sh = shape_of(sub)
    if theta is not None:
        sh.rope_enabled, sh.rope_theta = 1, theta
    b = budget_of(wl, percent, n_a)
    comp = Compressor(sh, b, extra_rows=decode_steps, keep_eps=True)
    comp.compress(Q, K, V, W)
    torch.cuda.synchronize()
    raw_o, sc_o = oracle_scores(oracle, wl, Q.cpu(), K.cpu())
    ok, worst = score_close(comp.scores.cpu().numpy(), sc_o, wl.group * wl.window)
    assert ok, f"score off by {worst:.3g} x tolerance"
    # routing fed by the oracle's scores must be bit-exact in Step 1, and in Step 3 given equal residuals
    sc32 = torch.from_numpy(sc_o.astype(np.float32)).to(DEV)
    tier = torch.empty_like(comp.tier)
    ret = torch.empty_like(comp.ret_idx)
    apx = torch.empty_like(comp.apx_idx)
    eps = torch.empty(len(units), b.n_pool, dtype=torch.float32, device=DEV)
    pool = torch.empty(len(units), b.n_pool, dtype=torch.int32, device=DEV)
    vec.vector_route(sh, b, sc32, K, V, W, tier, ret, apx, eps, pool, comp.ws)
    torch.cuda.synchronize()
    for j, u in enumerate(units):
        r = _oracle_route_unit(oracle, wl, b, sc_o[j].astype(np.float32), K[j].cpu(), V[j].cpu(), W[j].cpu(), theta)
        assert np.array_equal(pool[j].cpu().numpy(), r["pool_idx"]), f"unit {u}: pool differs"
        rows = torch.from_numpy(r["pool_idx"]).long()
        ok, worst = eps_close(eps[j].cpu().numpy(), r["eps"], K[j].cpu()[rows], V[j].cpu()[rows], W[j].cpu())
        assert ok, f"unit {u}: eps off by {worst:.3g} x bound"
        t2, r2, a2 = oracle.truncate(eps[j].cpu().numpy(), r["pool_idx"], b.n_apx, wl.N)
        assert np.array_equal(tier[j].cpu().numpy(), t2), f"unit {u}: tiers differ on identical residuals"
        assert np.array_equal(ret[j].cpu().numpy(), r2) and np.array_equal(apx[j].cpu().numpy(), a2)
    # end to end (device scores -> device routing) against the oracle end to end
    _assert_routing_agrees(oracle, sub, b, comp, K, V, W.cpu(), sc_o, list(range(len(units))), theta)
    # compaction is a pure gather of the device's own index lists
    c = comp.cache
    ri, ai = comp.ret_idx.long(), comp.apx_idx.long()
    for j in range(len(units)):
        assert torch.equal(c.ret_k[j, : b.n_ret], K[j][ri[j]]) and torch.equal(c.ret_v[j, : b.n_ret], V[j][ri[j]])
        assert torch.equal(c.apx_k[j, : b.n_apx], K[j][ai[j]])
        assert torch.equal(c.ret_pos[j, : b.n_ret], comp.ret_idx[j]) and torch.equal(c.apx_pos[j, : b.n_apx], comp.apx_idx[j])
        assert 2 * b.n_ret + b.n_apx == 2 * b.n_budget_pairs
    # decode steps over the mixed cache, appending the generated token each step
    sk, sq, wt = synth.all_head_params(wl, DEV)
    out = torch.empty(len(units), wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    out_bf = torch.empty(len(units), wl.group, wl.head_dim, dtype=torch.bfloat16, device=DEV)
    scale = 1.0 / np.sqrt(wl.head_dim)
    for step in range(decode_steps):
        q = synth.decode_q(wl, step, DEV, sq, units)
        comp.decode(q, W, out)
        comp.decode(q, W, out_bf)
        torch.cuda.synchronize()
        for j in range(len(units)):
            o_tok, o_fac = oracle.attend(q[j].cpu(), c.ret_k[j, : c.n_ret].cpu(), c.ret_v[j, : c.n_ret].cpu(),
                                         c.apx_k[j, : c.n_apx].cpu(), W[j].cpu(), scale,
                                         apx_pos=c.apx_pos[j, : c.n_apx].cpu().numpy(), rope=theta is not None,
                                         theta=theta or 10000.0)
            assert np.max(np.abs(o_tok - o_fac)) <= 1e-9 * max(1.0, np.max(np.abs(o_tok)))
            err = np.max(np.abs(out[j].cpu().double().numpy() - o_fac))
            assert err <= 2e-2, f"decode step {step} unit {units[j]}: abs err {err}"
            errb = np.abs(out_bf[j].cpu().double().numpy() - o_fac)
            assert np.all(errb <= 2e-2 + 2.0 ** -8 * np.abs(o_fac))
        if wl.dtype == "bf16" and wl.head_dim == 128 and theta is None:
            comp.decode(q, W, out, mode=1)              # per-tile reconstruction: sum_A p (W k) formed tile by tile
            torch.cuda.synchronize()
            for j in range(len(units)):
                o_tok, _ = oracle.attend(q[j].cpu(), c.ret_k[j, : c.n_ret].cpu(), c.ret_v[j, : c.n_ret].cpu(),
                                         c.apx_k[j, : c.n_apx].cpu(), W[j].cpu(), scale)
                err = np.max(np.abs(out[j].cpu().double().numpy() - o_tok))
                assert err <= 2e-2, f"per-tile decode step {step} unit {units[j]}: abs err {err}"
        kn, vn = synth.decode_kv(wl, step, DEV, sk, wt, units)
        comp.append(kn, vn, wl.N + step)


def test_pipeline_config0_all_units(oracle):
    _run_pipeline_case(oracle, synth.WORKLOADS[0], 25, decode_steps=8)


@pytest.mark.parametrize("percent", [10, 20, 40])
def test_pipeline_config1_all_units(oracle, percent):
    _run_pipeline_case(oracle, synth.WORKLOADS[1], percent, decode_steps=3)


def test_pipeline_eviction_only_and_ragged(oracle):
    wl = synth.shrink(synth.WORKLOADS[1], N=1531, n_kv_heads=2, n_q_heads=8, n_calib=2048)
    _run_pipeline_case(oracle, wl, 30, n_a=0)          # no approximation tier: plain eviction
    _run_pipeline_case(oracle, wl, 30)
    wl8 = synth.shrink(synth.WORKLOADS[4], N=3000, n_layers=2, n_kv_heads=1, n_q_heads=8, n_calib=2048)
    _run_pipeline_case(oracle, wl8, 12)                # g = 8, window 128


def test_pipeline_with_rotary_keys(oracle):
    """RoPE decoupling: stored keys are post-RoPE, the regressor input is the key turned back by its
    position, in the residual of Step 2 and in the reconstruction inside decode attention."""
    wl = synth.shrink(synth.WORKLOADS[1], N=1200, n_kv_heads=2, n_q_heads=8, n_calib=2048)
    _run_pipeline_case(oracle, wl, 30, theta=10000.0)
    _run_pipeline_case(oracle, synth.shrink(synth.WORKLOADS[0], N=700), 25, decode_steps=2, theta=500.0)    # fp32, d = 64
    # eight query heads per KV head, window 128, pools that end inside a 64-key half
    wl8 = synth.shrink(synth.WORKLOADS[4], N=3000, n_layers=2, n_kv_heads=1, n_q_heads=8, n_calib=2048)
    _run_pipeline_case(oracle, wl8, 12, theta=500000.0)
    _run_pipeline_case(oracle, wl8, 31, theta=500000.0)


@pytest.mark.parametrize("base,over,theta", [(1, {"N": 3000, "n_kv_heads": 2, "n_q_heads": 8}, 10000.0),
                                             (4, {"N": 131072 // 64, "n_layers": 1, "n_kv_heads": 1, "n_q_heads": 8}, 500000.0),
                                             (0, {"N": 500}, 10000.0)])
def test_residual_rope_parity(oracle, base, over, theta):
    wl = synth.shrink(synth.WORKLOADS[base], n_calib=1024, **over)
    K, V, _ = synth.context(wl, DEV)
    K = synth.rope_keys(K, theta)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    sh.rope_enabled, sh.rope_theta = 1, theta
    n_idx = wl.N // 3
    g = torch.Generator().manual_seed(7)
    idx = torch.stack([torch.randperm(wl.N, generator=g)[:n_idx].sort().values for _ in range(wl.units)])
    idx = idx.to(torch.int32).to(DEV)
    eps = torch.empty(wl.units, n_idx, dtype=torch.float32, device=DEV)
    vec.vector_residual(sh, K, V, W, wl.N, idx, n_idx, eps)
    got = eps.cpu().numpy()
    for u in range(wl.units):
        want = oracle.residual(K[u].cpu(), V[u].cpu(), W[u % W.shape[0]].cpu(), idx[u].cpu().numpy(), rope=True, theta=theta)
        plain = oracle.residual(K[u].cpu(), V[u].cpu(), W[u % W.shape[0]].cpu(), idx[u].cpu().numpy())
        rows = idx[u].long().cpu()
        ok, worst = eps_close(got[u], want, K[u].cpu()[rows], V[u].cpu()[rows], W[u % W.shape[0]].cpu())
        assert ok, f"unit {u}: eps off by {worst:.3g} x bound"
        assert np.median(plain / want) > 2.0          # the rotation matters on these inputs


def test_decode_rope_large_positions(oracle):
    """Key-only rows whose original positions reach 10^5 (tens of thousands of radians): the angle needs
    more than fp32 to come out right modulo a turn."""
    wl = synth.shrink(synth.WORKLOADS[1], N=2048, n_kv_heads=2, n_q_heads=8, n_calib=1024)
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    sh.rope_enabled, sh.rope_theta = 1, 10000.0
    _, sq, _ = synth.all_head_params(wl, DEV)
    q = synth.decode_q(wl, 0, DEV, sq)
    n_ret, n_apx = 300, 1000
    g = torch.Generator().manual_seed(11)
    pos = torch.stack([torch.randperm(131072, generator=g)[:wl.N].sort().values for _ in range(wl.units)]).to(torch.int32)
    cache = vec.Cache(K.clone(), V.clone(), K.flip(1).contiguous(), pos.to(DEV), pos.to(DEV).clone(), n_ret, n_apx)
    ws = vec.alloc_workspace(sh, budget_of(wl, 50))
    out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    vec.vector_decode_attn(sh, q, cache, W, out, 0, ws)
    torch.cuda.synchronize()
    for u in range(wl.units):
        _, o = oracle.attend(q[u].cpu(), cache.ret_k[u, :n_ret].cpu(), cache.ret_v[u, :n_ret].cpu(),
                             cache.apx_k[u, :n_apx].cpu(), W[u].cpu(), 1.0 / np.sqrt(wl.head_dim),
                             apx_pos=pos[u, :n_apx].numpy(), rope=True, theta=10000.0)
        _, o_plain = oracle.attend(q[u].cpu(), cache.ret_k[u, :n_ret].cpu(), cache.ret_v[u, :n_ret].cpu(),
                                   cache.apx_k[u, :n_apx].cpu(), W[u].cpu(), 1.0 / np.sqrt(wl.head_dim))
        assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2, u
        assert np.max(np.abs(o - o_plain)) > 0.1      # the rotation matters on these inputs


def test_decode_degenerate_pools(oracle):
    """Only retained rows, only key-only rows, and a single key."""
    wl = synth.shrink(synth.WORKLOADS[1], N=512, n_kv_heads=2, n_q_heads=8, n_calib=1024)
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    _, sq, _ = synth.all_head_params(wl, DEV)
    q = synth.decode_q(wl, 0, DEV, sq)
    b = budget_of(wl, 50)
    ws = vec.alloc_workspace(sh, b)
    out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    scale = 1.0 / np.sqrt(wl.head_dim)
    ipos = torch.arange(512, dtype=torch.int32, device=DEV).repeat(wl.units, 1).contiguous()
    for n_ret, n_apx in [(512, 0), (0, 512), (1, 0), (0, 1), (300, 1), (1, 300), (257, 255)]:
        cache = vec.Cache(K.clone(), V.clone(), K.flip(1).contiguous(), ipos, ipos.clone(), n_ret, n_apx)
        for mode in (0, 1):
            vec.vector_decode_attn(sh, q, cache, W, out, mode, ws)
            torch.cuda.synchronize()
            for u in range(wl.units):
                _, o = oracle.attend(q[u].cpu(), cache.ret_k[u, :n_ret].cpu(), cache.ret_v[u, :n_ret].cpu(),
                                     cache.apx_k[u, :n_apx].cpu(), W[u].cpu(), scale)
                assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2, (n_ret, n_apx, u, mode)


def test_decode_long_block_ranges(oracle):
    """Few units with long pools: every block's tile range wraps its shared-memory ring several times and
    crosses a unit boundary; g = 4 and g = 8; a pool end that leaves a key-only tile half empty."""
    for base, over, n_ret, n_apx in [(1, {"N": 8192, "n_kv_heads": 2, "n_q_heads": 8}, 3000, 6000 + 37),
                                     (4, {"N": 8192, "n_layers": 1, "n_kv_heads": 1, "n_q_heads": 8}, 4100, 4090)]:
        wl = synth.shrink(synth.WORKLOADS[base], n_calib=1024, **over)
        K, V, _ = synth.context(wl, DEV)
        W = calibrated_maps(wl).to(DEV)
        sh = shape_of(wl)
        _, sq, _ = synth.all_head_params(wl, DEV)
        q = synth.decode_q(wl, 0, DEV, sq)
        ws = vec.alloc_workspace(sh, budget_of(wl, 50))
        out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
        ipos = torch.arange(wl.N, dtype=torch.int32, device=DEV).repeat(wl.units, 1).contiguous()
        cache = vec.Cache(K.clone(), V.clone(), K.flip(1).contiguous(), ipos, ipos.clone(), n_ret, n_apx)
        out1 = torch.empty_like(out)
        vec.vector_decode_attn(sh, q, cache, W, out, 0, ws)
        vec.vector_decode_attn(sh, q, cache, W, out1, 1, ws)
        torch.cuda.synchronize()
        assert vec.vector_device_fault() == 0
        for u in range(wl.units):
            o_tok, o = oracle.attend(q[u].cpu(), cache.ret_k[u, :n_ret].cpu(), cache.ret_v[u, :n_ret].cpu(),
                                     cache.apx_k[u, :n_apx].cpu(), W[u].cpu(), 1.0 / np.sqrt(wl.head_dim))
            assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2, (base, u)
            assert np.max(np.abs(out1[u].cpu().double().numpy() - o_tok)) <= 2e-2, (base, u, "per tile")


@pytest.mark.parametrize("g", [1, 2, 3, 6])
def test_decode_every_group_size(oracle, g):
    """Query heads per KV head other than the configurations' 4 and 8: the merge kernel's block is 128 g threads
    and the MMA rows and columns beyond g are padding.  Both forms, three units, a ragged key-only tile."""
    wl = synth.shrink(synth.WORKLOADS[1], N=2048, n_kv_heads=3, n_q_heads=3 * g, n_calib=1024)
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    _, sq, _ = synth.all_head_params(wl, DEV)
    q = synth.decode_q(wl, 0, DEV, sq)
    ws = vec.alloc_workspace(sh, budget_of(wl, 50))
    ipos = torch.arange(wl.N, dtype=torch.int32, device=DEV).repeat(wl.units, 1).contiguous()
    n_ret, n_apx = 700, 1100 + 13
    cache = vec.Cache(K.clone(), V.clone(), K.flip(1).contiguous(), ipos, ipos.clone(), n_ret, n_apx)
    out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    out1 = torch.empty_like(out)
    vec.vector_decode_attn(sh, q, cache, W, out, 0, ws)
    vec.vector_decode_attn(sh, q, cache, W, out1, 1, ws)
    torch.cuda.synchronize()
    assert vec.vector_device_fault() == 0
    for u in range(wl.units):
        o_tok, o = oracle.attend(q[u].cpu(), cache.ret_k[u, :n_ret].cpu(), cache.ret_v[u, :n_ret].cpu(),
                                 cache.apx_k[u, :n_apx].cpu(), W[u].cpu(), 1.0 / np.sqrt(wl.head_dim))
        assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2, (g, u)
        assert np.max(np.abs(out1[u].cpu().double().numpy() - o_tok)) <= 2e-2, (g, u, "per tile")


@pytest.mark.parametrize("base,head_dim,N,Bp,n_a", [(0, 64, 777, 230, 100), (0, 128, 500, 61, 0), (1, 64, 900, 167, 167),
                                                    (1, 128, 1500, 514, 257)])
def test_compact_bit_exact(oracle, base, head_dim, N, Bp, n_a):
    """Compaction alone, every element type and head size (8, 16 and 32 pieces of 16 bytes per row), ragged
    and empty pools: the gathered rows and positions are copies, so the comparison is exact."""
    wl = synth.shrink(synth.WORKLOADS[base], N=N, head_dim=head_dim, n_kv_heads=3, n_q_heads=6, window=8)
    K, V, _ = synth.context(wl, DEV)
    sh = shape_of(wl)
    n_ret, n_apx, n_pool = Bp - n_a, 2 * n_a, Bp + n_a          # the planner's identities
    b = vec.Budget(N, Bp, n_a, n_pool, n_apx, n_ret, N - n_pool)
    g = torch.Generator().manual_seed(N)
    ret_idx = torch.stack([torch.randperm(N, generator=g)[:n_ret].sort().values for _ in range(wl.units)]).to(torch.int32)
    apx_idx = torch.stack([torch.randperm(N, generator=g)[:n_apx].sort().values for _ in range(wl.units)]).to(torch.int32)
    cache = vec.alloc_cache(sh, b, 2, DEV)
    vec.vector_compact(sh, b, K, V, ret_idx.to(DEV).reshape(wl.units, -1), apx_idx.to(DEV).reshape(wl.units, -1), cache)
    torch.cuda.synchronize()
    for u in range(wl.units):
        rk, rpos = oracle.gather_rows(K[u].cpu(), ret_idx[u].numpy())
        rv, _ = oracle.gather_rows(V[u].cpu(), ret_idx[u].numpy())
        ak, apos = oracle.gather_rows(K[u].cpu(), apx_idx[u].numpy())
        assert np.array_equal(cache.ret_k[u, :n_ret].cpu().double().numpy(), rk)
        assert np.array_equal(cache.ret_v[u, :n_ret].cpu().double().numpy(), rv)
        assert np.array_equal(cache.apx_k[u, :n_apx].cpu().double().numpy(), ak)
        assert np.array_equal(cache.ret_pos[u, :n_ret].cpu().numpy(), rpos)
        assert np.array_equal(cache.apx_pos[u, :n_apx].cpu().numpy(), apos)


def test_back_to_back_calls_repeat_bitwise(oracle):
    """The calls of the path are asynchronous and partly overlap (programmatic dependent launches inside
    route and decode): issued back to back without a host synchronisation, on the same buffers, they
    must leave bit-identical results every time."""
    wl = synth.shrink(synth.WORKLOADS[2], n_layers=8)
    K, V, Q = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh, b = shape_of(wl), budget_of(wl, 20)
    comp = Compressor(sh, b, extra_rows=1, keep_eps=True)
    _, sq, _ = synth.all_head_params(wl, DEV)
    q = synth.decode_q(wl, 0, DEV, sq)
    out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    snaps = []
    for _ in range(4):
        comp.compress(Q, K, V, W)
        comp.decode(q, W, out)
        snaps.append([t.clone() for t in (comp.scores, comp.pool_idx, comp.eps, comp.tier, comp.ret_idx, comp.apx_idx,
                                          comp.cache.ret_k, comp.cache.ret_v, comp.cache.apx_k, out)])
    torch.cuda.synchronize()
    assert vec.vector_device_fault() == 0
    names = ("scores", "pool_idx", "eps", "tier", "ret_idx", "apx_idx", "ret_k", "ret_v", "apx_k", "out")
    for r, later in enumerate(snaps[1:]):
        for name, first, again in zip(names, snaps[0], later):
            # bit patterns, not values: rows past the pools are never written and may hold NaNs
            bits = {2: torch.int16, 4: torch.int32}.get(first.element_size())
            a, b_ = (first.view(bits), again.view(bits)) if bits and first.is_floating_point() else (first, again)
            assert torch.equal(a, b_), (name, r + 1, int((a != b_).sum()))


def _sampled_units_case(oracle, wl, percent, sample, theta=None, fed_by_device_scores=()):
    """Whole workload on the device in the launch shape the benchmark times; the oracle checks the
    sampled units end to end, every unit is checked for the properties that hold at any size.
    With `theta` the stored keys are post-RoPE and RoPE decoupling is on.  The units listed in
    `fed_by_device_scores` skip the oracle's scorer (minutes per unit at the longest context): the
    oracle routes them from the device's own fp32 scores, so Step 1 must match bit for bit, the
    residuals within their rounding bound and Step 3 bit for bit on the device's residuals."""
    K, V, Q = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    sh = shape_of(wl)
    if theta is not None:
        K = synth.rope_keys(K, theta)
        sh.rope_enabled, sh.rope_theta = 1, theta
    b = budget_of(wl, percent)
    comp = Compressor(sh, b, extra_rows=1, keep_eps=True)
    comp.compress(Q, K, V, W)
    torch.cuda.synchronize()
    raw_o, sc_o = oracle_scores(oracle, wl, Q[sample].cpu(), K[sample].cpu())
    ok, worst = score_close(comp.scores[sample].cpu().numpy(), sc_o, wl.group * wl.window)
    assert ok, f"score off by {worst:.3g} x tolerance"
    tier_all = comp.tier
    # properties that hold at any size, on every unit
    assert torch.all((tier_all == 1).sum(1) == b.n_apx) and torch.all((tier_all == 2).sum(1) == b.n_ret)
    assert torch.all(tier_all[:, -wl.window:] > 0)
    assert torch.all(comp.ret_idx[:, 1:] > comp.ret_idx[:, :-1]) and torch.all(comp.apx_idx[:, 1:] > comp.apx_idx[:, :-1])
    emax_apx = torch.gather(comp.eps, 1, torch.searchsorted(comp.pool_idx, comp.apx_idx).clamp(max=b.n_pool - 1)).max(1).values
    emin_ret = torch.gather(comp.eps, 1, torch.searchsorted(comp.pool_idx, comp.ret_idx).clamp(max=b.n_pool - 1)).min(1).values
    assert torch.all(emax_apx <= emin_ret)
    # sampled units against the oracle end to end
    class _View:            # the slice of the compressor state the agreement check reads
        tier = tier_all[sample]
    LH = wl.n_layers * wl.n_kv_heads
    Ws = torch.stack([W[u % LH] for u in sample]).cpu()
    sub = synth.shrink(wl, batch=1, n_layers=1, n_kv_heads=len(sample), n_q_heads=len(sample) * wl.group)
    _assert_routing_agrees(oracle, sub, b, _View, K[sample], V[sample], Ws, sc_o, list(range(len(sample))), theta)
    _, sq, _ = synth.all_head_params(wl, DEV)
    q = synth.decode_q(wl, 0, DEV, sq)
    out = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
    comp.decode(q, W, out)
    torch.cuda.synchronize()
    assert vec.vector_device_fault() == 0
    c = comp.cache
    for j, u in enumerate(sample):
        _, o = oracle.attend(q[u].cpu(), c.ret_k[u, : c.n_ret].cpu(), c.ret_v[u, : c.n_ret].cpu(),
                             c.apx_k[u, : c.n_apx].cpu(), Ws[j], 1.0 / np.sqrt(wl.head_dim),
                             apx_pos=c.apx_pos[u, : c.n_apx].cpu().numpy(), rope=theta is not None, theta=theta or 10000.0)
        assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2
    for u in fed_by_device_scores:
        Wu = W[u % LH].cpu()
        r = _oracle_route_unit(oracle, wl, b, comp.scores[u].cpu().numpy(), K[u].cpu(), V[u].cpu(), Wu, theta)
        assert np.array_equal(comp.pool_idx[u].cpu().numpy(), r["pool_idx"]), f"unit {u}: pool differs"
        rows = torch.from_numpy(r["pool_idx"]).long()
        ok, worst = eps_close(comp.eps[u].cpu().numpy(), r["eps"], K[u].cpu()[rows], V[u].cpu()[rows], Wu)
        assert ok, f"unit {u}: eps off by {worst:.3g} x bound"
        t2, r2, a2 = oracle.truncate(comp.eps[u].cpu().numpy(), r["pool_idx"], b.n_apx, wl.N)
        assert np.array_equal(tier_all[u].cpu().numpy(), t2), f"unit {u}: tiers differ on identical residuals"
        assert np.array_equal(comp.ret_idx[u].cpu().numpy(), r2) and np.array_equal(comp.apx_idx[u].cpu().numpy(), a2)
        assert torch.equal(c.ret_k[u, : b.n_ret], K[u][comp.ret_idx[u].long()])
        assert torch.equal(c.ret_v[u, : b.n_ret], V[u][comp.ret_idx[u].long()])
        assert torch.equal(c.apx_k[u, : b.n_apx], K[u][comp.apx_idx[u].long()])
        _, o = oracle.attend(q[u].cpu(), c.ret_k[u, : c.n_ret].cpu(), c.ret_v[u, : c.n_ret].cpu(),
                             c.apx_k[u, : c.n_apx].cpu(), Wu, 1.0 / np.sqrt(wl.head_dim),
                             apx_pos=c.apx_pos[u, : c.n_apx].cpu().numpy(), rope=theta is not None, theta=theta or 10000.0)
        assert np.max(np.abs(out[u].cpu().double().numpy() - o)) <= 2e-2, u


def test_config2_shape_rope_decoupled_sampled_units(oracle):
    """Config-2 shape (8 of its layers: the decode grid is full, blocks start and end inside units) with
    post-RoPE keys: the tensor-core residual and decode kernels with RoPE decoupling, sampled units."""
    _sampled_units_case(oracle, synth.shrink(synth.WORKLOADS[2], n_layers=8), 20, [0, 37, 63], theta=500000.0)


def test_full_size_bench_configuration_sampled_units(oracle):
    """Config 2 at full size in the launch shape the benchmark times; the oracle checks sampled units."""
    _sampled_units_case(oracle, synth.WORKLOADS[2], 20, [0, 131, 255])


def test_config3_shape_sampled_units(oracle):
    """Batched serving shape (config 3: N = 16384, budget 10 %, several sequences), cut to 2 sequences x 4 layers."""
    _sampled_units_case(oracle, synth.shrink(synth.WORKLOADS[3], batch=2, n_layers=4), 10, [3, 40])


def test_config3_full_size_sampled_units(oracle):
    """Config 3 at full size (8 sequences x 32 layers x 8 KV heads = 2048 units, 17 GB of K and V) in the
    launch shape the benchmark times: decode blocks own about fourteen whole units each, two record slots
    per unit.  Units of the first, a middle and the last sequence against the oracle end to end."""
    _sampled_units_case(oracle, synth.WORKLOADS[3], 10, [3, 1029, 2047], fed_by_device_scores=[517, 1536])


def test_config4_shape_sampled_unit(oracle):
    """Long-context shape (config 4: N = 131072, 8 query heads per KV head, window 128, budget 5 %), one layer;
    the oracle scores one whole unit (1024 window rows x 131072 keys)."""
    _sampled_units_case(oracle, synth.shrink(synth.WORKLOADS[4], n_layers=1), 5, [5])


def test_config4_full_size_sampled_units(oracle):
    """Config 4 at full size (80 layers x 8 KV heads = 640 units, 43 GB of K and V) in the launch shape the
    benchmark times.  The oracle scores one whole unit (its scorer takes about half a minute per unit
    here); three more units are routed by the oracle from the device's scores and attended by it."""
    _sampled_units_case(oracle, synth.WORKLOADS[4], 5, [333], fed_by_device_scores=[0, 470, 639])
