"""Shared helpers of the parity tests: run the oracle unit by unit on the exact stored bits."""
import numpy as np
import torch

import paper_2605_23258_b200 as vec
from paper_2605_23258_b200 import synth


def shape_of(wl, batch=None, n_layers=None):
    return vec.Shape(wl.batch if batch is None else batch, wl.n_layers if n_layers is None else n_layers,
                     wl.n_q_heads, wl.n_kv_heads, wl.head_dim,
                     vec.VECTOR_BF16 if wl.dtype == "bf16" else vec.VECTOR_F32, wl.window, wl.pool_kernel)


def budget_of(wl, percent, n_a=-1):
    return vec.vector_plan_budget(wl.N, (wl.N * percent) // 100, n_a, wl.window)


def calibrated_maps(wl, device="cuda"):
    """W [LH][d][d] in the workload dtype (the bits both sides use), via the library's host solver.
    `device` is where the calibration draw is generated: it must be the device the context tensors are
    generated on, because the per-head parameters (channel scales, true map) come from that device's
    random stream."""
    from paper_2605_23258_b200.pipeline import calibrate_maps
    pairs = []
    for l in range(wl.n_layers):
        for h in range(wl.n_kv_heads):
            k, v = synth.calib_kv(wl, l, h, device)
            pairs.append((k.cpu(), v.cpu()))
    return calibrate_maps(pairs, wl.lam).to(wl.torch_dtype)


def oracle_scores(oracle, wl, Q, K):
    """Q [U][g][w][d], K [U][N][d] (cpu) -> raw, score float64 [U][N]."""
    scale = 1.0 / np.sqrt(wl.head_dim)
    raws, scs = [], []
    for u in range(K.shape[0]):
        r, s = oracle.score(Q[u], K[u], scale, wl.pool_kernel)
        raws.append(r), scs.append(s)
    return np.stack(raws), np.stack(scs)


def score_close(got, want, mass, rtol=1e-3):
    """|g - o| <= rtol * max(|o|, 1e-6 * mass) elementwise on the finite entries; infinities must match."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    inf_ok = np.array_equal(np.isinf(got), np.isinf(want)) and np.all(got[np.isinf(got)] > 0)
    fin = np.isfinite(want)
    err = np.abs(got[fin] - want[fin])
    tol = rtol * np.maximum(np.abs(want[fin]), 1e-6 * mass)
    return inf_ok and bool(np.all(err <= tol)), float(np.max(err / tol)) if err.size else 0.0


def eps_close(got, want, K_rows, V_rows, W):
    """Residual eps = sum_c r_c^2, r = v - W k, computed on the device with fp32 accumulation of exact
    bf16/fp32 products against the oracle's fp64.  Each r_c carries an absolute error of at most
    delta_c = 130 * 2^-23 * (|v_c| + sum_j |W_cj| |k_j|)   (d + 2 roundings of relative size 2^-23, a
    bound that also covers an accumulator that truncates instead of rounding), so
    |eps_gpu - eps| <= 2 sqrt(eps) ||delta|| + ||delta||^2, plus 2^-21 eps for the fp32 sum of squares."""
    K_rows, V_rows, W = (np.asarray(t.double().numpy() if hasattr(t, "double") else t, np.float64) for t in (K_rows, V_rows, W))
    delta = 130 * 2.0 ** -23 * (np.abs(V_rows) + np.abs(K_rows) @ np.abs(W).T)
    dn = np.sqrt((delta ** 2).sum(1))
    want = np.asarray(want, np.float64)
    tol = 2 * np.sqrt(want) * dn + dn ** 2 + 2.0 ** -21 * want
    err = np.abs(np.asarray(got, np.float64) - want)
    return bool(np.all(err <= tol)), float(np.max(err / tol))
