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


def calibrated_maps(wl, device="cpu"):
    """W [LH][d][d] in the workload dtype (the bits both sides use), via the library's host solver."""
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
