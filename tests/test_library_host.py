"""CPU-only checks of the C-ABI library: exports, host entry points, argument validation."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

import paper_2605_23258_b200 as vec
from paper_2605_23258_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2605_23258_b200.build import build
    build()


def test_every_declared_symbol_is_exported():
    text = open(os.path.join(ROOT, "include", "vector.h")).read()
    names = re.findall(r"VECTOR_API[^;(]*?\b(vector_\w+)\s*\(", text)
    assert len(names) >= 12 and len(set(names)) == len(names)
    lib = ctypes.CDLL(vec.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_plan_budget_matches_oracle(oracle):
    rng = np.random.default_rng(0)
    for _ in range(300):
        N = int(rng.integers(1, 5000))
        Bp = int(rng.integers(0, N + 1))
        n_a = int(rng.integers(-1, Bp + 2))
        w = int(rng.integers(0, 40))
        try:
            want = oracle.plan_budget(N, Bp, n_a, w)
        except oracle.OracleError:
            with pytest.raises(vec.VectorError):
                vec.vector_plan_budget(N, Bp, n_a, w)
            continue
        got = vec.vector_plan_budget(N, Bp, n_a, w)
        assert (got.n_tokens, got.n_budget_pairs, got.n_a, got.n_pool, got.n_apx, got.n_ret, got.n_evict) == \
               (want.n_tokens, want.n_budget_pairs, want.n_a, want.n_pool, want.n_apx, want.n_ret, want.n_evict)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_calibrate_matches_oracle(oracle, dtype):
    g = torch.Generator().manual_seed(3)
    n, d = 3000, 32
    K = (torch.randn(n, d, generator=g) * torch.exp(torch.rand(d, generator=g) * 2 - 0.7)).to(dtype)
    Wt = torch.randn(d, d, generator=g) / d ** 0.5
    V = (K.float() @ Wt.T + 0.3 * torch.randn(n, d, generator=g)).to(dtype)
    W, r2 = vec.vector_calibrate(K, V, 1e-4, want_r2=True)
    want = oracle.calibrate(K, V, 1e-4)
    assert np.max(np.abs(W.double().numpy() - want)) <= 2e-7 * max(1.0, np.max(np.abs(want)))
    Kd, Vd = K.double().numpy(), V.double().numpy()
    r2_ref = 1 - np.sum((Vd - Kd @ want.T) ** 2) / np.sum((Vd - Vd.mean(0)) ** 2)
    assert r2 == pytest.approx(r2_ref, abs=1e-9)


def test_calibrate_errors():
    K = torch.randn(64, 8)
    K[:, 3] = 0
    V = torch.randn(64, 8)
    with pytest.raises(vec.VectorError) as e:
        vec.vector_calibrate(K, V, 0.0)
    assert e.value.status == -6
    vec.vector_calibrate(K, V, 1e-3)
    with pytest.raises(ValueError):
        vec.vector_calibrate(K, V.double(), 1e-3)


def _shape(**kw):
    base = dict(batch=1, n_layers=1, n_q_heads=4, n_kv_heads=2, head_dim=64, dtype=vec.VECTOR_F32, window=32)
    base.update(kw)
    return vec.Shape(**base)


def test_device_calls_validate_before_touching_the_gpu():
    lib = binding.load_library()
    b = vec.vector_plan_budget(1024, 256, -1, 32)
    sh, bu = _shape()._c(), b._c()
    # null pointers
    assert lib.vector_score(ctypes.byref(sh), None, None, 1024, None, None, None, 0, None) == -1
    assert lib.vector_route(ctypes.byref(sh), ctypes.byref(bu), *([None] * 9), None, 0, None) == -1
    assert lib.vector_compact(ctypes.byref(sh), ctypes.byref(bu), None, None, None, None, None, None) == -1
    assert lib.vector_decode_attn(ctypes.byref(sh), None, None, None, None, 0, 0, None, 0, None) == -1
    # unsupported shapes
    for bad in (_shape(head_dim=96), _shape(n_q_heads=5), _shape(pool_kernel=4), _shape(window=0),
                _shape(n_q_heads=32, n_kv_heads=2), _shape(window=600)):
        assert lib.vector_score(ctypes.byref(bad._c()), 1, 1, 1024, 1, None, None, 0, None) == -2
    assert lib.vector_score(ctypes.byref(_shape(dtype=7)._c()), 1, 1, 1024, 1, None, None, 0, None) == -3
    # N shorter than the window; missing workspace
    assert lib.vector_score(ctypes.byref(sh), 1, 1, 16, 1, None, None, 0, None) == -2
    assert lib.vector_score(ctypes.byref(sh), 256, 256, 1024, 256, None, None, 0, None) == -5
    # the second scorer, the diagnostics and the per-tile decode mode check their arguments the same way
    assert lib.vector_score_keydiff(ctypes.byref(sh), None, 1024, None, None, 0, None) == -1
    assert lib.vector_score_keydiff(ctypes.byref(sh), 256, 0, 256, None, 0, None) == -2
    assert lib.vector_score_keydiff(ctypes.byref(sh), 256, 1024, 256, None, 0, None) == -5
    assert lib.vector_diagnostics(ctypes.byref(sh), ctypes.byref(bu), *([None] * 6), None) == -1
    c = binding._Cache(256, 256, 256, 256, 256, 8, 8, 4, 4)
    assert lib.vector_decode_attn(ctypes.byref(sh), 256, ctypes.byref(c), 256, 256, 0, 1, 256, 1 << 30, None) == -9   # mode 1: bf16/128 only
    assert lib.vector_decode_attn(ctypes.byref(sh), 256, ctypes.byref(c), 256, 256, 0, 2, 256, 1 << 30, None) == -2
    rope = _shape(rope_enabled=1, rope_theta=0.5)
    assert lib.vector_score(ctypes.byref(rope._c()), 1, 1, 1024, 1, None, None, 0, None) == -2                   # theta must exceed 1
    # inconsistent budget
    bad_b = vec.Budget(1024, 256, 128, 999, 256, 128, 640)._c()
    assert lib.vector_pool_select(ctypes.byref(sh), ctypes.byref(bad_b), 256, 256, None, 0, None) == -4
    assert vec.vector_status_string(-4) == "impossible tier sizes"
    assert vec.vector_workspace_bytes(_shape(), b) > 0
    assert vec.vector_workspace_bytes(_shape(head_dim=96), b) == 0


def test_synthetic_inputs_are_deterministic_and_shaped():
    wl = synth.shrink(synth.WORKLOADS[1], N=256, n_calib=64)
    K1, V1, Q1 = synth.context(wl, "cpu", units=[0, 5])
    K2, V2, Q2 = synth.context(wl, "cpu", units=[5])
    assert torch.equal(K1[1], K2[0]) and torch.equal(V1[1], V2[0]) and torch.equal(Q1[1], Q2[0])
    assert K1.shape == (2, 256, 128) and Q1.shape == (2, 4, 64, 128) and K1.dtype == torch.bfloat16
    assert not torch.equal(K1[0], K1[1])
    sk, sq, wt = synth.all_head_params(wl, "cpu")
    assert sk.shape == (8, 128) and float(sk.max()) > 8.0         # an outlier channel x20
    q = synth.decode_q(wl, 3, "cpu", sq)
    assert q.shape == (8, 4, 128)
    assert torch.equal(q[[2]], synth.decode_q(wl, 3, "cpu", sq, units=[2]))
