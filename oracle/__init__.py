"""ctypes front end of the VECTOR oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Loads ``liboracle.so`` (plain C, fp64, single-threaded; built from
``vector_oracle.c`` with gcc) and marshals numpy arrays into it.  Only tests,
the smoke check and the CPU-baseline leg of the benchmark may import this
package; the CUDA library and its Python binding never do.

Every function takes ONE unit = one (sequence, layer, KV head).  Tensors may be
numpy arrays or torch CPU tensors of any float dtype: they are widened to
float64 exactly (bf16 and fp32 are subsets of fp64), so the oracle computes on
the same stored bits the kernels read.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vector_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")

OK, ERR_ARG, ERR_BUDGET, ERR_SINGULAR = 0, -1, -2, -3


class OracleError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"oracle {where} failed with code {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no CUDA involved); returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_p_a_deploy.restype = ctypes.c_double
        _lib.oracle_p_a_deploy.argtypes = [ctypes.c_double, ctypes.c_double]
    return _lib


class _Budget(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("n_tokens", "n_budget_pairs", "n_a", "n_pool", "n_apx", "n_ret", "n_evict")]


@dataclass(frozen=True)
class Budget:
    n_tokens: int
    n_budget_pairs: int
    n_a: int
    n_pool: int
    n_apx: int
    n_ret: int
    n_evict: int


def _f64(x) -> np.ndarray:
    if hasattr(x, "detach"):                     # torch tensor (cpu)
        import torch
        x = x.detach().to("cpu", torch.float64).numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _f32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        import torch
        x = x.detach().to("cpu", torch.float32).numpy()
    return np.ascontiguousarray(x, dtype=np.float32)


def _i32(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().cpu().numpy()
    return np.ascontiguousarray(x, dtype=np.int32)


def _p(a: np.ndarray | None):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, where: str):
    if rc != OK:
        raise OracleError(rc, where)


def p_a_deploy(p_c: float, eps: float = 0.0) -> float:
    """Eq. (1) in real numbers."""
    return float(lib().oracle_p_a_deploy(p_c, eps))


def budget_pairs(n_tokens: int, budget_percent: int) -> int:
    """Bp = floor(N * percent / 100) in integer arithmetic."""
    return (int(n_tokens) * int(budget_percent)) // 100


def plan_budget(n_tokens: int, n_budget_pairs: int, n_a: int = -1, window: int = 0) -> Budget:
    b = _Budget()
    rc = lib().oracle_plan_budget(ctypes.c_int64(n_tokens), ctypes.c_int64(n_budget_pairs),
                                  ctypes.c_int64(n_a), ctypes.c_int32(window), ctypes.byref(b))
    _check(rc, "plan_budget")
    return Budget(*(getattr(b, f[0]) for f in _Budget._fields_))


def calibrate(K, V, lam: float) -> np.ndarray:
    """W [d_v][d_k] (y = W x) minimising sum ||W k - v||^2 + lam ||W||_F^2."""
    K, V = _f64(K), _f64(V)
    n, dk = K.shape
    dv = V.shape[1]
    W = np.empty((dv, dk), dtype=np.float64)
    rc = lib().oracle_calibrate(_p(K), _p(V), ctypes.c_int64(n), ctypes.c_int32(dk),
                                ctypes.c_int32(dv), ctypes.c_double(lam), _p(W))
    _check(rc, "calibrate")
    return W


def score(Q, K, scale: float, pool_kernel: int):
    """Q [g][w][d], K [N][d] -> (raw [N], score [N]) float64."""
    Q, K = _f64(Q), _f64(K)
    g, w, d = Q.shape
    N = K.shape[0]
    raw = np.empty(N, dtype=np.float64)
    sc = np.empty(N, dtype=np.float64)
    rc = lib().oracle_score(_p(Q), _p(K), ctypes.c_int32(g), ctypes.c_int32(w), ctypes.c_int32(d),
                            ctypes.c_int64(N), ctypes.c_double(scale), ctypes.c_int32(pool_kernel),
                            _p(raw), _p(sc))
    _check(rc, "score")
    return raw, sc


def score_keydiff(K) -> np.ndarray:
    """Key-geometry scorer: K [N][d] -> score [N] float64 (minus the cosine to the mean unit key)."""
    K = _f64(K)
    N, d = K.shape
    sc = np.empty(N, dtype=np.float64)
    rc = lib().oracle_score_keydiff(_p(K), ctypes.c_int32(d), ctypes.c_int64(N), _p(sc))
    _check(rc, "score_keydiff")
    return sc


def pool_select(score_f32, n_pool: int) -> np.ndarray:
    s = _f32(score_f32)
    out = np.empty(n_pool, dtype=np.int32)
    rc = lib().oracle_pool_select(_p(s), ctypes.c_int64(s.shape[0]), ctypes.c_int64(n_pool), _p(out))
    _check(rc, "pool_select")
    return out


def residual(K, V, W, idx, rope: bool = False, theta: float = 10000.0) -> np.ndarray:
    K, V, W, idx = _f64(K), _f64(V), _f64(W), _i32(idx)
    d = K.shape[1]
    eps = np.empty(idx.shape[0], dtype=np.float64)
    rc = lib().oracle_residual(_p(K), _p(V), _p(W), ctypes.c_int32(d), _p(idx),
                               ctypes.c_int64(idx.shape[0]), ctypes.c_int32(int(rope)),
                               ctypes.c_double(theta), _p(eps))
    _check(rc, "residual")
    return eps


def truncate(eps_f32, pool_idx, n_apx: int, N: int):
    """-> (tier uint8 [N], ret_idx, apx_idx) ; eps in pool order, fp32."""
    e, pool = _f32(eps_f32), _i32(pool_idx)
    n_pool = pool.shape[0]
    tier = np.empty(N, dtype=np.uint8)
    ret = np.empty(max(n_pool - n_apx, 0), dtype=np.int32)
    apx = np.empty(n_apx, dtype=np.int32)
    rc = lib().oracle_truncate(_p(e), _p(pool), ctypes.c_int64(n_pool), ctypes.c_int64(n_apx),
                               ctypes.c_int64(N), _p(tier), _p(ret), _p(apx))
    _check(rc, "truncate")
    return tier, ret, apx


def route(score_f32, K, V, W, n_pool: int, n_apx: int, rope: bool = False, theta: float = 10000.0):
    """Steps 1-3 -> dict(tier, ret_idx, apx_idx, eps (float64, pool order), pool_idx)."""
    s, K, V, W = _f32(score_f32), _f64(K), _f64(V), _f64(W)
    N, d = K.shape
    tier = np.empty(N, dtype=np.uint8)
    ret = np.empty(n_pool - n_apx, dtype=np.int32)
    apx = np.empty(n_apx, dtype=np.int32)
    eps = np.empty(n_pool, dtype=np.float64)
    pool = np.empty(n_pool, dtype=np.int32)
    rc = lib().oracle_route(_p(s), _p(K), _p(V), _p(W), ctypes.c_int64(N), ctypes.c_int32(d),
                            ctypes.c_int64(n_pool), ctypes.c_int64(n_apx), ctypes.c_int32(int(rope)),
                            ctypes.c_double(theta), _p(tier), _p(ret), _p(apx), _p(eps), _p(pool))
    _check(rc, "route")
    return dict(tier=tier, ret_idx=ret, apx_idx=apx, eps=eps, pool_idx=pool)


DIAG_FIELDS = ("E", "r2_approx", "mu_a", "sum_evicted_w", "sum_approximated_w", "w_bar", "w_star", "threshold")


def diagnostics(importance, tier, K, V, W) -> dict:
    """Distortion E, R^2 over the approximated set and the threshold of Proposition 1 for one routed unit."""
    imp, K, V, W = _f64(importance), _f64(K), _f64(V), _f64(W)
    t = np.ascontiguousarray(np.asarray(tier, dtype=np.uint8))
    N, d = K.shape
    out = np.empty(8, dtype=np.float64)
    rc = lib().oracle_diagnostics(_p(imp), _p(t), _p(K), _p(V), _p(W), ctypes.c_int64(N), ctypes.c_int32(d), _p(out))
    _check(rc, "diagnostics")
    return dict(zip(DIAG_FIELDS, out.tolist()))


def r2_global(K, V, W) -> dict:
    """K -> V predictability of a fixed map over a whole context (Section 3.1, "Empirical Evidence"):
    R^2 = 1 - sum_i ||v_i - W k_i||^2 / sum_i ||v_i - mean(v)||^2 over ALL tokens, the residual of each token
    taken by the residual step itself (identity index list)."""
    K, V, W = _f64(K), _f64(V), _f64(W)
    N = K.shape[0]
    eps = residual(K, V, W, np.arange(N, dtype=np.int32))
    ss_res = float(np.sum(eps))
    mean = np.zeros(V.shape[1])
    for i in range(N):
        mean += V[i]
    mean /= N
    ss_tot = 0.0
    for i in range(N):
        ss_tot += float(np.sum((V[i] - mean) ** 2))
    r2 = 1.0 - ss_res / ss_tot if ss_tot > 0.0 else (1.0 if ss_res == 0.0 else -np.inf)
    return dict(r2=r2, ss_res=ss_res, ss_tot=ss_tot, n=N)


def gather_rows(src, idx):
    """-> (rows [n_idx][d] float64, pos int32)."""
    src, idx = _f64(src), _i32(idx)
    d = src.shape[1]
    dst = np.empty((idx.shape[0], d), dtype=np.float64)
    pos = np.empty(idx.shape[0], dtype=np.int32)
    rc = lib().oracle_gather_rows(_p(src), ctypes.c_int32(d), _p(idx), ctypes.c_int64(idx.shape[0]),
                                  _p(dst), _p(pos))
    _check(rc, "gather_rows")
    return dst, pos


def attend(q, ret_k, ret_v, apx_k, W, scale: float, apx_pos=None, rope: bool = False,
           theta: float = 10000.0):
    """Mixed-cache attention -> (o_per_token [g][d], o_factored [g][d]) float64."""
    q, W = _f64(q), _f64(W)
    g, d = q.shape
    ret_k = _f64(ret_k).reshape(-1, d)
    ret_v = _f64(ret_v).reshape(-1, d)
    apx_k = _f64(apx_k).reshape(-1, d)
    n_ret, n_apx = ret_k.shape[0], apx_k.shape[0]
    pos = _i32(apx_pos) if apx_pos is not None else np.zeros(max(n_apx, 1), dtype=np.int32)
    o1 = np.empty((g, d), dtype=np.float64)
    o2 = np.empty((g, d), dtype=np.float64)
    rc = lib().oracle_attend(_p(q), ctypes.c_int32(g), ctypes.c_int32(d), _p(ret_k), _p(ret_v),
                             ctypes.c_int64(n_ret), _p(apx_k), _p(pos), ctypes.c_int64(n_apx), _p(W),
                             ctypes.c_double(scale), ctypes.c_int32(int(rope)), ctypes.c_double(theta),
                             _p(o1), _p(o2))
    _check(rc, "attend")
    return o1, o2


# ---- one map per layer (Section 5.1 calibrates the map layer-wise): the same steps on the keys and
# values concatenated over the layer's KV heads.  Tensors come head-major, [Hkv][N][d].
def concat_heads(X) -> np.ndarray:
    """[Hkv][N][d] -> [N][Hkv d]: a token's vector over the whole layer."""
    X = _f64(X)
    Hkv, N, d = X.shape
    return np.ascontiguousarray(X.transpose(1, 0, 2).reshape(N, Hkv * d))


def calibrate_layer(K, V, lam: float) -> np.ndarray:
    """K, V [Hkv][n][d] -> W [Hkv d][Hkv d] minimising sum ||W k - v||^2 + lam ||W||_F^2 over whole-layer vectors."""
    return calibrate(concat_heads(K), concat_heads(V), lam)


def layer_score(scores_per_head) -> np.ndarray:
    """The routing decision holds for a token of the layer: its score is the sum of its per-head base scores."""
    return np.asarray(scores_per_head, dtype=np.float64).sum(axis=0)


def residual_layer(K, V, W, idx) -> np.ndarray:
    """eps_i = || v_i - W k_i ||^2 over the whole-layer vectors; K, V [Hkv][N][d], W [Hkv d][Hkv d]."""
    return residual(concat_heads(K), concat_heads(V), W, idx)


def route_layer(layer_score_f32, K, V, W, n_pool: int, n_apx: int):
    """Steps 1-3 per layer: one tier per token for all heads.  Same dict as route()."""
    return route(layer_score_f32, concat_heads(K), concat_heads(V), W, n_pool, n_apx)


def attend_layer(q, ret_k, ret_v, apx_k, W, scale: float):
    """q [Hq][d]; ret_k, ret_v [Hkv][n_ret][d]; apx_k [Hkv][n_apx][d]; W [Hkv d][Hkv d]
    -> (o_per_token [Hq][d], o_factored [Hq][d]) float64."""
    q, W = _f64(q), _f64(W)
    Hq, d = q.shape
    Hkv = W.shape[0] // d
    def cat(X):
        X = _f64(X).reshape(Hkv, -1, d)
        return concat_heads(X) if X.shape[1] > 0 else np.zeros((0, Hkv * d))
    rk, rv, ak = cat(ret_k), cat(ret_v), cat(apx_k)
    o1 = np.empty((Hq, d), dtype=np.float64)
    o2 = np.empty((Hq, d), dtype=np.float64)
    rc = lib().oracle_attend_layer(_p(q), ctypes.c_int32(Hq), ctypes.c_int32(Hkv), ctypes.c_int32(d),
                                   _p(rk), _p(rv), ctypes.c_int64(rk.shape[0]), _p(ak), ctypes.c_int64(ak.shape[0]),
                                   _p(W), ctypes.c_double(scale), _p(o1), _p(o2))
    _check(rc, "attend_layer")
    return o1, o2


def rope_inverse(k, pos: int, theta: float = 10000.0) -> np.ndarray:
    k = _f64(k)
    out = np.empty_like(k)
    lib().oracle_rope_inverse(_p(k), ctypes.c_int32(k.shape[0]), ctypes.c_int64(pos),
                              ctypes.c_double(theta), _p(out))
    return out


def rope_forward(k, pos: int, theta: float = 10000.0) -> np.ndarray:
    k = _f64(k)
    out = np.empty_like(k)
    lib().oracle_rope_forward(_p(k), ctypes.c_int32(k.shape[0]), ctypes.c_int64(pos),
                              ctypes.c_double(theta), _p(out))
    return out
