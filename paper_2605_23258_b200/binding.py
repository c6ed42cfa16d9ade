"""ctypes binding of libvector: argument marshalling only.

Every function has the name and the argument order of its C entry point
(``include/vector.h``).  Tensors are ``torch`` tensors used as typed device (or,
for calibration, host) buffers; the binding checks dtype, device and
contiguity, passes raw pointers, and raises :class:`VectorError` on a non-zero
status.  There is no fallback: if the shared library is missing the import of
any entry point fails loudly.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

VECTOR_F32, VECTOR_BF16 = 0, 1
_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libvector.so")
_lib = None


class VectorError(RuntimeError):
    def __init__(self, status: int, where: str):
        text = load_library().vector_status_string(status).decode()
        extra = ""
        if status == -7:
            extra = f" (cudaError {load_library().vector_last_cuda_error()})"
        super().__init__(f"{where}: {text}{extra} [status {status}]")
        self.status = status


class _Shape(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("window", ctypes.c_int32), ("pool_kernel", ctypes.c_int32), ("sm_scale", ctypes.c_float),
                ("rope_enabled", ctypes.c_int32), ("rope_theta", ctypes.c_float)]


class _Budget(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in
                ("n_tokens", "n_budget_pairs", "n_a", "n_pool", "n_apx", "n_ret", "n_evict")]


class _Cache(ctypes.Structure):
    _fields_ = [("ret_k", ctypes.c_void_p), ("ret_v", ctypes.c_void_p), ("apx_k", ctypes.c_void_p),
                ("ret_pos", ctypes.c_void_p), ("apx_pos", ctypes.c_void_p),
                ("cap_ret", ctypes.c_int64), ("cap_apx", ctypes.c_int64),
                ("n_ret", ctypes.c_int64), ("n_apx", ctypes.c_int64)]


@dataclass
class Shape:
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: int
    window: int
    pool_kernel: int = 7
    sm_scale: float = 0.0
    rope_enabled: int = 0
    rope_theta: float = 10000.0

    @property
    def units(self) -> int:
        return self.batch * self.n_layers * self.n_kv_heads

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == VECTOR_BF16 else torch.float32

    def _c(self) -> _Shape:
        return _Shape(self.batch, self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim, self.dtype,
                      self.window, self.pool_kernel, self.sm_scale, self.rope_enabled, self.rope_theta)


@dataclass
class Budget:
    n_tokens: int
    n_budget_pairs: int
    n_a: int
    n_pool: int
    n_apx: int
    n_ret: int
    n_evict: int

    def _c(self) -> _Budget:
        return _Budget(self.n_tokens, self.n_budget_pairs, self.n_a, self.n_pool, self.n_apx, self.n_ret,
                       self.n_evict)


@dataclass
class Cache:
    """Device buffers of the mixed cache plus the row counts in use."""
    ret_k: torch.Tensor      # [U][cap_ret][d]
    ret_v: torch.Tensor      # [U][cap_ret][d]
    apx_k: torch.Tensor      # [U][cap_apx][d]
    ret_pos: torch.Tensor    # [U][cap_ret] int32
    apx_pos: torch.Tensor    # [U][cap_apx] int32
    n_ret: int
    n_apx: int

    def _c(self) -> _Cache:
        return _Cache(self.ret_k.data_ptr(), self.ret_v.data_ptr(), self.apx_k.data_ptr(),
                      self.ret_pos.data_ptr(), self.apx_pos.data_ptr(),
                      self.ret_k.shape[1], self.apx_k.shape[1], self.n_ret, self.n_apx)


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads libvector.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2605_23258_b200.build` "
                          "(nvcc, sm_100a). There is no fallback path.")
    lib = ctypes.CDLL(_LIB_PATH)
    P, I32, I64, SZ = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    SP, BP, CP = ctypes.POINTER(_Shape), ctypes.POINTER(_Budget), ctypes.POINTER(_Cache)
    lib.vector_status_string.restype = ctypes.c_char_p
    lib.vector_status_string.argtypes = [ctypes.c_int]
    lib.vector_last_cuda_error.restype = ctypes.c_int
    lib.vector_last_cuda_error.argtypes = []
    lib.vector_plan_budget.argtypes = [I64, I64, I64, I32, BP]
    lib.vector_calibrate.argtypes = [P, P, I64, I32, I32, I32, ctypes.c_double, P, P]
    lib.vector_workspace_bytes.restype = SZ
    lib.vector_workspace_bytes.argtypes = [SP, BP]
    lib.vector_score.argtypes = [SP, P, P, I64, P, P, P, SZ, P]
    lib.vector_score_keydiff.argtypes = [SP, P, I64, P, P, SZ, P]
    lib.vector_score_keydiff.restype = ctypes.c_int
    lib.vector_pool_select.argtypes = [SP, BP, P, P, P, SZ, P]
    lib.vector_residual.argtypes = [SP, P, P, P, I64, P, I64, P, P]
    lib.vector_truncate.argtypes = [SP, BP, P, P, P, P, P, P, SZ, P]
    lib.vector_route.argtypes = [SP, BP, P, P, P, P, P, P, P, P, P, P, SZ, P]
    lib.vector_compact.argtypes = [SP, BP, P, P, P, P, CP, P]
    lib.vector_diagnostics.argtypes = [SP, BP, P, P, P, P, P, P, P]
    lib.vector_diagnostics.restype = ctypes.c_int
    lib.vector_decode_attn.argtypes = [SP, P, CP, P, P, I32, I32, P, SZ, P]
    lib.vector_decode_scratch_bytes.restype = SZ
    lib.vector_decode_scratch_bytes.argtypes = [SP]
    lib.vector_decode_attn_static.argtypes = [SP, P, CP, P, P, I32, I32, P]
    lib.vector_decode_attn_static.restype = ctypes.c_int
    lib.vector_layer_workspace_bytes.restype = SZ
    lib.vector_layer_workspace_bytes.argtypes = [SP, BP]
    lib.vector_layer_scores.argtypes = [SP, P, I64, P, P]
    lib.vector_residual_layer.argtypes = [SP, P, P, P, I64, P, I64, P, P]
    lib.vector_route_layer.argtypes = [SP, BP, P, P, P, P, P, P, P, P, P, P, SZ, P]
    lib.vector_compact_layer.argtypes = [SP, BP, P, P, P, P, CP, P]
    lib.vector_decode_attn_layer.argtypes = [SP, P, CP, P, P, I32, P, SZ, P]
    lib.vector_r2_global_workspace_bytes.restype = SZ
    lib.vector_r2_global_workspace_bytes.argtypes = [SP, I64]
    lib.vector_r2_global.argtypes = [SP, P, P, P, I64, P, P, SZ, P]
    lib.vector_r2_global.restype = ctypes.c_int
    lib.vector_sync_check.argtypes = [P]
    lib.vector_sync_check.restype = ctypes.c_int
    for name in ("vector_layer_scores", "vector_residual_layer", "vector_route_layer", "vector_compact_layer",
                 "vector_decode_attn_layer"):
        getattr(lib, name).restype = ctypes.c_int
    for name in ("vector_plan_budget", "vector_calibrate", "vector_score", "vector_pool_select",
                 "vector_residual", "vector_truncate", "vector_route", "vector_compact", "vector_decode_attn"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def _check(rc: int, where: str):
    if rc != 0:
        raise VectorError(rc, where)


def _dev(t: torch.Tensor | None, dtype=None, name="tensor"):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ws(ws: torch.Tensor | None):
    if ws is None:
        return None, 0
    return _dev(ws, torch.uint8, "workspace"), ws.numel()


def vector_status_string(status: int) -> str:
    return load_library().vector_status_string(status).decode()


def vector_kernel_launches() -> int:
    """Kernels the library has launched so far in this process."""
    lib = load_library()
    lib.vector_kernel_launches.restype = ctypes.c_uint64
    lib.vector_kernel_launches.argtypes = []
    return int(lib.vector_kernel_launches())


def score_poly_share() -> float:
    """Share of the score passes' exponentials evaluated on the FMA pipe (vector_score_exp2_fma_share)."""
    lib = load_library()
    lib.vector_score_exp2_fma_share.restype = ctypes.c_float
    lib.vector_score_exp2_fma_share.argtypes = []
    return float(lib.vector_score_exp2_fma_share())


def vector_device_fault() -> int:
    """Synchronises the device; returns (and clears) the code of a kernel wait that gave up, 0 if none."""
    lib = load_library()
    lib.vector_device_fault.restype = ctypes.c_int
    return int(lib.vector_device_fault())


def vector_plan_budget(n_tokens: int, n_budget_pairs: int, n_a: int = -1, window: int = 0) -> Budget:
    b = _Budget()
    _check(load_library().vector_plan_budget(n_tokens, n_budget_pairs, n_a, window, ctypes.byref(b)),
           "vector_plan_budget")
    return Budget(*(getattr(b, f[0]) for f in _Budget._fields_))


def vector_calibrate(K: torch.Tensor, V: torch.Tensor, lam: float, want_r2: bool = False):
    """K [n][d_k], V [n][d_v] host tensors (fp32 or bf16) -> W fp32 [d_v][d_k] (and R^2)."""
    if K.is_cuda or V.is_cuda:
        raise ValueError("vector_calibrate works on host tensors")
    if K.dtype != V.dtype or K.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("K and V must both be fp32 or both bf16")
    K, V = K.contiguous(), V.contiguous()
    n, dk = K.shape
    dv = V.shape[1]
    W = torch.empty(dv, dk, dtype=torch.float32)
    r2 = ctypes.c_double(0.0)
    dt = VECTOR_BF16 if K.dtype == torch.bfloat16 else VECTOR_F32
    rc = load_library().vector_calibrate(K.data_ptr(), V.data_ptr(), n, dk, dv, dt, float(lam), W.data_ptr(),
                                         ctypes.cast(ctypes.byref(r2), ctypes.c_void_p) if want_r2 else None)
    _check(rc, "vector_calibrate")
    return (W, r2.value) if want_r2 else W


def vector_workspace_bytes(shape: Shape, budget: Budget) -> int:
    return int(load_library().vector_workspace_bytes(ctypes.byref(shape._c()), ctypes.byref(budget._c())))


def alloc_workspace(shape: Shape, budget: Budget, device="cuda") -> torch.Tensor:
    return torch.empty(vector_workspace_bytes(shape, budget), dtype=torch.uint8, device=device)


def alloc_cache(shape: Shape, budget: Budget, extra_rows: int = 0, device="cuda") -> Cache:
    """Empty mixed cache with room for `extra_rows` appended (generated) tokens per unit."""
    U, d, dt = shape.units, shape.head_dim, shape.torch_dtype
    cap_ret = max(budget.n_ret + extra_rows, 1)
    cap_apx = max(budget.n_apx, 1)
    return Cache(torch.empty(U, cap_ret, d, dtype=dt, device=device),
                 torch.empty(U, cap_ret, d, dtype=dt, device=device),
                 torch.empty(U, cap_apx, d, dtype=dt, device=device),
                 torch.empty(U, cap_ret, dtype=torch.int32, device=device),
                 torch.empty(U, cap_apx, dtype=torch.int32, device=device),
                 budget.n_ret, budget.n_apx)


def vector_score(shape: Shape, Q_obs, K, N: int, scores, raw_out=None, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_score(ctypes.byref(shape._c()), _dev(Q_obs, shape.torch_dtype, "Q_obs"),
                                     _dev(K, shape.torch_dtype, "K"), N, _dev(scores, torch.float32, "scores"),
                                     _dev(raw_out, torch.float32, "raw_out"), wp, wn, _stream(stream))
    _check(rc, "vector_score")


def vector_score_keydiff(shape: Shape, K, N: int, scores, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_score_keydiff(ctypes.byref(shape._c()), _dev(K, shape.torch_dtype, "K"), N,
                                             _dev(scores, torch.float32, "scores"), wp, wn, _stream(stream))
    _check(rc, "vector_score_keydiff")


def vector_pool_select(shape: Shape, budget: Budget, scores, pool_idx, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_pool_select(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                           _dev(scores, torch.float32, "scores"),
                                           _dev(pool_idx, torch.int32, "pool_idx"), wp, wn, _stream(stream))
    _check(rc, "vector_pool_select")


def vector_residual(shape: Shape, K, V, W, N: int, idx, n_idx: int, eps, stream=None):
    rc = load_library().vector_residual(ctypes.byref(shape._c()), _dev(K, shape.torch_dtype, "K"),
                                        _dev(V, shape.torch_dtype, "V"), _dev(W, shape.torch_dtype, "W"), N,
                                        _dev(idx, torch.int32, "idx"), n_idx, _dev(eps, torch.float32, "eps"),
                                        _stream(stream))
    _check(rc, "vector_residual")


def vector_truncate(shape: Shape, budget: Budget, eps, pool_idx, tier, ret_idx, apx_idx, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_truncate(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                        _dev(eps, torch.float32, "eps"), _dev(pool_idx, torch.int32, "pool_idx"),
                                        _dev(tier, torch.uint8, "tier"), _dev(ret_idx, torch.int32, "ret_idx"),
                                        _dev(apx_idx, torch.int32, "apx_idx"), wp, wn, _stream(stream))
    _check(rc, "vector_truncate")


def vector_route(shape: Shape, budget: Budget, scores, K, V, W, tier, ret_idx, apx_idx, eps_out=None,
                 pool_idx_out=None, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_route(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                     _dev(scores, torch.float32, "scores"), _dev(K, shape.torch_dtype, "K"),
                                     _dev(V, shape.torch_dtype, "V"), _dev(W, shape.torch_dtype, "W"),
                                     _dev(tier, torch.uint8, "tier"), _dev(ret_idx, torch.int32, "ret_idx"),
                                     _dev(apx_idx, torch.int32, "apx_idx"), _dev(eps_out, torch.float32, "eps_out"),
                                     _dev(pool_idx_out, torch.int32, "pool_idx_out"), wp, wn, _stream(stream))
    _check(rc, "vector_route")


DIAG_FIELDS = ("E", "r2_approx", "mu_a", "sum_evicted_w", "sum_approximated_w", "w_bar", "w_star", "threshold")


def vector_diagnostics(shape: Shape, budget: Budget, importance, tier, pool_idx, eps, V, out, stream=None):
    """out [U][8] fp32: the DIAG_FIELDS of every unit."""
    rc = load_library().vector_diagnostics(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                           _dev(importance, torch.float32, "importance"), _dev(tier, torch.uint8, "tier"),
                                           _dev(pool_idx, torch.int32, "pool_idx"), _dev(eps, torch.float32, "eps"),
                                           _dev(V, shape.torch_dtype, "V"), _dev(out, torch.float32, "out"), _stream(stream))
    _check(rc, "vector_diagnostics")


R2_FIELDS = ("r2", "ss_res", "ss_tot", "n")


def vector_r2_global_workspace_bytes(shape: Shape, N: int) -> int:
    return int(load_library().vector_r2_global_workspace_bytes(ctypes.byref(shape._c()), N))


def vector_r2_global(shape: Shape, K, V, W, N: int, out, ws, stream=None):
    """out [U][4] fp32: the R2_FIELDS of every unit over all N tokens."""
    wp, wn = _ws(ws)
    rc = load_library().vector_r2_global(ctypes.byref(shape._c()), _dev(K, shape.torch_dtype, "K"),
                                         _dev(V, shape.torch_dtype, "V"), _dev(W, shape.torch_dtype, "W"),
                                         N, _dev(out, torch.float32, "out"), wp, wn, _stream(stream))
    _check(rc, "vector_r2_global")


def vector_sync_check(stream=None):
    """Waits for the stream; raises VectorError(VECTOR_ERR_TIMEOUT) if a bounded wait inside a kernel gave up."""
    _check(load_library().vector_sync_check(_stream(stream)), "vector_sync_check")


def vector_compact(shape: Shape, budget: Budget, K, V, ret_idx, apx_idx, cache: Cache, stream=None):
    c = cache._c()
    rc = load_library().vector_compact(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                       _dev(K, shape.torch_dtype, "K"), _dev(V, shape.torch_dtype, "V"),
                                       _dev(ret_idx, torch.int32, "ret_idx"), _dev(apx_idx, torch.int32, "apx_idx"),
                                       ctypes.byref(c), _stream(stream))
    _check(rc, "vector_compact")


def vector_decode_attn(shape: Shape, q, cache: Cache, W, out, mode: int = 0, ws=None, stream=None):
    wp, wn = _ws(ws)
    c = cache._c()
    if out.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("out must be fp32 or bf16")
    out_dt = VECTOR_BF16 if out.dtype == torch.bfloat16 else VECTOR_F32
    rc = load_library().vector_decode_attn(ctypes.byref(shape._c()), _dev(q, shape.torch_dtype, "q"),
                                           ctypes.byref(c), _dev(W, shape.torch_dtype, "W"), _dev(out, None, "out"),
                                           out_dt, mode, wp, wn, _stream(stream))
    _check(rc, "vector_decode_attn")


# ---- one map per layer: scores, tiers and index lists per (sequence, layer); pools per head
def vector_layer_workspace_bytes(shape: Shape, budget: Budget) -> int:
    return int(load_library().vector_layer_workspace_bytes(ctypes.byref(shape._c()), ctypes.byref(budget._c())))


def vector_layer_scores(shape: Shape, scores, N: int, layer_scores, stream=None):
    rc = load_library().vector_layer_scores(ctypes.byref(shape._c()), _dev(scores, torch.float32, "scores"), N,
                                            _dev(layer_scores, torch.float32, "layer_scores"), _stream(stream))
    _check(rc, "vector_layer_scores")


def vector_residual_layer(shape: Shape, K, V, W_layer, N: int, idx, n_idx: int, eps, stream=None):
    rc = load_library().vector_residual_layer(ctypes.byref(shape._c()), _dev(K, shape.torch_dtype, "K"),
                                              _dev(V, shape.torch_dtype, "V"), _dev(W_layer, shape.torch_dtype, "W_layer"),
                                              N, _dev(idx, torch.int32, "idx"), n_idx, _dev(eps, torch.float32, "eps"),
                                              _stream(stream))
    _check(rc, "vector_residual_layer")


def vector_route_layer(shape: Shape, budget: Budget, layer_scores, K, V, W_layer, tier, ret_idx, apx_idx,
                       eps_out=None, pool_idx_out=None, ws=None, stream=None):
    wp, wn = _ws(ws)
    rc = load_library().vector_route_layer(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                           _dev(layer_scores, torch.float32, "layer_scores"),
                                           _dev(K, shape.torch_dtype, "K"), _dev(V, shape.torch_dtype, "V"),
                                           _dev(W_layer, shape.torch_dtype, "W_layer"), _dev(tier, torch.uint8, "tier"),
                                           _dev(ret_idx, torch.int32, "ret_idx"), _dev(apx_idx, torch.int32, "apx_idx"),
                                           _dev(eps_out, torch.float32, "eps_out"),
                                           _dev(pool_idx_out, torch.int32, "pool_idx_out"), wp, wn, _stream(stream))
    _check(rc, "vector_route_layer")


def vector_compact_layer(shape: Shape, budget: Budget, K, V, ret_idx, apx_idx, cache: Cache, stream=None):
    c = cache._c()
    rc = load_library().vector_compact_layer(ctypes.byref(shape._c()), ctypes.byref(budget._c()),
                                             _dev(K, shape.torch_dtype, "K"), _dev(V, shape.torch_dtype, "V"),
                                             _dev(ret_idx, torch.int32, "ret_idx"), _dev(apx_idx, torch.int32, "apx_idx"),
                                             ctypes.byref(c), _stream(stream))
    _check(rc, "vector_compact_layer")


def vector_decode_attn_layer(shape: Shape, q, cache: Cache, W_layer, out, ws=None, stream=None):
    wp, wn = _ws(ws)
    c = cache._c()
    if out.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("out must be fp32 or bf16")
    out_dt = VECTOR_BF16 if out.dtype == torch.bfloat16 else VECTOR_F32
    rc = load_library().vector_decode_attn_layer(ctypes.byref(shape._c()), _dev(q, shape.torch_dtype, "q"),
                                                 ctypes.byref(c), _dev(W_layer, shape.torch_dtype, "W_layer"),
                                                 _dev(out, None, "out"), out_dt, wp, wn, _stream(stream))
    _check(rc, "vector_decode_attn_layer")


VECTOR_STATIC_SCRATCH_BYTES = 16 << 20


def vector_decode_scratch_bytes(shape: Shape) -> int:
    """Bytes of split-KV scratch a decode call of this shape needs (0 for an unsupported shape)."""
    return int(load_library().vector_decode_scratch_bytes(ctypes.byref(shape._c())))


def vector_decode_attn_static(shape: Shape, q, cache: Cache, W, out, mode: int = 0, stream=None):
    """vector_decode_attn without a workspace argument and without any allocation.

    For callers that cannot get device memory when they call (their own pool owns the
    device, or a cudaMalloc stall is unacceptable inside the decode loop): the partial
    results go to a fixed VECTOR_STATIC_SCRATCH_BYTES array inside the library.  Shapes
    that need more raise VectorError (workspace).  Calls on one device share that array,
    so calls that overlap on the GPU race; make the first call per device at start-up.
    """
    c = cache._c()
    if out.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("out must be fp32 or bf16")
    out_dt = VECTOR_BF16 if out.dtype == torch.bfloat16 else VECTOR_F32
    rc = load_library().vector_decode_attn_static(ctypes.byref(shape._c()), _dev(q, shape.torch_dtype, "q"),
                                                  ctypes.byref(c), _dev(W, shape.torch_dtype, "W"),
                                                  _dev(out, None, "out"), out_dt, mode, _stream(stream))
    _check(rc, "vector_decode_attn_static")
