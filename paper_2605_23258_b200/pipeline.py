"""Buffer ownership and call order around the C-ABI: no arithmetic of the method here.

``Compressor`` allocates (through PyTorch) every buffer the device calls need
once, then ``compress`` issues vector_score -> vector_route -> vector_compact on
the current stream and ``decode`` issues vector_decode_attn.  ``calibrate_maps``
fans vector_calibrate (host least squares) out over host threads.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os

import torch

from . import binding as B


def calibrate_maps(kv_pairs, lam: float, threads: int | None = None, want_r2: bool = False):
    """kv_pairs: iterable of (K [n][d], V [n][d]) host tensors, one per (layer, KV head).
    Returns W fp32 [LH][d][d] (y = W x), and the list of R^2 when asked."""
    pairs = list(kv_pairs)
    threads = threads or min(len(pairs), os.cpu_count() or 1)
    with ThreadPoolExecutor(max_workers=max(threads, 1)) as ex:
        res = list(ex.map(lambda kv: B.vector_calibrate(kv[0], kv[1], lam, want_r2), pairs))
    if want_r2:
        return torch.stack([r[0] for r in res]), [r[1] for r in res]
    return torch.stack(res)


class Compressor:
    """Owns the device buffers of one (shape, budget) and issues the hot-path calls."""

    def __init__(self, shape: B.Shape, budget: B.Budget, extra_rows: int = 0, device="cuda",
                 keep_eps: bool = False):
        self.shape, self.budget, self.device = shape, budget, device
        U, N = shape.units, budget.n_tokens
        self.scores = torch.empty(U, N, dtype=torch.float32, device=device)
        self.tier = torch.empty(U, N, dtype=torch.uint8, device=device)
        self.ret_idx = torch.empty(U, max(budget.n_ret, 1), dtype=torch.int32, device=device)[:, :budget.n_ret]
        self.apx_idx = torch.empty(U, max(budget.n_apx, 1), dtype=torch.int32, device=device)[:, :budget.n_apx]
        self.ret_idx = self.ret_idx.contiguous()
        self.apx_idx = self.apx_idx.contiguous()
        self.eps = torch.empty(U, budget.n_pool, dtype=torch.float32, device=device) if keep_eps else None
        self.pool_idx = torch.empty(U, budget.n_pool, dtype=torch.int32, device=device) if keep_eps else None
        self.cache = B.alloc_cache(shape, budget, extra_rows, device)
        self.ws = B.alloc_workspace(shape, budget, device)

    def score(self, Q_obs, K):
        B.vector_score(self.shape, Q_obs, K, self.budget.n_tokens, self.scores, None, self.ws)

    def route(self, K, V, W):
        B.vector_route(self.shape, self.budget, self.scores, K, V, W, self.tier, self.ret_idx, self.apx_idx,
                       self.eps, self.pool_idx, self.ws)

    def compact(self, K, V):
        self.cache.n_ret, self.cache.n_apx = self.budget.n_ret, self.budget.n_apx
        B.vector_compact(self.shape, self.budget, K, V, self.ret_idx, self.apx_idx, self.cache)

    def compress(self, Q_obs, K, V, W):
        """Prefill-time compression of all units: score, route, compact (asynchronous)."""
        self.score(Q_obs, K)
        self.route(K, V, W)
        self.compact(K, V)
        return self.cache

    def append(self, k_new, v_new, pos: int):
        """Keeps a generated token in full: writes its row behind the retained pool."""
        c = self.cache
        if c.n_ret >= c.ret_k.shape[1]:
            raise ValueError("retained pool is full")
        c.ret_k[:, c.n_ret] = k_new
        c.ret_v[:, c.n_ret] = v_new
        c.ret_pos[:, c.n_ret] = pos
        c.n_ret += 1

    def decode(self, q, W, out, mode: int = 0):
        B.vector_decode_attn(self.shape, q, self.cache, W, out, mode, self.ws)
        return out
