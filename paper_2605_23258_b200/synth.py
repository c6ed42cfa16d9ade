"""Seeded synthetic workloads shaped like the paper's long-context KV caches.

Input generation only: nothing of the method's arithmetic lives here.  The
five workloads follow the benchmark configurations (Llama-3-8B / Mistral-7B /
Llama-3-70B KV geometry); they stand in for the long-context evaluation suites
the paper measures on, whose text and model weights are not available here.

Law of one unit (one sequence, layer, KV head), all draws from a torch Philox
generator keyed by (seed, workload, stream, layer, head, batch):
  sigma_K[c], sigma_Q[c] = exp(U(ln 0.5, ln 4))            per (layer, head)
  outlier key channels (a fraction of d) have sigma_K x 20  per (layer, head)
  W_true = N(0,1) / sqrt(d)                                  per (layer, head)
  K_i = sigma_K * z ;  Q = sigma_Q * z
  V_i = W_true K_i + s_i * z,  s_i per token: {0.05, 1.0} w.p. 1/2 ("two_level")
        or exp(U(ln 0.02, ln 2)) ("loguniform"), times a per-layer factor that
        runs linearly from layer_noise[0] to layer_noise[1] when given.
V is formed in fp32 from the fp32 key, then K, V, Q are rounded once to the
workload dtype; those rounded values are the inputs of every implementation.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import torch

SEED = 42

_STREAM = {"head": 1, "ctx": 2, "qobs": 3, "calib": 4, "dec_q": 5, "dec_kv": 6}


@dataclass(frozen=True)
class Workload:
    name: str
    wid: int
    batch: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                 # "fp32" | "bf16"
    N: int
    window: int
    pool_kernel: int
    budget_percents: tuple
    noise: str                 # "two_level" | "loguniform"
    layer_noise: tuple | None
    outlier_frac: float
    n_calib: int
    lam: float
    decode_steps: int

    @property
    def units(self) -> int:
        return self.batch * self.n_layers * self.n_kv_heads

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def unit_index(self, b: int, l: int, h: int) -> int:
        return (b * self.n_layers + l) * self.n_kv_heads + h

    def unit_coords(self, u: int):
        h = u % self.n_kv_heads
        l = (u // self.n_kv_heads) % self.n_layers
        b = u // (self.n_kv_heads * self.n_layers)
        return b, l, h


WORKLOADS = {
    0: Workload("config0_tiny_fp32", 0, 1, 1, 4, 2, 64, "fp32", 1024, 32, 7, (25,), "two_level", None, 0.0,
                4096, 1e-4, 8),
    1: Workload("config1_llama3_8b_layer_slice", 1, 1, 1, 32, 8, 128, "bf16", 8192, 64, 7, (10, 20, 40),
                "loguniform", None, 0.01, 16384, 1e-4, 128),
    2: Workload("config2_llama3_8b_32layers_n32768", 2, 1, 32, 32, 8, 128, "bf16", 32768, 64, 7, (20,),
                "loguniform", (0.05, 1.5), 0.01, 4096, 1e-4, 256),
    3: Workload("config3_mistral_7b_batch8_n16384", 3, 8, 32, 32, 8, 128, "bf16", 16384, 64, 7, (10,),
                "loguniform", (0.05, 1.5), 0.01, 4096, 1e-4, 512),
    4: Workload("config4_llama3_70b_80layers_n131072", 4, 1, 80, 64, 8, 128, "bf16", 131072, 128, 7, (5,),
                "loguniform", (0.05, 1.5), 0.02, 4096, 1e-4, 64),
}


def shrink(wl: Workload, **kw) -> Workload:
    """A smaller variant of a workload (same law) for parity tests."""
    return replace(wl, **kw)


def _mix(*ints: int) -> int:
    x = 0x9E3779B97F4A7C15
    for v in ints:
        x ^= (int(v) + 0x9E3779B97F4A7C15 + ((x << 6) & 0xFFFFFFFFFFFFFFFF) + (x >> 2)) & 0xFFFFFFFFFFFFFFFF
        x = (x * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        x ^= x >> 31
    return x & 0x7FFFFFFFFFFFFFFF


def _gen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(_mix(SEED, *key))
    return g


def _loguniform(shape, lo, hi, gen, device):
    u = torch.rand(shape, generator=gen, device=device, dtype=torch.float32)
    return torch.exp(math.log(lo) + u * (math.log(hi) - math.log(lo)))


def head_params(wl: Workload, l: int, h: int, device):
    """-> sigma_K [d], sigma_Q [d], W_true [d][d] (fp32) for one (layer, KV head)."""
    d = wl.head_dim
    gen = _gen(device, wl.wid, _STREAM["head"], l, h)
    sigma_k = _loguniform((d,), 0.5, 4.0, gen, device)
    sigma_q = _loguniform((d,), 0.5, 4.0, gen, device)
    w_true = torch.randn(d, d, generator=gen, device=device, dtype=torch.float32) / math.sqrt(d)
    if wl.outlier_frac > 0:
        n_out = max(1, round(wl.outlier_frac * d))
        perm = torch.randperm(d, generator=gen, device=device)
        sigma_k[perm[:n_out]] *= 20.0
    return sigma_k, sigma_q, w_true


def _layer_factor(wl: Workload, l: int) -> float:
    if wl.layer_noise is None:
        return 1.0
    lo, hi = wl.layer_noise
    return lo if wl.n_layers == 1 else lo + (hi - lo) * l / (wl.n_layers - 1)


def _kv(wl: Workload, gen, n: int, sigma_k, w_true, l: int, device):
    d = wl.head_dim
    k = torch.randn(n, d, generator=gen, device=device, dtype=torch.float32) * sigma_k
    if wl.noise == "two_level":
        pick = torch.rand(n, generator=gen, device=device) < 0.5
        s = torch.where(pick, torch.tensor(0.05, device=device), torch.tensor(1.0, device=device))
    else:
        s = _loguniform((n,), 0.02, 2.0, gen, device)
    s = s * _layer_factor(wl, l)
    z = torch.randn(n, d, generator=gen, device=device, dtype=torch.float32)
    v = k @ w_true.T + s[:, None] * z
    return k.to(wl.torch_dtype), v.to(wl.torch_dtype)


def unit_kv(wl: Workload, b: int, l: int, h: int, device, params=None):
    """Context K, V [N][d] of one unit in the workload dtype."""
    sigma_k, _, w_true = params if params is not None else head_params(wl, l, h, device)
    return _kv(wl, _gen(device, wl.wid, _STREAM["ctx"], l, h, b), wl.N, sigma_k, w_true, l, device)


def unit_qobs(wl: Workload, b: int, l: int, h: int, device, params=None):
    """Observation-window queries [g][w][d] of one unit."""
    _, sigma_q, _ = params if params is not None else head_params(wl, l, h, device)
    gen = _gen(device, wl.wid, _STREAM["qobs"], l, h, b)
    q = torch.randn(wl.group, wl.window, wl.head_dim, generator=gen, device=device, dtype=torch.float32)
    return (q * sigma_q).to(wl.torch_dtype)


def calib_kv(wl: Workload, l: int, h: int, device, params=None):
    """Calibration draw K, V [n_calib][d] for one (layer, KV head): separate seed, same law."""
    sigma_k, _, w_true = params if params is not None else head_params(wl, l, h, device)
    return _kv(wl, _gen(device, wl.wid, _STREAM["calib"], l, h), wl.n_calib, sigma_k, w_true, l, device)


def context(wl: Workload, device, units=None):
    """K, V [U'][N][d] and Q_obs [U'][g][w][d] for all units (or the listed unit indices)."""
    units = list(range(wl.units)) if units is None else list(units)
    K = torch.empty(len(units), wl.N, wl.head_dim, dtype=wl.torch_dtype, device=device)
    V = torch.empty_like(K)
    Q = torch.empty(len(units), wl.group, wl.window, wl.head_dim, dtype=wl.torch_dtype, device=device)
    cache = {}
    for j, u in enumerate(units):
        b, l, h = wl.unit_coords(u)
        if (l, h) not in cache:
            cache[(l, h)] = head_params(wl, l, h, device)
        K[j], V[j] = unit_kv(wl, b, l, h, device, cache[(l, h)])
        Q[j] = unit_qobs(wl, b, l, h, device, cache[(l, h)])
    return K, V, Q


# ---- one map per layer: values depend on the keys of all heads of the layer ------------------------
def layer_params(wl: Workload, l: int, device):
    """-> sigma_K [Hkv][d], sigma_Q [Hkv][d], W_true [Hkv d][Hkv d] (fp32) for one layer: the channel scales of
    its heads and a dense whole-layer map (cross-head blocks included)."""
    per_head = [head_params(wl, l, h, device) for h in range(wl.n_kv_heads)]
    D = wl.n_kv_heads * wl.head_dim
    gen = _gen(device, wl.wid, _STREAM["head"], l, 10**6)
    w_true = torch.randn(D, D, generator=gen, device=device, dtype=torch.float32) / math.sqrt(D)
    return torch.stack([p[0] for p in per_head]), torch.stack([p[1] for p in per_head]), w_true


def _layer_kv(wl: Workload, gen, n: int, sigma_k, w_true, l: int, device):
    Hkv, d = wl.n_kv_heads, wl.head_dim
    k = torch.randn(n, Hkv, d, generator=gen, device=device, dtype=torch.float32) * sigma_k[None]
    if wl.noise == "two_level":
        pick = torch.rand(n, generator=gen, device=device) < 0.5
        s = torch.where(pick, torch.tensor(0.05, device=device), torch.tensor(1.0, device=device))
    else:
        s = _loguniform((n,), 0.02, 2.0, gen, device)
    s = s * _layer_factor(wl, l)
    z = torch.randn(n, Hkv * d, generator=gen, device=device, dtype=torch.float32)
    v = k.reshape(n, Hkv * d) @ w_true.T + s[:, None] * z
    k = k.permute(1, 0, 2).contiguous().to(wl.torch_dtype)                       # [Hkv][n][d]
    v = v.reshape(n, Hkv, d).permute(1, 0, 2).contiguous().to(wl.torch_dtype)
    return k, v


def layer_kv(wl: Workload, b: int, l: int, device, params=None):
    """Context K, V [Hkv][N][d] of one (sequence, layer): V = W_true K + noise over whole-layer vectors."""
    sigma_k, _, w_true = params if params is not None else layer_params(wl, l, device)
    return _layer_kv(wl, _gen(device, wl.wid, _STREAM["ctx"], l, 10**6, b), wl.N, sigma_k, w_true, l, device)


def layer_calib_kv(wl: Workload, l: int, device, params=None):
    """Calibration draw K, V [Hkv][n_calib][d] for one layer: separate seed, same law."""
    sigma_k, _, w_true = params if params is not None else layer_params(wl, l, device)
    return _layer_kv(wl, _gen(device, wl.wid, _STREAM["calib"], l, 10**6), wl.n_calib, sigma_k, w_true, l, device)


def all_head_params(wl: Workload, device):
    """Stacked sigma_K [LH][d], sigma_Q [LH][d], W_true [LH][d][d]."""
    sk, sq, wt = [], [], []
    for l in range(wl.n_layers):
        for h in range(wl.n_kv_heads):
            a, b, c = head_params(wl, l, h, device)
            sk.append(a), sq.append(b), wt.append(c)
    return torch.stack(sk), torch.stack(sq), torch.stack(wt)


def decode_q(wl: Workload, step: int, device, sigma_q_all, units=None):
    """Decode-step queries [U'][g][d]."""
    units = torch.arange(wl.units) if units is None else torch.as_tensor(list(units))
    lh = (units % (wl.n_layers * wl.n_kv_heads)).to(device)
    gen = _gen(device, wl.wid, _STREAM["dec_q"], step)
    z = torch.randn(wl.units, wl.group, wl.head_dim, generator=gen, device=device, dtype=torch.float32)
    z = z[units.to(device)]
    return (z * sigma_q_all[lh][:, None, :]).to(wl.torch_dtype)


def decode_kv(wl: Workload, step: int, device, sigma_k_all, w_true_all, units=None):
    """K, V rows [U'][d] of the token generated at `step` (kept in full in the retained pool)."""
    units = torch.arange(wl.units) if units is None else torch.as_tensor(list(units))
    lh = (units % (wl.n_layers * wl.n_kv_heads)).to(device)
    gen = _gen(device, wl.wid, _STREAM["dec_kv"], step)
    zk = torch.randn(wl.units, wl.head_dim, generator=gen, device=device, dtype=torch.float32)[units.to(device)]
    zv = torch.randn(wl.units, wl.head_dim, generator=gen, device=device, dtype=torch.float32)[units.to(device)]
    k = zk * sigma_k_all[lh]
    layer = (lh // wl.n_kv_heads).to(torch.float32)
    if wl.layer_noise is None:
        fac = torch.ones_like(layer)
    else:
        lo, hi = wl.layer_noise
        fac = lo + (hi - lo) * layer / max(wl.n_layers - 1, 1)
    v = torch.einsum("uce,ue->uc", w_true_all[lh], k) + 0.5 * fac[:, None] * zv
    return k.to(wl.torch_dtype), v.to(wl.torch_dtype)


def rope_keys(K: torch.Tensor, theta: float = 10000.0, first_pos: int = 0) -> torch.Tensor:
    """Stored (post-RoPE) keys from pre-rotation keys K [..., n, d]: row i is turned by its position
    first_pos + i, half-split pairing (channel c with c + d/2, angle pos * theta^(-2c/d)).  Input
    shaping only: this is the model's positional encoding, applied in fp64 and rounded once."""
    d = K.shape[-1]
    h = d // 2
    pos = torch.arange(first_pos, first_pos + K.shape[-2], device=K.device, dtype=torch.float64)
    inv = torch.pow(torch.tensor(theta, dtype=torch.float64, device=K.device),
                    -2.0 * torch.arange(h, device=K.device, dtype=torch.float64) / d)
    ang = pos[:, None] * inv[None, :]
    cs, sn = torch.cos(ang), torch.sin(ang)
    x, y = K[..., :h].double(), K[..., h:].double()
    return torch.cat([x * cs - y * sn, x * sn + y * cs], dim=-1).to(K.dtype)
