"""One map per layer (Section 5.1: the map is calibrated layer-wise): the device path through the C-ABI
against the oracle on the same seeded inputs.  Scores, tiers and index lists are per (sequence, layer);
K, V, the cache pools and the queries keep the per-head layouts.

Tolerances as for the per-head path: layer scores 1e-3 relative (sums of per-head scores), Step 1
bit-exact on identical layer scores, residuals within the rounding bound of fp32 accumulation over
Hkv d products, Step 3 bit-exact on identical residuals, decode output within 2e-2."""
import numpy as np
import pytest
import torch

import paper_2605_23258_b200 as vec
from paper_2605_23258_b200 import synth

from helpers import budget_of, oracle_scores, score_close, shape_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _layer_inputs(wl):
    """K, V [B L Hkv][N][d], Q [B L Hkv][g][w][d], W_layer [L][Hkv d][Hkv d] in the workload dtype."""
    Ks, Vs, Qs, Ws = [], [], [], []
    for b in range(wl.batch):
        for l in range(wl.n_layers):
            params = synth.layer_params(wl, l, DEV)
            k, v = synth.layer_kv(wl, b, l, DEV, params)
            Ks.append(k), Vs.append(v)
            for h in range(wl.n_kv_heads):
                gen = torch.Generator(device=DEV).manual_seed(1000 * l + 10 * h + b)
                qh = torch.randn(wl.group, wl.window, wl.head_dim, generator=gen, device=DEV) * params[1][h]
                Qs.append(qh.to(wl.torch_dtype))
    for l in range(wl.n_layers):
        params = synth.layer_params(wl, l, DEV)
        kc, vc = synth.layer_calib_kv(wl, l, DEV, params)
        n = kc.shape[1]
        Kc = kc.permute(1, 0, 2).reshape(n, -1).contiguous().cpu()
        Vc = vc.permute(1, 0, 2).reshape(n, -1).contiguous().cpu()
        Ws.append(vec.vector_calibrate(Kc, Vc, wl.lam))           # host least squares on whole-layer rows
    return (torch.cat(Ks), torch.cat(Vs), torch.stack(Qs), torch.stack(Ws).to(wl.torch_dtype).to(DEV))


def _eps_bound(got, want, Kc, Vc, W):
    """|eps_gpu - eps| <= 2 sqrt(eps) ||delta|| + ||delta||^2 + 2^-20 eps with delta_c = (D + 2) 2^-23 (|v_c| + sum |W||k|):
    fp32 accumulation of exact products over D = Hkv d inputs, in any order."""
    D = Kc.shape[1]
    delta = (D + 2) * 2.0 ** -23 * (np.abs(Vc) + np.abs(Kc) @ np.abs(W).T)
    dn = np.sqrt((delta ** 2).sum(1))
    tol = 2 * np.sqrt(want) * dn + dn ** 2 + 2.0 ** -20 * want
    err = np.abs(np.asarray(got, np.float64) - want)
    return bool(np.all(err <= tol)), float(np.max(err / tol))


@pytest.mark.parametrize("base,over,percent", [
    (1, {"N": 1500, "n_kv_heads": 4, "n_q_heads": 16, "n_calib": 2048, "n_layers": 2}, 30),       # bf16 d=128: tensor-core residual
    (1, {"N": 700, "n_kv_heads": 8, "n_q_heads": 32, "n_calib": 2048, "batch": 2}, 20),           # 8 heads, two sequences: MMA decode
    (1, {"N": 3000, "n_kv_heads": 8, "n_q_heads": 16, "n_calib": 2048}, 30),                      # many tiles and splits, g = 2
    (0, {"N": 600, "n_calib": 1024, "n_layers": 2}, 25),                                          # fp32 d=64: CUDA-core kernels
    (4, {"N": 900, "n_layers": 1, "n_kv_heads": 2, "n_q_heads": 16, "window": 32, "n_calib": 1024}, 30),   # g = 8
])
def test_layer_map_pipeline(oracle, base, over, percent):
    wl = synth.shrink(synth.WORKLOADS[base], **over)
    K, V, Q, W = _layer_inputs(wl)
    sh, b = shape_of(wl), budget_of(wl, percent)
    U, Hkv, N, d, g = wl.units, wl.n_kv_heads, wl.N, wl.head_dim, wl.group
    UL = U // Hkv
    ws = torch.empty(max(vec.vector_workspace_bytes(sh, b), vec.vector_layer_workspace_bytes(sh, b)), dtype=torch.uint8, device=DEV)
    scores = torch.empty(U, N, dtype=torch.float32, device=DEV)
    vec.vector_score(sh, Q, K, N, scores, None, ws)
    lsc = torch.empty(UL, N, dtype=torch.float32, device=DEV)
    vec.vector_layer_scores(sh, scores, N, lsc)
    tier = torch.empty(UL, N, dtype=torch.uint8, device=DEV)
    ret = torch.empty(UL, b.n_ret, dtype=torch.int32, device=DEV)
    apx = torch.empty(UL, b.n_apx, dtype=torch.int32, device=DEV)
    eps = torch.empty(UL, b.n_pool, dtype=torch.float32, device=DEV)
    pool = torch.empty(UL, b.n_pool, dtype=torch.int32, device=DEV)
    vec.vector_route_layer(sh, b, lsc, K, V, W, tier, ret, apx, eps, pool, ws)
    cache = vec.alloc_cache(sh, b, 0, DEV)
    vec.vector_compact_layer(sh, b, K, V, ret, apx, cache)
    torch.cuda.synchronize()
    assert vec.vector_device_fault() == 0

    # layer scores: the oracle's per-head scores summed
    _, sc_o = oracle_scores(oracle, wl, Q.cpu(), K.cpu())
    lsc_o = np.stack([oracle.layer_score(sc_o[ul * Hkv:(ul + 1) * Hkv]) for ul in range(UL)])
    ok, worst = score_close(lsc.cpu().numpy(), lsc_o, Hkv * g * wl.window)
    assert ok, f"layer score off by {worst:.3g} x tolerance"

    # routing fed by the oracle's layer scores: Step 1 bit-exact, residuals within bound, Step 3 bit-exact on device residuals
    lsc32 = torch.from_numpy(lsc_o.astype(np.float32)).to(DEV)
    tier2, ret2, apx2 = torch.empty_like(tier), torch.empty_like(ret), torch.empty_like(apx)
    eps2, pool2 = torch.empty_like(eps), torch.empty_like(pool)
    vec.vector_route_layer(sh, b, lsc32, K, V, W, tier2, ret2, apx2, eps2, pool2, ws)
    torch.cuda.synchronize()
    Kc, Vc = K.cpu(), V.cpu()
    for ul in range(UL):
        l = ul % wl.n_layers
        Ku, Vu, Wl = Kc[ul * Hkv:(ul + 1) * Hkv], Vc[ul * Hkv:(ul + 1) * Hkv], W[l].cpu()
        r = oracle.route_layer(lsc_o[ul].astype(np.float32), Ku, Vu, Wl, b.n_pool, b.n_apx)
        assert np.array_equal(pool2[ul].cpu().numpy(), r["pool_idx"]), f"(sequence, layer) {ul}: pool differs"
        rows = torch.from_numpy(r["pool_idx"]).long()
        Kcat = oracle.concat_heads(Ku)[rows.numpy()]
        Vcat = oracle.concat_heads(Vu)[rows.numpy()]
        ok, worst = _eps_bound(eps2[ul].cpu().numpy(), r["eps"], Kcat, Vcat, Wl.double().numpy())
        assert ok, f"(sequence, layer) {ul}: eps off by {worst:.3g} x bound"
        t3, r3, a3 = oracle.truncate(eps2[ul].cpu().numpy(), r["pool_idx"], b.n_apx, N)
        assert np.array_equal(tier2[ul].cpu().numpy(), t3) and np.array_equal(ret2[ul].cpu().numpy(), r3)
        assert np.array_equal(apx2[ul].cpu().numpy(), a3)
        # end to end (device scores): at least 99.9 % of the tokens routed alike
        agree = np.mean(tier[ul].cpu().numpy() == r["tier"])
        assert agree >= 0.999 or N < 2000 and agree >= 1 - 4 / N, (ul, agree)

    # compaction: every head of a layer holds the rows its layer's lists name
    for u in range(U):
        ul = u // Hkv
        assert torch.equal(cache.ret_k[u, : b.n_ret], K[u][ret[ul].long()]) and torch.equal(cache.ret_v[u, : b.n_ret], V[u][ret[ul].long()])
        assert torch.equal(cache.apx_k[u, : b.n_apx], K[u][apx[ul].long()])
        assert torch.equal(cache.ret_pos[u, : b.n_ret], ret[ul]) and torch.equal(cache.apx_pos[u, : b.n_apx], apx[ul])

    # decode attention with the layer's map
    gen = torch.Generator(device=DEV).manual_seed(7)
    q = (torch.randn(U, g, d, generator=gen, device=DEV) * 2.0).to(wl.torch_dtype)
    out = torch.empty(U, g, d, dtype=torch.float32, device=DEV)
    vec.vector_decode_attn_layer(sh, q, cache, W, out, ws)
    out_bf = torch.empty(U, g, d, dtype=torch.bfloat16, device=DEV)
    vec.vector_decode_attn_layer(sh, q, cache, W, out_bf, ws)
    torch.cuda.synchronize()
    scale = 1.0 / np.sqrt(d)
    for ul in range(UL):
        l = ul % wl.n_layers
        sl = slice(ul * Hkv, (ul + 1) * Hkv)
        o_tok, o_fac = oracle.attend_layer(q[sl].reshape(Hkv * g, d).cpu(), cache.ret_k[sl, : b.n_ret].cpu(),
                                           cache.ret_v[sl, : b.n_ret].cpu(), cache.apx_k[sl, : b.n_apx].cpu(), W[l].cpu(), scale)
        assert np.max(np.abs(o_tok - o_fac)) <= 1e-9 * max(1.0, np.max(np.abs(o_tok)))
        got = out[sl].reshape(Hkv * g, d).cpu().double().numpy()
        assert np.max(np.abs(got - o_fac)) <= 2e-2, (ul, float(np.max(np.abs(got - o_fac))))
        gotb = out_bf[sl].reshape(Hkv * g, d).cpu().double().numpy()
        assert np.all(np.abs(gotb - o_fac) <= 2e-2 + 2.0 ** -8 * np.abs(o_fac))
