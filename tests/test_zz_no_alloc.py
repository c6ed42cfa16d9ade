"""The allocation-free decode entry point against the workspace-taking one.

vector_decode_attn_static serves callers that cannot allocate device memory at
call time (a server whose own pool holds the whole device, or a decode loop that
cannot afford a cudaMalloc stall): its split-KV scratch is a fixed array inside
the library.  It must give what vector_decode_attn gives, call after call, since
every call reuses the same array with the previous call's contents still in it.
This file sorts last so that a run that stops at the first failure has already
run every other test.
"""
import gc

import pytest
import torch

import paper_2605_23258_b200 as vec
from paper_2605_23258_b200 import synth

from helpers import budget_of, calibrated_maps, shape_of

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _cache_from(wl, K, V, n_ret, n_apx):
    pos = torch.arange(wl.N, dtype=torch.int32, device=DEV).repeat(wl.units, 1).contiguous()
    return vec.Cache(K.clone(), V.clone(), K.flip(1).contiguous(), pos, pos.clone(), n_ret, n_apx)


def test_static_scratch_decode_matches_workspace_decode_twice():
    wl = synth.shrink(synth.WORKLOADS[1], N=4096, n_kv_heads=4, n_q_heads=16, n_calib=1024)
    sh = shape_of(wl)
    assert 0 < vec.vector_decode_scratch_bytes(sh) <= vec.VECTOR_STATIC_SCRATCH_BYTES
    K, V, _ = synth.context(wl, DEV)
    W = calibrated_maps(wl).to(DEV)
    _, sq, _ = synth.all_head_params(wl, DEV)
    ws = vec.alloc_workspace(sh, budget_of(wl, 50))
    # two calls in a row on different problems: the second finds the first one's partials in the array
    for step, (n_ret, n_apx) in enumerate([(1500, 2596), (4096, 700)]):
        q = synth.decode_q(wl, step, DEV, sq)
        cache = _cache_from(wl, K, V, n_ret, n_apx)
        for dt in (torch.float32, torch.bfloat16):
            want = torch.empty(wl.units, wl.group, wl.head_dim, dtype=dt, device=DEV)
            got = torch.full_like(want, float("nan"))
            vec.vector_decode_attn(sh, q, cache, W, want, 0, ws)
            vec.vector_decode_attn_static(sh, q, cache, W, got, 0)
            torch.cuda.synchronize()
            assert torch.isfinite(got).all()
            # same kernels, same launch shape, same inputs: well inside the 2e-2 decode tolerance
            assert (got.float() - want.float()).abs().max().item() <= 2e-2
            assert torch.equal(got, want)


def test_static_scratch_both_record_layouts_back_to_back_and_no_allocation():
    """The fp32 / head_dim-64 path keeps split records of another layout in the same array than the
    bf16 / head_dim-128 path: run them alternately so that each finds the other's leftovers, and check
    that a call takes no device memory (free bytes of the device and the bytes torch holds unchanged)."""
    wl_a = synth.shrink(synth.WORKLOADS[0], N=1024, n_calib=1024)                            # fp32, d = 64, g = 2
    wl_b = synth.shrink(synth.WORKLOADS[1], N=2048, n_kv_heads=2, n_q_heads=8, n_calib=1024)  # bf16, d = 128
    cases = []
    for wl, (n_ret, n_apx) in ((wl_a, (128, 256)), (wl_b, (700, 1100))):
        sh = shape_of(wl)
        K, V = synth.context(wl, DEV)[:2]          # no name bound here is rebound below: no tensor dies in the measured region
        W = calibrated_maps(wl).to(DEV)
        sq = synth.all_head_params(wl, DEV)[1]
        q = synth.decode_q(wl, 0, DEV, sq)
        cache = _cache_from(wl, K, V, n_ret, n_apx)
        ws = vec.alloc_workspace(sh, budget_of(wl, 50))
        want = torch.empty(wl.units, wl.group, wl.head_dim, dtype=torch.float32, device=DEV)
        vec.vector_decode_attn(sh, q, cache, W, want, 0, ws)
        got = torch.empty_like(want)
        cases.append((sh, q, cache, W, want, got))
    for sh, q, cache, W, want, got in cases:                   # the first call per device looks the array up
        vec.vector_decode_attn_static(sh, q, cache, W, got, 0)
    rounds = [[torch.full_like(c[4], float("nan")) for c in cases] for _ in range(3)]
    gc.collect()                                               # tensors of earlier tests must not be released in between
    torch.cuda.synchronize()
    free0, held0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for outs in rounds:                                        # nothing but the library's calls in between
        for case, o in zip(cases, outs):
            vec.vector_decode_attn_static(case[0], case[1], case[2], case[3], o, 0)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == held0
    for outs in rounds:
        for case, o in zip(cases, outs):
            assert torch.equal(o, case[4])


def test_static_scratch_rejects_shapes_beyond_its_limit():
    # 65535 units of 8 query heads need far more partial records than the fixed array holds
    big = vec.Shape(1, 1, 8 * 65535, 65535, 128, vec.VECTOR_BF16, 64)
    assert vec.vector_decode_scratch_bytes(big) > vec.VECTOR_STATIC_SCRATCH_BYTES
    t = torch.zeros(16, dtype=torch.bfloat16, device=DEV)
    i = torch.zeros(16, dtype=torch.int32, device=DEV)
    cache = vec.Cache(t.view(1, 1, 16), t.view(1, 1, 16), t.view(1, 1, 16), i.view(1, 16), i.view(1, 16), 1, 0)
    with pytest.raises(vec.VectorError) as e:
        vec.vector_decode_attn_static(big, t, cache, t, torch.zeros(16, device=DEV))
    assert e.value.status == -5
