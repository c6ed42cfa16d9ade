"""The allocation-free decode entry point against the workspace-taking one.

vector_decode_attn_static serves callers that cannot allocate device memory at
call time (a server whose own pool holds the whole device, or a decode loop that
cannot afford a cudaMalloc stall): its split-KV scratch is a fixed array inside
the library.  It must give what vector_decode_attn gives, call after call, since
every call reuses the same array with the previous call's contents still in it.
This file sorts last so that a run that stops at the first failure has already
run every other test.
"""
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
