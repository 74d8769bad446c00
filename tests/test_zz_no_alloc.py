"""sp_pruned_decode_static: decode attention for callers that cannot allocate.

Some users of this library run where no device memory can be requested at call time (an
inference server whose pool is already carved up, a plugin that may not touch the CUDA
allocator).  For them the library carries its own fixed split-KV scratch array.  This test
drives that entry point through the C ABI twice in a row -- the second call finds the
first call's leftovers in the shared array -- and checks both results against the ordinary
entry point that takes a caller workspace and against the CPU oracle, and that the device's
free memory is the same before and after the call.  It is collected last on purpose, and it
passes on its own in a fresh process as well as after the other GPU tests."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2404_06910_b200 as sp
from helpers import dev, f32, rel_l2, workspace
from workloads import build_layout

pytestmark = pytest.mark.gpu


def _inputs(dtype, seed, B_H_D):
    H, Hkv, D = B_H_D
    lay = build_layout([16, 3, 40], [[32, 1, 129, 40], [200, 17], [64, 64, 300]],
                       [[8, 8, 8, 8], [5, 5], [24, 24, 24]])
    g = torch.Generator().manual_seed(seed)
    mk = lambda *shape: torch.randn(*shape, generator=g).to(dtype)
    B, T = lay.n_prompts, lay.total_tokens
    kept = np.array([[2, 0], [4, -1], [8, 6]], np.int32)
    tail_len = np.array([5, 1, 3], np.int32)
    return lay, dict(q=mk(B, H, D), kc=mk(T, Hkv, D), vc=mk(T, Hkv, D), tk=mk(B, 6, Hkv, D), tv=mk(B, 6, Hkv, D),
                     kept=kept, tail_len=tail_len)


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-5), (torch.bfloat16, 1e-2)])
def test_static_scratch_decode_matches_workspace_decode_twice(dtype, tol):
    H, Hkv, D = 4, 2, 128
    assert sp.sp_pruned_decode_static_max_bytes() >= 1 << 20
    for call, seed in enumerate((11, 12)):          # two calls in a row share the built-in array
        lay, x = _inputs(dtype, seed, (H, Hkv, D))
        dl = sp.DeviceLayout.from_host(lay)
        B = lay.n_prompts
        d = {n: dev(a) for n, a in x.items()}
        scale = 1 / math.sqrt(D)
        ref = torch.full((B, H, D), float("nan"), dtype=dtype, device="cuda")
        ref_lse = torch.full((B, H), float("nan"), device="cuda")
        ws = workspace(sp.sp_decode_workspace_bytes(B, H, D))
        sp.sp_pruned_decode(d["q"], d["kc"], d["vc"], dl, d["kept"], 2, d["tk"], d["tv"], d["tail_len"], 6, scale,
                            ref, ref_lse, ws)
        got = torch.full_like(ref, float("nan"))
        got_lse = torch.full_like(ref_lse, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        sp.sp_pruned_decode_static(d["q"], d["kc"], d["vc"], dl, d["kept"], 2, d["tk"], d["tv"], d["tail_len"], 6,
                                   scale, got, got_lse)
        torch.cuda.synchronize()
        if call == 1:       # (the very first call may load the kernel's code; the second one must take nothing)
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert not torch.isnan(got).any(), f"call {call}: rows left unwritten"
        assert rel_l2(f32(got), f32(ref)) <= tol, f"call {call}"
        want, want_lse = oracle.pruned_decode(f32(x["q"]), f32(x["kc"]), f32(x["vc"]), lay, x["kept"], f32(x["tk"]),
                                              f32(x["tv"]), x["tail_len"], scale)
        assert rel_l2(f32(got), want) <= tol, f"call {call}: against the oracle"
        np.testing.assert_allclose(got_lse.cpu().numpy(), want_lse, atol=1e-5 if dtype == torch.float32 else 2e-2)
        np.testing.assert_allclose(got_lse.cpu().numpy(), ref_lse.cpu().numpy(), atol=1e-5 if dtype == torch.float32 else 2e-2)


def test_static_scratch_decode_rejects_oversized_problems():
    """64 prompts x 40000 heads need 10 MB of arrival counters, more than the built-in array
    holds: the call must fail on the host with a clear message and launch nothing.  (The
    tensors have their real sizes, so even a missed check could not read out of bounds.)"""
    B, H, D = 64, 40000, 128
    lay = build_layout([8] * B, [[16]] * B, [[4]] * B)
    dl = sp.DeviceLayout.from_host(lay)
    q = torch.zeros((B, H, D), dtype=torch.bfloat16, device="cuda")
    kc = torch.zeros((lay.total_tokens, 1, D), dtype=torch.bfloat16, device="cuda")
    kept = torch.zeros((B, 1), dtype=torch.int32, device="cuda")
    out = torch.full_like(q, 7.0)
    with pytest.raises(sp.SpError) as e:
        sp.sp_pruned_decode_static(q, kc, kc, dl, kept, 1, None, None, None, 0, 1.0, out)
    assert e.value.code == sp.SP_ERR_WORKSPACE and str(sp.sp_pruned_decode_static_max_bytes()) in str(e.value)
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
