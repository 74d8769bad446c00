"""The prefill with the rotation of Q folded in (Section 3.2.2, footnote on RoPE) against the oracle
(rotation, then fork-join attention) and against the two-call path of the library, which it must equal."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2404_06910_b200 as sp
from helpers import dev, f32, rel_l2, workspace
from workloads import build_layout, draw_lengths, get_config

pytestmark = pytest.mark.gpu


def _randn(shape, seed, std=1.0):
    g = torch.Generator()
    g.manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).bfloat16()


def _fused(q, k, v, lay, pos, pairing, base=10000.0):
    dl = sp.DeviceLayout.from_host(lay)
    T, H, D = q.shape
    qd = dev(q)
    q0 = qd.clone()
    out = torch.full_like(qd, float("nan"))
    lse = torch.full((H, T), float("nan"), device="cuda")
    ws = workspace(sp.sp_prefill_rope_workspace_bytes(dl, H, D, sp.SP_BF16))
    sp.sp_superpose_prefill_rope(qd, dev(k), dev(v), dl, dev(pos), base, pairing, 1 / math.sqrt(D), out, lse, ws)
    sp.sp_check_status(ws)
    assert torch.equal(qd, q0), "q must not be modified"
    return out, lse


def _two_calls(q, k, v, lay, pos, pairing, base=10000.0):
    dl = sp.DeviceLayout.from_host(lay)
    T, H, D = q.shape
    qd = dev(q)
    sp.sp_rope_apply(qd, dev(pos), H, D, base=base, pairing=pairing)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full((H, T), float("nan"), device="cuda")
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.SP_BF16))
    sp.sp_superpose_prefill(qd, dev(k), dev(v), dl, 1 / math.sqrt(D), out, lse, ws)
    sp.sp_check_status(ws)
    return out, lse, qd


@pytest.mark.parametrize("pairing", [sp.SP_ROPE_HALF_SPLIT, sp.SP_ROPE_INTERLEAVED])
@pytest.mark.parametrize("H,Hkv", [(4, 4), (4, 2)])
def test_prefill_rope_fused(pairing, H, Hkv):
    # several query tiles per path, ragged tails, a one-row path, tiles with 32- and 64-row boxes
    lay = build_layout([21, 40], [[37, 290, 9, 130], [150, 1, 61]], [[5, 7, 3, 11], [9, 2, 6]])
    T, D = lay.total_tokens, 128
    q, k, v = _randn((T, H, D), 31), _randn((T, Hkv, D), 32), _randn((T, Hkv, D), 33)
    g = torch.Generator()
    g.manual_seed(34)
    pos = (torch.rand(T, generator=g) * 900).float()          # real-valued positions, any order
    out_f, lse_f = _fused(q, k, v, lay, pos, pairing)
    out_u, lse_u, q_rot = _two_calls(q, k, v, lay, pos, pairing)
    assert not torch.isnan(out_f.float()).any(), "rows left unwritten"
    assert torch.equal(out_f, out_u) and torch.equal(lse_f, lse_u), "fused and two-call paths differ"
    # the oracle: rotation in fp64 angles, the rotated query rounded to bf16 as the stored tensor is
    q_ref = torch.from_numpy(oracle.rope(f32(q), pos.numpy(), pairing=pairing)).bfloat16()
    assert np.all(np.abs(f32(q_rot) - f32(q_ref)) <= np.abs(f32(q_ref)) * 2.0 ** -7 + 1e-6)
    ref_o, ref_l = oracle.prefill(f32(q_ref), f32(k), f32(v), lay, 1 / math.sqrt(D))
    got = f32(out_f)
    assert rel_l2(got, ref_o) <= 1e-2
    num = np.linalg.norm((got - ref_o).reshape(T, -1), axis=1)
    den = np.linalg.norm(ref_o.reshape(T, -1), axis=1) + 1e-6
    assert (num / den).max() <= 2e-2
    np.testing.assert_allclose(lse_f.cpu().numpy(), ref_l, atol=2e-2)


def test_prefill_rope_fused_larger_batch_equals_two_calls():
    lay = draw_lengths(get_config("cfg2"), n_prompts=6)
    T, H, D = lay.total_tokens, 8, 128
    q, k, v = _randn((T, H, D), 41, D ** -0.5), _randn((T, H, D), 42, D ** -0.5), _randn((T, H, D), 43)
    g = torch.Generator()
    g.manual_seed(44)
    pos = (torch.rand(T, generator=g) * 3000).float()
    out_f, lse_f = _fused(q, k, v, lay, pos, sp.SP_ROPE_HALF_SPLIT)
    out_u, lse_u, _ = _two_calls(q, k, v, lay, pos, sp.SP_ROPE_HALF_SPLIT)
    assert torch.equal(out_f, out_u) and torch.equal(lse_f, lse_u)


def test_prefill_rope_rejects_what_it_does_not_serve():
    lay = build_layout([8], [[20]], [[4]])
    dl = sp.DeviceLayout.from_host(lay)
    T = lay.total_tokens
    pos = torch.arange(T, dtype=torch.float32, device="cuda")
    for dtype, D in ((torch.float32, 128), (torch.bfloat16, 64)):
        q = torch.zeros((T, 2, D), dtype=dtype, device="cuda")
        out = torch.zeros_like(q)
        ws = workspace(1 << 20)
        with pytest.raises(sp.SpError) as e:
            sp.sp_superpose_prefill_rope(q, q, q, dl, pos, 10000.0, 0, 0.1, out, None, ws)
        assert e.value.code == sp.SP_ERR_UNSUPPORTED
    q = torch.zeros((T, 2, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros_like(q)
    small = workspace(sp.sp_prefill_workspace_bytes(dl, 2, 128, sp.SP_BF16))     # no room for the table
    with pytest.raises(sp.SpError) as e:
        sp.sp_superpose_prefill_rope(q, q, q, dl, pos, 10000.0, 0, 0.1, out, None, small)
    assert e.value.code == sp.SP_ERR_WORKSPACE
    with pytest.raises(sp.SpError) as e:
        sp.sp_superpose_prefill_rope(q, q, q, dl, pos, 10000.0, 7, 0.1, out, None, workspace(1 << 20))
    assert e.value.code == sp.SP_ERR_INVALID_ARG
