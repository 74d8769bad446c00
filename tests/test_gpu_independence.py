"""Path independence on the device (Section 3.2: a path sees its prompt's preamble and itself,
never another path).  The oracle has this property by construction (pinned on the CPU); here
the CUDA kernels are held to it bit for bit: changing one document's Q / K / V, even to Inf or
NaN, must leave every other path's and the preamble's rows of `out` and `lse` unchanged."""
import math

import numpy as np
import pytest
import torch

import paper_2404_06910_b200 as sp
from helpers import dev, workspace
from workloads import build_layout

pytestmark = pytest.mark.gpu

TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _randn(shape, dtype, seed, std=1.0):
    g = torch.Generator()
    g.manual_seed(seed)
    return (torch.randn(*shape, generator=g) * std).to(TDT[dtype])


def _layout():
    # ragged on purpose: document ends fall inside 16-key MMA steps and inside TMA boxes, so the
    # rows that follow a path's last key in shared memory belong to its neighbour
    return build_layout([21, 40],
                        [[37, 130, 9, 77], [150, 3, 61]],
                        [[5, 7, 3, 11], [9, 2, 6]])


def _path_rows(lay, i):
    return np.arange(lay.path_start[i], lay.path_start[i] + lay.doc_len[i] + lay.qry_len[i])


def _run_prefill(q, k, v, lay, rows):
    dl = sp.DeviceLayout.from_host(lay)
    T, H, D = q.shape
    out = torch.zeros((T, H, D), dtype=q.dtype, device="cuda")
    lse = torch.zeros((H, T), device="cuda")
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.dtype_code(q)))
    sp.sp_superpose_prefill(dev(q), dev(k), dev(v), dl, 1 / math.sqrt(D), out, lse, ws, rows=rows)
    sp.sp_check_status(ws)
    return out.cpu(), lse.cpu()


# tensor-core kernel (bf16, 128), query-only kernel (bf16, 128, query rows), SIMT kernel (the rest)
@pytest.mark.parametrize("dtype,D,rows", [("bf16", 128, sp.SP_ROWS_ALL), ("bf16", 128, sp.SP_ROWS_QUERY_ONLY),
                                          ("f32", 64, sp.SP_ROWS_ALL), ("bf16", 64, sp.SP_ROWS_ALL)])
@pytest.mark.parametrize("kind", ["finite", "non_finite"])
def test_prefill_paths_do_not_see_each_other(dtype, D, rows, kind):
    lay = _layout()
    T, H, Hkv = lay.total_tokens, 4, 2
    q, k, v = _randn((T, H, D), dtype, 900), _randn((T, Hkv, D), dtype, 901), _randn((T, Hkv, D), dtype, 902)
    out0, lse0 = _run_prefill(q, k, v, lay, rows)
    for j in (1, 2, 5):                                   # a path of each prompt, one of them tiny
        q2, k2, v2 = q.clone(), k.clone(), v.clone()
        r = torch.from_numpy(_path_rows(lay, j))
        if kind == "finite":
            q2[r], k2[r], v2[r] = q2[r] * -1.5 + 0.25, k2[r] * 2.0 - 0.5, v2[r] * -3.0 + 1.0
        else:
            q2[r], k2[r] = float("nan"), float("inf")
            v2[r] = float("nan")
            v2[r[::2]] = float("-inf")
        out1, lse1 = _run_prefill(q2, k2, v2, lay, rows)
        keep = np.ones(T, dtype=bool)
        keep[r.numpy()] = False
        assert torch.equal(out0[keep], out1[keep]), f"path {j} ({kind}) leaked into another path's output"
        assert torch.equal(lse0[:, keep], lse1[:, keep])


def test_prefill_ignores_rows_outside_every_segment():
    """Packed rows that belong to no segment (gaps between segments) may hold anything."""
    base = build_layout([16], [[45, 70]], [[6, 9]])
    # the same segments with 5 unused rows after each of them
    gap = 5
    import copy
    lay = copy.deepcopy(base)
    lay.path_start = (base.path_start + gap * (1 + np.arange(base.n_paths))).astype(np.int32)
    lay.total_tokens = base.total_tokens + gap * (base.n_paths + 1)
    T, H, D = lay.total_tokens, 2, 128
    used = np.zeros(T, dtype=bool)
    used[:16] = True
    for i in range(lay.n_paths):
        used[_path_rows(lay, i)] = True
    q, k, v = _randn((T, H, D), "bf16", 910), _randn((T, H, D), "bf16", 911), _randn((T, H, D), "bf16", 912)
    out0, lse0 = _run_prefill(q, k, v, lay, sp.SP_ROWS_ALL)
    q2, k2, v2 = q.clone(), k.clone(), v.clone()
    q2[~used], k2[~used], v2[~used] = float("nan"), float("nan"), float("nan")
    out1, lse1 = _run_prefill(q2, k2, v2, lay, sp.SP_ROWS_ALL)
    assert torch.equal(out0[used], out1[used]) and torch.equal(lse0[:, used], lse1[:, used])


@pytest.mark.parametrize("dtype,D", [("bf16", 128), ("f32", 64)])
@pytest.mark.parametrize("kind", ["finite", "non_finite"])
def test_decode_sees_only_kept_paths(dtype, D, kind):
    """The decode attention reads the preamble, the kept paths and the tail: a path that was
    pruned may change (or hold Inf / NaN) without any effect, bit for bit."""
    lay = _layout()
    B, T, H, Hkv, cap = lay.n_prompts, lay.total_tokens, 4, 2, 3
    kc, vc = _randn((T, Hkv, D), dtype, 920), _randn((T, Hkv, D), dtype, 921)
    q = _randn((B, H, D), dtype, 922)
    tk, tv = _randn((B, cap, Hkv, D), dtype, 923), _randn((B, cap, Hkv, D), dtype, 924)
    kept = np.array([[3, 0], [4, -1]], np.int32)           # pruned: paths 1, 2 (prompt 0) and 5, 6 (prompt 1)
    tl = np.array([2, 3], np.int32)
    dl = sp.DeviceLayout.from_host(lay)

    def run(kc_, vc_):
        out = torch.zeros((B, H, D), dtype=TDT[dtype], device="cuda")
        lse = torch.zeros((B, H), device="cuda")
        ws = workspace(sp.sp_decode_workspace_bytes(B, H, D))
        sp.sp_pruned_decode(dev(q), dev(kc_), dev(vc_), dl, dev(kept), 2, dev(tk), dev(tv), dev(tl), cap,
                            1 / math.sqrt(D), out, lse, ws)
        sp.sp_check_status(ws)
        return out.cpu(), lse.cpu()

    out0, lse0 = run(kc, vc)
    for j in (1, 2, 5, 6):
        k2, v2 = kc.clone(), vc.clone()
        r = torch.from_numpy(_path_rows(lay, j))
        if kind == "finite":
            k2[r], v2[r] = k2[r] * 2.0 - 0.5, v2[r] * -3.0 + 1.0
        else:
            k2[r], v2[r] = float("inf"), float("nan")
        out1, lse1 = run(k2, v2)
        assert torch.equal(out0, out1) and torch.equal(lse0, lse1), f"pruned path {j} ({kind}) reached the decode output"
