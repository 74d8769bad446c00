"""Layouts that contradict themselves must come back as an error, never as an access outside the
caller's tensors.  With a host mirror of the index arrays the host refuses the call; without one
the device-side checks skip what cannot be trusted and report SP_ERR_LAYOUT through the
workspace status word.  Every tensor here is allocated far larger than the declared layout
needs, so that even a missed check would stay inside allocated memory."""
import copy
import math
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import paper_2404_06910_b200 as sp
from helpers import workspace
from workloads import build_layout

pytestmark = pytest.mark.gpu

H, D, SLACK = 2, 128, 4096


def _tensors(T):
    g = torch.Generator().manual_seed(3)
    mk = lambda: torch.randn(T + SLACK, H, D, generator=g).bfloat16().cuda()
    return mk(), mk(), mk()


def _bad_layouts():
    base = build_layout([16], [[100, 40, 70]], [[8, 8, 8]])
    a = copy.deepcopy(base)                      # a path that starts beyond the declared T
    a.path_start = base.path_start.copy(); a.path_start[2] = base.total_tokens + 5
    b = copy.deepcopy(base)                      # a document longer than max_path_len allows
    b.doc_len = base.doc_len.copy(); b.doc_len[1] = 100000
    c = copy.deepcopy(base)                      # negative length
    c.qry_len = base.qry_len.copy(); c.qry_len[0] = -3
    d = copy.deepcopy(base)                      # two paths on the same rows
    d.path_start = base.path_start.copy(); d.path_start[1] = base.path_start[0] + 10
    return base, {"start_beyond_T": a, "length_over_max": b, "negative_length": c, "overlap": d}


class _Fixed:
    """A layout whose host scalars stay those of the consistent layout."""
    def __init__(self, lay, ref):
        self.__dict__.update(lay.__dict__)
        self.max_pre_len, self.max_path_len = ref.max_pre_len, ref.max_path_len


@pytest.mark.parametrize("name", ["start_beyond_T", "length_over_max", "negative_length", "overlap"])
def test_host_mirror_refuses_inconsistent_layouts(name):
    base, bad = _bad_layouts()
    q, k, v = _tensors(base.total_tokens)
    dl = sp.DeviceLayout.from_host(_Fixed(bad[name], base), mirror=True)
    out = torch.full_like(q, 7.0)
    ws = workspace(sp.sp_prefill_workspace_bytes(sp.DeviceLayout.from_host(base), H, D, sp.SP_BF16))
    with pytest.raises(sp.SpError) as e:
        sp.sp_superpose_prefill(q, k, v, dl, 1 / math.sqrt(D), out, None, ws)
    assert e.value.code == sp.SP_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())              # nothing was launched


@pytest.mark.parametrize("rows", [sp.SP_ROWS_ALL, sp.SP_ROWS_QUERY_ONLY])
@pytest.mark.parametrize("name", ["start_beyond_T", "length_over_max", "negative_length"])
def test_device_checks_skip_and_report_without_a_mirror(name, rows):
    base, bad = _bad_layouts()
    T = base.total_tokens
    q, k, v = _tensors(T)
    good_dl = sp.DeviceLayout.from_host(base, mirror=False)
    ws = workspace(sp.sp_prefill_workspace_bytes(good_dl, H, D, sp.SP_BF16))
    ref = torch.full_like(q, 7.0)
    sp.sp_superpose_prefill(q, k, v, good_dl, 1 / math.sqrt(D), ref, None, ws, rows=rows)
    sp.sp_check_status(ws)
    dl = sp.DeviceLayout.from_host(_Fixed(bad[name], base), mirror=False)
    out = torch.full_like(q, 7.0)
    sp.sp_superpose_prefill(q, k, v, dl, 1 / math.sqrt(D), out, None, ws, rows=rows)
    with pytest.raises(sp.SpError) as e:
        sp.sp_check_status(ws)
    assert e.value.code == sp.SP_ERR_LAYOUT
    assert bool((out[T:] == 7.0).all())          # nothing beyond the declared rows was written
    # the segments that are consistent were still computed, the broken one was left alone
    broken = {"start_beyond_T": 2, "length_over_max": 1, "negative_length": 0}[name]
    for i in range(base.n_paths):
        r = slice(int(base.path_start[i]), int(base.path_start[i] + base.doc_len[i] + base.qry_len[i]))
        if i != broken and name != "start_beyond_T":
            assert torch.equal(out[r], ref[r])
    # and the next consistent call clears the word
    sp.sp_superpose_prefill(q, k, v, good_dl, 1 / math.sqrt(D), out, None, ws, rows=rows)
    sp.sp_check_status(ws)
    assert torch.equal(out[:T], ref[:T])


def test_decode_skips_kept_paths_outside_the_cache():
    base, bad = _bad_layouts()
    T = base.total_tokens
    _, k, v = _tensors(T)
    q = torch.randn(1, H, D, generator=torch.Generator().manual_seed(4)).bfloat16().cuda()
    kept = torch.tensor([[2, 0]], dtype=torch.int32, device="cuda")
    ws = workspace(sp.sp_decode_workspace_bytes(1, H, D))

    def run(lay, kept_):
        out = torch.zeros((1, H, D), dtype=torch.bfloat16, device="cuda")
        sp.sp_pruned_decode(q, k[:T], v[:T], sp.DeviceLayout.from_host(lay, mirror=False), kept_, 2, None, None, None, 0,
                            1 / math.sqrt(D), out, None, ws)
        torch.cuda.synchronize()
        return out

    want = run(base, torch.tensor([[-1, 0]], dtype=torch.int32, device="cuda"))     # path 2 simply not kept
    got = run(_Fixed(bad["start_beyond_T"], base), kept)                             # path 2 kept but out of range
    assert torch.equal(got, want)


def test_debug_build_finds_overlapping_segments_and_passes_parity():
    """The library built with -DSP_DEBUG_BOUNDS looks at every pair of segments on the device: two
    paths on the same rows come back as SP_ERR_LAYOUT without a host mirror.  The same build runs
    the ragged-edge parity cases unchanged.  (A child process, because the library is chosen when
    the package is imported.)"""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SP_B200_DEBUG_BOUNDS="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                        os.path.join(root, "tests", "test_gpu_layout_checks.py") + "::test_overlap_reported_by_debug_build",
                        os.path.join(root, "tests", "test_gpu_parity.py"), "-k",
                        "overlap_reported or prefill_ragged_edges or query_only_ragged or decode_small"],
                       env=env, capture_output=True, text=True, timeout=900, cwd=root)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "skipped" not in r.stdout.splitlines()[-1]


def test_overlap_reported_by_debug_build():
    if os.environ.get("SP_B200_DEBUG_BOUNDS") != "1":
        pytest.skip("runs in the child process of the test above, under the debug build")
    assert sp.LIB_PATH.endswith("libsp_b200_debug.so")
    base, bad = _bad_layouts()
    q, k, v = _tensors(base.total_tokens)
    ws = workspace(sp.sp_prefill_workspace_bytes(sp.DeviceLayout.from_host(base), H, D, sp.SP_BF16))
    out = torch.full_like(q, 7.0)
    sp.sp_superpose_prefill(q, k, v, sp.DeviceLayout.from_host(_Fixed(bad["overlap"], base), mirror=False),
                            1 / math.sqrt(D), out, None, ws)
    with pytest.raises(sp.SpError) as e:
        sp.sp_check_status(ws)
    assert e.value.code == sp.SP_ERR_LAYOUT
