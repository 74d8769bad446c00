"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header
declares, rejects bad arguments before any launch, and its host-side position
assignment agrees with the oracle.  No compute call needs a GPU here."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2404_06910_b200 as sp
from workloads import CONFIGS, draw_lengths
from helpers import positions_for

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "sp.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert len(names) >= 12
    raw = ctypes.CDLL(sp.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), f"{n} declared in include/sp.h but not exported"
    assert set(names) == set(sp.EXPORTS)
    assert sp.sp_version().startswith("sp-b200")


def test_binding_has_a_function_per_symbol():
    for n in _declared_functions():
        if n != "sp_last_error":
            assert callable(getattr(sp, n)), n


@pytest.mark.parametrize("cfg", CONFIGS[:4], ids=lambda c: c.name)
def test_host_positions_match_oracle(cfg):
    lay = draw_lengths(cfg, n_prompts=min(cfg.n_prompts, 4))
    got, nxt = positions_for(lay, lambda P, L, Q: sp.sp_positions(P, L, Q))
    ref, nref = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q))
    np.testing.assert_array_equal(got, ref)            # both round the fp64 value once to fp32
    np.testing.assert_allclose(nxt, nref, rtol=1e-15)


def test_host_positions_variants_match_oracle():
    L = [7, 0, 33, 12]
    for scheme, name in ((sp.SP_POS_EQUILIBRIUM, "equilibrium"), (sp.SP_POS_LEFT_ALIGNED, "left")):
        for q_mode in (0, 1):
            got, S, nxt = sp.sp_positions(5, L, 3, scheme=scheme, q_mode=q_mode)
            ref, Sr, nr = oracle.positions(5, L, 3, scheme=name, q_mode=q_mode)
            np.testing.assert_array_equal(got, ref.astype(np.float32))
            assert S == pytest.approx(Sr, rel=1e-15) and nxt == pytest.approx(nr, rel=1e-15)
    got, S, _ = sp.sp_positions(0, [], 0)
    assert got.size == 0 and S == 0.0


def _rc(fn, *args):
    return fn(*args)


def test_invalid_arguments_are_rejected_on_the_host():
    lib = sp.lib
    # sp_positions
    L = np.array([3, -1], np.int32)
    pos = np.zeros(16, np.float32)
    assert lib.sp_positions(0, 0, 2, 2, L.ctypes.data, 1, pos.ctypes.data, None, None) == sp.SP_ERR_INVALID_ARG
    assert b"doc_len" in lib.sp_last_error()
    assert lib.sp_positions(7, 0, 2, 0, None, 1, pos.ctypes.data, None, None) == sp.SP_ERR_INVALID_ARG
    # sp_rope_apply: odd rot_dim, bad dtype, short stride (all before any launch)
    assert lib.sp_rope_apply(256, 256, 4, 64, 1, 64, 63, 10000.0, 0, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_rope_apply(256, 256, 4, 64, 1, 64, 64, 10000.0, 0, 9, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_rope_apply(256, 256, 4, 32, 1, 64, 64, 10000.0, 0, 0, None) == sp.SP_ERR_INVALID_ARG
    # sp_prune_topk: k <= 0
    assert lib.sp_prune_topk(256, 256, 1, 0, 256, None, None) == sp.SP_ERR_INVALID_ARG
    assert b"k must be" in lib.sp_last_error()
    # sp_path_scores: vocab > ld, missing workspace
    assert lib.sp_path_scores(256, 8, 256, 256, 4, 1, 16, None, None, 256, None, None, 0, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_path_scores(256, 16, 256, 256, 4, 1, 16, None, None, 256, None, None, 0, 0, None) == sp.SP_ERR_WORKSPACE
    # layouts
    lay = sp.binding._CLayout(1, 1, 256, 256, 256, 256, 256, 256, 10, 2, 8)
    ref = ctypes.byref(lay)
    # head_dim unsupported / heads not divisible / NULL layout / missing workspace
    assert lib.sp_superpose_prefill(256, 256, 256, ref, 4, 4, 96, 1.0, 0, 256, None, None, 0, 0, None) == sp.SP_ERR_UNSUPPORTED
    assert lib.sp_superpose_prefill(256, 256, 256, ref, 4, 3, 64, 1.0, 0, 256, None, None, 0, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_superpose_prefill(256, 256, 256, None, 4, 4, 64, 1.0, 0, 256, None, None, 0, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_superpose_prefill(256, 256, 256, ref, 4, 4, 64, 1.0, 0, 256, None, None, 0, 0, None) == sp.SP_ERR_WORKSPACE
    assert lib.sp_superpose_prefill(264, 256, 256, ref, 4, 4, 64, 1.0, 0, 256, None, 256, 1 << 20, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_superpose_prefill(256, 256, 256, ref, 4, 4, 64, 1.0, 5, 256, None, 256, 1 << 20, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_pruned_decode(256, 256, 256, ref, 256, 1, None, None, None, 0, 0, 4, 4, 64, 1.0, 256, None,
                                None, 0, 0, None) == sp.SP_ERR_WORKSPACE
    assert lib.sp_pruned_decode(256, 256, 256, ref, None, 1, None, None, None, 0, 0, 4, 4, 64, 1.0, 256, None,
                                256, 1 << 20, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_pruned_decode(256, 256, 256, ref, 256, 1, None, None, None, 4, 0, 4, 4, 64, 1.0, 256, None,
                                256, 1 << 20, 0, None) == sp.SP_ERR_INVALID_ARG   # tail_cap > 0, NULL tail
    bad = sp.binding._CLayout(-1, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0)
    assert lib.sp_pruned_decode(256, 256, 256, ctypes.byref(bad), 256, 1, None, None, None, 0, 0, 4, 4, 64, 1.0,
                                256, None, 256, 1 << 20, 0, None) == sp.SP_ERR_INVALID_ARG
    assert lib.sp_check_status(None, None) == sp.SP_ERR_INVALID_ARG


def test_workspace_sizes_are_sane():
    lib = sp.lib
    assert lib.sp_path_scores_workspace_bytes(1000) >= 256 + 4000
    assert lib.sp_decode_workspace_bytes(1, 32, 128) % 256 == 0
    assert lib.sp_decode_workspace_bytes(64, 32, 128) >= 256
    assert lib.sp_prefill_workspace_bytes(1, 20, 32, 184, 32, 128, sp.SP_BF16) >= 256


def test_next_round_layout_moves_kept_documents_into_the_prefix():
    import numpy as np
    from workloads import build_layout, next_round_layout
    lay = build_layout([3, 0], [[10, 20, 30], [5, 6]], [[4, 4, 4], [2, 2]])
    nxt = next_round_layout(lay, np.array([[2, 0], [4, -1]]))
    assert list(nxt.pre_len) == [3 + 30 + 10, 6]
    assert list(nxt.doc_len) == [20, 5] and list(nxt.qry_len) == [4, 2]
    assert list(nxt.prompt_path_off) == [0, 1, 2]
    assert nxt.total_tokens == 43 + 24 + 6 + 7
