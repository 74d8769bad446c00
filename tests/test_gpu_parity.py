"""GPU parity: every entry point of the C ABI against the CPU oracle, element by element on
the same seeded inputs, at sizes that span several tiles and ragged tails, plus edge cases.

Tolerances (stated by the target): attention outputs rel-L2 <= 1e-2 for bf16 and <= 1e-5
for fp32; |sum_t row_logp| within 1e-3 * query length; top-k indices bit-exact."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2404_06910_b200 as sp
from helpers import dev, f32, positions_for, rel_l2, workspace
from workloads import (CONFIGS, build_layout, draw_decode_inputs, draw_lengths, draw_logits,
                       draw_prior_weight, draw_qkv, draw_targets, next_round_layout)

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 1e-2}
TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


def _rng(seed):
    g = torch.Generator()
    g.manual_seed(seed)
    return g


def _randn(shape, dtype, seed, std=1.0):
    return (torch.randn(*shape, generator=_rng(seed)) * std).to(TDT[dtype])


# ------------------------------------------------------------------------- RoPE
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("pairing", [0, 1])
@pytest.mark.parametrize("H,D,rot", [(4, 64, 64), (32, 128, 128), (3, 128, 64), (2, 24, 12)])
def test_rope_parity(dtype, pairing, H, D, rot):
    n = 301
    x = _randn((n, H, D), dtype, 7)
    pos = (torch.rand(n, generator=_rng(8)) * 700).float()
    ref = oracle.rope(f32(x), pos.numpy(), rot_dim=rot, pairing=pairing)
    xd = dev(x)
    sp.sp_rope_apply(xd, dev(pos), H, D, rot_dim=rot, pairing=pairing)
    got = f32(xd)
    if dtype == "f32":
        np.testing.assert_allclose(got, ref, rtol=0, atol=4e-6)
    else:   # one bf16 rounding of the fp32 result
        assert np.all(np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 * 1.02 + 1e-6)


def test_rope_strided_tokens_and_empty():
    H, D, n, ld = 4, 64, 9, 4 * 64 * 3
    buf = _randn((n, ld), "f32", 3)
    pos = torch.arange(n).float() * 1.5
    ref = buf.clone().numpy()
    ref[:, :H * D] = oracle.rope(ref[:, :H * D].reshape(n, H, D).copy(), pos.numpy()).reshape(n, H * D)
    bd = dev(buf)
    sp.sp_rope_apply(bd, dev(pos), H, D, ld_token=ld)
    np.testing.assert_allclose(f32(bd), ref, atol=4e-6)
    sp.sp_rope_apply(bd, dev(pos), H, D, n_tokens=0)      # no-op


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rope_pair_equals_two_calls(dtype):
    """Queries and keys of a step rotated in one launch: bit-identical to two single calls, also
    with different head counts, a strided key tensor and an unaligned (scalar-path) shape."""
    for (Hq, Hk, D, rot, n, ldk) in [(32, 8, 128, 128, 301, None), (4, 4, 64, 32, 5, 3 * 4 * 64), (3, 1, 24, 12, 9, None)]:
        xq, xk = _randn((n, Hq, D), dtype, 70), _randn((n, (ldk or Hk * D)), dtype, 71)
        pos = (torch.rand(n, generator=_rng(72)) * 900).float()
        q1, k1 = dev(xq), dev(xk)
        sp.sp_rope_apply(q1, dev(pos), Hq, D, rot_dim=rot)
        sp.sp_rope_apply(k1, dev(pos), Hk, D, rot_dim=rot, ld_token=ldk)
        q2, k2 = dev(xq), dev(xk)
        sp.sp_rope_apply_pair(q2, Hq, k2, Hk, dev(pos), D, rot_dim=rot, ld_k=ldk)
        assert torch.equal(q1, q2) and torch.equal(k1, k2)
        ref = oracle.rope(f32(xq), pos.numpy(), rot_dim=rot)
        tol = 4e-6 if dtype == "f32" else None
        if tol:
            np.testing.assert_allclose(f32(q2), ref, rtol=0, atol=tol)
        else:
            assert np.all(np.abs(f32(q2) - ref) <= np.abs(ref) * 2.0 ** -8 * 1.02 + 1e-6)


# ------------------------------------------------------------------------- prefill
def _prefill_gpu(q, k, v, lay, scale, rows=sp.SP_ROWS_ALL, poison=True):
    dl = sp.DeviceLayout.from_host(lay)
    T, H, D = q.shape
    qd, kd, vd = dev(q), dev(k), dev(v)
    out = torch.full_like(qd, float("nan")) if poison else torch.zeros_like(qd)
    lse = torch.full((H, T), float("nan"), device="cuda")
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.dtype_code(qd)))
    sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out, lse, ws, rows=rows)
    sp.sp_check_status(ws)
    return f32(out), lse.cpu().numpy()


def _check_prefill(lay, H, Hkv, D, dtype, seed, std=1.0, scale=None, q_row_gain=None):
    T = lay.total_tokens
    q = _randn((T, H, D), dtype, seed, std)
    if q_row_gain is not None:
        q = (q.float() * torch.from_numpy(q_row_gain).float()[:, None, None]).to(q.dtype)
    k = _randn((T, Hkv, D), dtype, seed + 1, std)
    v = _randn((T, Hkv, D), dtype, seed + 2)
    scale = 1 / math.sqrt(D) if scale is None else scale
    ref_o, ref_l = oracle.prefill(f32(q), f32(k), f32(v), lay, scale)
    got_o, got_l = _prefill_gpu(q, k, v, lay, scale)
    assert not np.isnan(got_o).any(), "rows left unwritten"
    assert rel_l2(got_o, ref_o) <= TOL[dtype]
    np.testing.assert_allclose(got_l, ref_l, atol=1e-5 if dtype == "f32" else 2e-2)
    # per-row check too, so that a single bad row cannot hide in the norm
    num = np.linalg.norm((got_o - ref_o).reshape(T, -1), axis=1)
    den = np.linalg.norm(ref_o.reshape(T, -1), axis=1) + 1e-6
    assert (num / den).max() <= 2 * TOL[dtype]
    return q, k, v, got_o, got_l


@pytest.mark.parametrize("cfg", CONFIGS[:2], ids=lambda c: c.name)
def test_prefill_config_full(cfg):
    lay = draw_lengths(cfg)
    q, k, v = draw_qkv(cfg, lay)
    scale = 1 / math.sqrt(cfg.head_dim)
    ref_o, ref_l = oracle.prefill(f32(q), f32(k), f32(v), lay, scale)
    got_o, got_l = _prefill_gpu(q, k, v, lay, scale)
    assert rel_l2(got_o, ref_o) <= TOL[cfg.dtype]
    np.testing.assert_allclose(got_l, ref_l, atol=1e-5 if cfg.dtype == "f32" else 2e-2)


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16", 128)])
def test_prefill_ragged_edges(dtype, D):
    """Lengths around tile edges, empty preamble, empty documents, single rows."""
    lay = build_layout([0, 5, 16, 130],
                       [[1, 15, 16], [17, 127, 0], [128, 129], [300, 2, 64]],
                       [[1, 1, 2], [3, 1, 8], [7, 24], [33, 1, 64]])
    _check_prefill(lay, 4, 2, D, dtype, 100, std=1.0)


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("bf16", 128)])
def test_prefill_fewer_rows_than_one_tile(dtype, D):
    """Whole problems smaller than a single tile (the tensor is shorter than a TMA box)."""
    for pre, docs, qrys in (([3], [[5]], [[2]]), ([0], [[0]], [[1]]), ([1, 2], [[1], [0, 3]], [[1], [1, 1]])):
        lay = build_layout(pre, docs, qrys)
        _check_prefill(lay, 2, 2, D, dtype, 900 + lay.total_tokens)


def test_prefill_one_tile_items_follow_long_items():
    """Work items with a single key tile (no preamble, a path shorter than one tile) right after
    items with three key tiles in the same persistent block: warps whose rows are masked out of
    the long item's last tile run ahead into the short item, which must not disturb the hand-off
    of the long item's row sums.  With 2 heads a block's next item is 148 tiles further on."""
    docs, qrys = [], []
    for _ in range(3):
        docs += [184] * 74 + [12] * 148          # 74 paths of 192 rows (2 tiles each), 148 of 20 rows
        qrys += [8] * 74 + [8] * 148
    lay = build_layout([0], [docs], [qrys])
    # the middle third's queries are 6x larger, so its row sums and maxima differ widely from
    # those of the items that used the same hand-off slot before and after
    gain = np.ones(lay.total_tokens, dtype=np.float32)
    gain[lay.total_tokens // 3: 2 * lay.total_tokens // 3] = 6.0
    for rep in range(3):
        _check_prefill(lay, 2, 2, 128, "bf16", 4242 + rep, q_row_gain=gain)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_prefill_peaky_scores_and_planted_keys(dtype):
    """Unscaled N(0,1) q.k (sharp softmax) and one dominant key per row: masking or
    rescaling mistakes cannot hide behind a near-uniform softmax."""
    D, H = 128, 2
    lay = build_layout([40], [[200, 77]], [[24, 24]])
    _check_prefill(lay, H, H, D, dtype, 200, std=1.0, scale=0.35)
    T = lay.total_tokens
    q = _randn((T, H, D), dtype, 300, 0.05)
    k = _randn((T, H, D), dtype, 301, 0.05)
    v = _randn((T, H, D), dtype, 302)
    g = np.random.default_rng(5)
    for r in range(T):                      # plant: row r's query matches one allowed key strongly
        c = int(g.integers(0, r + 1)) if r < 40 else int(g.integers(0, 40))
        q[r] = (k[c].float() * 60).to(q.dtype)
    ref_o, _ = oracle.prefill(f32(q), f32(k), f32(v), lay, 1.0)
    got_o, _ = _prefill_gpu(q, k, v, lay, 1.0)
    assert rel_l2(got_o, ref_o) <= TOL[dtype]


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("bf16", 128)])
def test_prefill_query_only_rows(dtype, D):
    lay = build_layout([9, 33], [[50, 140], [7]], [[8, 8], [24]])
    H = 2
    T = lay.total_tokens
    q, k, v = (_randn((T, H, D), dtype, s) for s in (11, 12, 13))
    scale = 1 / math.sqrt(D)
    ref_o, ref_l = oracle.prefill(f32(q), f32(k), f32(v), lay, scale)
    got_o, got_l = _prefill_gpu(q, k, v, lay, scale, rows=sp.SP_ROWS_QUERY_ONLY)
    is_q = np.zeros(T, bool)
    for i in range(lay.n_paths):
        s = lay.path_start[i] + lay.doc_len[i]
        is_q[s:s + lay.qry_len[i]] = True
    assert np.isnan(got_o[~is_q]).all(), "non-query rows must stay untouched"
    assert rel_l2(got_o[is_q], ref_o[is_q]) <= TOL[dtype]
    np.testing.assert_allclose(got_l[:, is_q], ref_l[:, is_q], atol=1e-5 if dtype == "f32" else 2e-2)


def _query_row_mask(lay):
    is_q = np.zeros(lay.total_tokens, bool)
    for i in range(lay.n_paths):
        s = lay.path_start[i] + lay.doc_len[i]
        is_q[s:s + lay.qry_len[i]] = True
    return is_q


@pytest.mark.parametrize("case", ["ragged", "long_queries", "no_preamble_short", "many_paths"])
def test_prefill_query_only_ragged(case):
    """Query rows only (bf16, head_dim 128): query lengths around and beyond the 32-row item,
    empty documents and preambles, items of one or two key tiles behind longer ones, grouped
    heads; per-row check, untouched non-query rows, and bit-identical repeats."""
    rng = np.random.default_rng(11)
    if case == "ragged":
        lay = build_layout([0, 5, 40, 130], [[1, 15, 16, 31], [17, 127, 0], [128, 129], [300, 2, 64]],
                           [[1, 1, 2, 32], [3, 33, 8], [7, 24], [31, 1, 64]])
        H, Hkv = 4, 2
    elif case == "long_queries":
        lay = build_layout([33], [[200, 10, 0]], [[100, 65, 140]])
        H, Hkv = 2, 2
    elif case == "no_preamble_short":
        # items with one key tile (<= 32 keys in all) mixed with long ones, 2 heads
        docs = [int(x) for x in rng.integers(0, 20, 300)]
        docs[::7] = [250] * len(docs[::7])
        lay = build_layout([0], [docs], [[int(x) for x in rng.integers(1, 12, 300)]])
        H, Hkv = 2, 1
    else:
        lay = build_layout([32] * 3, [[int(x) for x in rng.integers(64, 257, 40)] for _ in range(3)], [[24] * 40] * 3)
        H, Hkv = 8, 8
    T, D = lay.total_tokens, 128
    q, k, v = _randn((T, H, D), "bf16", 21), _randn((T, Hkv, D), "bf16", 22), _randn((T, Hkv, D), "bf16", 23)
    gain = np.ones(T, np.float32)
    gain[T // 3: 2 * T // 3] = 4.0
    q = (q.float() * torch.from_numpy(gain)[:, None, None]).to(q.dtype)
    scale = 1 / math.sqrt(D)
    ref_o, ref_l = oracle.prefill(f32(q), f32(k), f32(v), lay, scale)
    got_o, got_l = _prefill_gpu(q, k, v, lay, scale, rows=sp.SP_ROWS_QUERY_ONLY)
    is_q = _query_row_mask(lay)
    assert np.isnan(got_o[~is_q]).all(), "non-query rows must stay untouched"
    assert not np.isnan(got_o[is_q]).any(), "query rows left unwritten"
    num = np.linalg.norm((got_o - ref_o)[is_q].reshape(int(is_q.sum()), -1), axis=1)
    den = np.linalg.norm(ref_o[is_q].reshape(int(is_q.sum()), -1), axis=1) + 1e-6
    assert rel_l2(got_o[is_q], ref_o[is_q]) <= TOL["bf16"]
    assert (num / den).max() <= 5 * TOL["bf16"]
    np.testing.assert_allclose(got_l[:, is_q], ref_l[:, is_q], atol=2e-2)
    for _ in range(3):
        again_o, again_l = _prefill_gpu(q, k, v, lay, scale, rows=sp.SP_ROWS_QUERY_ONLY)
        np.testing.assert_array_equal(again_o[is_q], got_o[is_q])
        np.testing.assert_array_equal(again_l[:, is_q], got_l[:, is_q])


def test_prefill_is_deterministic():
    cfg = CONFIGS[1]
    lay = draw_lengths(cfg)
    q, k, v = draw_qkv(cfg, lay)
    a, la = _prefill_gpu(q, k, v, lay, 0.0884)
    for _ in range(5):
        b, lb = _prefill_gpu(q, k, v, lay, 0.0884)
        np.testing.assert_array_equal(a, b)
        np.testing.assert_array_equal(la, lb)


@pytest.mark.parametrize("case", ["mixed", "tiny_items", "preamble_only", "merged_documents"])
def test_prefill_random_ragged_layouts(case):
    """Random segment lengths (empty documents and preambles included), grouped-query heads,
    items of every size next to each other in the persistent blocks' work lists."""
    rng = np.random.default_rng(3)
    if case == "mixed":
        lay = build_layout(list(rng.integers(0, 70, 4)), [list(rng.integers(0, 300, 30)) for _ in range(4)],
                           [list(rng.integers(1, 40, 30)) for _ in range(4)])
        H, Hkv = 8, 2
    elif case == "tiny_items":
        lay = build_layout([0] * 4, [list(rng.integers(0, 30, 200)) for _ in range(4)],
                           [list(rng.integers(1, 8, 200)) for _ in range(4)])
        H, Hkv = 4, 4
    elif case == "merged_documents":
        # superposition factor > 1 (Appendix ablation): several documents share a path, so paths
        # run to many query tiles and long causal key ranges
        lay = build_layout([48, 0], [list(rng.integers(500, 1000, 5)), list(rng.integers(300, 700, 4))],
                           [[32] * 5, [24] * 4])
        H, Hkv = 4, 2
    else:
        lay = build_layout([700, 1, 129], [[], [], []], [[], [], []])
        H, Hkv = 4, 1
    gain = np.ones(lay.total_tokens, dtype=np.float32)
    gain[lay.total_tokens // 3: 2 * lay.total_tokens // 3] = 5.0
    _check_prefill(lay, H, Hkv, 128, "bf16", 77, q_row_gain=gain)


# ------------------------------------------------------------------------- path scores
def _scores_gpu(logits, tgt, off, prior, weight, with_rows=True):
    R = logits.shape[0]
    n_paths = len(off) - 1
    scores = torch.full((n_paths,), float("nan"), device="cuda")
    rows = torch.full((R,), float("nan"), device="cuda") if with_rows else None
    ws = workspace(sp.sp_path_scores_workspace_bytes(R))
    sp.sp_path_scores(dev(logits), dev(tgt), dev(off), scores,
                      None if prior is None else dev(prior), None if weight is None else dev(weight),
                      rows, ws)
    return scores.cpu().numpy(), None if rows is None else rows.cpu().numpy()


@pytest.mark.parametrize("cfg", CONFIGS[:2], ids=lambda c: c.name)
def test_path_scores_config_full(cfg):
    lay = draw_lengths(cfg)
    logits = draw_logits(cfg, lay)
    tgt = draw_targets(cfg, lay)
    prior, weight = draw_prior_weight(cfg, lay)
    off = lay.query_row_offsets()
    ref_s, ref_r = oracle.path_scores(f32(logits), tgt, off, prior, weight)
    got_s, got_r = _scores_gpu(logits, tgt, off, prior, weight)
    np.testing.assert_allclose(got_r, ref_r, atol=1e-3)
    sums_got = np.add.reduceat(got_r, off[:-1])
    sums_ref = np.add.reduceat(ref_r, off[:-1])
    assert np.all(np.abs(sums_got - sums_ref) <= 1e-3 * lay.qry_len)
    assert np.all(np.abs(got_s - ref_s) <= 1e-3 * lay.qry_len * weight + 1e-6)
    # reproducible bit for bit, with or without the row output
    again, _ = _scores_gpu(logits, tgt, off, prior, weight, with_rows=False)
    np.testing.assert_array_equal(got_s, again)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 7, 8, 1000, 4099, 50432])
def test_path_scores_vocab_edges(dtype, V):
    qlens = [1, 3, 0, 5]
    off = np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32)
    logits = _randn((int(off[-1]), V), dtype, 40 + V, 3.0)
    g = np.random.default_rng(V)
    tgt = g.integers(0, V, size=int(off[-1])).astype(np.int32)
    tgt[[0, 3]] = -1
    ref_s, ref_r = oracle.path_scores(f32(logits), tgt, off)
    got_s, got_r = _scores_gpu(logits, tgt, off, None, None)
    np.testing.assert_allclose(got_r, ref_r, atol=1e-4)
    np.testing.assert_allclose(got_s, ref_s, atol=1e-3)
    assert got_s[2] == 0.0                      # a path with no rows scores its prior (0)


def test_path_scores_unaligned_rows_and_large_offsets():
    V, ld = 1003, 1011                          # odd stride: rows are not 16-byte aligned
    buf = _randn((6, ld), "bf16", 77, 3.0)
    logits = buf[:, :V]
    off = np.array([0, 6], np.int32)
    tgt = np.array([5, 1002, 0, 17, -1, 400], np.int32)
    ref_s, ref_r = oracle.path_scores(f32(logits), tgt, off)
    scores = torch.zeros(1, device="cuda")
    rows = torch.zeros(6, device="cuda")
    sp.sp_path_scores(dev(buf)[:, :V], dev(tgt), dev(off), scores, row_logp=rows)
    np.testing.assert_allclose(rows.cpu().numpy(), ref_r, atol=1e-4)
    # logits far from zero: the running maximum must carry the scale
    shifted = (f32(logits) * 0 + 3.0e4).astype(np.float32)
    shifted[:, ::7] += 11.0
    ref_s, ref_r = oracle.path_scores(shifted, tgt, off)
    got_s, got_r = _scores_gpu(torch.from_numpy(shifted), tgt, off, None, None)
    np.testing.assert_allclose(got_r, ref_r, atol=1e-3)


# ------------------------------------------------------------------------- top-k
def _topk_gpu(scores, ppo, k):
    B = len(ppo) - 1
    idx = torch.full((B, k), -7, dtype=torch.int32, device="cuda")
    post = torch.full((B, k), float("nan"), device="cuda")
    sp.sp_prune_topk(dev(scores), dev(ppo), k, idx, post)
    return idx.cpu().numpy(), post.cpu().numpy()


@pytest.mark.parametrize("n,k", [(4, 1), (20, 2), (100, 4), (400, 8), (33, 33), (5, 9), (1000, 64)])
def test_topk_bit_exact(n, k):
    g = np.random.default_rng(n * 31 + k)
    ppo = np.array([0, n, n, 2 * n + 3], np.int32)
    s = g.standard_normal(int(ppo[-1])).astype(np.float32)
    s[g.integers(0, len(s), size=len(s) // 4)] = s[0]        # many exact ties
    ref_i, ref_p = oracle.prune_topk(s, ppo, k)
    got_i, got_p = _topk_gpu(s, ppo, k)
    np.testing.assert_array_equal(got_i, ref_i)
    np.testing.assert_allclose(got_p, ref_p, rtol=2e-5, atol=1e-9)


def test_topk_nan_inf_and_signed_zero():
    ppo = np.array([0, 8, 12], np.int32)
    s = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1.0, np.nan, 0.0,
                  np.nan, np.nan, -np.inf, -np.inf], np.float32)
    ref_i, ref_p = oracle.prune_topk(s[:8].copy(), ppo[:2], 8)
    got_i, got_p = _topk_gpu(s, ppo, 8)
    np.testing.assert_array_equal(got_i[0], ref_i[0])
    assert list(got_i[0]) == [3, 5, 0, 1, 7, 4, 2, 6]
    ref_i2, ref_p2 = oracle.prune_topk(s, ppo, 8)
    np.testing.assert_array_equal(got_i, ref_i2)
    np.testing.assert_array_equal(got_p[1], ref_p2[1])           # all -inf / NaN: posterior 0


# ------------------------------------------------------------------------- decode
def _decode_case(lay, H, Hkv, D, dtype, k, kept, tail_cap, tail_len, seed, scale=None, std=1.0):
    B, T = lay.n_prompts, lay.total_tokens
    kc = _randn((T, Hkv, D), dtype, seed, std)
    vc = _randn((T, Hkv, D), dtype, seed + 1)
    q = _randn((B, H, D), dtype, seed + 2, std)
    tk = _randn((B, max(tail_cap, 1), Hkv, D), dtype, seed + 3, std)
    tv = _randn((B, max(tail_cap, 1), Hkv, D), dtype, seed + 4)
    scale = 1 / math.sqrt(D) if scale is None else scale
    kept = np.asarray(kept, np.int32).reshape(B, k)
    tl = np.asarray(tail_len, np.int32)
    ref_o, ref_l = oracle.pruned_decode(f32(q), f32(kc), f32(vc), lay, kept, f32(tk), f32(tv), tl, scale)
    dl = sp.DeviceLayout.from_host(lay)
    out = torch.full((B, H, D), float("nan"), dtype=TDT[dtype], device="cuda")
    lse = torch.full((B, H), float("nan"), device="cuda")
    ws = workspace(sp.sp_decode_workspace_bytes(B, H, D))
    args = (dev(q), dev(kc), dev(vc), dl, dev(kept), k,
            dev(tk) if tail_cap else None, dev(tv) if tail_cap else None, dev(tl) if tail_cap else None,
            tail_cap, scale, out, lse, ws)
    sp.sp_pruned_decode(*args)
    sp.sp_check_status(ws)
    got_o, got_l = f32(out), lse.cpu().numpy()
    assert rel_l2(got_o, ref_o) <= TOL[dtype]
    fin = np.isfinite(ref_l)
    np.testing.assert_allclose(got_l[fin], ref_l[fin], atol=1e-5 if dtype == "f32" else 2e-2)
    np.testing.assert_array_equal(got_l[~fin], ref_l[~fin])
    out2 = torch.full_like(out, float("nan"))
    sp.sp_pruned_decode(*args[:11], out2, lse, ws)      # same workspace again: bit-identical
    np.testing.assert_array_equal(f32(out2), got_o)
    return got_o


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16", 128)])
def test_decode_small_batches_split_kv(dtype, D):
    lay = build_layout([16, 3], [[32, 1, 129, 40], [200, 17]], [[8, 8, 8, 8], [5, 5]])
    _decode_case(lay, 4, 2, D, dtype, 2, [[2, 0], [4, -1]], 6, [6, 1], 500)
    _decode_case(lay, 4, 4, D, dtype, 4, [[3, 2, 1, 0], [5, 4, -1, -1]], 0, [0, 0], 510)   # k = N, no tail
    _decode_case(lay, 2, 1, D, dtype, 1, [[-1], [-1]], 3, [0, 2], 520)                     # nothing kept


def test_decode_no_keys_at_all():
    lay = build_layout([0, 4], [[5], [6]], [[2], [2]])
    got = _decode_case(lay, 2, 2, 64, "f32", 1, [[-1], [1]], 2, [0, 1], 530)
    assert np.all(got[0] == 0.0)


@pytest.mark.parametrize("cfg", CONFIGS[:2], ids=lambda c: c.name)
def test_decode_config_steps(cfg):
    """The config's decode loop: kept paths from the oracle's top-k, tail growing by one
    token per step (the new token attends to itself)."""
    lay = draw_lengths(cfg)
    _, kc, vc = draw_qkv(cfg, lay)
    steps = min(cfg.decode_steps, 5)
    q, tk, tv = draw_decode_inputs(cfg, lay.n_prompts, steps)
    scores = np.random.default_rng(cfg.seed).standard_normal(lay.n_paths).astype(np.float32)
    kept, _ = oracle.prune_topk(scores, lay.prompt_path_off, cfg.top_k)
    dl = sp.DeviceLayout.from_host(lay)
    B, H, D = lay.n_prompts, cfg.n_heads, cfg.head_dim
    ws = workspace(sp.sp_decode_workspace_bytes(B, H, D))
    kcd, vcd, tkd, tvd, keptd = dev(kc), dev(vc), dev(tk), dev(tv), dev(kept)
    scale = 1 / math.sqrt(D)
    for t in range(steps):
        tl = np.full(B, t + 1, np.int32)
        ref_o, _ = oracle.pruned_decode(f32(q[t]), f32(kc), f32(vc), lay, kept, f32(tk), f32(tv), tl, scale)
        out = torch.empty((B, H, D), dtype=TDT[cfg.dtype], device="cuda")
        sp.sp_pruned_decode(dev(q[t]), kcd, vcd, dl, keptd, cfg.top_k, tkd, tvd, dev(tl), steps, scale, out, None, ws)
        assert rel_l2(f32(out), ref_o) <= TOL[cfg.dtype]


# ------------------------------------------------------------------------- whole chain
@pytest.mark.parametrize("cfg", CONFIGS[:2], ids=lambda c: c.name)
def test_chain_rope_prefill_scores_topk_decode(cfg):
    """One pass of the hot path, each stage fed by the previous stage's device output,
    against the same chain in the oracle."""
    lay = draw_lengths(cfg)
    B, H, Hkv, D = lay.n_prompts, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    q, k, v = draw_qkv(cfg, lay)
    if cfg.positions == "equilibrium":
        pos, nxt = positions_for(lay, lambda P, L, Q: sp.sp_positions(P, L, Q))
        pos_ref, _ = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q))
    else:
        pos, nxt = positions_for(lay, lambda P, L, Q: sp.sp_positions(P, L, Q, scheme=sp.SP_POS_LEFT_ALIGNED))
        pos_ref, _ = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q, scheme="left"))
    np.testing.assert_array_equal(pos, pos_ref)
    scale = 1 / math.sqrt(D)
    dl = sp.DeviceLayout.from_host(lay)
    qd, kd, vd, posd = dev(q), dev(k), dev(v), dev(pos)
    sp.sp_rope_apply(qd, posd, H, D, base=cfg.rope_base)
    sp.sp_rope_apply(kd, posd, Hkv, D, base=cfg.rope_base)
    out = torch.empty_like(qd)
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.dtype_code(qd)))
    sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out, None, ws)
    # oracle chain (rounding the rotated tensors to the storage type, as the device does)
    rnd = (lambda a: a) if cfg.dtype == "f32" else (lambda a: torch.from_numpy(a).bfloat16().float().numpy())
    q_r = rnd(oracle.rope(f32(q), pos_ref, base=cfg.rope_base))
    k_r = rnd(oracle.rope(f32(k), pos_ref, base=cfg.rope_base))
    ref_o, _ = oracle.prefill(q_r, k_r, f32(v), lay, scale)
    assert rel_l2(f32(out), ref_o) <= TOL[cfg.dtype] * (1 if cfg.dtype == "bf16" else 3)

    logits, tgt = draw_logits(cfg, lay), draw_targets(cfg, lay)
    prior, weight = draw_prior_weight(cfg, lay)
    off = lay.query_row_offsets()
    scores = torch.empty(lay.n_paths, device="cuda")
    ws2 = workspace(sp.sp_path_scores_workspace_bytes(logits.shape[0]))
    sp.sp_path_scores(dev(logits), dev(tgt), dev(off), scores, dev(prior), dev(weight), None, ws2)
    kept = torch.empty((B, cfg.top_k), dtype=torch.int32, device="cuda")
    post = torch.empty((B, cfg.top_k), device="cuda")
    sp.sp_prune_topk(scores, dl.prompt_path_off, cfg.top_k, kept, post)
    ref_s, _ = oracle.path_scores(f32(logits), tgt, off, prior, weight)
    ref_kept, ref_post = oracle.prune_topk(ref_s, lay.prompt_path_off, cfg.top_k)
    tol = 1e-3 * cfg.qry_len * float(weight.max())
    for b in range(B):       # bit-exact where the k-th / (k+1)-th gap exceeds twice the tolerance
        lo, hi = lay.prompt_path_off[b], lay.prompt_path_off[b + 1]
        srt = np.sort(ref_s[lo:hi])[::-1]
        gaps = np.abs(np.diff(srt[:cfg.top_k + 1]))
        if gaps.size == 0 or gaps.min() > 2 * tol:
            np.testing.assert_array_equal(kept[b].cpu().numpy(), ref_kept[b])
        else:
            assert set(kept[b].cpu().numpy()) <= set(np.where(ref_s[lo:hi] >= srt[cfg.top_k - 1] - 2 * tol)[0] + lo)
    np.testing.assert_allclose(post.cpu().numpy(), ref_post, rtol=5e-3, atol=1e-6)

    steps = 3
    dq, tk, tv = draw_decode_inputs(cfg, B, steps)
    tkd, tvd = dev(tk), dev(tv)
    ws3 = workspace(sp.sp_decode_workspace_bytes(B, H, D))
    kept_h = kept.cpu().numpy()
    tk_ref, tv_ref = f32(tk).copy(), f32(tv)
    for t in range(steps):
        tpos = np.asarray(nxt + t, np.float32)          # task / response positions continue with step 1
        qt = dev(dq[t])
        sp.sp_rope_apply(qt, dev(tpos), H, D, base=cfg.rope_base)
        sp.sp_rope_apply(tkd[:, t], dev(tpos), Hkv, D, n_tokens=B, ld_token=steps * Hkv * D, base=cfg.rope_base)
        o = torch.empty((B, H, D), dtype=TDT[cfg.dtype], device="cuda")
        tl = np.full(B, t + 1, np.int32)
        sp.sp_pruned_decode(qt, kd, vd, dl, kept, cfg.top_k, tkd, tvd, dev(tl), steps, scale, o, None, ws3)
        qt_ref = rnd(oracle.rope(f32(dq[t]), tpos, base=cfg.rope_base))
        tk_ref[:, t] = rnd(oracle.rope(np.ascontiguousarray(tk_ref[:, t]), tpos, base=cfg.rope_base))
        ref_d, _ = oracle.pruned_decode(qt_ref, k_r, f32(v), lay, kept_h, tk_ref, tv_ref, tl, scale)
        assert rel_l2(f32(o), ref_d) <= TOL[cfg.dtype] * (1 if cfg.dtype == "bf16" else 3)


def test_iterative_superposition_rounds():
    """Section 4.3's iterative variant, t = 3 rounds with k = 2: each round is a fork-join prefill
    over the remaining documents behind a shared prefix that has grown by the documents kept so
    far, scored and pruned; the response then attends to the final prefix plus the last kept paths.
    Every round's device results are checked against the oracle on the same layout."""
    cfg = CONFIGS[1]
    H, Hkv, D, k_top = 8, 4, 128, 2
    rng = np.random.default_rng(99)
    lay = build_layout([20, 7], [list(rng.integers(40, 200, 9)), list(rng.integers(40, 200, 7))], [[12] * 9, [12] * 7])
    scale = 1 / math.sqrt(D)
    for rnd_no in range(3):
        B, T = lay.n_prompts, lay.total_tokens
        q, k, v = _randn((T, H, D), "bf16", 50 + rnd_no), _randn((T, Hkv, D), "bf16", 60 + rnd_no), _randn((T, Hkv, D), "bf16", 70 + rnd_no)
        pos, _ = positions_for(lay, lambda P, L, Q: sp.sp_positions(P, L, Q))
        pos_ref, _ = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q))
        np.testing.assert_array_equal(pos, pos_ref)
        dl = sp.DeviceLayout.from_host(lay)
        qd, kd, vd = dev(q), dev(k), dev(v)
        sp.sp_rope_apply(qd, dev(pos), H, D)
        sp.sp_rope_apply(kd, dev(pos), Hkv, D)
        out = torch.full_like(qd, float("nan"))
        ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.SP_BF16))
        sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out, None, ws)
        sp.sp_check_status(ws)
        bf = lambda a: torch.from_numpy(a).bfloat16().float().numpy()
        q_r, k_r = bf(oracle.rope(f32(q), pos_ref)), bf(oracle.rope(f32(k), pos_ref))
        ref_o, _ = oracle.prefill(q_r, k_r, f32(v), lay, scale)
        assert rel_l2(f32(out), ref_o) <= TOL["bf16"]
        # the same round in cached mode (query rows only) agrees on the query rows
        out_q = torch.full_like(qd, float("nan"))
        sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out_q, None, ws, rows=sp.SP_ROWS_QUERY_ONLY)
        is_q = _query_row_mask(lay)
        assert rel_l2(f32(out_q)[is_q], ref_o[is_q]) <= TOL["bf16"]

        R = int(lay.qry_len.sum())
        logits = _randn((R, 777), "bf16", 80 + rnd_no, 3.0)
        tgt = rng.integers(0, 777, R).astype(np.int32)
        off = lay.query_row_offsets()
        weight = (1.0 / np.maximum(lay.qry_len, 1)).astype(np.float32)
        prior = rng.normal(-2.5, 0.25, lay.n_paths).astype(np.float32)
        scores = torch.empty(lay.n_paths, device="cuda")
        sp.sp_path_scores(dev(logits), dev(tgt), dev(off), scores, dev(prior), dev(weight), None,
                          workspace(sp.sp_path_scores_workspace_bytes(R)))
        ref_s, _ = oracle.path_scores(f32(logits), tgt, off, prior, weight)
        np.testing.assert_allclose(scores.cpu().numpy(), ref_s, atol=1e-3)
        kept = torch.empty((B, k_top), dtype=torch.int32, device="cuda")
        sp.sp_prune_topk(scores, dl.prompt_path_off, k_top, kept)
        ref_kept, _ = oracle.prune_topk(scores.cpu().numpy(), lay.prompt_path_off, k_top)
        np.testing.assert_array_equal(kept.cpu().numpy(), ref_kept)     # same scores in: bit-exact
        if rnd_no < 2:
            nxt = next_round_layout(lay, ref_kept)
            assert nxt.n_paths == lay.n_paths - B * k_top
            assert nxt.total_tokens == lay.total_tokens - sum(int(lay.qry_len[i]) for i in ref_kept.ravel())
            lay = nxt
    # response step on the last round's tensors: prefix (preamble + 4 documents kept earlier) + 2 kept paths
    dq, tk, tv = _randn((B, H, D), "bf16", 90), _randn((B, 1, Hkv, D), "bf16", 91), _randn((B, 1, Hkv, D), "bf16", 92)
    o = torch.empty((B, H, D), dtype=torch.bfloat16, device="cuda")
    tl = np.ones(B, np.int32)
    sp.sp_pruned_decode(dev(dq), kd, vd, dl, kept, k_top, dev(tk), dev(tv), dev(tl), 1, scale, o, None,
                        workspace(sp.sp_decode_workspace_bytes(B, H, D)))
    ref_d, _ = oracle.pruned_decode(f32(dq), k_r, f32(v), lay, ref_kept, f32(tk), f32(tv), tl, scale)
    assert rel_l2(f32(o), ref_d) <= TOL["bf16"]


# ------------------------------------------------------------------------- ALiBi variants
def _slopes(H):
    return np.array([2.0 ** (-8.0 * (h + 1) / H) for h in range(H)], np.float32)


@pytest.mark.parametrize("dtype,D,rows", [("f32", 64, "all"), ("bf16", 64, "all"), ("bf16", 128, "all"), ("bf16", 128, "query"),
                                          ("f32", 128, "query")])
def test_prefill_alibi_parity(dtype, D, rows):
    """Fork-join prefill with the ALiBi bias at equilibrium (fractional) positions, every kernel
    that serves the entry point: fp32 / head_dim 64 SIMT, bf16 tensor-core, bf16 query-only."""
    rng = np.random.default_rng(5)
    lay = build_layout([0, 40, 130], [[1, 15, 70, 200], [17, 127, 0], [128, 300]],
                       [[9, 9, 9, 9], [33, 33, 33], [24, 24]])
    H, Hkv, T = 4, 2, lay.total_tokens
    pos, _ = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q))
    slopes = _slopes(H) * 4.0
    q, k, v = _randn((T, H, D), dtype, 31), _randn((T, Hkv, D), dtype, 32), _randn((T, Hkv, D), dtype, 33)
    scale = 1 / math.sqrt(D)
    ref_o, ref_l = oracle.prefill(f32(q), f32(k), f32(v), lay, scale, pos=pos, slopes=slopes)
    plain_o, _ = oracle.prefill(f32(q), f32(k), f32(v), lay, scale)
    assert rel_l2(plain_o, ref_o) > 0.05, "the bias must matter in this test"
    dl = sp.DeviceLayout.from_host(lay)
    qd = dev(q)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full((H, T), float("nan"), device="cuda")
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.dtype_code(qd)))
    mode = sp.SP_ROWS_ALL if rows == "all" else sp.SP_ROWS_QUERY_ONLY
    sp.sp_superpose_prefill_alibi(qd, dev(k), dev(v), dl, dev(pos), dev(slopes), scale, out, lse, ws, rows=mode)
    sp.sp_check_status(ws)
    sel = np.ones(T, bool) if rows == "all" else _query_row_mask(lay)
    got_o, got_l = f32(out), lse.cpu().numpy()
    assert np.isnan(got_o[~sel]).all() and not np.isnan(got_o[sel]).any()
    assert rel_l2(got_o[sel], ref_o[sel]) <= TOL[dtype]
    num = np.linalg.norm((got_o - ref_o)[sel].reshape(int(sel.sum()), -1), axis=1)
    den = np.linalg.norm(ref_o[sel].reshape(int(sel.sum()), -1), axis=1) + 1e-6
    assert (num / den).max() <= 2 * TOL[dtype]
    np.testing.assert_allclose(got_l[:, sel], ref_l[:, sel], atol=2e-5 if dtype == "f32" else 2e-2)


@pytest.mark.parametrize("dtype,D", [("f32", 64), ("bf16", 128)])
def test_decode_alibi_parity(dtype, D):
    lay = build_layout([16, 3], [[32, 1, 129, 40], [200, 17]], [[8, 8, 8, 8], [5, 5]])
    B, H, Hkv, T, k_top, cap = 2, 4, 2, lay.total_tokens, 2, 6
    kc, vc = _randn((T, Hkv, D), dtype, 41), _randn((T, Hkv, D), dtype, 42)
    q = _randn((B, H, D), dtype, 43)
    tk, tv = _randn((B, cap, Hkv, D), dtype, 44), _randn((B, cap, Hkv, D), dtype, 45)
    kept = np.array([[2, 0], [4, -1]], np.int32)
    tl = np.array([6, 1], np.int32)
    cpos, nxt = positions_for(lay, lambda P, L, Q: oracle.positions(P, L, Q))
    tpos = (nxt[:, None] + np.arange(cap)[None, :]).astype(np.float32)
    qpos = tpos[np.arange(B), tl - 1].copy()
    slopes = _slopes(H) * 4.0
    scale = 1 / math.sqrt(D)
    ref_o, ref_l = oracle.pruned_decode(f32(q), f32(kc), f32(vc), lay, kept, f32(tk), f32(tv), tl, scale,
                                        q_pos=qpos, cache_pos=cpos, tail_pos=tpos, slopes=slopes)
    plain_o, _ = oracle.pruned_decode(f32(q), f32(kc), f32(vc), lay, kept, f32(tk), f32(tv), tl, scale)
    assert rel_l2(plain_o, ref_o) > 0.05
    dl = sp.DeviceLayout.from_host(lay)
    out = torch.full((B, H, D), float("nan"), dtype=TDT[dtype], device="cuda")
    lse = torch.full((B, H), float("nan"), device="cuda")
    ws = workspace(sp.sp_decode_workspace_bytes(B, H, D))
    sp.sp_pruned_decode_alibi(dev(q), dev(kc), dev(vc), dl, dev(kept), k_top, dev(tk), dev(tv), dev(tl), cap,
                              dev(qpos), dev(cpos), dev(tpos), dev(slopes), scale, out, lse, ws)
    sp.sp_check_status(ws)
    assert rel_l2(f32(out), ref_o) <= TOL[dtype]
    np.testing.assert_allclose(lse.cpu().numpy(), ref_l, atol=2e-5 if dtype == "f32" else 2e-2)


# ------------------------------------------------------------------------- decode with the rotation folded in
@pytest.mark.parametrize("dtype,D", [("f32", 64), ("f32", 128), ("bf16", 64), ("bf16", 128)])
@pytest.mark.parametrize("pairing", [0, 1])
@pytest.mark.parametrize("H,Hkv", [(4, 4), (4, 2), (8, 2)])
def test_decode_rope_fused(dtype, D, pairing, H, Hkv):
    """sp_pruned_decode_rope against the oracle's rope followed by its decode, over three steps
    (so that keys rotated and written back by earlier steps are read again), and the stored
    tail keys against the stand-alone rotation."""
    lay = build_layout([16, 3, 0], [[32, 1, 129, 40], [200, 17], [5]], [[8, 8, 8, 8], [5, 5], [2]])
    B, T, cap, k = lay.n_prompts, lay.total_tokens, 4, 2
    kc, vc = _randn((T, Hkv, D), dtype, 700), _randn((T, Hkv, D), dtype, 701)
    tk, tv = _randn((B, cap, Hkv, D), dtype, 703), _randn((B, cap, Hkv, D), dtype, 704)
    kept = np.array([[2, 0], [4, -1], [-1, -1]], np.int32)
    dl = sp.DeviceLayout.from_host(lay)
    scale = 1 / math.sqrt(D)
    rnd = (lambda a: a) if dtype == "f32" else (lambda a: torch.from_numpy(a).bfloat16().float().numpy())
    tkd, kcd, vcd, tvd, keptd = dev(tk), dev(kc), dev(vc), dev(tv), dev(kept)
    tk_ref = f32(tk).copy()                                   # oracle's tail: rows rotated as the steps go
    tk_sep = dev(tk)                                          # rotated by the stand-alone kernel
    for step in range(3):
        q = _randn((B, H, D), dtype, 710 + step)
        pos = np.array([301.25 + step, 17.5 + 2 * step, 3.0 + step], np.float32)
        tl = np.array([step + 1, step + 1, step + 1 if step else 0], np.int32)   # prompt 2 has no tail at step 0
        out = torch.full((B, H, D), float("nan"), dtype=TDT[dtype], device="cuda")
        lse = torch.full((B, H), float("nan"), device="cuda")
        sp.sp_pruned_decode_rope(dev(q), kcd, vcd, dl, keptd, k, tkd, tvd, dev(tl), cap, dev(pos), scale, out, lse,
                                 pairing=pairing)
        torch.cuda.synchronize()
        # oracle: rotate q and each prompt's newest tail row, then decode
        q_ref = rnd(oracle.rope(f32(q), pos, pairing=pairing))
        for b in range(B):
            if tl[b] > 0:
                r = tl[b] - 1
                tk_ref[b, r] = rnd(oracle.rope(np.ascontiguousarray(tk_ref[b, r][None]), pos[b:b + 1], pairing=pairing))[0]
                sp.sp_rope_apply(tk_sep[b, r], dev(pos[b:b + 1]), Hkv, D, n_tokens=1, pairing=pairing)
        ref_o, ref_l = oracle.pruned_decode(q_ref, f32(kc), f32(vc), lay, kept, tk_ref, f32(tv), tl, scale)
        assert rel_l2(f32(out), ref_o) <= TOL[dtype]
        fin = np.isfinite(ref_l)
        np.testing.assert_allclose(lse.cpu().numpy()[fin], ref_l[fin], atol=1e-5 if dtype == "f32" else 2e-2)
        # the rows written back: what the stand-alone rotation stores, up to one rounding of the last place
        got_t, sep_t = f32(tkd), f32(tk_sep)
        for b in range(B):
            rows = slice(0, int(tl[b]))
            tol = 2e-6 if dtype == "f32" else 2.0 ** -7
            assert np.all(np.abs(got_t[b, rows] - sep_t[b, rows]) <= np.abs(sep_t[b, rows]) * tol + 2e-6)
            np.testing.assert_array_equal(got_t[b, int(tl[b]):], f32(tk)[b, int(tl[b]):])    # later rows untouched


def test_decode_rope_rejects_wide_groups():
    lay = build_layout([4], [[8]], [[2]])
    dl = sp.DeviceLayout.from_host(lay)
    q = dev(_randn((1, 8, 64), "f32", 1))
    kc = dev(_randn((lay.total_tokens, 1, 64), "f32", 2))
    tk = dev(_randn((1, 1, 1, 64), "f32", 3))
    with pytest.raises(sp.SpError) as e:
        sp.sp_pruned_decode_rope(q, kc, kc, dl, dev(np.array([[0]], np.int32)), 1, tk, tk, dev(np.array([1], np.int32)), 1,
                                 dev(np.array([5.0], np.float32)), 0.125, torch.empty_like(q))
    assert e.value.code == sp.SP_ERR_UNSUPPORTED


@pytest.mark.parametrize("H,Hkv", [(8, 1), (8, 2), (6, 3), (6, 2), (3, 1), (32, 8)])
def test_decode_grouped_heads(H, Hkv):
    """Query heads that share a KV head are served by one block per group of 4, 2 or 1 heads."""
    lay = build_layout([16, 3], [[32, 1, 129, 40], [200, 17]], [[8, 8, 8, 8], [5, 5]])
    _decode_case(lay, H, Hkv, 128, "bf16", 2, [[2, 0], [4, -1]], 6, [6, 1], 540)
    _decode_case(lay, H, Hkv, 64, "f32", 2, [[3, 1], [5, 4]], 2, [0, 2], 541)


def test_decode_long_sequences_many_splits():
    """Few (prompt, head) pairs and thousands of keys: the largest cluster (16 blocks) and many loop trips."""
    lay = build_layout([64], [[2000, 1500, 3000]], [[32, 32, 32]])
    _decode_case(lay, 2, 2, 128, "bf16", 3, [[2, 0, 1]], 40, [37], 550)
    _decode_case(lay, 1, 1, 64, "f32", 2, [[1, 2]], 8, [8], 551)


def test_prefill_pair_variant_in_child_process():
    """The experimental two-tiles-per-block prefill (shared K/V stages) is chosen by an environment
    variable when the library is first used, so it runs in a child process: the ragged, sub-tile,
    peaky, random-layout, determinism and ALiBi prefill cases against the oracle."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SP_B200_PREFILL_PAIR="1")
    r = subprocess.run([sys.executable, "-m", "pytest", "-q", "-x", "-m", "gpu", "-p", "no:cacheprovider",
                        os.path.join(root, "tests", "test_gpu_parity.py"), os.path.join(root, "tests", "test_gpu_independence.py"),
                        "-k", "(prefill and not query and not pair_variant) or paths_do_not or rows_outside"],
                       env=env, capture_output=True, text=True, timeout=1200, cwd=root)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout
