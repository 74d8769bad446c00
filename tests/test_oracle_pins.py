"""Pins of the CPU oracle against things other than itself: closed forms, invariants the
paper states, library routines (torch SDPA / log_softmax), and brute force built from
the DAG reachability definition.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from workloads import build_layout

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ---------------------------------------------------------------- O1 positions
def _read_golden(name):
    rec = {}
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rec[key] = [Fraction(v) for v in vals]
    return rec


def test_positions_worked_example():
    """Eq. 1 + Algorithm 1 on the hand-derived fixture."""
    g = _read_golden("equilibrium_positions_L2_L4.txt")
    pos, S, nxt = oracle.positions(int(g["P"][0]), [int(x) for x in g["L"]], int(g["Q"][0]))
    assert S == pytest.approx(float(g["S"][0]), rel=1e-15)
    np.testing.assert_allclose(pos, [float(x) for x in g["pos"]], rtol=1e-15)
    assert nxt == pytest.approx(float(g["next"][0]), rel=1e-15)


def test_positions_equal_lengths_are_classical():
    """Equal lengths: harmonic mean = L, step 1, i.e. the integer positions of a classical
    prompt p + d_i + q, and identical to left alignment."""
    P, L, Q, N = 5, 7, 3, 4
    pos, S, nxt = oracle.positions(P, [L] * N, Q)
    left, Sl, nl = oracle.positions(P, [L] * N, Q, scheme="left")
    assert S == L and Sl == L and nxt == P + L + Q
    expect = list(range(P)) + N * list(range(P, P + L + Q))
    np.testing.assert_array_equal(pos, expect)
    np.testing.assert_array_equal(left, expect)


def test_positions_harmonic_mean_properties():
    """S <= arithmetic mean; every document's next slot P + L_i * s_i is the same P + S;
    documents start right after the preamble; steps are S / L_i."""
    P, Q = 11, 4
    L = rng.integers(1, 300, size=20)
    pos, S, _ = oracle.positions(P, L, Q)
    assert S == pytest.approx(len(L) / np.sum(1.0 / L), rel=1e-14)
    assert S <= L.mean() + 1e-12
    r = P
    for Li in L:
        d = pos[r:r + Li]
        assert d[0] == P
        if Li > 1:
            np.testing.assert_allclose(np.diff(d), S / Li, rtol=1e-12)
        assert d[-1] + S / Li == pytest.approx(P + S, rel=1e-13)
        np.testing.assert_allclose(pos[r + Li:r + Li + Q], P + S + np.arange(Q), rtol=1e-13)
        r += Li + Q
    # literal reading of Algorithm 3: the query starts on document 1's last position
    lit, _, _ = oracle.positions(P, L, Q, q_mode=1)
    assert lit[P + L[0]] == pytest.approx(pos[P + L[0] - 1])


def test_positions_left_aligned():
    P, Q, L = 4, 2, [3, 9, 5]
    pos, S, _ = oracle.positions(P, L, Q, scheme="left")
    r = P
    for Li in L:
        np.testing.assert_array_equal(pos[r:r + Li], P + np.arange(Li))
        np.testing.assert_array_equal(pos[r + Li:r + Li + Q], P + 9 + np.arange(Q))
        r += Li + Q


# ---------------------------------------------------------------- O2 RoPE
def _rope_complex(x, pos, base, pairing):
    """Textbook RoPE as a complex multiplication (independent formulation)."""
    n, H, D = x.shape
    m = np.arange(D // 2)
    theta = pos.astype(np.float64)[:, None] * base ** (-2.0 * m / D)
    rot = np.exp(1j * theta)[:, None, :]
    x = x.astype(np.float64)
    if pairing == 0:
        z = (x[..., :D // 2] + 1j * x[..., D // 2:]) * rot
        return np.concatenate([z.real, z.imag], axis=-1)
    z = (x[..., 0::2] + 1j * x[..., 1::2]) * rot
    out = np.empty_like(x)
    out[..., 0::2], out[..., 1::2] = z.real, z.imag
    return out


@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_matches_textbook_integer_and_fractional(pairing):
    x = rng.standard_normal((9, 3, 16)).astype(np.float32)
    for pos in (np.arange(9, dtype=np.float32), (np.arange(9) * 4 / 3 + 0.25).astype(np.float32)):
        got = oracle.rope(x, pos, pairing=pairing)
        np.testing.assert_allclose(got, _rope_complex(x, pos, 10000.0, pairing), rtol=0, atol=2e-6)


def test_rope_identity_norm_and_relative_shift():
    x = rng.standard_normal((6, 2, 32)).astype(np.float32)
    np.testing.assert_array_equal(oracle.rope(x, np.zeros(6, np.float32)), x)
    pos = np.array([0.5, 1.75, 3.0, 7.25, 8.0, 11.5], np.float32)
    y = oracle.rope(x, pos)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-6)
    # <R(a)q, R(b)k> depends only on a - b, for real-valued shifts too
    q, k = x[:3], x[3:]
    pa, pb = pos[:3], pos[3:]
    d0 = np.einsum("nhd,nhd->nh", oracle.rope(q, pa), oracle.rope(k, pb))
    c = np.float32(2.625)
    d1 = np.einsum("nhd,nhd->nh", oracle.rope(q, pa + c), oracle.rope(k, pb + c))
    np.testing.assert_allclose(d0, d1, atol=2e-5)
    # partial rotation leaves the tail untouched
    z = oracle.rope(x, pos, rot_dim=16)
    np.testing.assert_array_equal(z[..., 16:], x[..., 16:])
    np.testing.assert_allclose(z[..., :16], oracle.rope(np.ascontiguousarray(x[..., :16]), pos), atol=1e-6)


# ---------------------------------------------------------------- O3 prefill
def _rand_qkv(T, H, Hkv, D, scale=1.0):
    q = (rng.standard_normal((T, H, D)) * scale).astype(np.float32)
    k = (rng.standard_normal((T, Hkv, D)) * scale).astype(np.float32)
    v = rng.standard_normal((T, Hkv, D)).astype(np.float32)
    return q, k, v


def _dense_masked_attention(q, k, v, mask, scale):
    """softmax(scale q k^T + mask) v with a dense boolean [T, T] mask, fp64, per head."""
    T, H, D = q.shape
    g = H // k.shape[1]
    out = np.zeros((T, H, D))
    lse = np.zeros((H, T))
    for h in range(H):
        s = scale * q[:, h].astype(np.float64) @ k[:, h // g].astype(np.float64).T
        s = np.where(mask, s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        den = e.sum(axis=1, keepdims=True)
        out[:, h] = (e / den) @ v[:, h // g].astype(np.float64)
        lse[h] = (m + np.log(den))[:, 0]
    return out, lse


def _dag_mask(lay):
    """Mask from the definition: row of segment v sees segment u iff the segment DAG
    (preamble -> doc_i -> query_i) has a path u -> v; causal inside a segment."""
    seg_of, segs, edges = np.full(lay.total_tokens, -1), [], []
    for b in range(lay.n_prompts):
        pre = len(segs)
        segs.append((lay.pre_start[b], lay.pre_len[b]))
        for i in range(lay.prompt_path_off[b], lay.prompt_path_off[b + 1]):
            d = len(segs)
            segs.append((lay.path_start[i], lay.doc_len[i]))
            segs.append((lay.path_start[i] + lay.doc_len[i], lay.qry_len[i]))
            edges += [(pre, d), (d, d + 1)]
    for s, (lo, n) in enumerate(segs):
        seg_of[lo:lo + n] = s
    S = len(segs)
    adj = np.zeros((S, S), dtype=np.int64)
    for u, v in edges:
        adj[u, v] = 1
    reach, power = np.zeros_like(adj), np.eye(S, dtype=np.int64)
    for _ in range(S):
        power = (power @ adj > 0).astype(np.int64)
        reach |= power
    T = lay.total_tokens
    r, c = np.arange(T)[:, None], np.arange(T)[None, :]
    same = seg_of[r] == seg_of[c]
    return (reach[seg_of[c], seg_of[r]] > 0) | (same & (c <= r))


def test_prefill_brute_force_dag_mask():
    lay = build_layout([5, 0, 3], [[4, 1, 7], [6, 2], [0, 5]], [[3, 3, 3], [2, 2], [4, 1]])
    q, k, v = _rand_qkv(lay.total_tokens, 4, 2, 8)
    out, lse = oracle.prefill(q, k, v, lay, 0.4)
    ref_o, ref_l = _dense_masked_attention(q, k, v, _dag_mask(lay), 0.4)
    np.testing.assert_allclose(out, ref_o, atol=2e-6)
    np.testing.assert_allclose(lse, ref_l, atol=2e-6)
    # allowed-pair counter of the layout agrees with the mask
    assert lay.allowed_pairs() == int(_dag_mask(lay).sum())


def test_prefill_single_path_is_causal_attention():
    """A classical prompt is the linked-list special case: N = 1 must equal ordinary causal
    attention over p + d + q (checked against torch SDPA)."""
    P, L, Q, H, D = 6, 9, 4, 3, 16
    lay = build_layout([P], [[L]], [[Q]])
    q, k, v = _rand_qkv(P + L + Q, H, H, D)
    out, _ = oracle.prefill(q, k, v, lay, 1 / math.sqrt(D))
    tq, tk, tv = (torch.from_numpy(a).double().permute(1, 0, 2)[None] for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2)
    np.testing.assert_allclose(out, ref.numpy(), atol=2e-6)


def test_prefill_paths_are_independent_and_permutable():
    P, Ls, Q, H, D = 4, [5, 8, 3], 2, 2, 8
    lay = build_layout([P], [Ls], [[Q] * 3])
    q, k, v = _rand_qkv(lay.total_tokens, H, H, D)
    out, lse = oracle.prefill(q, k, v, lay, 0.3)

    def seg(i):
        return slice(lay.path_start[i], lay.path_start[i] + Ls[i] + Q)

    # perturb document 1: preamble rows and paths 0, 2 stay bit-identical
    k2, v2 = k.copy(), v.copy()
    k2[seg(1)] += 1.0
    v2[seg(1)] -= 2.0
    out2, lse2 = oracle.prefill(q, k2, v2, lay, 0.3)
    for s in (slice(0, P), seg(0), seg(2)):
        np.testing.assert_array_equal(out[s], out2[s])
        np.testing.assert_array_equal(lse[:, s], lse2[:, s])
    assert not np.allclose(out[seg(1)], out2[seg(1)])
    # permute the documents: path outputs permute with them
    perm = [2, 0, 1]
    lay_p = build_layout([P], [[Ls[i] for i in perm]], [[Q] * 3])
    gather = np.concatenate([np.arange(P)] + [np.arange(seg(i).start, seg(i).stop) for i in perm])
    out_p, lse_p = oracle.prefill(q[gather], k[gather], v[gather], lay_p, 0.3)
    np.testing.assert_array_equal(out_p, out[gather])
    np.testing.assert_array_equal(lse_p, lse[:, gather])


def test_prefill_degenerate_rows():
    lay = build_layout([3], [[2, 4]], [[2, 2]])
    q, k, v = _rand_qkv(lay.total_tokens, 2, 1, 8)
    # all value rows equal -> every output equals that row
    v[:] = v[0]
    out, lse = oracle.prefill(q, k, v, lay, 0.7)
    np.testing.assert_allclose(out, np.broadcast_to(np.repeat(v[:1], 2, axis=1), out.shape), atol=1e-6)
    # a row with a single key (first preamble row): LSE is its score
    s00 = 0.7 * float(q[0, 1].astype(np.float64) @ k[0, 0].astype(np.float64))
    assert lse[1, 0] == pytest.approx(s00, abs=1e-6)
    # row subset = same rows of the full result
    rows = np.array([0, 4, 7, lay.total_tokens - 1])
    sub, lsub = oracle.prefill(q, k, v, lay, 0.7, rows=rows)
    np.testing.assert_array_equal(sub[rows], out[rows])
    np.testing.assert_array_equal(lsub[:, rows], lse[:, rows])


# ---------------------------------------------------------------- O4 path scores
# ---------------------------------------------------------------------- ALiBi bias (prefill)
def _alibi_slopes(H):
    return np.array([2.0 ** (-8.0 * (h + 1) / H) for h in range(H)], np.float32)


def test_prefill_alibi_single_path_is_textbook_alibi():
    """One path, integer positions 0..n-1: causal attention with the additive bias
    -slope_h * (i - j), checked against torch SDPA given that bias as an explicit mask."""
    P, L, Q, H, D = 5, 8, 3, 4, 16
    n = P + L + Q
    lay = build_layout([P], [[L]], [[Q]])
    q, k, v = _rand_qkv(n, H, H, D)
    slopes = _alibi_slopes(H)
    pos = np.arange(n, dtype=np.float32)
    out, _ = oracle.prefill(q, k, v, lay, 1 / math.sqrt(D), pos=pos, slopes=slopes)
    i, j = torch.arange(n)[:, None], torch.arange(n)[None, :]
    bias = -torch.from_numpy(slopes).double()[:, None, None] * (i - j).double()
    bias = bias.masked_fill(j > i, float("-inf"))
    tq, tk, tv = (torch.from_numpy(a).double().permute(1, 0, 2)[None] for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=bias[None])[0].permute(1, 0, 2)
    np.testing.assert_allclose(out, ref.numpy(), atol=2e-6)


def test_prefill_alibi_fork_join_dense_and_invariances():
    lay = build_layout([5, 0, 3], [[4, 1, 7], [6, 2], [0, 5]], [[3, 3, 3], [2, 2], [4, 4]])
    T, H = lay.total_tokens, 4
    q, k, v = _rand_qkv(T, H, 2, 8)
    slopes = _alibi_slopes(H)
    # fractional positions, as the equilibrium assignment produces
    pos = np.concatenate([oracle.positions(int(lay.pre_len[b]), lay.doc_len[lay.prompt_path_off[b]:lay.prompt_path_off[b + 1]],
                                           int(lay.qry_len[lay.prompt_path_off[b]]))[0] for b in range(3)]).astype(np.float32)
    assert pos.shape == (T,) and np.any(pos != np.round(pos))
    out, lse = oracle.prefill(q, k, v, lay, 0.4, pos=pos, slopes=slopes)
    mask = _dag_mask(lay)
    dist = np.abs(pos.astype(np.float64)[:, None] - pos.astype(np.float64)[None, :])
    for h in range(H):              # dense reference, one head at a time: scores + bias matrix
        sc = 0.4 * q[:, h].astype(np.float64) @ k[:, h // 2].astype(np.float64).T - float(slopes[h]) * dist
        sc = np.where(mask, sc, -np.inf)
        m = sc.max(axis=1, keepdims=True)
        e = np.exp(sc - m)
        np.testing.assert_allclose(out[:, h], (e / e.sum(1, keepdims=True)) @ v[:, h // 2].astype(np.float64), atol=2e-6)
        np.testing.assert_allclose(lse[h], (m + np.log(e.sum(1, keepdims=True)))[:, 0], atol=2e-6)
    plain, plain_l = oracle.prefill(q, k, v, lay, 0.4)
    zero, zero_l = oracle.prefill(q, k, v, lay, 0.4, pos=pos, slopes=np.zeros(H, np.float32))
    np.testing.assert_array_equal(zero, plain)                      # zero slopes: no bias
    same, _ = oracle.prefill(q, k, v, lay, 0.4, pos=np.full(T, 3.25, np.float32), slopes=slopes)
    np.testing.assert_allclose(same, plain, atol=1e-6)              # all tokens at one position: no bias
    shifted, _ = oracle.prefill(q, k, v, lay, 0.4, pos=pos + 64.0, slopes=slopes)
    np.testing.assert_allclose(shifted, out, atol=1e-5)             # only distances matter
    assert np.abs(out - plain).max() > 1e-3                         # and the bias does something


def test_prefill_alibi_steep_slope_attends_to_itself():
    """slope -> infinity: every key but the row's own (distance 0) is suppressed, so out = v."""
    lay = build_layout([3], [[4, 2]], [[2, 2]])
    T = lay.total_tokens
    q, k, v = _rand_qkv(T, 2, 2, 8)
    pos = oracle.positions(3, [4, 2], 2)[0].astype(np.float32)
    out, _ = oracle.prefill(q, k, v, lay, 0.3, pos=pos, slopes=np.full(2, 1e4, np.float32))
    np.testing.assert_allclose(out, v, atol=1e-6)


def test_decode_alibi_dense_and_matches_prefill_row():
    lay, H, Hkv, D, q, kc, vc, tk, tv = _decode_setup()
    slopes = _alibi_slopes(H)
    cpos = (np.arange(lay.total_tokens) * 0.75 + 1.0).astype(np.float32)
    tpos = np.array([[40.0, 41.0, 42.0], [30.5, 31.5, 32.5]], np.float32)
    qpos = np.array([42.0, 30.5], np.float32)
    kept = np.array([[2, 0], [4, -1]], np.int32)
    tl = np.array([3, 1], np.int32)
    out, lse = oracle.pruned_decode(q, kc, vc, lay, kept, tk, tv, tl, 0.35, q_pos=qpos, cache_pos=cpos, tail_pos=tpos, slopes=slopes)
    for b in range(2):
        rows = list(range(lay.pre_start[b], lay.pre_start[b] + lay.pre_len[b]))
        for i in kept[b]:
            if i >= 0:
                rows += list(range(lay.path_start[i], lay.path_start[i] + lay.doc_len[i] + lay.qry_len[i]))
        kpos = np.concatenate([cpos[rows], tpos[b, :tl[b]]]).astype(np.float64)
        for h in range(H):
            keys = np.concatenate([kc[rows, h // 2], tk[b, :tl[b], h // 2]]).astype(np.float64)
            vals = np.concatenate([vc[rows, h // 2], tv[b, :tl[b], h // 2]]).astype(np.float64)
            sc = 0.35 * keys @ q[b, h].astype(np.float64) - float(slopes[h]) * np.abs(float(qpos[b]) - kpos)
            e = np.exp(sc - sc.max())
            np.testing.assert_allclose(out[b, h], (e / e.sum()) @ vals, atol=2e-6)
            assert lse[b, h] == pytest.approx(sc.max() + math.log(e.sum()), abs=2e-6)
    plain, _ = oracle.pruned_decode(q, kc, vc, lay, kept, tk, tv, tl, 0.35)
    zero, _ = oracle.pruned_decode(q, kc, vc, lay, kept, tk, tv, tl, 0.35, q_pos=qpos, cache_pos=cpos, tail_pos=tpos,
                                   slopes=np.zeros(H, np.float32))
    np.testing.assert_array_equal(zero, plain)
    # k = 1: the decoded token is the last row of an ALiBi prefill over p + d_i + q_i + [itself]
    i = 1
    P, L, Q = int(lay.pre_len[0]), int(lay.doc_len[i]), int(lay.qry_len[i])
    o1, _ = oracle.pruned_decode(q, kc, vc, lay, np.array([[i], [-1]], np.int32), tk, tv, np.array([1, 1], np.int32), 0.5,
                                 q_pos=qpos, cache_pos=cpos, tail_pos=tpos, slopes=slopes)
    ext = build_layout([P], [[L]], [[Q + 1]])
    rows = list(range(P)) + list(range(lay.path_start[i], lay.path_start[i] + L + Q))
    q_ext = np.zeros((ext.total_tokens, H, D), np.float32)
    q_ext[-1] = q[0]
    pos_ext = np.concatenate([cpos[rows], [qpos[0]]]).astype(np.float32)
    tpos1 = tpos.copy(); tpos1[0, 0] = qpos[0]
    o1, _ = oracle.pruned_decode(q, kc, vc, lay, np.array([[i], [-1]], np.int32), tk, tv, np.array([1, 1], np.int32), 0.5,
                                 q_pos=qpos, cache_pos=cpos, tail_pos=tpos1, slopes=slopes)
    o_ext, _ = oracle.prefill(q_ext, np.concatenate([kc[rows], tk[0, :1]]), np.concatenate([vc[rows], tv[0, :1]]), ext, 0.5,
                              pos=pos_ext, slopes=slopes)
    np.testing.assert_allclose(o1[0], o_ext[-1], atol=1e-6)


def test_path_scores_match_log_softmax_gather():
    V, qlens = 97, [3, 5, 1, 4]
    off = np.concatenate([[0], np.cumsum(qlens)]).astype(np.int32)
    logits = (rng.standard_normal((off[-1], V)) * 3).astype(np.float32)
    tgt = rng.integers(0, V, size=off[-1]).astype(np.int32)
    tgt[off[1:] - 1] = -1
    prior = rng.standard_normal(4).astype(np.float32)
    weight = (1.0 / np.array(qlens)).astype(np.float32)
    scores, row_logp = oracle.path_scores(logits, tgt, off, prior, weight)
    lsm = torch.log_softmax(torch.from_numpy(logits).double(), dim=-1).numpy()
    ref_rows = np.where(tgt >= 0, lsm[np.arange(len(tgt)), np.maximum(tgt, 0)], 0.0)
    np.testing.assert_allclose(row_logp, ref_rows, atol=1e-6)
    ref = np.array([weight[i] * ref_rows[off[i]:off[i + 1]].sum() + prior[i] for i in range(4)])
    np.testing.assert_allclose(scores, ref, atol=1e-6)
    # defaults: weight 1, prior 0
    s2, _ = oracle.path_scores(logits, tgt, off)
    np.testing.assert_allclose(s2, [ref_rows[off[i]:off[i + 1]].sum() for i in range(4)], atol=1e-5)


def test_path_scores_closed_forms():
    V = 64
    off = np.array([0, 2, 4], np.int32)
    logits = np.full((4, V), 1.5, np.float32)
    tgt = np.array([3, 9, 0, -1], np.int32)
    scores, rows = oracle.path_scores(logits, tgt, off)
    np.testing.assert_allclose(rows, [-math.log(V)] * 3 + [0.0], rtol=1e-7)
    np.testing.assert_allclose(scores, [-2 * math.log(V), -math.log(V)], rtol=1e-7)
    # a per-row constant changes nothing; a dominant target logit gives ~0
    lg = (rng.standard_normal((4, V)) * 2).astype(np.float64)
    a, _ = oracle.path_scores(lg, tgt, off)
    b, _ = oracle.path_scores(lg + np.array([[5.0], [-3.0], [100.0], [1.0]]), tgt, off)
    np.testing.assert_allclose(a, b, atol=2e-5)
    lg[0, 3] = 80.0
    _, r = oracle.path_scores(lg, tgt, off)
    assert abs(r[0]) < 1e-6


# ---------------------------------------------------------------- O5 top-k
def test_topk_matches_full_sort_and_shift_invariance():
    ppo = np.array([0, 7, 7, 12], np.int32)
    s = rng.standard_normal(12).astype(np.float32)
    idx, post = oracle.prune_topk(s, ppo, 3)
    for b in range(3):
        lo, hi = ppo[b], ppo[b + 1]
        order = lo + np.argsort(-s[lo:hi], kind="stable")
        want = list(order[:3]) + [-1] * (3 - min(3, hi - lo))
        assert list(idx[b]) == want
        if hi > lo:
            p = np.exp(s[lo:hi].astype(np.float64) - s[lo:hi].max())
            p /= p.sum()
            np.testing.assert_allclose(post[b, :min(3, hi - lo)], p[order[:3] - lo], rtol=1e-6)
    # the constant C of Eq. 2 is irrelevant: shifting all scores changes nothing
    idx2, post2 = oracle.prune_topk(s + np.float32(4.0), ppo, 3)
    np.testing.assert_array_equal(idx, idx2)
    np.testing.assert_allclose(post, post2, atol=1e-6)
    # k = N: posterior sums to one
    _, pall = oracle.prune_topk(s, ppo, 7)
    assert pall[0].sum() == pytest.approx(1.0, abs=1e-6)


def test_topk_ties_nan_and_short_prompts():
    ppo = np.array([0, 5], np.int32)
    s = np.array([1.0, 2.0, 2.0, np.nan, 2.0], np.float32)
    idx, post = oracle.prune_topk(s, ppo, 5)
    assert list(idx[0]) == [1, 2, 4, 0, 3]          # ties by index, NaN last
    assert post[0, 4] == 0.0 and post[0].sum() == pytest.approx(1.0, abs=1e-6)
    idx, _ = oracle.prune_topk(s, ppo, 8)
    assert list(idx[0][5:]) == [-1, -1, -1]
    with pytest.raises(ValueError):
        oracle.prune_topk(s, ppo, 0)


def test_topk_posterior_when_no_score_is_finite():
    """Cases the paper is silent on, expected values written out by hand from the reading taken
    (NaN ranks below every number and counts as -inf; equal scores keep the lower id first; the
    posterior of a prompt with no score above -inf is zero everywhere, not NaN)."""
    ninf, nan = -np.inf, np.nan
    idx, post = oracle.prune_topk(np.array([ninf, nan, ninf], np.float32), np.array([0, 3], np.int32), 3)
    assert idx.tolist() == [[0, 2, 1]] and post.tolist() == [[0.0, 0.0, 0.0]]
    idx, post = oracle.prune_topk(np.array([nan, nan], np.float32), np.array([0, 2], np.int32), 1)
    assert idx.tolist() == [[0]] and post.tolist() == [[0.0]]
    # one finite score among -inf and NaN takes the whole posterior
    idx, post = oracle.prune_topk(np.array([ninf, 3.0, ninf, nan], np.float32), np.array([0, 4], np.int32), 2)
    assert idx.tolist() == [[1, 0]] and post.tolist() == [[1.0, 0.0]]
    # two prompts side by side: the degenerate one does not disturb its neighbour
    idx, post = oracle.prune_topk(np.array([ninf, ninf, 0.0, 0.0], np.float32), np.array([0, 2, 4], np.int32), 2)
    assert idx.tolist() == [[0, 1], [2, 3]] and post.tolist() == [[0.0, 0.0], [0.5, 0.5]]


def test_positions_with_empty_documents_and_empty_preamble():
    """Eq. 1 with a zero-length document (it has no term in the harmonic mean and no rows of its
    own; its query copy still starts at P + S like every other) and with no preamble
    (max of the empty set + 1 = 0).  Expected values derived by hand:
    L = {0, 2, 4}: S = 2 / (1/2 + 1/4) = 8/3, steps 4/3 and 2/3, queries at 2 + 8/3 = 14/3."""
    pos, S, nxt = oracle.positions(2, [0, 2, 4], 1)
    want = [0, 1,                      # preamble
            14 / 3,                    # empty document: only its query copy
            2, 10 / 3, 14 / 3,         # document of 2 (step 4/3), query
            2, 8 / 3, 10 / 3, 4, 14 / 3]
    np.testing.assert_allclose(pos, want, rtol=0, atol=1e-12)
    assert S == pytest.approx(8 / 3, abs=1e-12) and nxt == pytest.approx(17 / 3, abs=1e-12)
    pos, S, nxt = oracle.positions(0, [2, 4], 1)
    np.testing.assert_allclose(pos, [0, 4 / 3, 8 / 3, 0, 2 / 3, 4 / 3, 2, 8 / 3], rtol=0, atol=1e-12)
    assert nxt == pytest.approx(11 / 3, abs=1e-12)
    # every document empty: S = 0, the queries follow the preamble directly
    pos, S, nxt = oracle.positions(3, [0, 0], 2)
    assert pos.tolist() == [0, 1, 2, 3, 4, 3, 4] and S == 0.0 and nxt == 5.0


# ---------------------------------------------------------------- O6 decode
def _decode_setup():
    lay = build_layout([3, 2], [[4, 2, 5], [3, 6]], [[2, 2, 2], [3, 3]])
    H, Hkv, D = 4, 2, 8
    _, kc, vc = _rand_qkv(lay.total_tokens, H, Hkv, D)
    q = rng.standard_normal((2, H, D)).astype(np.float32)
    tk = rng.standard_normal((2, 3, Hkv, D)).astype(np.float32)
    tv = rng.standard_normal((2, 3, Hkv, D)).astype(np.float32)
    return lay, H, Hkv, D, q, kc, vc, tk, tv


def _dense_decode(qb, keys, vals, scale):
    s = scale * keys.astype(np.float64) @ qb.astype(np.float64)
    m = s.max()
    p = np.exp(s - m)
    return (p / p.sum()) @ vals.astype(np.float64), m + math.log(p.sum())


def test_decode_is_dense_softmax_over_the_kept_union():
    lay, H, Hkv, D, q, kc, vc, tk, tv = _decode_setup()
    kept = np.array([[2, 0], [4, -1]], np.int32)
    tl = np.array([3, 1], np.int32)
    out, lse = oracle.pruned_decode(q, kc, vc, lay, kept, tk, tv, tl, 0.35)
    for b in range(2):
        rows = list(range(lay.pre_start[b], lay.pre_start[b] + lay.pre_len[b]))
        for i in kept[b]:
            if i >= 0:
                rows += list(range(lay.path_start[i], lay.path_start[i] + lay.doc_len[i] + lay.qry_len[i]))
        for h in range(H):
            keys = np.concatenate([kc[rows, h // 2], tk[b, :tl[b], h // 2]])
            vals = np.concatenate([vc[rows, h // 2], tv[b, :tl[b], h // 2]])
            o, l = _dense_decode(q[b, h], keys, vals, 0.35)
            np.testing.assert_allclose(out[b, h], o, atol=2e-6)
            assert lse[b, h] == pytest.approx(l, abs=2e-6)
    # order of the kept paths does not matter (caches are simply concatenated)
    out2, _ = oracle.pruned_decode(q, kc, vc, lay, kept[:, ::-1].copy(), tk, tv, tl, 0.35)
    np.testing.assert_allclose(out, out2, atol=1e-6)


def test_decode_keep_one_equals_classical_prefill_row():
    """k = 1: decoding one token over p + d_i + q_i + [itself] is the last row of causal
    attention on that sequence, i.e. of the prefill on a layout whose path is one row longer."""
    lay, H, Hkv, D, q, kc, vc, tk, tv = _decode_setup()
    i = 1
    kept = np.array([[i], [-1]], np.int32)
    out, lse = oracle.pruned_decode(q, kc, vc, lay, kept, tk, tv, np.array([1, 1], np.int32), 0.5)
    P, L, Q = int(lay.pre_len[0]), int(lay.doc_len[i]), int(lay.qry_len[i])
    ext = build_layout([P], [[L]], [[Q + 1]])
    rows = list(range(P)) + list(range(lay.path_start[i], lay.path_start[i] + L + Q))
    k_ext = np.concatenate([kc[rows], tk[0, :1]])
    v_ext = np.concatenate([vc[rows], tv[0, :1]])
    q_ext = np.zeros((ext.total_tokens, H, D), np.float32)
    q_ext[-1] = q[0]
    o_ext, l_ext = oracle.prefill(q_ext, k_ext, v_ext, ext, 0.5)
    np.testing.assert_allclose(out[0], o_ext[-1], atol=1e-6)
    np.testing.assert_allclose(lse[0], l_ext[:, -1], atol=1e-6)


def test_decode_split_merge_identity():
    """Attention over A u B equals the LSE-weighted combination of attention over A and B
    (the identity a split-KV kernel relies on)."""
    lay, H, Hkv, D, q, kc, vc, tk, tv = _decode_setup()
    none = np.array([[-1], [-1]], np.int32)
    tl0 = np.zeros(2, np.int32)
    oa, la = oracle.pruned_decode(q, kc, vc, lay, np.array([[0], [3]], np.int32), tk, tv, tl0, 0.4)
    ob, lb = oracle.pruned_decode(q, kc, vc, lay, np.array([[1], [4]], np.int32), tk, tv, tl0, 0.4)
    op, lp = oracle.pruned_decode(q, kc, vc, lay, none, tk, tv, tl0, 0.4)        # preamble only
    oab, lab = oracle.pruned_decode(q, kc, vc, lay, np.array([[0, 1], [3, 4]], np.int32), tk, tv, tl0, 0.4)
    # A = pre + path a, B = pre + path b; A u B counted once => subtract the preamble part
    wa, wb, wp = np.exp(la.astype(np.float64)), np.exp(lb.astype(np.float64)), np.exp(lp.astype(np.float64))
    den = wa + wb - wp
    merged = (wa[..., None] * oa + wb[..., None] * ob - wp[..., None] * op) / den[..., None]
    np.testing.assert_allclose(oab, merged, atol=5e-6)
    np.testing.assert_allclose(lab, np.log(den), atol=5e-6)
