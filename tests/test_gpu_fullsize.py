"""Full-size parity: the workloads at their stated sizes, launched exactly as bench.py
launches them, checked on sampled outputs that the oracle computes one by one (whole sampled
paths / prompts are cut out of the packed arrays and given to the oracle as small problems).
Every row is additionally checked for having been written (NaN poison)."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2404_06910_b200 as sp
from helpers import dev, f32, rel_l2, sub_problem, workspace
from workloads import (CONFIGS, draw_decode_inputs, draw_lengths, draw_logits, draw_prior_weight, draw_qkv,
                       draw_targets)

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", CONFIGS[2:], ids=lambda c: c.name)
def test_full_size_sampled(cfg):
    rng = np.random.default_rng(cfg.seed)
    lay = draw_lengths(cfg)
    B, H, Hkv, D = lay.n_prompts, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
    scale = 1 / math.sqrt(D)
    dl = sp.DeviceLayout.from_host(lay)

    # ---- prefill: all rows on the GPU, sampled prompts/paths in the oracle -------------
    q, k, v = draw_qkv(cfg, lay)
    qd, kd, vd = dev(q), dev(k), dev(v)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full((H, lay.total_tokens), float("nan"), device="cuda")
    ws = workspace(sp.sp_prefill_workspace_bytes(dl, H, D, sp.SP_BF16))
    sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out, lse, ws)
    sp.sp_check_status(ws)
    assert not bool(torch.isnan(out).any()), "prefill left rows unwritten"
    assert not bool(torch.isnan(lse).any())
    prompts = sorted(set([0, B - 1] + list(rng.integers(0, B, size=2))))
    for b in prompts:
        p0, p1 = int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])
        lens = lay.doc_len[p0:p1]
        paths = sorted(set([p0, p1 - 1, p0 + int(lens.argmax()), p0 + int(lens.argmin()),
                            int(rng.integers(p0, p1))]))
        sub, rows, _ = sub_problem(lay, b, paths)
        ref_o, ref_l = oracle.prefill(f32(q[rows]), f32(k[rows]), f32(v[rows]), sub, scale)
        got_o = f32(out[torch.from_numpy(rows).cuda()])
        got_l = lse[:, torch.from_numpy(rows).cuda()].cpu().numpy()
        assert rel_l2(got_o, ref_o) <= 1e-2
        num = np.linalg.norm((got_o - ref_o).reshape(len(rows), -1), axis=1)
        den = np.linalg.norm(ref_o.reshape(len(rows), -1), axis=1) + 1e-6
        assert (num / den).max() <= 5e-2
        np.testing.assert_allclose(got_l, ref_l, atol=2e-2)
    # ---- the same prompts in cached / online mode: only query rows are produced -----------
    out_q = torch.full_like(qd, float("nan"))
    lse_q = torch.full((H, lay.total_tokens), float("nan"), device="cuda")
    sp.sp_superpose_prefill(qd, kd, vd, dl, scale, out_q, lse_q, ws, rows=sp.SP_ROWS_QUERY_ONLY)
    sp.sp_check_status(ws)
    is_q = np.zeros(lay.total_tokens, bool)
    for i in range(lay.n_paths):
        s0 = lay.path_start[i] + lay.doc_len[i]
        is_q[s0:s0 + lay.qry_len[i]] = True
    is_qd = torch.from_numpy(is_q).cuda()
    assert not bool(torch.isnan(out_q[is_qd]).any()), "query rows left unwritten"
    assert bool(torch.isnan(out_q[~is_qd]).all()), "non-query rows must stay untouched"
    # both modes compute the same rows from the same inputs: they must agree to bf16 rounding
    diff = (out_q[is_qd].float() - out[is_qd].float()).abs().max().item()
    assert diff <= 2e-2 * out[is_qd].float().abs().max().item()
    for b in prompts[:2]:
        p0, p1 = int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])
        paths = sorted(set([p0, p1 - 1, int(rng.integers(p0, p1))]))
        sub, rows, _ = sub_problem(lay, b, paths)
        ref_o, ref_l = oracle.prefill(f32(q[rows]), f32(k[rows]), f32(v[rows]), sub, scale)
        sel = is_q[rows]
        got_o = f32(out_q[torch.from_numpy(rows).cuda()])
        got_l = lse_q[:, torch.from_numpy(rows).cuda()].cpu().numpy()
        assert rel_l2(got_o[sel], ref_o[sel]) <= 1e-2
        np.testing.assert_allclose(got_l[:, sel], ref_l[:, sel], atol=2e-2)
    del out, lse, qd, out_q, lse_q

    # ---- decode: all prompts on the GPU, sampled prompts in the oracle -----------------
    scores = rng.standard_normal(lay.n_paths).astype(np.float32)
    kept, _ = oracle.prune_topk(scores, lay.prompt_path_off, cfg.top_k)
    got_kept = torch.empty((B, cfg.top_k), dtype=torch.int32, device="cuda")
    sp.sp_prune_topk(dev(scores), dl.prompt_path_off, cfg.top_k, got_kept)
    np.testing.assert_array_equal(got_kept.cpu().numpy(), kept)          # bit-exact at full size
    steps = cfg.decode_steps
    dq, tk, tv = draw_decode_inputs(cfg, B, steps)
    tkd, tvd = dev(tk), dev(tv)
    wsd = workspace(sp.sp_decode_workspace_bytes(B, H, D))
    for t in (0, steps - 1):
        tl = np.full(B, t + 1, np.int32)
        o = torch.full((B, H, D), float("nan"), dtype=torch.bfloat16, device="cuda")
        sp.sp_pruned_decode(dev(dq[t]), kd, vd, dl, got_kept, cfg.top_k, tkd, tvd, dev(tl), steps, scale, o, None, wsd)
        sp.sp_check_status(wsd)
        assert not bool(torch.isnan(o).any())
        for b in prompts[:3]:
            sub, rows, remap = sub_problem(lay, b, kept[b])
            sub_kept = np.array([[remap[int(i)] for i in kept[b]]], np.int32)
            ref, _ = oracle.pruned_decode(f32(dq[t][b:b + 1]), f32(k[rows]), f32(v[rows]), sub, sub_kept,
                                          f32(tk[b:b + 1]), f32(tv[b:b + 1]), tl[:1], scale)
            assert rel_l2(f32(o[b:b + 1]), ref) <= 1e-2
    del kd, vd, tkd, tvd, q, k, v

    # ---- path scores: all rows on the GPU, sampled paths in the oracle -----------------
    logits = draw_logits(cfg, lay)
    tgt = draw_targets(cfg, lay)
    prior, weight = draw_prior_weight(cfg, lay)
    off = lay.query_row_offsets()
    R = logits.shape[0]
    got_s = torch.full((lay.n_paths,), float("nan"), device="cuda")
    got_r = torch.full((R,), float("nan"), device="cuda")
    sp.sp_path_scores(dev(logits), dev(tgt), dev(off), got_s, dev(prior), dev(weight), got_r,
                      workspace(sp.sp_path_scores_workspace_bytes(R)))
    got_s, got_r = got_s.cpu().numpy(), got_r.cpu().numpy()
    assert not np.isnan(got_s).any() and not np.isnan(got_r).any()
    for i in sorted(set([0, lay.n_paths - 1] + list(rng.integers(0, lay.n_paths, size=6)))):
        a, b_ = int(off[i]), int(off[i + 1])
        ref_s, ref_r = oracle.path_scores(f32(logits[a:b_]), tgt[a:b_], np.array([0, b_ - a], np.int32),
                                          prior[i:i + 1], weight[i:i + 1])
        np.testing.assert_allclose(got_r[a:b_], ref_r, atol=1e-3)
        assert abs(got_s[i] - ref_s[0]) <= 1e-3 * (b_ - a) * weight[i] + 1e-6
