#!/usr/bin/env python
"""Benchmark of the superposition-prompting hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic prompts:
  RoPE(Q), RoPE(K) -> fork-join prefill -> path scores -> top-k -> decode_steps x
  (pruned decode with the rotation of the new q and k rows folded in).
`value` is the prefill's useful TFLOP/s counted over the WHOLE step time (inputs resident
in HBM); `roofline` describes the prefill kernel (the one the metric is named after),
`roofline_decode` the decode kernel, `kernels` every stage; times are medians over the timed
steps.  After the default workload (cfg2) the two other large single-GPU workloads (cfg3,
cfg4) are measured in the same process and reported under `workloads`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

N > 1: started as a plain script, bench.py starts N ranks of itself (torch.distributed.run on
127.0.0.1); started by torchrun it uses the ranks it is given.  Every rank runs its own batch
(independent prompts, no data-path collective); the time is the max over ranks and `value`
the aggregate ("weak" scaling).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import (draw_decode_inputs, draw_lengths, draw_logits, draw_prior_weight,  # noqa: E402
                       draw_qkv, draw_targets, get_config)

METRIC = "superposition prefill useful TFLOP/s over the whole hot-path step"
UNIT = "TFLOP/s"
PREFILL_LAUNCHES = 2           # kernels sp_superpose_prefill launches per call (tile plan + attention)
# dram__bytes_read.sum + dram__bytes_write.sum from the ncu captures summarised under profiles/,
# per unit of work (the captures run a smaller case; traffic grows in proportion to the units).
# Each entry names the hash of the kernel sources it was taken from: after a kernel change the
# figure is withheld (null in the JSON line) until the capture is repeated.
NCU_TRAFFIC = {
    ("prefill", "cfg2_batched_serving"): {"bytes_per_unit": 2602638512.0 / 74087, "unit": "token",
                                          "capture": "the cfg2 shape with 20 prompts (74 087 tokens), one launch",
                                          "source_hash": "84bbcbe117cf"},
    ("decode", "cfg3_llama2_7b"): {"bytes_per_unit": 109603584.0 / 6548, "unit": "gathered key",
                                   "capture": "cfg3 (8 prompts, 6 548 keys per launch), two launches averaged",
                                   "source_hash": "18396a4613a6"},
}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def rank_seed(cfg, rank: int) -> int:
    """Every rank draws its own prompts (data parallel over independent prompts)."""
    return cfg.seed + 1000 * rank


def max_over_ranks(values, dist=None, device="cpu"):
    """Per-rank timings -> the slowest rank's (the job's) timings, on every rank."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def aggregate_value(flop_per_rank: float, ms: float, world: int) -> float:
    """Whole-job useful TFLOP/s: every rank does flop_per_rank in the (max-over-ranks) time."""
    return world * flop_per_rank / (ms * 1e-3) / 1e12


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


def positions_all(lay, fn):
    pos = np.zeros(lay.total_tokens, dtype=np.float32)
    nxt = np.zeros(lay.n_prompts, dtype=np.float64)
    for b in range(lay.n_prompts):
        p0, p1 = int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])
        q = int(lay.qry_len[p0]) if p1 > p0 else 0
        p, _, n = fn(int(lay.pre_len[b]), lay.doc_len[p0:p1], q)
        lo, hi = lay.prompt_row_range(b)
        pos[lo:hi] = p
        nxt[b] = n
    return pos, nxt


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True).start()
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        for ln in list(self.lines):
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------
class HotPath:
    """Device buffers and the launch sequence of one step, through the C-ABI binding."""

    def __init__(self, cfg, seed, sp, device, n_prompts=None, decode_steps=None):
        self.cfg, self.sp = cfg, sp
        t0 = time.time()
        self.lay = lay = draw_lengths(cfg, seed=seed, n_prompts=n_prompts)
        B, H, Hkv, D = lay.n_prompts, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim
        self.B, self.H, self.Hkv, self.D = B, H, Hkv, D
        self.tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
        self.steps_dec = cfg.decode_steps if decode_steps is None else decode_steps
        # host inputs (pinned: they are also the source of the end-to-end copies)
        self.h_q, self.h_k, self.h_v = draw_qkv(cfg, lay, seed=seed, pin=True)
        self.h_logits = draw_logits(cfg, lay, seed=seed, pin=True)
        self.h_tgt = torch.from_numpy(draw_targets(cfg, lay, seed=seed)).pin_memory()
        prior, weight = draw_prior_weight(cfg, lay, seed=seed)
        self.h_dq, self.h_tk, self.h_tv = draw_decode_inputs(cfg, B, self.steps_dec, seed=seed, pin=True)
        scheme = sp.SP_POS_EQUILIBRIUM if cfg.positions == "equilibrium" else sp.SP_POS_LEFT_ALIGNED
        pos, nxt = positions_all(lay, lambda P, L, Q: sp.sp_positions(P, L, Q, scheme=scheme))
        self.h_pos = torch.from_numpy(pos).pin_memory()
        tpos = (nxt[None, :] + np.arange(self.steps_dec)[:, None]).astype(np.float32)   # [steps, B]
        self.gen_s = time.time() - t0

        dv = lambda t: t.to(device, non_blocking=True)
        self.dl = sp.DeviceLayout.from_host(lay, device)
        self.q, self.k, self.v = dv(self.h_q), dv(self.h_k), dv(self.h_v)
        self.out = torch.empty_like(self.q)
        self.logits, self.tgt, self.pos = dv(self.h_logits), dv(self.h_tgt), dv(self.h_pos)
        self.row_off = torch.from_numpy(lay.query_row_offsets()).to(device)
        self.prior, self.weight = torch.from_numpy(prior).to(device), torch.from_numpy(weight).to(device)
        self.scores = torch.empty(lay.n_paths, device=device)
        self.kept = torch.empty((B, cfg.top_k), dtype=torch.int32, device=device)
        self.post = torch.empty((B, cfg.top_k), device=device)
        self.dq, self.tk, self.tv = dv(self.h_dq), dv(self.h_tk), dv(self.h_tv)
        self.tpos = torch.from_numpy(tpos).to(device)
        self.tail_len = (torch.arange(1, self.steps_dec + 1, dtype=torch.int32)[:, None]
                         .expand(self.steps_dec, B).contiguous().to(device))
        self.dec_out = torch.empty((self.steps_dec, B, H, D), dtype=self.tdt, device=device)
        ws = lambda n: torch.zeros(max(int(n), 256), dtype=torch.uint8, device=device)
        self.ws_pre = ws(sp.sp_prefill_workspace_bytes(self.dl, H, D, sp.dtype_code(self.q)))
        self.ws_sc = ws(sp.sp_path_scores_workspace_bytes(self.logits.shape[0]))
        self.ws_dec = ws(sp.sp_decode_workspace_bytes(B, H, D))
        self.scale = 1.0 / math.sqrt(D)
        self.h_dec_out = torch.empty(self.dec_out.shape, dtype=self.tdt).pin_memory()
        self.h_kept = torch.empty(self.kept.shape, dtype=torch.int32).pin_memory()
        torch.cuda.synchronize()

        # algorithmic work per step
        eb = cfg.elt_bytes
        T = lay.total_tokens
        self.pairs = lay.allowed_pairs()
        self.flop_prefill = 4.0 * D * H * self.pairs
        self.bytes_prefill = float(T) * (2 * H + 2 * Hkv) * D * eb
        self.bytes_rope = 2.0 * T * (H + Hkv) * D * eb
        # query-only mode: K, V of every token read once, Q read and O written for query rows only
        rq = float(lay.qry_len.sum())
        pairs_q = 0
        for b in range(B):
            for i in range(int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])):
                L, Q = int(lay.doc_len[i]), int(lay.qry_len[i])
                pairs_q += Q * (int(lay.pre_len[b]) + L) + Q * (Q + 1) // 2
        self.flop_query_only = 4.0 * D * H * pairs_q
        self.bytes_query_only = (2.0 * rq * H + 2.0 * T * Hkv) * D * eb
        scored = int((self.h_tgt >= 0).sum())
        self.bytes_scores = float(scored) * cfg.vocab * eb
        self.bytes_decode = None        # needs the kept set: filled after the first step
        # kernels launched per step (ours): rope x2, prefill, row_logp + path_sum, top-k,
        # per decode step rope (q and the new key in one launch) + decode
        self.fused_rope = (H // Hkv) in (1, 2, 4)
        self.launches = 2 + PREFILL_LAUNCHES + 2 + 1 + self.steps_dec * (1 if self.fused_rope else 2)
        self.decode_graph = None
        self.kv_sets = [(self.k, self.v)]

    def decode_bytes(self):
        kept = self.kept.cpu().numpy()
        lay = self.lay
        tot = 0
        for b in range(self.B):
            n = int(lay.pre_len[b]) + sum(int(lay.doc_len[i] + lay.qry_len[i]) for i in kept[b] if i >= 0)
            tot += sum(n + t + 1 for t in range(self.steps_dec))
        return float(tot) * 2 * self.Hkv * self.D * self.cfg.elt_bytes

    def h2d(self):
        nb = 0
        for d, h in ((self.q, self.h_q), (self.k, self.h_k), (self.v, self.h_v), (self.logits, self.h_logits),
                     (self.tgt, self.h_tgt), (self.pos, self.h_pos), (self.dq, self.h_dq), (self.tk, self.h_tk),
                     (self.tv, self.h_tv)):
            d.copy_(h, non_blocking=True)
            nb += h.numel() * h.element_size()
        return nb

    def d2h(self):
        self.h_dec_out.copy_(self.dec_out, non_blocking=True)
        self.h_kept.copy_(self.kept, non_blocking=True)
        return self.h_dec_out.numel() * self.h_dec_out.element_size() + self.h_kept.numel() * 4

    def step(self, ev=None):
        """Launches one pass.  ev (optional): list that receives CUDA events at stage edges."""
        sp, cfg = self.sp, self.cfg
        H, Hkv, D, B = self.H, self.Hkv, self.D, self.B
        mark = (lambda: None) if ev is None else (lambda: (ev.append(torch.cuda.Event(enable_timing=True)), ev[-1].record()))
        mark()
        sp.sp_rope_apply(self.q, self.pos, H, D, base=cfg.rope_base)       # two launches stream slightly better
        sp.sp_rope_apply(self.k, self.pos, Hkv, D, base=cfg.rope_base)     # than one over both tensors
        mark()
        sp.sp_superpose_prefill(self.q, self.k, self.v, self.dl, self.scale, self.out, None, self.ws_pre)
        mark()
        sp.sp_path_scores(self.logits, self.tgt, self.row_off, self.scores, self.prior, self.weight, None, self.ws_sc)
        mark()
        sp.sp_prune_topk(self.scores, self.dl.prompt_path_off, cfg.top_k, self.kept, self.post)
        mark()
        if self.decode_graph is not None:
            self.decode_graph.replay()
        else:
            self.decode_loop()
        mark()

    def make_kv_sets(self, l2_bytes):
        """A decode step reads only the kept paths' KV (about 100 MB on the smaller workloads),
        which would stay in the 126 MB L2 if every step re-read the same buffers.  A real
        model has one cache per layer, so consecutive decode launches read different memory:
        rotate over enough copies of the cache to exceed twice the L2."""
        keys = self.lay.max_pre_len + self.cfg.top_k * float(np.mean(self.lay.doc_len + self.lay.qry_len))
        per_step = max(1.0, self.B * keys * 2 * self.Hkv * self.D * self.cfg.elt_bytes)
        n = int(min(8, max(1, math.ceil(2.0 * l2_bytes / per_step))))
        self.kv_sets = [(self.k, self.v)] + [(self.k.clone(), self.v.clone()) for _ in range(n - 1)]

    def decode_loop(self, with_rope=True):
        sp, cfg = self.sp, self.cfg
        H, Hkv, D, B = self.H, self.Hkv, self.D, self.B
        ld = self.steps_dec * Hkv * D
        for t in range(self.steps_dec):
            kc, vc = self.kv_sets[t % len(self.kv_sets)]
            if with_rope and self.fused_rope:
                # one launch per token: the new query and key rows are rotated inside the decode kernel
                sp.sp_pruned_decode_rope(self.dq[t], kc, vc, self.dl, self.kept, cfg.top_k, self.tk, self.tv,
                                         self.tail_len[t], self.steps_dec, self.tpos[t], self.scale, self.dec_out[t],
                                         None, base=cfg.rope_base)
                continue
            if with_rope:
                sp.sp_rope_apply_pair(self.dq[t], H, self.tk[:, t], Hkv, self.tpos[t], D, n_tokens=B, ld_k=ld,
                                      base=cfg.rope_base)
            sp.sp_pruned_decode(self.dq[t], kc, vc, self.dl, self.kept, cfg.top_k, self.tk, self.tv,
                                self.tail_len[t], self.steps_dec, self.scale, self.dec_out[t], None, self.ws_dec)

    def capture_decode_graph(self):
        """The decode loop is launch-bound (3 small launches per token): replay it from a CUDA
        graph.  kept_idx is read on the device, so the captured graph stays valid when the
        kept set changes."""
        self.kept.fill_(-1)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.decode_loop()                      # warm-up outside capture (first-call set-up)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            self.decode_loop()
        self.decode_graph = g


STAGES = ("rope", "prefill", "path_scores", "topk", "decode")
PREFILL_SOURCES = ("prefill_tc.cu", "prefill_plan.cuh", "tc_ptx.cuh")
DECODE_SOURCES = ("decode.cu",)


def source_hash(names) -> str:
    """Short hash of kernel source files: a captured ncu figure is only quoted while the kernel
    it was taken from is unchanged."""
    import hashlib
    h = hashlib.sha256()
    for n in names:
        with open(os.path.join(ROOT, "paper_2404_06910_b200", "csrc", n), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def captured_traffic(kernel: str, workload: str, sources, units: float):
    """dram bytes per launch from the ncu capture summarised under profiles/, scaled to this
    launch by the units processed (tokens for the prefill, gathered keys for the decode);
    None when there is no capture for this workload or the kernel changed since."""
    ent = NCU_TRAFFIC.get((kernel, workload))
    if ent is None or ent["source_hash"] != source_hash(sources):
        return None, None
    return ent["bytes_per_unit"] * units, (f"scaled by units from the capture of {ent['capture']} "
                                           f"({ent['bytes_per_unit']:.1f} B per {ent['unit']})")


def full_causal_pairs(lay) -> int:
    """(query, key) pairs a plain causal mask over each prompt's packed rows would admit."""
    tot = 0
    for b in range(lay.n_prompts):
        lo, hi = lay.prompt_row_range(b)
        n = hi - lo
        tot += n * (n + 1) // 2
    return tot


def measure_workload(cfg, sp, device, args, rank, dist, peaks, steps, warmup, with_e2e, l2_bytes):
    """Times `steps` passes of the whole hot path on one workload; returns the per-kernel
    figures (medians over the timed steps) and, for the rank's own use, the step time."""
    hp = HotPath(cfg, rank_seed(cfg, rank), sp, device, args.prompts, args.decode_steps)
    hp.make_kv_sets(l2_bytes)
    if not args.no_graph:
        hp.capture_decode_graph()
    flush = None
    if hp.bytes_prefill < 2 * l2_bytes:          # small workload: flush L2 between steps
        flush = torch.empty(2 * l2_bytes, dtype=torch.uint8, device=device)

    def sync():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        hp.step()
        if flush is not None:
            flush.zero_()
    sync()
    hp.bytes_decode = hp.decode_bytes()

    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0:
        sampler.start()
    all_ev = []
    sync()
    for _ in range(steps):
        ev = []
        hp.step(ev)
        all_ev.append(ev)
        if flush is not None:
            flush.zero_()
    sync()
    clocks = sampler.stop() if rank == 0 else None
    per_step = np.array([[ev[i].elapsed_time(ev[i + 1]) for i in range(len(STAGES))] for ev in all_ev])
    totals = np.array([ev[0].elapsed_time(ev[-1]) for ev in all_ev])
    stage_ms = np.median(per_step, axis=0)
    ms_per_step = float(np.median(totals))

    def timed(fn, reps=5, per=1):
        fn(); torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            if flush is not None:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / per)
        return float(np.median(ts))

    def graph_of(fn):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
        return g

    # decode kernel alone (no rotation of the new rows), replayed from a graph: the per-launch
    # figure of that kernel; cold = KV sets rotate (as in the step), warm = one set re-read
    n_dec = hp.steps_dec
    plain_loop = lambda: hp.decode_loop(with_rope=False)
    dec_cold_ms = timed(plain_loop if args.no_graph else graph_of(plain_loop).replay, per=n_dec)
    sets = hp.kv_sets
    hp.kv_sets = sets[:1]
    dec_warm_ms = timed(plain_loop if args.no_graph else graph_of(plain_loop).replay, per=n_dec)
    hp.kv_sets = sets
    # the decode step as an application without CUDA graphs would issue it: eager launches
    dec_eager_ms = timed(lambda: hp.decode_loop(), reps=3, per=n_dec)

    # cached / online mode of the prefill (only the query rows of every path are produced): timed
    # on its own, it is not part of the step
    qo_ms = None
    if cfg.dtype == "bf16":
        qo_ms = timed(lambda: sp.sp_superpose_prefill(hp.q, hp.k, hp.v, hp.dl, hp.scale, hp.out, None, hp.ws_pre,
                                                      rows=sp.SP_ROWS_QUERY_ONLY))

    # end to end: pinned host -> device copies of every input, the pass, device -> host results
    e2e = None
    if with_e2e:
        e2e_steps = max(1, min(steps, 3))
        hp.h2d(); hp.step(); hp.d2h(); sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            bi = hp.h2d()
            hp.step()
            bo = hp.d2h()
        e1.record()
        sync()
        e2e = {"ms": e0.elapsed_time(e1) / e2e_steps, "steps": e2e_steps, "h2d": bi, "d2h": bo}

    tf = lambda flop, ms: flop / (ms * 1e-3) / 1e12
    gb = lambda byt, ms: byt / (ms * 1e-3) / 1e9
    ms = dict(zip(STAGES, (float(x) for x in stage_ms)))
    hbm = peaks["hbm_gbs"]
    pre_gbs, pre_tf = gb(hp.bytes_prefill, ms["prefill"]), tf(hp.flop_prefill, ms["prefill"])
    ai = hp.flop_prefill / hp.bytes_prefill
    bound_tf = min(peaks["bf16_tflops_sustained"], ai * hbm / 1e3)
    dec_bytes = hp.bytes_decode / n_dec
    kernels = {
        "rope": {"ms": ms["rope"], "gbs": gb(hp.bytes_rope, ms["rope"]), "frac_hbm": gb(hp.bytes_rope, ms["rope"]) / hbm},
        "prefill": {"ms": ms["prefill"], "useful_tflops": pre_tf, "gbs": pre_gbs,
                    "frac_bf16_burst": pre_tf / peaks["bf16_tflops"],
                    "frac_bf16_sustained": pre_tf / peaks["bf16_tflops_sustained"],
                    "arith_intensity": ai, "binding_roofline_tflops": bound_tf, "frac_binding": pre_tf / bound_tf},
        "path_scores": {"ms": ms["path_scores"], "gbs": gb(hp.bytes_scores, ms["path_scores"]),
                        "frac_hbm": gb(hp.bytes_scores, ms["path_scores"]) / hbm},
        "topk": {"ms": ms["topk"]},
        "prefill_query_only": None if qo_ms is None else {
            "ms": qo_ms, "useful_tflops": tf(hp.flop_query_only, qo_ms), "gbs": gb(hp.bytes_query_only, qo_ms),
            "frac_hbm": gb(hp.bytes_query_only, qo_ms) / hbm,
            "note": "SP_ROWS_QUERY_ONLY (cached preamble/doc KV, Algorithm 3's query batch); not part of the step"},
        "decode": {"ms": ms["decode"], "steps": n_dec, "us_per_token": ms["decode"] / n_dec * 1e3,
                   "gbs": gb(hp.bytes_decode, ms["decode"]), "frac_hbm": gb(hp.bytes_decode, ms["decode"]) / hbm,
                   "kernel_only_us_cold": dec_cold_ms * 1e3, "kernel_only_frac_hbm_cold": gb(dec_bytes, dec_cold_ms) / hbm,
                   "kernel_only_us_warm": dec_warm_ms * 1e3, "kernel_only_gbs_warm": gb(dec_bytes, dec_warm_ms),
                   "ungraphed_us_per_token": dec_eager_ms * 1e3, "kv_sets": len(hp.kv_sets),
                   "launches_per_token": 1 if hp.fused_rope else 2,
                   "includes": ("one launch per token (the new query and key rows are rotated inside the decode kernel)"
                                if hp.fused_rope else "1 rope launch (q and the new key) + 1 decode launch per token")
                               + ("" if args.no_graph else ", replayed from a CUDA graph"),
                   "warm_note": "warm = the same KV set re-read by every launch (may sit in L2): not compared with the HBM peak"},
    }
    T = hp.lay.total_tokens
    keys_per_launch = dec_bytes / (2.0 * hp.Hkv * hp.D * cfg.elt_bytes)
    tr_p, tr_p_note = captured_traffic("prefill", cfg.name, PREFILL_SOURCES, float(T))
    tr_d, tr_d_note = captured_traffic("decode", cfg.name, DECODE_SOURCES, keys_per_launch)
    roof_prefill = {"kernel": "prefill_tc_kernel (sp_superpose_prefill)", "bound": "hbm", "achieved": pre_gbs,
                    "peak": hbm, "unit": "GB/s", "frac": pre_gbs / hbm, "traffic": tr_p, "traffic_note": tr_p_note,
                    "peak_source": peaks["source"], "algorithmic_bytes": hp.bytes_prefill, "launch_ms": ms["prefill"],
                    "useful_tflops": pre_tf, "frac_bf16_sustained": pre_tf / peaks["bf16_tflops_sustained"],
                    "why_hbm": f"arithmetic intensity {ai:.1f} flop/B is below the ridge of the measured peaks"}
    roof_decode = {"kernel": "decode_cluster_kernel (sp_pruned_decode)", "bound": "hbm", "achieved": gb(dec_bytes, dec_cold_ms),
                   "peak": hbm, "unit": "GB/s", "frac": gb(dec_bytes, dec_cold_ms) / hbm, "traffic": tr_d,
                   "traffic_note": tr_d_note, "peak_source": peaks["source"], "algorithmic_bytes": dec_bytes,
                   "launch_ms": dec_cold_ms, "launches_per_step": n_dec}
    res = {
        "workload": cfg.name, "ms_per_step": ms_per_step, "steps": steps, "warmup": warmup,
        "value": tf(hp.flop_prefill, ms_per_step), "frac_bf16_sustained": pre_tf / peaks["bf16_tflops_sustained"],
        "config": {"workload": cfg.name, "prompts_per_gpu": hp.B, "paths": hp.lay.n_paths,
                   "tokens": T, "heads": hp.H, "head_dim": hp.D, "vocab": cfg.vocab,
                   "top_k": cfg.top_k, "decode_steps": n_dec, "allowed_pairs": hp.pairs,
                   "decode_kv_sets": len(hp.kv_sets),
                   "l2": "inputs larger than L2" if flush is None else "L2 flushed between steps",
                   "timing": "median over the timed steps, CUDA events on the launching stream"},
        "useful_vs_full_causal": hp.pairs / max(1, full_causal_pairs(hp.lay)),
        "roofline": roof_prefill, "roofline_decode": roof_decode, "kernels": kernels,
        "flop_prefill": hp.flop_prefill, "launches_per_step": hp.launches, "input_generation_s": hp.gen_s,
        "clocks": clocks, "e2e": e2e,
    }
    del hp, flush
    torch.cuda.empty_cache()
    return res


def run_ours(args):
    import paper_2404_06910_b200 as sp          # raises if the CUDA library is missing
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    peaks = load_peaks()
    l2_bytes = torch.cuda.get_device_properties(device).L2_cache_size
    cfg = get_config(args.workload)
    main = measure_workload(cfg, sp, device, args, rank, dist, peaks, args.steps, args.warmup, not args.no_e2e, l2_bytes)
    # the other large single-GPU workloads, in the same process: fewer steps, no host-copy leg
    extra = []
    if not args.no_extra and args.prompts is None and cfg.name.startswith("cfg2"):
        for name in ("cfg3", "cfg4"):
            extra.append(measure_workload(get_config(name), sp, device, args, rank, dist, peaks,
                                          max(3, min(args.steps, 5)), 3, False, l2_bytes))

    e2e_ms = main["e2e"]["ms"] if main["e2e"] else float("nan")
    ms_per_step, e2e_ms = max_over_ranks([main["ms_per_step"], e2e_ms], dist, device)
    if rank == 0:
        def brief(w):
            k = w["kernels"]
            return {"workload": w["workload"], "ms_per_step": w["ms_per_step"], "steps": w["steps"],
                    "value": w["value"], "tokens": w["config"]["tokens"], "allowed_pairs": w["config"]["allowed_pairs"],
                    "useful_vs_full_causal": w["useful_vs_full_causal"], "roofline": w["roofline"],
                    "roofline_decode": w["roofline_decode"], "kernels": k}
        line = {
            "metric": METRIC, "value": aggregate_value(main["flop_prefill"], ms_per_step, world), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "frac_bf16_sustained": main["frac_bf16_sustained"],
            "config": dict(main["config"], parallelism=f"dp{world} (independent prompts per GPU, no collective)"),
            "useful_vs_full_causal": main["useful_vs_full_causal"],
            "roofline": main["roofline"], "roofline_decode": main["roofline_decode"], "kernels": main["kernels"],
            "workloads": [brief(w) for w in extra],
            "e2e": None if not main["e2e"] else {
                "value": aggregate_value(main["flop_prefill"], e2e_ms, world), "unit": UNIT, "ms_per_step": e2e_ms,
                "steps": main["e2e"]["steps"], "h2d_bytes_per_step": main["e2e"]["h2d"],
                "d2h_bytes_per_step": main["e2e"]["d2h"]},
            "gpu_launches": main["launches_per_step"] * args.steps,
            "clocks": main["clocks"],
            "input_generation_s": main["input_generation_s"],
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = cpu_baseline(cfg, steps=1, warmup=0, budget_s=15.0)[0]
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------
def run_widened(args):
    """Timings of the rows beyond the first path (not part of the step, printed as one JSON line):
    the ALiBi variants of the prefill and the decode on the chosen workload, and an iterative
    superposition workload (Section 4.3: t rounds, the k documents kept in a round join the
    shared prefix of the next) with document lengths around the paper's multi-hop setting
    (Appendix D: 20 documents, about 121 tokens each)."""
    import paper_2404_06910_b200 as sp
    from workloads import build_layout, next_round_layout
    device = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    peaks = load_peaks()
    hbm = peaks["hbm_gbs"]
    cfg = get_config(args.workload)
    hp = HotPath(cfg, cfg.seed, sp, device, args.prompts, args.decode_steps)
    H, D, B = hp.H, hp.D, hp.B

    def timed(fn, reps=7, per=1):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / per)
        return float(np.median(ts))

    gb = lambda byt, ms: byt / (ms * 1e-3) / 1e9
    slopes = torch.tensor([2.0 ** (-8.0 * (h + 1) / H) for h in range(H)], dtype=torch.float32, device=device)
    plain_ms = timed(lambda: sp.sp_superpose_prefill(hp.q, hp.k, hp.v, hp.dl, hp.scale, hp.out, None, hp.ws_pre))
    alibi_ms = timed(lambda: sp.sp_superpose_prefill_alibi(hp.q, hp.k, hp.v, hp.dl, hp.pos, slopes, hp.scale, hp.out,
                                                           None, hp.ws_pre))
    # the rotation of Q folded into the prefill (sp_superpose_prefill_rope) against the two calls it replaces
    ws_rope = torch.zeros(sp.sp_prefill_rope_workspace_bytes(hp.dl, H, D, sp.SP_BF16), dtype=torch.uint8, device=device)
    rope_q_ms = timed(lambda: sp.sp_rope_apply(hp.q, hp.pos, H, D, base=cfg.rope_base))
    fused_ms = timed(lambda: sp.sp_superpose_prefill_rope(hp.q, hp.k, hp.v, hp.dl, hp.pos, cfg.rope_base,
                                                          sp.SP_ROPE_HALF_SPLIT, hp.scale, hp.out, None, ws_rope))
    rope_fused = {"workload": cfg.name, "rope_q_ms": rope_q_ms, "prefill_ms": plain_ms, "two_calls_ms": rope_q_ms + plain_ms,
                  "prefill_rope_ms": fused_ms,
                  "note": "sp_superpose_prefill_rope = (cos, sin) table kernel + tile plan + prefill kernel that rotates each "
                          "query tile in shared memory; K is rotated by sp_rope_apply in both paths"}
    del ws_rope
    hp.step()
    torch.cuda.synchronize()
    hp.bytes_decode = hp.decode_bytes()
    n_dec = hp.steps_dec
    tail_pos = hp.tpos.t().contiguous()                                # [B, steps]
    def dec_plain():
        for t in range(n_dec):
            sp.sp_pruned_decode(hp.dq[t], hp.k, hp.v, hp.dl, hp.kept, cfg.top_k, hp.tk, hp.tv, hp.tail_len[t], n_dec,
                                hp.scale, hp.dec_out[t], None, hp.ws_dec)
    def dec_alibi():
        for t in range(n_dec):
            sp.sp_pruned_decode_alibi(hp.dq[t], hp.k, hp.v, hp.dl, hp.kept, cfg.top_k, hp.tk, hp.tv, hp.tail_len[t],
                                      n_dec, hp.tpos[t], hp.pos, tail_pos, slopes, hp.scale, hp.dec_out[t], None, hp.ws_dec)
    dplain_ms, dalibi_ms = timed(dec_plain, reps=3, per=n_dec), timed(dec_alibi, reps=3, per=n_dec)
    alibi = {"workload": cfg.name,
             "prefill_ms": plain_ms, "prefill_alibi_ms": alibi_ms, "prefill_alibi_frac_hbm": gb(hp.bytes_prefill, alibi_ms) / hbm,
             "decode_us": dplain_ms * 1e3, "decode_alibi_us": dalibi_ms * 1e3,
             "decode_alibi_frac_hbm": gb(hp.bytes_decode / n_dec, dalibi_ms) / hbm,
             "note": "decode launches issued eagerly, one KV set"}
    del hp
    torch.cuda.empty_cache()

    # iterative superposition: lengths ~ U{60..180} (mean 120), 20 documents, preamble 32, query 24
    rng = np.random.default_rng(20240410 + 77)
    n_prompts, n_docs, k_keep, rounds = 64, 20, 2, 3
    lay = build_layout([32] * n_prompts, [rng.integers(60, 181, size=n_docs) for _ in range(n_prompts)],
                       [[24] * n_docs] * n_prompts)
    iters = []
    for r in range(rounds):
        T = lay.total_tokens
        g = torch.Generator(device=device); g.manual_seed(100 + r)
        q, k, v = (torch.randn(T, H, D, device=device, generator=g).mul_(D ** -0.5).bfloat16() for _ in range(3))
        out = torch.empty_like(q)
        dl = sp.DeviceLayout.from_host(lay, device)
        ws = torch.zeros(max(256, sp.sp_prefill_workspace_bytes(dl, H, D, sp.SP_BF16)), dtype=torch.uint8, device=device)
        ms = timed(lambda: sp.sp_superpose_prefill(q, k, v, dl, D ** -0.5, out, None, ws))
        byt, flop = 4.0 * T * H * D * 2, 4.0 * D * H * lay.allowed_pairs()
        iters.append({"round": r, "prefix_len": int(lay.max_pre_len), "paths_per_prompt": int(lay.n_paths // n_prompts),
                      "tokens": int(T), "prefill_ms": ms, "frac_hbm": gb(byt, ms) / hbm,
                      "useful_tflops": flop / (ms * 1e-3) / 1e12, "arith_intensity": flop / byt})
        # the k kept documents of every prompt (here: its first k remaining paths) join the prefix
        kept = np.stack([np.arange(lay.prompt_path_off[b], lay.prompt_path_off[b] + k_keep) for b in range(n_prompts)])
        lay = next_round_layout(lay, kept)
        del q, k, v, out
        torch.cuda.empty_cache()
    # grouped query heads: the cfg2 decode shape with 8 KV heads under the 32 query heads (one block owns
    # a KV head and 4 of its query heads, so each K / V row is read once per group)
    lay_g = draw_lengths(cfg)
    Bg, Hkv_g, n_g = lay_g.n_prompts, 8, 8
    g = torch.Generator(device=device); g.manual_seed(8)
    mk = lambda *shape: torch.randn(*shape, device=device, generator=g).mul_(D ** -0.5).bfloat16()
    kc_sets = [(mk(lay_g.total_tokens, Hkv_g, D), mk(lay_g.total_tokens, Hkv_g, D)) for _ in range(4)]   # > 2 x L2 in rotation
    qg, tkg, tvg = mk(n_g, Bg, H, D), mk(Bg, n_g, Hkv_g, D), mk(Bg, n_g, Hkv_g, D)
    dl_g = sp.DeviceLayout.from_host(lay_g, device)
    kept_g = torch.stack([torch.arange(2, dtype=torch.int32) + int(lay_g.prompt_path_off[b]) for b in range(Bg)]).to(device)
    tl_g = torch.arange(1, n_g + 1, dtype=torch.int32)[:, None].expand(n_g, Bg).contiguous().to(device)
    out_g = torch.empty((n_g, Bg, H, D), dtype=torch.bfloat16, device=device)
    ws_g = torch.zeros(max(256, sp.sp_decode_workspace_bytes(Bg, H, D)), dtype=torch.uint8, device=device)
    def dec_gqa():
        for t in range(n_g):
            kc, vc = kc_sets[t % len(kc_sets)]
            sp.sp_pruned_decode(qg[t], kc, vc, dl_g, kept_g, 2, tkg, tvg, tl_g[t], n_g, D ** -0.5, out_g[t], None, ws_g)
    gqa_ms = timed(dec_gqa, reps=5, per=n_g)
    keys_g = sum(int(lay_g.pre_len[b]) + sum(int(lay_g.doc_len[i] + lay_g.qry_len[i]) for i in kept_g[b].tolist()) for b in range(Bg)) \
        + Bg * (n_g + 1) / 2.0
    bytes_g = keys_g * 2 * Hkv_g * D * 2
    gqa = {"shape": "cfg2 lengths, 64 prompts, 32 query heads over 8 KV heads, k = 2", "decode_us": gqa_ms * 1e3,
           "algorithmic_mb": bytes_g / 1e6, "frac_hbm": gb(bytes_g, gqa_ms) / hbm,
           "note": "bytes counted once per KV head; launches issued eagerly, KV sets rotating"}
    del kc_sets, qg, tkg, tvg, out_g
    torch.cuda.empty_cache()

    # bf16 with head_dim 64 (served by the fp32-arithmetic SIMT kernel): a smaller batch of the cfg2 shape
    lay64 = draw_lengths(get_config("cfg2"), n_prompts=8)
    T64, H64, D64 = lay64.total_tokens, 32, 64
    g = torch.Generator(device=device); g.manual_seed(64)
    q, k, v = (torch.randn(T64, H64, D64, device=device, generator=g).mul_(D64 ** -0.5).bfloat16() for _ in range(3))
    out = torch.empty_like(q)
    dl64 = sp.DeviceLayout.from_host(lay64, device)
    ws64 = torch.zeros(max(256, sp.sp_prefill_workspace_bytes(dl64, H64, D64, sp.SP_BF16)), dtype=torch.uint8, device=device)
    ms64 = timed(lambda: sp.sp_superpose_prefill(q, k, v, dl64, D64 ** -0.5, out, None, ws64), reps=3)
    flop64 = 4.0 * D64 * H64 * lay64.allowed_pairs()
    simt = {"shape": "cfg2 lengths, 8 prompts, 32 heads x 64, bf16", "tokens": int(T64), "prefill_ms": ms64,
            "useful_tflops": flop64 / (ms64 * 1e-3) / 1e12, "frac_hbm": gb(4.0 * T64 * H64 * D64 * 2, ms64) / hbm,
            "note": "warp per (row, head), fp32 FMA arithmetic, no tensor cores"}
    del q, k, v, out
    print(json.dumps({"widened": True, "alibi": alibi, "rope_folded_into_prefill": rope_fused, "decode_grouped_heads": gqa,
                      "bf16_head_dim_64": simt,
                      "iterative": {"prompts": n_prompts, "documents": n_docs, "kept_per_round": k_keep, "rounds": iters,
                                    "data": "synthetic, lengths U{60..180}"}}))


# ---------------------------------------------------------------------------------------
def oracle_sample_pass(cfg, n_prompts):
    """Returns a closure that runs the whole hot path in the CPU oracle on the first n_prompts
    prompts of the workload, and the useful prefill FLOPs of that sample."""
    import oracle
    from workloads.tensors import to_f32_numpy
    lay = draw_lengths(cfg, n_prompts=n_prompts)
    B = lay.n_prompts
    q, k, v = (to_f32_numpy(t) for t in draw_qkv(cfg, lay))
    logits = to_f32_numpy(draw_logits(cfg, lay))
    tgt = draw_targets(cfg, lay)
    prior, weight = draw_prior_weight(cfg, lay)
    steps = cfg.decode_steps
    dq, tk, tv = (to_f32_numpy(t) for t in draw_decode_inputs(cfg, B, steps))
    scheme = "equilibrium" if cfg.positions == "equilibrium" else "left"
    scale = 1.0 / math.sqrt(cfg.head_dim)

    def run():
        pos, nxt = positions_all(lay, lambda P, L, Q: oracle.positions(P, L, Q, scheme=scheme))
        qr = oracle.rope(q, pos, base=cfg.rope_base)
        kr = oracle.rope(k, pos, base=cfg.rope_base)
        oracle.prefill(qr, kr, v, lay, scale)
        s, _ = oracle.path_scores(logits, tgt, lay.query_row_offsets(), prior, weight)
        kept, _ = oracle.prune_topk(s, lay.prompt_path_off, cfg.top_k)
        tkr = tk.copy()
        for t in range(steps):
            tp = (nxt + t).astype(np.float32)
            qt = oracle.rope(dq[t], tp, base=cfg.rope_base)
            tkr[:, t] = oracle.rope(np.ascontiguousarray(tkr[:, t]), tp, base=cfg.rope_base)
            oracle.pruned_decode(qt, kr, v, lay, kept, tkr, tv, np.full(B, t + 1, np.int32), scale)

    flop = 4.0 * cfg.head_dim * cfg.n_heads * lay.allowed_pairs()
    return run, flop, B


def cpu_baseline(cfg, steps, warmup, budget_s):
    """Times the oracle, as it stands, on a bounded sample: whole prompts of the workload,
    as many as fit the time budget (calibrated on one prompt)."""
    import oracle
    run1, _, _ = oracle_sample_pass(cfg, 1)
    t0 = time.perf_counter()
    run1()
    t1 = max(time.perf_counter() - t0, 1e-3)
    n = int(max(1, min(cfg.n_prompts, budget_s / max(1, steps + warmup) / t1)))
    run, flop, n = oracle_sample_pass(cfg, n)
    for _ in range(warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(steps):
        run()
    dt = (time.perf_counter() - t0) / steps
    return ({"value": flop / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
             "sample": f"whole hot path (rope, prefill, scores, top-k, {cfg.decode_steps} decode steps) on the "
                       f"first {n} of {cfg.n_prompts} prompts of {cfg.name}, all heads",
             "ms_per_sample": dt * 1e3}, dt)


def run_reference(args):
    """Times the CPU oracle (as it stands) on the host cores; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg = get_config(args.workload)
    base, dt = cpu_baseline(cfg, args.steps, args.warmup, budget_s=150.0)
    line = {"impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": cfg.name, "sample": base["sample"]},
            "cpu_baseline": base,
            "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def launcher_command(n_gpus: int, argv):
    """`bench.py --gpus N` started as a plain script: the command that starts N ranks of it on this
    node (one per GPU), rendezvous on the loopback address."""
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the decode loop eagerly instead of replaying a CUDA graph")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg (profiling aid)")
    ap.add_argument("--widened", action="store_true", help="time the ALiBi variants and an iterative-superposition workload instead of the step")
    ap.add_argument("--no-extra", action="store_true", help="skip the cfg3 / cfg4 passes that follow the default workload")
    ap.add_argument("--prompts", type=int, default=None, help="override the prompts per GPU (profiling aid)")
    ap.add_argument("--decode-steps", type=int, default=None, help="override the decode steps (profiling aid)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(subprocess.call(launcher_command(args.gpus, sys.argv[1:])))
    if args.widened:
        run_widened(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
