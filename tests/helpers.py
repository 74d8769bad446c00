"""Test utilities: error metrics, sub-problem extraction for sampled parity, device upload."""
from __future__ import annotations

import numpy as np
import torch

from workloads import build_layout


def rel_l2(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(got - ref) / (den if den > 0 else 1.0))


def f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float32).contiguous().numpy()


def sub_problem(lay, b: int, path_ids):
    """Layout holding only prompt b's preamble and the given (global) paths, the packed-row
    gather that extracts it, and the map old path id -> new path id."""
    path_ids = [int(i) for i in path_ids]
    P = int(lay.pre_len[b])
    sub = build_layout([P], [[int(lay.doc_len[i]) for i in path_ids]],
                       [[int(lay.qry_len[i]) for i in path_ids]])
    rows = [np.arange(lay.pre_start[b], lay.pre_start[b] + P)]
    for i in path_ids:
        rows.append(np.arange(lay.path_start[i], lay.path_start[i] + lay.doc_len[i] + lay.qry_len[i]))
    return sub, np.concatenate(rows).astype(np.int64), {old: new for new, old in enumerate(path_ids)}


def positions_for(lay, positions_fn):
    """Packed float32 positions of every prompt of a layout, from a per-prompt function
    (pre_len, doc_lens, qry_len) -> (pos, S, next)."""
    out = np.zeros(lay.total_tokens, dtype=np.float32)
    nxt = np.zeros(lay.n_prompts, dtype=np.float64)
    for b in range(lay.n_prompts):
        p0, p1 = int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])
        q = int(lay.qry_len[p0]) if p1 > p0 else 0
        pos, _, n = positions_fn(int(lay.pre_len[b]), lay.doc_len[p0:p1], q)
        lo, hi = lay.prompt_row_range(b)
        out[lo:hi] = pos
        nxt[b] = n
    return out, nxt


def dev(a, dtype=None):
    if isinstance(a, np.ndarray):
        a = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        a = a.to(dtype)
    return a.to("cuda").contiguous()


def workspace(nbytes: int):
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")
