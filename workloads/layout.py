"""Ragged fork-join packing: where each segment's rows sit in the packed arrays.

Packed row order inside one prompt is path-major,
    [ preamble | doc_0 query_0 | doc_1 query_1 | ... ],
and prompts follow each other.  This is bookkeeping only.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from .configs import Config


@dataclass
class Layout:
    n_prompts: int
    n_paths: int
    prompt_path_off: np.ndarray   # int32 [B+1]
    pre_start: np.ndarray         # int32 [B]
    pre_len: np.ndarray           # int32 [B]
    path_start: np.ndarray        # int32 [NP]  first packed row of doc_i (query_i follows)
    doc_len: np.ndarray           # int32 [NP]
    qry_len: np.ndarray           # int32 [NP]
    total_tokens: int             # T

    @property
    def max_pre_len(self) -> int:
        return int(self.pre_len.max()) if self.n_prompts else 0

    @property
    def max_path_len(self) -> int:
        return int((self.doc_len + self.qry_len).max()) if self.n_paths else 0

    def prompt_row_range(self, b: int):
        """[first, last) packed rows of prompt b."""
        lo = int(self.pre_start[b])
        p1 = int(self.prompt_path_off[b + 1])
        p0 = int(self.prompt_path_off[b])
        if p1 > p0:
            hi = int(self.path_start[p1 - 1] + self.doc_len[p1 - 1] + self.qry_len[p1 - 1])
        else:
            hi = lo + int(self.pre_len[b])
        return lo, hi

    def query_row_offsets(self) -> np.ndarray:
        """int32 [NP+1]: path i's query rows occupy [off[i], off[i+1]) of a
        path-major [R, V] logits array."""
        off = np.zeros(self.n_paths + 1, dtype=np.int32)
        np.cumsum(self.qry_len, out=off[1:])
        return off

    def allowed_pairs(self) -> int:
        """Number of (query row, key row) pairs the fork-join mask admits."""
        total = 0
        for b in range(self.n_prompts):
            P = int(self.pre_len[b])
            total += P * (P + 1) // 2
            for i in range(int(self.prompt_path_off[b]), int(self.prompt_path_off[b + 1])):
                n = int(self.doc_len[i] + self.qry_len[i])
                total += n * P + n * (n + 1) // 2
        return total


def build_layout(pre_lens, doc_lens, qry_lens) -> Layout:
    """pre_lens: [B]; doc_lens, qry_lens: list (per prompt) of per-path lengths."""
    B = len(pre_lens)
    ppo = [0]
    pre_start, path_start, dl, ql = [], [], [], []
    row = 0
    for b in range(B):
        pre_start.append(row)
        row += int(pre_lens[b])
        for L, Q in zip(doc_lens[b], qry_lens[b]):
            path_start.append(row)
            dl.append(int(L))
            ql.append(int(Q))
            row += int(L) + int(Q)
        ppo.append(len(path_start))
    i32 = lambda a: np.asarray(a, dtype=np.int32).reshape(-1)
    return Layout(B, len(path_start), i32(ppo), i32(pre_start), i32(pre_lens),
                  i32(path_start), i32(dl), i32(ql), row)


def draw_lengths(cfg: Config, seed: int | None = None, n_prompts: int | None = None) -> Layout:
    """Document lengths ~ U{doc_len_min..doc_len_max}, independent per prompt."""
    rng = np.random.default_rng(cfg.seed if seed is None else seed)
    B = cfg.n_prompts if n_prompts is None else n_prompts
    docs = [rng.integers(cfg.doc_len_min, cfg.doc_len_max + 1, size=cfg.n_docs) for _ in range(B)]
    qrys = [np.full(cfg.n_docs, cfg.qry_len) for _ in range(B)]
    return build_layout([cfg.pre_len] * B, docs, qrys)


def next_round_layout(lay: Layout, kept: np.ndarray) -> Layout:
    """Iterative superposition (Section 4.3): the documents kept in this round (global path
    ids per prompt, -1 = none) join the prompt's shared prefix, in the order given; every other
    path stays a path of the next round, with its own copy of the query."""
    kept = np.asarray(kept).reshape(lay.n_prompts, -1)
    pre, docs, qrys = [], [], []
    for b in range(lay.n_prompts):
        p0, p1 = int(lay.prompt_path_off[b]), int(lay.prompt_path_off[b + 1])
        chosen = [int(i) for i in kept[b] if p0 <= int(i) < p1]
        pre.append(int(lay.pre_len[b]) + sum(int(lay.doc_len[i]) for i in chosen))
        rest = [i for i in range(p0, p1) if i not in chosen]
        docs.append([int(lay.doc_len[i]) for i in rest])
        qrys.append([int(lay.qry_len[i]) for i in rest])
    return build_layout(pre, docs, qrys)
