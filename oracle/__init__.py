"""ctypes front-end of the CPU oracle (``sp_oracle.c``).

TEST INFRASTRUCTURE: only the test-suite, the smoke check and the CPU-baseline /
reference leg of the benchmark may import this package.  It shares nothing with the
CUDA library.  Arrays are numpy, float32 / int32 / int64 on the host.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sp_oracle.c")
_LIB = os.path.join(_HERE, "libsp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain C, OpenMP over independent rows/paths)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-fno-fast-math", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.spo_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().spo_num_threads())


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a, ct=ctypes.c_void_p):
    return None if a is None else a.ctypes.data_as(ct)


def _check(rc, name):
    if rc != 0:
        raise ValueError(f"oracle {name} rejected its arguments (code {rc})")


def positions(P: int, doc_lens, Q: int, scheme: str = "equilibrium", q_mode: int = 0):
    """Packed positions of one prompt (float64), S, and the first position after the query."""
    L = _i32(doc_lens)
    n = int(P + L.sum() + len(L) * Q)
    pos = np.zeros(n, dtype=np.float64)
    S = ctypes.c_double()
    nxt = ctypes.c_double()
    rc = _load().spo_positions(ctypes.c_int({"equilibrium": 0, "left": 1}[scheme]), ctypes.c_int(q_mode),
                               ctypes.c_int(P), ctypes.c_int(len(L)), _p(L), ctypes.c_int(Q),
                               _p(pos), ctypes.byref(S), ctypes.byref(nxt))
    _check(rc, "positions")
    return pos, S.value, nxt.value


def rope(x, pos, rot_dim=None, base=10000.0, pairing=0):
    """x: [n, H, D] float32 (copied); pos: [n] float32.  Returns the rotated copy."""
    x = _f32(x).copy()
    n, H, D = x.shape
    pos = _f32(pos)
    assert pos.shape == (n,)
    rc = _load().spo_rope(_p(x), _p(pos), ctypes.c_int64(n), ctypes.c_int64(H * D), ctypes.c_int(H),
                          ctypes.c_int(D), ctypes.c_int(D if rot_dim is None else rot_dim),
                          ctypes.c_double(base), ctypes.c_int(pairing))
    _check(rc, "rope")
    return x


def _lay_args(lay):
    arrs = [_i32(lay.prompt_path_off), _i32(lay.pre_start), _i32(lay.pre_len),
            _i32(lay.path_start), _i32(lay.doc_len), _i32(lay.qry_len)]
    return arrs, [ctypes.c_int(lay.n_prompts)] + [_p(a) for a in arrs]


def prefill(q, k, v, lay, scale, rows=None, want_lse=True, pos=None, slopes=None):
    """q [T,H,D], k/v [T,Hkv,D] float32.  Returns (out [T,H,D], lse [H,T]).
    With ``rows`` (int64 list) only those packed rows are computed; the rest stay 0.
    With ``pos`` [T] and ``slopes`` [H] the scores get the ALiBi bias -slope * |pos_q - pos_k|."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    T, H, D = q.shape
    Hkv = k.shape[1]
    assert T == lay.total_tokens and k.shape == (T, Hkv, D) and v.shape == k.shape
    out = np.zeros_like(q)
    lse = np.zeros((H, T), dtype=np.float32) if want_lse else None
    keep, largs = _lay_args(lay)
    r = None if rows is None else np.ascontiguousarray(rows, dtype=np.int64)
    ps = None if pos is None else _f32(pos)
    sl = None if slopes is None else _f32(slopes)
    assert (ps is None) == (sl is None) and (ps is None or (ps.shape == (T,) and sl.shape == (H,)))
    rc = _load().spo_prefill_alibi(_p(q), _p(k), _p(v), *largs, ctypes.c_int64(T), ctypes.c_int(H),
                                   ctypes.c_int(Hkv), ctypes.c_int(D), ctypes.c_double(scale), _p(ps), _p(sl),
                                   _p(r), ctypes.c_int64(0 if r is None else len(r)), _p(out), _p(lse))
    _check(rc, "prefill")
    return out, lse


def path_scores(logits, targets, row_off, prior=None, weight=None, want_row_logp=True):
    logits = _f32(logits)
    R, V = logits.shape
    targets, row_off = _i32(targets), _i32(row_off)
    n_paths = len(row_off) - 1
    scores = np.zeros(n_paths, dtype=np.float32)
    row_logp = np.zeros(R, dtype=np.float32) if want_row_logp else None
    pr = None if prior is None else _f32(prior)
    w = None if weight is None else _f32(weight)
    rc = _load().spo_path_scores(_p(logits), ctypes.c_int64(V), _p(targets), _p(row_off),
                                 ctypes.c_int(n_paths), ctypes.c_int(V), _p(pr), _p(w),
                                 _p(scores), _p(row_logp))
    _check(rc, "path_scores")
    return scores, row_logp


def prune_topk(scores, prompt_path_off, k):
    scores, ppo = _f32(scores), _i32(prompt_path_off)
    B = len(ppo) - 1
    idx = np.zeros((B, k), dtype=np.int32)
    post = np.zeros((B, k), dtype=np.float32)
    rc = _load().spo_prune_topk(_p(scores), _p(ppo), ctypes.c_int(B), ctypes.c_int(k), _p(idx), _p(post))
    _check(rc, "prune_topk")
    return idx, post


def pruned_decode(q, k_cache, v_cache, lay, kept_idx, tail_k, tail_v, tail_len, scale,
                  q_pos=None, cache_pos=None, tail_pos=None, slopes=None):
    """q [B,H,D]; caches [T,Hkv,D]; tail_k/v [B,cap,Hkv,D]; kept_idx [B,k]; tail_len [B].
    ALiBi: q_pos [B], cache_pos [T], tail_pos [B,cap], slopes [H] (all or none)."""
    q, k_cache, v_cache = _f32(q), _f32(k_cache), _f32(v_cache)
    B, H, D = q.shape
    Hkv = k_cache.shape[1]
    kept_idx = _i32(kept_idx).reshape(B, -1)
    k = kept_idx.shape[1]
    if tail_k is None:
        tail_k = np.zeros((B, 1, Hkv, D), dtype=np.float32)
        tail_v = np.zeros((B, 1, Hkv, D), dtype=np.float32)
        tail_len = np.zeros(B, dtype=np.int32)
    tail_k, tail_v, tail_len = _f32(tail_k), _f32(tail_v), _i32(tail_len)
    cap = tail_k.shape[1]
    out = np.zeros((B, H, D), dtype=np.float32)
    lse = np.zeros((B, H), dtype=np.float32)
    keep, largs = _lay_args(lay)
    qp = None if slopes is None else _f32(q_pos)
    cp = None if slopes is None else _f32(cache_pos)
    tp = None if slopes is None else (_f32(tail_pos) if tail_pos is not None else np.zeros((B, cap), dtype=np.float32))
    sl = None if slopes is None else _f32(slopes)
    assert sl is None or (qp.shape == (B,) and cp.shape == (k_cache.shape[0],) and tp.shape == (B, cap) and sl.shape == (H,))
    rc = _load().spo_pruned_decode_alibi(_p(q), _p(k_cache), _p(v_cache), *largs, _p(kept_idx), ctypes.c_int(k),
                                         _p(tail_k), _p(tail_v), _p(tail_len), ctypes.c_int(cap),
                                         ctypes.c_int(H), ctypes.c_int(Hkv), ctypes.c_int(D),
                                         ctypes.c_double(scale), _p(qp), _p(cp), _p(tp), _p(sl), _p(out), _p(lse))
    _check(rc, "pruned_decode")
    return out, lse
