"""ctypes binding of libsp_b200.so (declared in include/sp.h).

Argument marshalling only: every function forwards raw device pointers and sizes to the
C ABI entry point of the same name.  torch is used for device memory and streams.
There is no fallback: if the CUDA library is missing, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# SP_B200_DEBUG_BOUNDS=1 selects the twin built with -DSP_DEBUG_BOUNDS (extra device-side layout checks)
LIB_PATH = os.path.join(_HERE, "libsp_b200_debug.so" if os.environ.get("SP_B200_DEBUG_BOUNDS") == "1" else "libsp_b200.so")

SP_OK = 0
SP_ERR_INVALID_ARG, SP_ERR_UNSUPPORTED, SP_ERR_WORKSPACE, SP_ERR_CUDA, SP_ERR_TIMEOUT, SP_ERR_LAYOUT = 1, 2, 3, 4, 5, 6
SP_F32, SP_BF16 = 0, 1
SP_ROWS_ALL, SP_ROWS_QUERY_ONLY = 0, 1
SP_POS_EQUILIBRIUM, SP_POS_LEFT_ALIGNED = 0, 1
SP_ROPE_HALF_SPLIT, SP_ROPE_INTERLEAVED = 0, 1

EXPORTS = (
    "sp_last_error", "sp_version", "sp_positions", "sp_rope_apply",
    "sp_prefill_workspace_bytes", "sp_superpose_prefill",
    "sp_path_scores_workspace_bytes", "sp_path_scores", "sp_prune_topk",
    "sp_decode_workspace_bytes", "sp_pruned_decode", "sp_check_status",
    "sp_pruned_decode_static_max_bytes", "sp_pruned_decode_static",
    "sp_superpose_prefill_alibi", "sp_pruned_decode_alibi", "sp_rope_apply_pair", "sp_pruned_decode_rope",
    "sp_prefill_rope_workspace_bytes", "sp_superpose_prefill_rope",
)


class SpError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"sp status {code}: {message}")
        self.code = code


class _CLayoutHost(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("prompt_path_off", "pre_start", "pre_len", "path_start", "doc_len", "qry_len")]


class _CLayout(ctypes.Structure):
    _fields_ = [
        ("n_prompts", ctypes.c_int32), ("n_paths", ctypes.c_int32),
        ("prompt_path_off", ctypes.c_void_p), ("pre_start", ctypes.c_void_p),
        ("pre_len", ctypes.c_void_p), ("path_start", ctypes.c_void_p),
        ("doc_len", ctypes.c_void_p), ("qry_len", ctypes.c_void_p),
        ("total_tokens", ctypes.c_int64),
        ("max_pre_len", ctypes.c_int32), ("max_path_len", ctypes.c_int32),
        ("host_mirror", ctypes.POINTER(_CLayoutHost)),
    ]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2404_06910_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    c_int, c_i64, c_f, c_d, vp, sz = (ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_double,
                                      ctypes.c_void_p, ctypes.c_size_t)
    lp = ctypes.POINTER(_CLayout)
    lib.sp_last_error.restype = ctypes.c_char_p
    lib.sp_version.restype = ctypes.c_char_p
    lib.sp_positions.argtypes = [c_int, c_int, c_int, c_int, vp, c_int, vp, ctypes.POINTER(c_d), ctypes.POINTER(c_d)]
    lib.sp_rope_apply.argtypes = [vp, vp, c_i64, c_i64, c_int, c_int, c_int, c_d, c_int, c_int, vp]
    lib.sp_rope_apply_pair.argtypes = [vp, c_i64, c_int, vp, c_i64, c_int, vp, c_i64, c_int, c_int, c_d, c_int, c_int, vp]
    lib.sp_prefill_workspace_bytes.argtypes = [c_int] * 7
    lib.sp_prefill_workspace_bytes.restype = sz
    lib.sp_superpose_prefill.argtypes = [vp, vp, vp, lp, c_int, c_int, c_int, c_f, c_int, vp, vp, vp, sz, c_int, vp]
    lib.sp_prefill_rope_workspace_bytes.argtypes = [c_int, c_int, c_int, c_int, c_i64, c_int, c_int, c_int]
    lib.sp_prefill_rope_workspace_bytes.restype = sz
    lib.sp_superpose_prefill_rope.argtypes = [vp, vp, vp, lp, vp, c_d, c_int, c_int, c_int, c_int, c_f, vp, vp, vp, sz,
                                              c_int, vp]
    lib.sp_path_scores_workspace_bytes.argtypes = [c_i64]
    lib.sp_path_scores_workspace_bytes.restype = sz
    lib.sp_path_scores.argtypes = [vp, c_i64, vp, vp, c_i64, c_int, c_int, vp, vp, vp, vp, vp, sz, c_int, vp]
    lib.sp_prune_topk.argtypes = [vp, vp, c_int, c_int, vp, vp, vp]
    lib.sp_decode_workspace_bytes.argtypes = [c_int, c_int, c_int]
    lib.sp_decode_workspace_bytes.restype = sz
    lib.sp_pruned_decode.argtypes = [vp, vp, vp, lp, vp, c_int, vp, vp, vp, c_int, c_i64, c_int, c_int, c_int,
                                     c_f, vp, vp, vp, sz, c_int, vp]
    lib.sp_check_status.argtypes = [vp, vp]
    lib.sp_pruned_decode_static_max_bytes.restype = sz
    lib.sp_pruned_decode_static.argtypes = [vp, vp, vp, lp, vp, c_int, vp, vp, vp, c_int, c_i64, c_int, c_int, c_int,
                                            c_f, vp, vp, c_int, vp]
    lib.sp_superpose_prefill_alibi.argtypes = [vp, vp, vp, lp, vp, vp, c_int, c_int, c_int, c_f, c_int, vp, vp, vp, sz,
                                               c_int, vp]
    lib.sp_pruned_decode_alibi.argtypes = [vp, vp, vp, lp, vp, c_int, vp, vp, vp, c_int, c_i64, vp, vp, vp, vp, c_int,
                                           c_int, c_int, c_f, vp, vp, vp, sz, c_int, vp]
    lib.sp_pruned_decode_rope.argtypes = [vp, vp, vp, lp, vp, c_int, vp, vp, vp, c_int, c_i64, vp, c_d, c_int, c_int,
                                          c_int, c_int, c_f, vp, vp, c_int, vp]
    for name in EXPORTS:
        getattr(lib, name)          # raises AttributeError if a declared symbol is not exported
    return lib


lib = _load()


def _check(rc: int):
    if rc != SP_OK:
        raise SpError(rc, lib.sp_last_error().decode())


def dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return SP_F32
    if t.dtype == torch.bfloat16:
        return SP_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t):
    if t is None:
        return None
    assert t.is_contiguous(), "tensors must be contiguous"
    return t.data_ptr()


def _nbytes(t):
    return 0 if t is None else t.numel() * t.element_size()


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


@dataclass
class DeviceLayout:
    """sp_layout with its index arrays resident on the device."""
    c: _CLayout
    arrays: tuple          # keeps the device tensors alive
    n_prompts: int
    n_paths: int
    total_tokens: int
    max_pre_len: int
    max_path_len: int

    @property
    def prompt_path_off(self):
        return self.arrays[0]

    @staticmethod
    def from_host(lay, device="cuda", mirror: bool = True) -> "DeviceLayout":
        """mirror: also hand the host copies of the index arrays to the library, which then
        validates the whole layout on the host in every call."""
        host = tuple(np.ascontiguousarray(a, dtype=np.int32) for a in (lay.prompt_path_off, lay.pre_start, lay.pre_len,
                                                                       lay.path_start, lay.doc_len, lay.qry_len))
        arrs = tuple(torch.from_numpy(a).to(device) for a in host)
        hm = _CLayoutHost(*[a.ctypes.data for a in host]) if mirror else None
        c = _CLayout(lay.n_prompts, lay.n_paths, *[a.data_ptr() for a in arrs],
                     lay.total_tokens, lay.max_pre_len, lay.max_path_len,
                     ctypes.pointer(hm) if mirror else None)
        return DeviceLayout(c, arrs + host + (hm,), lay.n_prompts, lay.n_paths, lay.total_tokens,
                            lay.max_pre_len, lay.max_path_len)


def sp_version() -> str:
    return lib.sp_version().decode()


def sp_positions(pre_len: int, doc_lens, qry_len: int, scheme: int = SP_POS_EQUILIBRIUM, q_mode: int = 0):
    """Host call.  Returns (pos float32 [P + sum(L) + N*Q], S, next_pos)."""
    L = np.ascontiguousarray(doc_lens, dtype=np.int32)
    pos = np.empty(int(pre_len + L.sum() + len(L) * qry_len), dtype=np.float32)
    S, nxt = ctypes.c_double(), ctypes.c_double()
    _check(lib.sp_positions(scheme, q_mode, pre_len, len(L), L.ctypes.data, qry_len, pos.ctypes.data,
                            ctypes.byref(S), ctypes.byref(nxt)))
    return pos, S.value, nxt.value


def sp_rope_apply(x: torch.Tensor, pos: torch.Tensor, n_heads: int, head_dim: int, *, n_tokens=None,
                  ld_token=None, rot_dim=None, base: float = 10000.0, pairing: int = SP_ROPE_HALF_SPLIT,
                  stream=None):
    """In place on x ([n_tokens, n_heads, head_dim] with token stride ld_token elements)."""
    n = pos.numel() if n_tokens is None else n_tokens
    ld = n_heads * head_dim if ld_token is None else ld_token
    _check(lib.sp_rope_apply(x.data_ptr(), pos.data_ptr(), n, ld, n_heads, head_dim,
                             head_dim if rot_dim is None else rot_dim, base, pairing, dtype_code(x),
                             _stream(stream)))


def sp_rope_apply_pair(xq: torch.Tensor, n_heads_q: int, xk: torch.Tensor, n_heads_k: int, pos: torch.Tensor,
                       head_dim: int, *, n_tokens=None, ld_q=None, ld_k=None, rot_dim=None, base: float = 10000.0,
                       pairing: int = SP_ROPE_HALF_SPLIT, stream=None):
    """sp_rope_apply on a step's queries and keys (same positions) in one launch, in place."""
    n = pos.numel() if n_tokens is None else n_tokens
    _check(lib.sp_rope_apply_pair(xq.data_ptr(), n_heads_q * head_dim if ld_q is None else ld_q, n_heads_q,
                                  xk.data_ptr(), n_heads_k * head_dim if ld_k is None else ld_k, n_heads_k,
                                  pos.data_ptr(), n, head_dim, head_dim if rot_dim is None else rot_dim, base,
                                  pairing, dtype_code(xq), _stream(stream)))


def sp_prefill_workspace_bytes(lay: DeviceLayout, n_heads: int, head_dim: int, dtype: int) -> int:
    return int(lib.sp_prefill_workspace_bytes(lay.n_prompts, lay.n_paths, lay.max_pre_len, lay.max_path_len,
                                              n_heads, head_dim, dtype))


def sp_superpose_prefill(q, k, v, lay: DeviceLayout, scale: float, out, lse=None, ws=None,
                         rows: int = SP_ROWS_ALL, stream=None):
    T, H, D = q.shape
    Hkv = k.shape[1]
    _check(lib.sp_superpose_prefill(_ptr(q), _ptr(k), _ptr(v), ctypes.byref(lay.c), H, Hkv, D, scale, rows,
                                    _ptr(out), _ptr(lse), _ptr(ws), _nbytes(ws), dtype_code(q), _stream(stream)))


def sp_superpose_prefill_alibi(q, k, v, lay: DeviceLayout, pos, slopes, scale: float, out, lse=None, ws=None,
                               rows: int = SP_ROWS_ALL, stream=None):
    """sp_superpose_prefill with the ALiBi bias -slopes[h] * |pos[q] - pos[k]| (pos fp32 [T], slopes fp32 [H])."""
    T, H, D = q.shape
    Hkv = k.shape[1]
    _check(lib.sp_superpose_prefill_alibi(_ptr(q), _ptr(k), _ptr(v), ctypes.byref(lay.c), _ptr(pos), _ptr(slopes), H,
                                          Hkv, D, scale, rows, _ptr(out), _ptr(lse), _ptr(ws), _nbytes(ws),
                                          dtype_code(q), _stream(stream)))


def sp_prefill_rope_workspace_bytes(lay: DeviceLayout, n_heads: int, head_dim: int, dtype: int) -> int:
    return int(lib.sp_prefill_rope_workspace_bytes(lay.n_prompts, lay.n_paths, lay.max_pre_len, lay.max_path_len,
                                                   lay.total_tokens, n_heads, head_dim, dtype))


def sp_superpose_prefill_rope(q, k, v, lay: DeviceLayout, pos, base: float, pairing: int, scale: float, out, lse=None,
                              ws=None, stream=None):
    """sp_superpose_prefill over all rows with the rotation of the (unrotated) q folded in; k already rotated."""
    T, H, D = q.shape
    Hkv = k.shape[1]
    _check(lib.sp_superpose_prefill_rope(_ptr(q), _ptr(k), _ptr(v), ctypes.byref(lay.c), _ptr(pos), base, pairing, H,
                                         Hkv, D, scale, _ptr(out), _ptr(lse), _ptr(ws), _nbytes(ws), dtype_code(q),
                                         _stream(stream)))


def sp_path_scores_workspace_bytes(n_rows: int) -> int:
    return int(lib.sp_path_scores_workspace_bytes(n_rows))


def sp_path_scores(logits, targets, row_off, scores, prior=None, weight=None, row_logp=None, ws=None,
                   stream=None):
    R, V = logits.shape
    _check(lib.sp_path_scores(logits.data_ptr(), logits.stride(0) if R else V, _ptr(targets), _ptr(row_off), R,
                              row_off.numel() - 1, V, _ptr(prior), _ptr(weight), _ptr(scores), _ptr(row_logp),
                              _ptr(ws), _nbytes(ws), dtype_code(logits), _stream(stream)))


def sp_prune_topk(scores, prompt_path_off, k: int, kept_idx, kept_post=None, stream=None):
    _check(lib.sp_prune_topk(_ptr(scores), _ptr(prompt_path_off), prompt_path_off.numel() - 1, k,
                             _ptr(kept_idx), _ptr(kept_post), _stream(stream)))


def sp_decode_workspace_bytes(n_prompts: int, n_heads: int, head_dim: int) -> int:
    return int(lib.sp_decode_workspace_bytes(n_prompts, n_heads, head_dim))


def sp_pruned_decode(q, k_cache, v_cache, lay: DeviceLayout, kept_idx, k: int, tail_k, tail_v, tail_len,
                     tail_cap: int, scale: float, out, lse=None, ws=None, max_keys: int = 0, stream=None):
    B, H, D = q.shape
    Hkv = k_cache.shape[1]
    _check(lib.sp_pruned_decode(_ptr(q), _ptr(k_cache), _ptr(v_cache), ctypes.byref(lay.c), _ptr(kept_idx), k,
                                _ptr(tail_k), _ptr(tail_v), _ptr(tail_len), tail_cap, max_keys, H, Hkv, D, scale,
                                _ptr(out), _ptr(lse), _ptr(ws), _nbytes(ws), dtype_code(q), _stream(stream)))


def sp_pruned_decode_alibi(q, k_cache, v_cache, lay: DeviceLayout, kept_idx, k: int, tail_k, tail_v, tail_len,
                           tail_cap: int, q_pos, cache_pos, tail_pos, slopes, scale: float, out, lse=None, ws=None,
                           max_keys: int = 0, stream=None):
    """sp_pruned_decode with the ALiBi bias: q_pos fp32 [B], cache_pos fp32 [T], tail_pos fp32 [B, tail_cap],
    slopes fp32 [H]."""
    B, H, D = q.shape
    Hkv = k_cache.shape[1]
    _check(lib.sp_pruned_decode_alibi(_ptr(q), _ptr(k_cache), _ptr(v_cache), ctypes.byref(lay.c), _ptr(kept_idx), k,
                                      _ptr(tail_k), _ptr(tail_v), _ptr(tail_len), tail_cap, max_keys, _ptr(q_pos),
                                      _ptr(cache_pos), _ptr(tail_pos), _ptr(slopes), H, Hkv, D, scale, _ptr(out),
                                      _ptr(lse), _ptr(ws), _nbytes(ws), dtype_code(q), _stream(stream)))


def sp_pruned_decode_rope(q, k_cache, v_cache, lay: DeviceLayout, kept_idx, k: int, tail_k, tail_v, tail_len,
                          tail_cap: int, q_pos, scale: float, out, lse=None, base: float = 10000.0,
                          pairing: int = SP_ROPE_HALF_SPLIT, max_keys: int = 0, stream=None):
    """One decode step with the rotary embedding folded in: q and the newest tail key row arrive
    unrotated and are rotated at q_pos (fp32 [B]); the key row is written back rotated."""
    B, H, D = q.shape
    Hkv = k_cache.shape[1]
    _check(lib.sp_pruned_decode_rope(_ptr(q), _ptr(k_cache), _ptr(v_cache), ctypes.byref(lay.c), _ptr(kept_idx), k,
                                     _ptr(tail_k), _ptr(tail_v), _ptr(tail_len), tail_cap, max_keys, _ptr(q_pos),
                                     base, pairing, H, Hkv, D, scale, _ptr(out), _ptr(lse), dtype_code(q),
                                     _stream(stream)))


def sp_pruned_decode_static_max_bytes() -> int:
    return int(lib.sp_pruned_decode_static_max_bytes())


def sp_pruned_decode_static(q, k_cache, v_cache, lay: DeviceLayout, kept_idx, k: int, tail_k, tail_v, tail_len,
                            tail_cap: int, scale: float, out, lse=None, max_keys: int = 0, stream=None):
    """sp_pruned_decode for callers that cannot provide a workspace: the split-KV scratch is a
    fixed array inside the library (see include/sp.h for its limit and sharing rules)."""
    B, H, D = q.shape
    Hkv = k_cache.shape[1]
    _check(lib.sp_pruned_decode_static(_ptr(q), _ptr(k_cache), _ptr(v_cache), ctypes.byref(lay.c), _ptr(kept_idx),
                                       k, _ptr(tail_k), _ptr(tail_v), _ptr(tail_len), tail_cap, max_keys, H, Hkv,
                                       D, scale, _ptr(out), _ptr(lse), dtype_code(q), _stream(stream)))


def sp_check_status(ws, stream=None) -> None:
    _check(lib.sp_check_status(_ptr(ws), _stream(stream)))
