"""Thin Python binding of the C ABI in ``include/tailsieve.h``.

Argument marshalling only: every function takes torch CUDA tensors (device
memory) plus sizes, passes raw pointers and the current stream to the shared
library, and raises :class:`TailSieveError` on a non-zero status.  There is no
CPU path and no fallback: without the compiled library, or with tensors that
are not on a CUDA device, the calls fail loudly.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtailsieve.so")

TS_OK = 0
EXPORTED_SYMBOLS = (
    "ts_attn_workspace_bytes", "ts_splitkv_workspace_bytes", "ts_decode_attn", "ts_verify_attn",
    "ts_decode_attn_splitkv", "ts_lse_merge", "ts_accept_workspace_bytes", "ts_accept_greedy",
    "ts_accept_greedy_noalloc", "ts_sample_workspace_bytes", "ts_accept_sample", "ts_accept_sample_penalized", "ts_accept_sample_proposal", "ts_kv_append", "ts_rope_kv_append",
    "ts_set_attn_timing_events", "ts_status_string",
)


class TailSieveError(RuntimeError):
    pass


class ts_attn_params(ctypes.Structure):
    _fields_ = [
        ("num_seqs", ctypes.c_int32), ("q_len", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
        ("num_pages", ctypes.c_int32), ("max_pages_per_seq", ctypes.c_int32),
        ("kv_page_stride", ctypes.c_int64), ("kv_token_stride", ctypes.c_int64),
        ("kv_head_stride", ctypes.c_int64), ("scale", ctypes.c_float),
    ]


_lib = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """dlopen the CUDA library (building it is the job of ``build.py``); raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise TailSieveError(f"{path} not found: build it with `python -m paper_2608_22788_b200.build`")
    lib = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    pp = ctypes.POINTER(ts_attn_params)
    lib.ts_attn_workspace_bytes.restype = sz
    lib.ts_attn_workspace_bytes.argtypes = [pp]
    lib.ts_splitkv_workspace_bytes.restype = sz
    lib.ts_splitkv_workspace_bytes.argtypes = [pp]
    for name in ("ts_decode_attn", "ts_verify_attn"):
        f = getattr(lib, name)
        f.restype = ctypes.c_int
        f.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.ts_decode_attn_splitkv.restype = ctypes.c_int
    lib.ts_decode_attn_splitkv.argtypes = [pp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.ts_lse_merge.restype = ctypes.c_int
    lib.ts_lse_merge.argtypes = [pp, i32, vp, vp, vp, vp, vp]
    lib.ts_accept_workspace_bytes.restype = sz
    lib.ts_accept_workspace_bytes.argtypes = [i32, i32, i32]
    lib.ts_accept_greedy.restype = ctypes.c_int
    lib.ts_accept_greedy.argtypes = [vp, i64, vp, i32, i32, i32, vp, vp, vp, vp, sz, vp]
    lib.ts_accept_greedy_noalloc.restype = ctypes.c_int
    lib.ts_accept_greedy_noalloc.argtypes = [vp, i64, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.ts_sample_workspace_bytes.restype = sz
    lib.ts_sample_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.ts_accept_sample.restype = ctypes.c_int
    lib.ts_accept_sample.argtypes = [vp, i64, vp, vp, i32, i32, i32, ctypes.c_float, i32, ctypes.c_float, vp, vp, vp, sz, vp]
    lib.ts_accept_sample_penalized.restype = ctypes.c_int
    lib.ts_accept_sample_penalized.argtypes = [vp, i64, vp, vp, i32, i32, i32, ctypes.c_float, i32, ctypes.c_float,
                                               ctypes.c_float, vp, i64, vp, vp, vp, sz, vp]
    lib.ts_accept_sample_proposal.restype = ctypes.c_int
    lib.ts_accept_sample_proposal.argtypes = [vp, i64, vp, vp, i64, vp, i32, i32, i32, ctypes.c_float, i32, ctypes.c_float,
                                              ctypes.c_float, vp, i64, vp, vp, vp, sz, vp]
    lib.ts_kv_append.restype = ctypes.c_int
    lib.ts_kv_append.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp]
    lib.ts_rope_kv_append.restype = ctypes.c_int
    lib.ts_rope_kv_append.argtypes = [pp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.ts_set_attn_timing_events.restype = ctypes.c_int
    lib.ts_set_attn_timing_events.argtypes = [vp, vp]
    lib.ts_status_string.restype = ctypes.c_char_p
    lib.ts_status_string.argtypes = [ctypes.c_int]
    if path == LIB_PATH:
        _lib = lib
    return lib


def status_string(code: int) -> str:
    return load_library().ts_status_string(int(code)).decode()


def _check(code: int, what: str) -> None:
    if code != TS_OK:
        raise TailSieveError(f"{what} failed: {status_string(code)} ({code})")


def _ptr(t: Optional[torch.Tensor], what: str) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise TailSieveError(f"{what} must be a CUDA tensor (this library has no CPU path)")
    if not t.is_contiguous():
        raise TailSieveError(f"{what} must be contiguous")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


@dataclass
class AttnGeometry:
    """Shape of one attention call; mirrors ``ts_attn_params`` field by field."""
    num_seqs: int
    q_len: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    kv_page_stride: int
    kv_token_stride: int
    kv_head_stride: int
    scale: float

    def c_struct(self) -> ts_attn_params:
        return ts_attn_params(self.num_seqs, self.q_len, self.num_q_heads, self.num_kv_heads, self.head_dim,
                              self.page_size, self.num_pages, self.max_pages_per_seq, self.kv_page_stride,
                              self.kv_token_stride, self.kv_head_stride, self.scale)


def attn_workspace_bytes(geom: AttnGeometry) -> int:
    p = geom.c_struct()
    return int(load_library().ts_attn_workspace_bytes(ctypes.byref(p)))


def splitkv_workspace_bytes(geom: AttnGeometry) -> int:
    p = geom.c_struct()
    return int(load_library().ts_splitkv_workspace_bytes(ctypes.byref(p)))


def accept_workspace_bytes(num_seqs: int, gamma: int, vocab: int) -> int:
    return int(load_library().ts_accept_workspace_bytes(num_seqs, gamma, vocab))


def _attn_call(name, geom, q, k_pool, v_pool, block_table, kv_lens, out, workspace):
    lib = load_library()
    p = geom.c_struct()
    rc = getattr(lib, name)(ctypes.byref(p), _ptr(q, "q"), _ptr(k_pool, "k_pool"), _ptr(v_pool, "v_pool"),
                            _ptr(block_table, "block_table"), _ptr(kv_lens, "kv_lens"), _ptr(out, "out"),
                            _ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
    _check(rc, name)
    return out


def ts_decode_attn(geom, q, k_pool, v_pool, block_table, kv_lens, out, workspace):
    """Single-token decode attention; ``out`` bf16 ``[B, 1, Hq, D]`` is written and returned."""
    return _attn_call("ts_decode_attn", geom, q, k_pool, v_pool, block_table, kv_lens, out, workspace)


def ts_verify_attn(geom, q, k_pool, v_pool, block_table, kv_lens, out, workspace):
    """Speculative-verify attention (``q_len = 1 + gamma``); ``out`` bf16 ``[B, q_len, Hq, D]``."""
    return _attn_call("ts_verify_attn", geom, q, k_pool, v_pool, block_table, kv_lens, out, workspace)


def ts_decode_attn_splitkv(geom, q, k_pool, v_pool, block_table, kv_lens, max_splits, partial_o, partial_lse,
                           num_splits, workspace):
    """Split-KV attention: fills ``partial_o``, ``partial_lse`` and ``num_splits`` (see the header)."""
    lib = load_library()
    p = geom.c_struct()
    rc = lib.ts_decode_attn_splitkv(ctypes.byref(p), _ptr(q, "q"), _ptr(k_pool, "k_pool"), _ptr(v_pool, "v_pool"),
                                    _ptr(block_table, "block_table"), _ptr(kv_lens, "kv_lens"), int(max_splits),
                                    _ptr(partial_o, "partial_o"), _ptr(partial_lse, "partial_lse"),
                                    _ptr(num_splits, "num_splits"), _ptr(workspace, "workspace"),
                                    workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "ts_decode_attn_splitkv")
    return partial_o, partial_lse, num_splits


def ts_lse_merge(geom, max_splits, partial_o, partial_lse, num_splits, out):
    """Log-sum-exp merge of split results into bf16 ``out``."""
    lib = load_library()
    p = geom.c_struct()
    rc = lib.ts_lse_merge(ctypes.byref(p), int(max_splits), _ptr(partial_o, "partial_o"),
                          _ptr(partial_lse, "partial_lse"), _ptr(num_splits, "num_splits"), _ptr(out, "out"),
                          _stream())
    _check(rc, "ts_lse_merge")
    return out


def ts_accept_greedy(logits, draft, target_argmax, accept_len, out_tokens, workspace, row_stride=None):
    """Greedy draft acceptance over bf16 ``logits [B, gamma+1, V]`` and int32 ``draft [B, gamma]``."""
    lib = load_library()
    B, R, V = logits.shape
    gamma = R - 1
    stride = int(row_stride) if row_stride is not None else int(logits.stride(1))
    rc = lib.ts_accept_greedy(_ptr(logits, "logits"), stride, _ptr(draft, "draft") if gamma > 0 else None,
                              B, gamma, V, _ptr(target_argmax, "target_argmax"), _ptr(accept_len, "accept_len"),
                              _ptr(out_tokens, "out_tokens"), _ptr(workspace, "workspace"),
                              workspace.numel() * workspace.element_size(), _stream())
    _check(rc, "ts_accept_greedy")
    return target_argmax, accept_len, out_tokens


def ts_set_attn_timing_events(start_event: Optional[torch.cuda.Event], stop_event: Optional[torch.cuda.Event]) -> None:
    """Have later attention calls record the two events around their attention kernel (None = off).

    The events must already exist on the device (``torch.cuda.Event(enable_timing=True)`` creates
    its handle lazily: record it once before passing it here).
    """
    lib = load_library()
    a = start_event.cuda_event if start_event is not None else None
    b = stop_event.cuda_event if stop_event is not None else None
    _check(lib.ts_set_attn_timing_events(a, b), "ts_set_attn_timing_events")


def ts_accept_greedy_noalloc(logits, draft, target_argmax, accept_len, out_tokens, row_stride=None):
    """``ts_accept_greedy`` for callers with no scratch to give: same results, no workspace argument.

    The library keeps the intermediate keys in a fixed 512 KB device array of its own, so this call
    works for at most 1024 rows (``B * (gamma + 1)``) and must not overlap on the GPU with another
    call of itself (all calls on a device share that array).  Larger batches raise
    ``TailSieveError`` (TS_ERR_UNSUPPORTED) without launching anything.
    """
    lib = load_library()
    B, R, V = logits.shape
    gamma = R - 1
    stride = int(row_stride) if row_stride is not None else int(logits.stride(1))
    rc = lib.ts_accept_greedy_noalloc(_ptr(logits, "logits"), stride, _ptr(draft, "draft") if gamma > 0 else None,
                                      B, gamma, V, _ptr(target_argmax, "target_argmax"),
                                      _ptr(accept_len, "accept_len"), _ptr(out_tokens, "out_tokens"), _stream())
    _check(rc, "ts_accept_greedy_noalloc")
    return target_argmax, accept_len, out_tokens


def sample_workspace_bytes(num_seqs: int, gamma: int, vocab: int, top_k: int) -> int:
    return int(load_library().ts_sample_workspace_bytes(num_seqs, gamma, vocab, top_k))


def ts_accept_sample(logits, draft, uniforms, accept_len, out_tokens, workspace, *, temperature: float, top_k: int,
                     top_p: float, row_stride=None, presence_penalty: float = 0.0, seen=None, draft_probs=None):
    """Lossless draft acceptance under temperature / top-k / top-p sampling (see the header).

    With ``presence_penalty`` (and optionally ``seen``, a uint8 bitmap ``[B, >= V/8]`` of the tokens
    each sequence has generated so far) the call goes through ``ts_accept_sample_penalized``; with
    ``draft_probs`` (float32 ``[B, gamma, >= V]``, the distributions the drafts were sampled from)
    through ``ts_accept_sample_proposal``.
    """
    lib = load_library()
    B, R, V = logits.shape
    gamma = R - 1
    stride = int(row_stride) if row_stride is not None else int(logits.stride(1))
    if draft_probs is not None:
        if draft_probs.dtype != torch.float32 or draft_probs.dim() != 3 or draft_probs.shape[0] != B \
                or draft_probs.shape[1] != gamma or draft_probs.stride(2) != 1:
            raise TailSieveError("draft_probs must be float32 [num_seqs, gamma, vocab] with unit inner stride")
        if gamma > 1 and draft_probs.stride(0) != gamma * draft_probs.stride(1):
            raise TailSieveError("draft_probs rows must be evenly strided")
        seen_stride = 0
        if seen is not None:
            if seen.dtype != torch.uint8 or seen.dim() != 2 or seen.shape[0] != B:
                raise TailSieveError("seen must be a uint8 bitmap [num_seqs, bytes]")
            seen_stride = int(seen.stride(0))
        q_stride = int(draft_probs.stride(1)) if gamma > 0 else V
        rc = lib.ts_accept_sample_proposal(_ptr(logits, "logits"), stride, _ptr(draft, "draft") if gamma > 0 else None,
                                           _ptr(draft_probs, "draft_probs") if gamma > 0 else None, q_stride,
                                           _ptr(uniforms, "uniforms"), B, gamma, V, float(temperature), int(top_k),
                                           float(top_p), float(presence_penalty), _ptr(seen, "seen"), seen_stride,
                                           _ptr(accept_len, "accept_len"), _ptr(out_tokens, "out_tokens"),
                                           _ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                           _stream())
        _check(rc, "ts_accept_sample_proposal")
        return accept_len, out_tokens
    if presence_penalty == 0.0 and seen is None:
        rc = lib.ts_accept_sample(_ptr(logits, "logits"), stride, _ptr(draft, "draft") if gamma > 0 else None,
                                  _ptr(uniforms, "uniforms"), B, gamma, V, float(temperature), int(top_k), float(top_p),
                                  _ptr(accept_len, "accept_len"), _ptr(out_tokens, "out_tokens"),
                                  _ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream())
        _check(rc, "ts_accept_sample")
        return accept_len, out_tokens
    seen_stride = 0
    if seen is not None:
        if seen.dtype != torch.uint8 or seen.dim() != 2 or seen.shape[0] != B:
            raise TailSieveError("seen must be a uint8 bitmap [num_seqs, bytes]")
        seen_stride = int(seen.stride(0))
    rc = lib.ts_accept_sample_penalized(_ptr(logits, "logits"), stride, _ptr(draft, "draft") if gamma > 0 else None,
                                        _ptr(uniforms, "uniforms"), B, gamma, V, float(temperature), int(top_k),
                                        float(top_p), float(presence_penalty), _ptr(seen, "seen"), seen_stride,
                                        _ptr(accept_len, "accept_len"), _ptr(out_tokens, "out_tokens"),
                                        _ptr(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                        _stream())
    _check(rc, "ts_accept_sample_penalized")
    return accept_len, out_tokens


def ts_kv_append(geom, new_k, new_v, k_pool, v_pool, block_table, kv_lens):
    """Write this step's K/V rows ``[B, q_len, Hkv, D]`` into the paged pools (before attention)."""
    lib = load_library()
    p = geom.c_struct()
    rc = lib.ts_kv_append(ctypes.byref(p), _ptr(new_k, "new_k"), _ptr(new_v, "new_v"), _ptr(k_pool, "k_pool"),
                          _ptr(v_pool, "v_pool"), _ptr(block_table, "block_table"), _ptr(kv_lens, "kv_lens"), _stream())
    _check(rc, "ts_kv_append")


def ts_rope_kv_append(geom, q_in, q_out, new_k, new_v, k_pool, v_pool, block_table, kv_lens, inv_freq):
    """Rotate this step's Q rows (into ``q_out``) and K rows with the rotary embedding of their
    positions, and write the rotated K and the V rows into the paged pools (before attention)."""
    lib = load_library()
    p = geom.c_struct()
    rc = lib.ts_rope_kv_append(ctypes.byref(p), _ptr(q_in, "q_in"), _ptr(q_out, "q_out"), _ptr(new_k, "new_k"),
                               _ptr(new_v, "new_v"), _ptr(k_pool, "k_pool"), _ptr(v_pool, "v_pool"),
                               _ptr(block_table, "block_table"), _ptr(kv_lens, "kv_lens"), _ptr(inv_freq, "inv_freq"),
                               _stream())
    _check(rc, "ts_rope_kv_append")
