"""CPU fp64 oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Thin ctypes front end for ``ts_oracle.c`` (plain C, fp64, OpenMP over
(sequence, head)).  Only ``tests/``, the smoke check and the benchmark's
CPU-baseline leg may import this package; the CUDA library and its Python
binding never do, and share no code with it.

The C file is compiled on first use (``gcc -O2 -fopenmp -shared``) into
``oracle/libts_oracle.so``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ts_oracle.c")
_LIB = os.path.join(_HERE, "libts_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle's C file if the shared object is missing or stale."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c_i32p = ctypes.POINTER(ctypes.c_int32)
        c_u16p = ctypes.POINTER(ctypes.c_uint16)
        c_f64p = ctypes.POINTER(ctypes.c_double)
        lib.ora_paged_attention.restype = ctypes.c_int
        lib.ora_paged_attention.argtypes = [
            c_u16p, c_u16p, c_u16p, c_i32p, c_i32p, c_i32p, c_i32p,
            ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_double, c_f64p, c_f64p, ctypes.c_int]
        lib.ora_lse_merge.restype = ctypes.c_int
        lib.ora_lse_merge.argtypes = [c_f64p, c_f64p, c_i32p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                      ctypes.c_int, c_f64p, c_f64p]
        lib.ora_accept_greedy.restype = ctypes.c_int
        lib.ora_accept_greedy.argtypes = [c_u16p, ctypes.c_int64, c_i32p, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, c_i32p, c_i32p, c_i32p, ctypes.c_int]
        lib.ora_accept_sample.restype = ctypes.c_int
        lib.ora_accept_sample.argtypes = [c_u16p, ctypes.c_int64, c_i32p, c_f64p, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_double,
                                          c_i32p, c_i32p, c_i32p, c_f64p, ctypes.POINTER(ctypes.c_uint8),
                                          ctypes.c_int64, ctypes.c_double, ctypes.POINTER(ctypes.c_float),
                                          ctypes.c_int64]
        lib.ora_rope.restype = ctypes.c_int
        lib.ora_rope.argtypes = [c_u16p, ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_float),
                                 ctypes.c_int64, ctypes.c_int, ctypes.c_int, c_f64p]
        lib.ora_max_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray], ctype):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def max_threads() -> int:
    return int(_load().ora_max_threads())


def paged_attention(q, k_pool, v_pool, block_table, kv_lens, *, num_kv_heads: int, page_size: int,
                    kv_page_stride: int, kv_token_stride: int, kv_head_stride: int, scale: float,
                    key_begin=None, key_end=None, nthreads: int = 0):
    """fp64 attention over a paged cache.

    ``q``: uint16 bf16 bits ``[B, q_len, Hq, D]``; pools: uint16, any shape, addressed through
    the three strides (in elements).  Returns ``(out [B,q_len,Hq,D], lse [B,q_len,Hq])`` as
    float64.  ``key_begin``/``key_end`` (int32 ``[B]``) restrict the key set per sequence.
    """
    lib = _load()
    q = np.ascontiguousarray(q, dtype=np.uint16)
    k_pool = np.ascontiguousarray(k_pool, dtype=np.uint16)
    v_pool = np.ascontiguousarray(v_pool, dtype=np.uint16)
    block_table = np.ascontiguousarray(block_table, dtype=np.int32)
    kv_lens = np.ascontiguousarray(kv_lens, dtype=np.int32)
    B, q_len, Hq, D = q.shape
    assert block_table.ndim == 2 and block_table.shape[0] == B
    kb = None if key_begin is None else np.ascontiguousarray(key_begin, dtype=np.int32)
    ke = None if key_end is None else np.ascontiguousarray(key_end, dtype=np.int32)
    out = np.empty((B, q_len, Hq, D), dtype=np.float64)
    lse = np.empty((B, q_len, Hq), dtype=np.float64)
    rc = lib.ora_paged_attention(
        _p(q, ctypes.c_uint16), _p(k_pool, ctypes.c_uint16), _p(v_pool, ctypes.c_uint16),
        _p(block_table, ctypes.c_int32), _p(kv_lens, ctypes.c_int32), _p(kb, ctypes.c_int32),
        _p(ke, ctypes.c_int32), B, q_len, Hq, num_kv_heads, D, page_size, block_table.shape[1],
        kv_page_stride, kv_token_stride, kv_head_stride, float(scale),
        _p(out, ctypes.c_double), _p(lse, ctypes.c_double), int(nthreads))
    if rc != 0:
        raise RuntimeError(f"ora_paged_attention failed ({rc})")
    return out, lse


def attention_batch(batch, key_begin=None, key_end=None, nthreads: int = 0, seqs=None):
    """Run :func:`paged_attention` on a ``workloads.AttnBatch`` (optionally a subset of sequences)."""
    q, bt, lens = batch.q, batch.block_table, batch.kv_lens
    if seqs is not None:
        seqs = np.asarray(seqs, dtype=np.int64)
        q, bt, lens = q[seqs], bt[seqs], lens[seqs]
    return paged_attention(q, batch.k_pool, batch.v_pool, bt, lens,
                           num_kv_heads=batch.num_kv_heads, page_size=batch.page_size,
                           kv_page_stride=batch.kv_page_stride, kv_token_stride=batch.kv_token_stride,
                           kv_head_stride=batch.kv_head_stride, scale=batch.scale,
                           key_begin=key_begin, key_end=key_end, nthreads=nthreads)


def lse_merge(partial_o, partial_lse, num_splits):
    """Merge ``partial_o [B,S,R,D]`` / ``partial_lse [B,S,R]`` (any float dtype; promoted to fp64)."""
    lib = _load()
    po = np.ascontiguousarray(partial_o, dtype=np.float64)
    pl = np.ascontiguousarray(partial_lse, dtype=np.float64)
    ns = np.ascontiguousarray(num_splits, dtype=np.int32)
    B, S, R, D = po.shape
    assert pl.shape == (B, S, R) and ns.shape == (B,)
    out = np.empty((B, R, D), dtype=np.float64)
    out_lse = np.empty((B, R), dtype=np.float64)
    rc = lib.ora_lse_merge(_p(po, ctypes.c_double), _p(pl, ctypes.c_double), _p(ns, ctypes.c_int32),
                           B, S, R, D, _p(out, ctypes.c_double), _p(out_lse, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ora_lse_merge failed ({rc})")
    return out, out_lse


def accept_greedy(logits, draft, nthreads: int = 0):
    """Greedy draft acceptance.  ``logits``: uint16 bf16 bits ``[B, gamma+1, V]``; ``draft``: int
    ``[B, gamma]``.  Returns ``(target_argmax [B,gamma+1], accept_len [B], out_tokens [B,gamma+1])``."""
    lib = _load()
    logits = np.ascontiguousarray(logits, dtype=np.uint16)
    B, R, V = logits.shape
    gamma = R - 1
    draft = np.ascontiguousarray(draft, dtype=np.int32).reshape(B, gamma)
    tgt = np.empty((B, R), dtype=np.int32)
    acc = np.empty((B,), dtype=np.int32)
    out = np.empty((B, R), dtype=np.int32)
    rc = lib.ora_accept_greedy(_p(logits, ctypes.c_uint16), V, _p(draft, ctypes.c_int32), B, gamma, V,
                               _p(tgt, ctypes.c_int32), _p(acc, ctypes.c_int32), _p(out, ctypes.c_int32),
                               int(nthreads))
    if rc != 0:
        raise RuntimeError(f"ora_accept_greedy failed ({rc})")
    return tgt, acc, out


def accept_sample(logits, draft, uniforms, *, temperature: float, top_k: int, top_p: float,
                  seen=None, presence_penalty: float = 0.0, draft_probs=None):
    """Lossless acceptance under temperature / top-k / top-p sampling; drafts are point proposals
    unless ``draft_probs`` (float32 ``[B, gamma, V]``, the distributions they were drawn from) is given.

    ``logits``: uint16 bf16 bits ``[B, gamma+1, V]``; ``draft``: int ``[B, gamma]``; ``uniforms``:
    float ``[B, gamma+1, 2]`` in [0, 1).  Returns ``(accept_len [B], out_tokens [B,gamma+1],
    kept_ids [B,gamma+1,top_k], kept_p [B,gamma+1,top_k])``.

    ``seen``: optional uint8 bitmap ``[B, >= ceil(V/8)]`` (bit ``v & 7`` of byte ``v >> 3``) of the
    tokens each sequence has generated so far; with ``presence_penalty`` their logits, and those of
    the earlier drafts of the block, are lowered by the penalty before the top-k selection.
    """
    lib = _load()
    logits = np.ascontiguousarray(logits, dtype=np.uint16)
    B, R, V = logits.shape
    gamma = R - 1
    draft = np.ascontiguousarray(draft, dtype=np.int32).reshape(B, gamma)
    u = np.ascontiguousarray(uniforms, dtype=np.float64).reshape(B, R, 2)
    sb, sstride = None, 0
    if seen is not None:
        sb = np.ascontiguousarray(seen, dtype=np.uint8)
        assert sb.ndim == 2 and sb.shape[0] == B and sb.shape[1] * 8 >= V
        sstride = sb.shape[1]
    qd, qstride = None, 0
    if draft_probs is not None:
        qd = np.ascontiguousarray(draft_probs, dtype=np.float32)
        assert qd.shape == (B, gamma, V)
        qstride = V
    acc = np.empty((B,), dtype=np.int32)
    out = np.empty((B, R), dtype=np.int32)
    ids = np.empty((B, R, top_k), dtype=np.int32)
    pp = np.empty((B, R, top_k), dtype=np.float64)
    rc = lib.ora_accept_sample(_p(logits, ctypes.c_uint16), V, _p(draft, ctypes.c_int32), _p(u, ctypes.c_double),
                               B, gamma, V, float(temperature), int(top_k), float(top_p),
                               _p(acc, ctypes.c_int32), _p(out, ctypes.c_int32), _p(ids, ctypes.c_int32),
                               _p(pp, ctypes.c_double), _p(sb, ctypes.c_uint8), int(sstride), float(presence_penalty),
                               _p(qd, ctypes.c_float), int(qstride))
    if rc != 0:
        raise RuntimeError(f"ora_accept_sample failed ({rc})")
    return acc, out, ids, pp


def rope(x, pos, inv_freq):
    """Rotary position embedding ("rotate-half" pairing) of bf16 rows.

    ``x``: uint16 bf16 bits ``[rows, heads, D]``; ``pos``: int ``[rows]``; ``inv_freq``: float32
    ``[D/2]``.  Returns float64 ``[rows, heads, D]`` (not rounded).
    """
    lib = _load()
    x = np.ascontiguousarray(x, dtype=np.uint16)
    rows, heads, D = x.shape
    pos = np.ascontiguousarray(pos, dtype=np.int64).reshape(rows)
    f = np.ascontiguousarray(inv_freq, dtype=np.float32).reshape(D // 2)
    out = np.empty((rows, heads, D), dtype=np.float64)
    rc = lib.ora_rope(_p(x, ctypes.c_uint16), _p(pos, ctypes.c_int64), _p(f, ctypes.c_float), rows, heads, D,
                      _p(out, ctypes.c_double))
    if rc != 0:
        raise RuntimeError(f"ora_rope failed ({rc})")
    return out
