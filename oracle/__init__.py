"""fp64 CPU oracle for prefix+suffix scoring (ctypes front end of ``rpx_oracle.c``).

TEST INFRASTRUCTURE ONLY.  Callers are the tests, the smoke check and the benchmark's
CPU-baseline / reference legs.  Nothing in the product package imports this module and this
module imports nothing from the product package.

Arrays are numpy: bf16 tensors are carried as ``uint16`` bit patterns, fp32 tensors as
``float32``; results come back as ``float64``.  What each routine computes, and the passages of
the paper it follows, are stated at the top of ``rpx_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "rpx_oracle.c")
_LIB = os.path.join(_HERE, "librpx_oracle.so")
_lock = threading.Lock()
_lib = None

BF16, F32 = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc + OpenMP next to its source; returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + f".tmp{os.getpid()}"
            subprocess.check_call(
                ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32, i64, dbl, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_double, ctypes.c_void_p
        lib.rpx_oracle_num_threads.restype = ctypes.c_int
        lib.rpx_oracle_attn_rows.restype = ctypes.c_int
        lib.rpx_oracle_attn_rows.argtypes = [vp, vp, vp, ctypes.c_int, i64, i64, i64, vp, i32, i32, i32,
                                             i32, dbl, vp, i64, vp, vp]
        lib.rpx_oracle_logprob_rows.restype = ctypes.c_int
        lib.rpx_oracle_logprob_rows.argtypes = [vp, i64, vp, ctypes.c_int, vp, vp, i64, i32, i32, vp, vp]
        lib.rpx_oracle_entropy_rows.restype = ctypes.c_int
        lib.rpx_oracle_entropy_rows.argtypes = [vp, i64, vp, ctypes.c_int, vp, i64, i32, i32, vp]
        lib.rpx_oracle_slot.restype = i64
        lib.rpx_oracle_slot.argtypes = [vp, i32, i32, i32, i32]
        lib.rpx_oracle_cache_image.restype = ctypes.c_int
        lib.rpx_oracle_cache_image.argtypes = [vp, vp, ctypes.c_int, i64, i64, vp, i32, i32, i32, vp, i32,
                                               i32, i64, vp, vp]
        lib.rpx_oracle_logprob_backward.restype = ctypes.c_int
        lib.rpx_oracle_logprob_backward.argtypes = [vp, i64, vp, ctypes.c_int, vp, vp, i64, i32, i32, vp, vp]
        lib.rpx_oracle_attn_backward.restype = ctypes.c_int
        lib.rpx_oracle_attn_backward.argtypes = [vp, vp, vp, ctypes.c_int, i64, i64, i64, vp, i32, i32, i32, i32, dbl,
                                                 vp, vp, vp, vp]
        _lib = lib
    return _lib


def num_threads() -> int:
    """Threads the OpenMP loops will use (what the CPU baseline reports as ``cores``)."""
    return int(_load().rpx_oracle_num_threads())


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.uint16:
        return BF16
    if a.dtype == np.float32:
        return F32
    raise TypeError(f"oracle takes uint16 (bf16 bits) or float32 arrays, got {a.dtype}")


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _tok_stride(a: np.ndarray) -> int:
    """Token stride in elements of a [tokens, heads, d] array whose heads are contiguous."""
    assert a.ndim == 3 and a.strides[2] == a.itemsize and a.strides[1] == a.shape[2] * a.itemsize
    return a.strides[0] // a.itemsize


def attn_rows(q, k, v, cu_seqlens, rows, scale=None):
    """Monolithic causal GQA attention rows.

    q [T, H_q, d], k/v [T, H_kv, d]: whole sequences (prompt then response) packed by
    ``cu_seqlens`` (int32 [B+1]).  ``rows`` is int32 [n, 3] of (sequence, position, query head).
    Returns (out float64 [n, d], lse float64 [n]).
    """
    lib = _load()
    code = _dtype_code(q)
    assert _dtype_code(k) == code and _dtype_code(v) == code
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    rows = np.ascontiguousarray(rows, dtype=np.int32).reshape(-1, 3)
    hq, d = q.shape[1], q.shape[2]
    hkv = k.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    out = np.empty((rows.shape[0], d), dtype=np.float64)
    lse = np.empty((rows.shape[0],), dtype=np.float64)
    rc = lib.rpx_oracle_attn_rows(_ptr(q), _ptr(k), _ptr(v), code, _tok_stride(q), _tok_stride(k),
                                  _tok_stride(v), _ptr(cu), cu.shape[0] - 1, hq, hkv, d, float(scale),
                                  _ptr(rows), rows.shape[0], _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError(f"rpx_oracle_attn_rows failed with {rc}")
    return out, lse


def all_rows(cu_seqlens, num_q_heads: int) -> np.ndarray:
    """Every (sequence, position, head) triple of a packed batch, token-major then head."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    trip = []
    for s in range(cu.shape[0] - 1):
        n = int(cu[s + 1] - cu[s])
        pos = np.repeat(np.arange(n, dtype=np.int32), num_q_heads)
        hd = np.tile(np.arange(num_q_heads, dtype=np.int32), n)
        trip.append(np.stack([np.full_like(pos, s), pos, hd], axis=1))
    return np.concatenate(trip, axis=0) if trip else np.zeros((0, 3), np.int32)


def logprob_rows(hidden, w, target_ids, rows=None):
    """Monolithic log-softmax + gather.  hidden [N, H], w [V, H], target_ids int32 [N].

    ``rows`` (int64 row numbers) defaults to every row.  Returns (logprob, lse) float64 [n].
    """
    lib = _load()
    code = _dtype_code(hidden)
    assert _dtype_code(w) == code
    assert hidden.ndim == 2 and w.ndim == 2 and hidden.shape[1] == w.shape[1]
    assert hidden.strides[1] == hidden.itemsize and w.flags.c_contiguous
    ids = np.ascontiguousarray(target_ids, dtype=np.int32)
    if rows is None:
        rows = np.arange(hidden.shape[0], dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    lp = np.empty((rows.shape[0],), dtype=np.float64)
    lse = np.empty((rows.shape[0],), dtype=np.float64)
    rc = lib.rpx_oracle_logprob_rows(_ptr(hidden), hidden.strides[0] // hidden.itemsize, _ptr(w), code,
                                     _ptr(ids), _ptr(rows), rows.shape[0], hidden.shape[1], w.shape[0],
                                     _ptr(lp), _ptr(lse))
    if rc != 0:
        raise MemoryError(f"rpx_oracle_logprob_rows failed with {rc}")
    return lp, lse


def entropy_rows(hidden, w, rows=None):
    """Entropy (nats) of softmax(hidden[n] . w^T) per row, from the definition -sum p ln p in fp64."""
    lib = _load()
    code = _dtype_code(hidden)
    assert _dtype_code(w) == code and hidden.ndim == 2 and w.ndim == 2 and hidden.shape[1] == w.shape[1]
    assert hidden.strides[1] == hidden.itemsize and w.flags.c_contiguous
    if rows is None:
        rows = np.arange(hidden.shape[0], dtype=np.int64)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    ent = np.empty((rows.shape[0],), dtype=np.float64)
    rc = lib.rpx_oracle_entropy_rows(_ptr(hidden), hidden.strides[0] // hidden.itemsize, _ptr(w), code, _ptr(rows),
                                     rows.shape[0], hidden.shape[1], w.shape[0], _ptr(ent))
    if rc != 0:
        raise MemoryError(f"rpx_oracle_entropy_rows failed with {rc}")
    return ent


def slot(block_table, s: int, t: int, block_size: int = 16) -> int:
    """Physical cache slot of prefix position ``t`` of sequence ``s``."""
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    return int(_load().rpx_oracle_slot(_ptr(bt), bt.shape[1], int(s), int(t), int(block_size)))


def cache_image(k, v, cu_seqlens, block_table, num_blocks: int, block_size: int = 16, sentinel: int = 0x7FC1):
    """Expected (k_cache, v_cache) uint16 [num_blocks, H_kv, block_size, d] after the prefix pass.

    Slots no prefix token maps to keep ``sentinel``.  k/v are the PREFIX-packed tensors.
    """
    lib = _load()
    code = _dtype_code(k)
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    bt = np.ascontiguousarray(block_table, dtype=np.int32)
    hkv, d = k.shape[1], k.shape[2]
    kc = np.full((num_blocks, hkv, block_size, d), sentinel, dtype=np.uint16)
    vc = np.full((num_blocks, hkv, block_size, d), sentinel, dtype=np.uint16)
    rc = lib.rpx_oracle_cache_image(_ptr(k), _ptr(v), code, _tok_stride(k), _tok_stride(v), _ptr(cu),
                                    cu.shape[0] - 1, hkv, d, _ptr(bt), bt.shape[1], block_size, num_blocks,
                                    _ptr(kc), _ptr(vc))
    if rc != 0:
        raise ValueError(f"rpx_oracle_cache_image failed with {rc}")
    return kc, vc


def logprob_backward(hidden, w, target_ids, upstream, want_dw: bool = False):
    """Gradient of sum_n upstream[n] * logprob[n] with respect to hidden (and to w when asked), from the definition
    dL/dz = upstream * (onehot(target) - softmax(z)) in fp64.  hidden [N, H], w [V, H], target_ids int32 [N],
    upstream float64 [N].  Returns dhidden float64 [N, H] (and dw float64 [V, H])."""
    lib = _load()
    code = _dtype_code(hidden)
    assert _dtype_code(w) == code and hidden.ndim == 2 and w.ndim == 2 and hidden.shape[1] == w.shape[1]
    assert hidden.strides[1] == hidden.itemsize and w.flags.c_contiguous
    ids = np.ascontiguousarray(target_ids, dtype=np.int32)
    g = np.ascontiguousarray(upstream, dtype=np.float64)
    n, hdim = hidden.shape
    assert ids.shape == (n,) and g.shape == (n,)
    dh = np.empty((n, hdim), dtype=np.float64)
    dw = np.empty((w.shape[0], hdim), dtype=np.float64) if want_dw else None
    rc = lib.rpx_oracle_logprob_backward(_ptr(hidden), hidden.strides[0] // hidden.itemsize, _ptr(w), code, _ptr(ids),
                                         _ptr(g), n, hdim, w.shape[0], _ptr(dh), _ptr(dw) if want_dw else None)
    if rc != 0:
        raise MemoryError(f"rpx_oracle_logprob_backward failed with {rc}")
    return (dh, dw) if want_dw else dh


def attn_backward(q, k, v, cu_seqlens, dout, scale=None):
    """Gradients of sum(dout * O) for monolithic causal GQA attention over whole sequences (prompt then response).
    q [T, H_q, d], k/v [T, H_kv, d] packed by cu_seqlens; dout float64 [T, H_q, d].
    Returns (dq [T, H_q, d], dk [T, H_kv, d], dv [T, H_kv, d]) in float64."""
    lib = _load()
    code = _dtype_code(q)
    assert _dtype_code(k) == code and _dtype_code(v) == code
    cu = np.ascontiguousarray(cu_seqlens, dtype=np.int32)
    hq, d = q.shape[1], q.shape[2]
    hkv = k.shape[1]
    total = int(cu[-1])
    assert q.shape[0] == total and k.shape[0] == total and v.shape[0] == total
    do = np.ascontiguousarray(dout, dtype=np.float64)
    assert do.shape == (total, hq, d)
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    dq = np.empty((total, hq, d), dtype=np.float64)
    dk = np.empty((total, hkv, d), dtype=np.float64)
    dv = np.empty((total, hkv, d), dtype=np.float64)
    rc = lib.rpx_oracle_attn_backward(_ptr(q), _ptr(k), _ptr(v), code, _tok_stride(q), _tok_stride(k), _tok_stride(v),
                                      _ptr(cu), cu.shape[0] - 1, hq, hkv, d, float(scale), _ptr(do), _ptr(dq), _ptr(dk),
                                      _ptr(dv))
    if rc != 0:
        raise ValueError(f"rpx_oracle_attn_backward failed with {rc}")
    return dq, dk, dv
