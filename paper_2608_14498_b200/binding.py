"""ctypes binding of ``librpx.so`` (the C ABI declared in ``include/rpx.h``).

Only argument marshalling happens here: torch tensors supply device pointers and the current
stream; every step of the scoring path runs inside the CUDA library.  If the library is missing
the functions raise — there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "librpx.so")
_lib = None

RPX_BF16, RPX_F32 = 0, 1
BLOCK_SIZE = 16
STATIC_SCRATCH_BYTES = 8 << 20

EXPORTS = (
    "rpx_prefix_attn",
    "rpx_suffix_attn",
    "rpx_chunk_attn",
    "rpx_token_logprobs",
    "rpx_token_logprobs_entropy",
    "rpx_token_logprobs_shard",
    "rpx_token_logprobs_merge",
    "rpx_token_logprobs_static",
    "rpx_token_logprobs_backward",
    "rpx_token_logprobs_backward_full",
    "rpx_token_logprobs_backward_workspace_bytes",
    "rpx_set_lm_head_pairing",
    "rpx_get_lm_head_pairing",
    "rpx_attn_backward",
    "rpx_attn_backward_workspace_bytes",
    "rpx_prefix_attn_workspace_bytes",
    "rpx_suffix_attn_workspace_bytes",
    "rpx_token_logprobs_workspace_bytes",
    "rpx_selftest_bounded_wait",
    "rpx_set_sm_budget",
    "rpx_get_sm_budget",
    "rpx_status_string",
    "rpx_version",
)


class RpxError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class AttnDesc(ctypes.Structure):
    _fields_ = [
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float),
        ("dtype", ctypes.c_int32),
    ]


class KvCache(ctypes.Structure):
    _fields_ = [
        ("k_cache", ctypes.c_void_p),
        ("v_cache", ctypes.c_void_p),
        ("num_blocks", ctypes.c_int64),
        ("block_size", ctypes.c_int32),
        ("block_table", ctypes.c_void_p),
        ("block_table_stride", ctypes.c_int32),
    ]


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load librpx.so (built in-tree by ``paper_2608_14498_b200.build``); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2608_14498_b200.build` "
            "(there is no CPU or eager fallback)"
        )
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.rpx_prefix_attn.restype = i32
    lib.rpx_prefix_attn.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, i64, i64, i64, vp, i32, i64, i32,
                                    ctypes.POINTER(KvCache), vp, vp, vp, sz, vp, vp]
    lib.rpx_suffix_attn.restype = i32
    lib.rpx_suffix_attn.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, i64, i64, i64, vp, vp, i32, i64, i32,
                                    i32, ctypes.POINTER(KvCache), vp, vp, vp, sz, vp, vp]
    lib.rpx_chunk_attn.restype = i32
    lib.rpx_chunk_attn.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, i64, i64, i64, vp, vp, i32, i64, i32,
                                    i32, ctypes.POINTER(KvCache), vp, vp, vp, sz, vp, vp]
    lib.rpx_token_logprobs.restype = i32
    lib.rpx_token_logprobs.argtypes = [vp, i64, vp, vp, i64, i32, i32, i32, vp, vp, vp, sz, vp, vp]
    lib.rpx_token_logprobs_entropy.restype = i32
    lib.rpx_token_logprobs_entropy.argtypes = [vp, i64, vp, vp, i64, i32, i32, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.rpx_token_logprobs_shard.restype = i32
    lib.rpx_token_logprobs_shard.argtypes = [vp, i64, vp, vp, i64, i32, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.rpx_token_logprobs_merge.restype = i32
    lib.rpx_token_logprobs_merge.argtypes = [vp, i32, vp, i64, i32, vp, vp, vp, vp, vp]
    lib.rpx_token_logprobs_static.restype = i32
    lib.rpx_token_logprobs_static.argtypes = [vp, i64, vp, vp, i64, i32, i32, vp, vp, vp, vp]
    lib.rpx_token_logprobs_backward.restype = i32
    lib.rpx_token_logprobs_backward.argtypes = [vp, i64, vp, vp, vp, vp, i64, i32, i32, i32, vp, vp, sz, vp, vp]
    lib.rpx_token_logprobs_backward_full.restype = i32
    lib.rpx_token_logprobs_backward_full.argtypes = [vp, i64, vp, vp, vp, vp, i64, i32, i32, i32, vp, vp, i32, vp, sz, vp, vp]
    lib.rpx_token_logprobs_backward_workspace_bytes.restype = sz
    lib.rpx_token_logprobs_backward_workspace_bytes.argtypes = [i64, i32, i32, i32]
    lib.rpx_attn_backward.restype = i32
    lib.rpx_attn_backward.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, i64, i64, i64, vp, vp, vp, vp, vp, vp, i32,
                                      i64, i32, vp, vp, vp, i32, vp, sz, vp, vp]
    lib.rpx_attn_backward_workspace_bytes.restype = sz
    lib.rpx_attn_backward_workspace_bytes.argtypes = [ctypes.POINTER(AttnDesc), i64]
    lib.rpx_prefix_attn_workspace_bytes.restype = sz
    lib.rpx_prefix_attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnDesc), i64]
    lib.rpx_suffix_attn_workspace_bytes.restype = sz
    lib.rpx_suffix_attn_workspace_bytes.argtypes = [ctypes.POINTER(AttnDesc), i64]
    lib.rpx_token_logprobs_workspace_bytes.restype = sz
    lib.rpx_token_logprobs_workspace_bytes.argtypes = [i64, i32, i32, i32]
    lib.rpx_selftest_bounded_wait.restype = i32
    lib.rpx_selftest_bounded_wait.argtypes = [i64, vp, vp]
    lib.rpx_set_sm_budget.restype = i32
    lib.rpx_set_sm_budget.argtypes = [i32]
    lib.rpx_get_sm_budget.restype = i32
    lib.rpx_get_sm_budget.argtypes = []
    lib.rpx_set_lm_head_pairing.restype = i32
    lib.rpx_set_lm_head_pairing.argtypes = [i32]
    lib.rpx_get_lm_head_pairing.restype = i32
    lib.rpx_get_lm_head_pairing.argtypes = []
    lib.rpx_status_string.restype = ctypes.c_char_p
    lib.rpx_status_string.argtypes = [i32]
    lib.rpx_version.restype = i32
    lib.rpx_version.argtypes = []
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load_library().rpx_status_string(int(status)).decode()


def version() -> int:
    return int(load_library().rpx_version())


# ------------------------------------------------------------------ helpers (torch side)
def _torch():
    import torch

    return torch


def _dtype_code(t) -> int:
    torch = _torch()
    if t.dtype == torch.bfloat16:
        return RPX_BF16
    if t.dtype == torch.float32:
        return RPX_F32
    raise TypeError(f"rpx tensors are bfloat16 or float32, got {t.dtype}")


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_ptr(stream) -> int:
    torch = _torch()
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _tok_stride(t) -> int:
    if t.dim() != 3:
        raise ValueError("expected a [tokens, heads, head_dim] tensor")
    if t.shape[0] <= 1:
        return t.shape[1] * t.shape[2]
    if t.stride(2) != 1 or t.stride(1) != t.shape[2]:
        raise ValueError("expected a [tokens, heads, head_dim] tensor with contiguous heads")
    return t.stride(0)


def _workspace(nbytes: int, device, workspace):
    torch = _torch()
    if workspace is not None:
        if workspace.numel() * workspace.element_size() < nbytes:
            raise ValueError(f"workspace too small: need {nbytes} bytes")
        return workspace
    return torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)


def _in_call_context(fn):
    """Runs a wrapper with its first tensor's device current (the library launches on the current device) and,
    when ``stream=`` is given, with that stream current, so that outputs and temporary workspaces the wrapper
    allocates belong to the stream the kernels run on."""
    import functools

    @functools.wraps(fn)
    def call(*args, **kwargs):
        torch = _torch()
        first = args[0] if args else next(iter(kwargs.values()))
        stream = kwargs.get("stream")
        with torch.cuda.device(first.device):
            if stream is None:
                return fn(*args, **kwargs)
            with torch.cuda.stream(stream):
                return fn(*args, **kwargs)
    return call


def _desc(q, k, softmax_scale: float) -> AttnDesc:
    return AttnDesc(q.shape[1], k.shape[1], q.shape[2], float(softmax_scale), _dtype_code(q))


def _cache_struct(cache) -> KvCache:
    k_cache, v_cache, block_table = cache
    torch = _torch()
    if k_cache.dtype != torch.bfloat16 or v_cache.dtype != torch.bfloat16 or block_table.dtype != torch.int32:
        raise TypeError("cache pools are bfloat16 and the block table is int32")
    if not (k_cache.is_contiguous() and v_cache.is_contiguous()) or block_table.stride(1) != 1:
        raise ValueError("cache pools must be contiguous [blocks, kv_heads, 16, head_dim]")
    return KvCache(k_cache.data_ptr(), v_cache.data_ptr(), k_cache.shape[0], k_cache.shape[2],
                   block_table.data_ptr(), block_table.stride(0))


def prefix_attn_workspace_bytes(num_q_heads, num_kv_heads, head_dim, dtype_code, total_tokens) -> int:
    d = AttnDesc(num_q_heads, num_kv_heads, head_dim, 0.0, dtype_code)
    return int(load_library().rpx_prefix_attn_workspace_bytes(ctypes.byref(d), int(total_tokens)))


def suffix_attn_workspace_bytes(num_q_heads, num_kv_heads, head_dim, dtype_code, total_tokens) -> int:
    d = AttnDesc(num_q_heads, num_kv_heads, head_dim, 0.0, dtype_code)
    return int(load_library().rpx_suffix_attn_workspace_bytes(ctypes.byref(d), int(total_tokens)))


def attn_backward_workspace_bytes(num_q_heads, num_kv_heads, head_dim, total_tokens) -> int:
    desc = AttnDesc(num_q_heads, num_kv_heads, head_dim, 0.0, RPX_BF16)
    return int(load_library().rpx_attn_backward_workspace_bytes(ctypes.byref(desc), int(total_tokens)))


def token_logprobs_workspace_bytes(n_tokens, hidden_dim, vocab, dtype_code) -> int:
    return int(load_library().rpx_token_logprobs_workspace_bytes(int(n_tokens), int(hidden_dim), int(vocab),
                                                                 int(dtype_code)))


def selftest_bounded_wait(limit_cycles: int, device_status, stream=None) -> None:
    """rpx_selftest_bounded_wait: a wait that must time out and report RPX_ERR_TIMEOUT in device_status."""
    rc = load_library().rpx_selftest_bounded_wait(int(limit_cycles), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_selftest_bounded_wait")


def set_sm_budget(sms: int) -> None:
    """rpx_set_sm_budget: cap the persistent kernels' grids at ``sms`` CTAs (0 = no cap), process-wide."""
    rc = load_library().rpx_set_sm_budget(int(sms))
    if rc != 0:
        raise RpxError(rc, "rpx_set_sm_budget")


def set_lm_head_pairing(on: bool) -> None:
    """Process-wide choice of the LM-head kernel: CTA pairs (cta_group::2) when ``on``."""
    rc = load_library().rpx_set_lm_head_pairing(1 if on else 0)
    if rc != 0:
        raise RpxError(rc, "rpx_set_lm_head_pairing")


def get_lm_head_pairing() -> bool:
    return bool(load_library().rpx_get_lm_head_pairing())


def get_sm_budget() -> int:
    return int(load_library().rpx_get_sm_budget())


# ------------------------------------------------------------------ the three calls
@_in_call_context
def prefix_attn(q, k, v, cu_seqlens, max_seqlen: int, cache: Optional[Tuple] = None, softmax_scale: float = 0.0,
                out=None, lse=None, return_lse: bool = False, workspace=None, device_status=None, stream=None):
    """rpx_prefix_attn: causal GQA attention over packed prompts, writing the paged KV cache.

    q [T, H_q, d], k/v [T, H_kv, d] device tensors; cu_seqlens int32 [B+1] on the device;
    cache = (k_cache, v_cache, block_table) or None.  Returns out (and lse when asked).
    """
    torch = _torch()
    lib = load_library()
    desc = _desc(q, k, softmax_scale)
    total = q.shape[0]
    if out is None:
        out = torch.empty((total, q.shape[1], q.shape[2]), dtype=q.dtype, device=q.device)
    if lse is None and return_lse:
        lse = torch.empty((total, q.shape[1]), dtype=torch.float32, device=q.device)
    ws = _workspace(int(lib.rpx_prefix_attn_workspace_bytes(ctypes.byref(desc), total)), q.device, workspace)
    cs = _cache_struct(cache) if cache is not None else None
    rc = lib.rpx_prefix_attn(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _tok_stride(q), _tok_stride(k),
                             _tok_stride(v), _ptr(cu_seqlens), cu_seqlens.shape[0] - 1, total, int(max_seqlen),
                             ctypes.byref(cs) if cs is not None else None, _ptr(out), _ptr(lse), _ptr(ws),
                             ws.numel() * ws.element_size(), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_prefix_attn")
    return (out, lse) if return_lse else out


@_in_call_context
def suffix_attn(q, k, v, cu_seqlens_suffix, prefix_lens, max_suffix_len: int, max_prefix_len: int, cache: Tuple,
                softmax_scale: float = 0.0, out=None, lse=None, return_lse: bool = False, workspace=None,
                device_status=None, stream=None):
    """rpx_suffix_attn: response queries over [cached prefix KV ; causal self]."""
    torch = _torch()
    lib = load_library()
    desc = _desc(q, k, softmax_scale)
    total = q.shape[0]
    if out is None:
        out = torch.empty((total, q.shape[1], q.shape[2]), dtype=q.dtype, device=q.device)
    if lse is None and return_lse:
        lse = torch.empty((total, q.shape[1]), dtype=torch.float32, device=q.device)
    ws = _workspace(int(lib.rpx_suffix_attn_workspace_bytes(ctypes.byref(desc), total)), q.device, workspace)
    cs = _cache_struct(cache)
    rc = lib.rpx_suffix_attn(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _tok_stride(q), _tok_stride(k),
                             _tok_stride(v), _ptr(cu_seqlens_suffix), _ptr(prefix_lens),
                             cu_seqlens_suffix.shape[0] - 1, total, int(max_suffix_len), int(max_prefix_len),
                             ctypes.byref(cs), _ptr(out), _ptr(lse), _ptr(ws), ws.numel() * ws.element_size(),
                             _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_suffix_attn")
    return (out, lse) if return_lse else out


@_in_call_context
def chunk_attn(q, k, v, cu_seqlens_chunk, cached_lens, max_chunk_len: int, max_cached_len: int, cache: Tuple,
                softmax_scale: float = 0.0, out=None, lse=None, return_lse: bool = False, workspace=None,
                device_status=None, stream=None):
    """rpx_chunk_attn: the next chunk of every prompt over [cached earlier chunks ; causal self], appending
    the chunk's K/V to the cache (cached_lens must be multiples of the 16-token block)."""
    torch = _torch()
    lib = load_library()
    desc = _desc(q, k, softmax_scale)
    total = q.shape[0]
    if out is None:
        out = torch.empty((total, q.shape[1], q.shape[2]), dtype=q.dtype, device=q.device)
    if lse is None and return_lse:
        lse = torch.empty((total, q.shape[1]), dtype=torch.float32, device=q.device)
    ws = _workspace(int(lib.rpx_suffix_attn_workspace_bytes(ctypes.byref(desc), total)), q.device, workspace)
    cs = _cache_struct(cache)
    rc = lib.rpx_chunk_attn(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _tok_stride(q), _tok_stride(k),
                             _tok_stride(v), _ptr(cu_seqlens_chunk), _ptr(cached_lens),
                             cu_seqlens_chunk.shape[0] - 1, total, int(max_chunk_len), int(max_cached_len),
                             ctypes.byref(cs), _ptr(out), _ptr(lse), _ptr(ws), ws.numel() * ws.element_size(),
                             _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_chunk_attn")
    return (out, lse) if return_lse else out


@_in_call_context
def token_logprobs(hidden, w_vocab, target_ids, logprobs=None, lse=None, return_lse: bool = False, workspace=None,
                   device_status=None, stream=None, entropy=None):
    """rpx_token_logprobs: log p(target) per row from hidden [N, H] and W [V, H]; logits never stored.

    ``entropy`` (float32 [N], optional) additionally receives the entropy of each row's next-token
    distribution from the same pass (rpx_token_logprobs_entropy)."""
    torch = _torch()
    lib = load_library()
    code = _dtype_code(hidden)
    if _dtype_code(w_vocab) != code:
        raise TypeError("hidden and w_vocab must share an element type")
    if hidden.dim() != 2 or hidden.stride(1) != 1 or not w_vocab.is_contiguous():
        raise ValueError("hidden must be [N, H] with contiguous rows and w_vocab contiguous [V, H]")
    n, hdim = hidden.shape
    vocab = w_vocab.shape[0]
    if logprobs is None:
        logprobs = torch.empty((n,), dtype=torch.float32, device=hidden.device)
    if lse is None and return_lse:
        lse = torch.empty((n,), dtype=torch.float32, device=hidden.device)
    ws = _workspace(int(lib.rpx_token_logprobs_workspace_bytes(n, hdim, vocab, code)), hidden.device, workspace)
    row_stride = hidden.stride(0) if n > 1 else hdim
    if entropy is None:
        rc = lib.rpx_token_logprobs(_ptr(hidden), row_stride, _ptr(w_vocab), _ptr(target_ids), n, hdim, vocab, code,
                                    _ptr(logprobs), _ptr(lse), _ptr(ws), ws.numel() * ws.element_size(),
                                    _ptr(device_status), _stream_ptr(stream))
    else:
        rc = lib.rpx_token_logprobs_entropy(_ptr(hidden), row_stride, _ptr(w_vocab), _ptr(target_ids), n, hdim, vocab,
                                            code, _ptr(logprobs), _ptr(lse), _ptr(entropy), _ptr(ws),
                                            ws.numel() * ws.element_size(), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_token_logprobs")
    return (logprobs, lse) if return_lse else logprobs


def token_logprobs_backward_workspace_bytes(n_tokens, hidden_dim, vocab, dtype_code=RPX_BF16) -> int:
    return int(load_library().rpx_token_logprobs_backward_workspace_bytes(int(n_tokens), int(hidden_dim), int(vocab),
                                                                          int(dtype_code)))


@_in_call_context
def token_logprobs_backward(hidden, w_vocab, target_ids, lse, upstream, dhidden=None, workspace=None, device_status=None,
                            stream=None, dw=None, want_dw: bool = False, accumulate_dw: bool = False,
                            want_dhidden: bool = True):
    """rpx_token_logprobs_backward(_full): d(sum upstream * logprobs) / d hidden, bf16 [N, H], and - with ``want_dw`` or a
    ``dw`` buffer - d / d w_vocab, float32 [V, H] (added to ``dw`` when ``accumulate_dw``).

    ``lse`` is the forward call's lse output for the same rows, ``upstream`` float32 [N].  Returns dhidden, or
    (dhidden, dw) when the weight gradient was asked for (dhidden is None with ``want_dhidden=False``)."""
    torch = _torch()
    lib = load_library()
    if _dtype_code(hidden) != RPX_BF16 or _dtype_code(w_vocab) != RPX_BF16:
        raise TypeError("the LM-head backward pass takes bfloat16 tensors only")
    if hidden.dim() != 2 or hidden.stride(1) != 1 or not w_vocab.is_contiguous():
        raise ValueError("hidden must be [N, H] with contiguous rows and w_vocab contiguous [V, H]")
    if lse.dtype != torch.float32 or upstream.dtype != torch.float32:
        raise TypeError("lse and upstream are float32")
    n, hdim = hidden.shape
    vocab = w_vocab.shape[0]
    if dhidden is None and want_dhidden:
        dhidden = torch.empty((n, hdim), dtype=torch.bfloat16, device=hidden.device)
    with_dw = want_dw or dw is not None
    if with_dw:
        if dw is None:
            if accumulate_dw:
                raise ValueError("accumulate_dw needs the dw buffer to add to")
            dw = torch.empty((vocab, hdim), dtype=torch.float32, device=hidden.device)
        if dw.dtype != torch.float32 or not dw.is_contiguous() or tuple(dw.shape) != (vocab, hdim):
            raise ValueError("dw is a contiguous float32 [V, H] tensor")
    ws = _workspace(int(lib.rpx_token_logprobs_backward_workspace_bytes(n, hdim, vocab, RPX_BF16)), hidden.device, workspace)
    rc = lib.rpx_token_logprobs_backward_full(_ptr(hidden), hidden.stride(0) if n > 1 else hdim, _ptr(w_vocab),
                                              _ptr(target_ids), _ptr(lse), _ptr(upstream), n, hdim, vocab, RPX_BF16,
                                              _ptr(dhidden), _ptr(dw), 1 if accumulate_dw else 0, _ptr(ws),
                                              ws.numel() * ws.element_size(), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_token_logprobs_backward_full")
    return (dhidden, dw) if with_dw else dhidden


@_in_call_context
def attn_backward(q, k, v, out, dout, lse, cu_seqlens, max_seqlen: int, q_begin=None, q_end=None, softmax_scale: float = 0.0,
                  dq=None, dk=None, dv=None, accumulate_dkv: bool = False, workspace=None, device_status=None, stream=None):
    """rpx_attn_backward: gradients of causal GQA attention over packed whole sequences.

    q [T, H_q, d], k/v [T, H_kv, d], out/dout [T, H_q, d] bfloat16; lse float32 [T, H_q] from the forward pass;
    q_begin / q_end (int32 [B], optional) restrict the query rows that take part.  Returns float32 (dq, dk, dv);
    with ``accumulate_dkv`` the call's dk, dv are added to the given buffers."""
    torch = _torch()
    lib = load_library()
    if any(_dtype_code(t) != RPX_BF16 for t in (q, k, v, out, dout)):
        raise TypeError("the attention backward pass takes bfloat16 tensors only")
    if lse.dtype != torch.float32 or not lse.is_contiguous() or not out.is_contiguous() or not dout.is_contiguous():
        raise ValueError("out, dout and lse (float32) must be contiguous")
    desc = _desc(q, k, softmax_scale)
    total = q.shape[0]
    if dq is None:
        dq = torch.empty(tuple(q.shape), dtype=torch.float32, device=q.device)
    if accumulate_dkv and (dk is None or dv is None):
        raise ValueError("accumulate_dkv needs the dk and dv buffers to add to")
    if dk is None:
        dk = torch.empty(tuple(k.shape), dtype=torch.float32, device=q.device)
    if dv is None:
        dv = torch.empty(tuple(v.shape), dtype=torch.float32, device=q.device)
    for t in (dq, dk, dv):
        if t.dtype != torch.float32 or not t.is_contiguous():
            raise ValueError("dq, dk, dv are contiguous float32 tensors")
    ws = _workspace(int(lib.rpx_attn_backward_workspace_bytes(ctypes.byref(desc), total)), q.device, workspace)
    rc = lib.rpx_attn_backward(ctypes.byref(desc), _ptr(q), _ptr(k), _ptr(v), _tok_stride(q), _tok_stride(k),
                               _tok_stride(v), _ptr(out), _ptr(dout), _ptr(lse), _ptr(cu_seqlens), _ptr(q_begin),
                               _ptr(q_end), cu_seqlens.shape[0] - 1, total, int(max_seqlen), _ptr(dq), _ptr(dk), _ptr(dv),
                               1 if accumulate_dkv else 0, _ptr(ws), ws.numel() * ws.element_size(), _ptr(device_status),
                               _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_attn_backward")
    return dq, dk, dv


@_in_call_context
def token_logprobs_static(hidden, w_vocab, target_ids, logprobs, lse=None, device_status=None, stream=None):
    """rpx_token_logprobs_static: the same log-probs, for callers that cannot allocate device memory.

    Nothing is allocated on this path, not even by torch: ``logprobs`` (float32 [N]) must be passed
    in, and the partial records go to a fixed array inside the library.  Use it where the device
    allocator is out of reach (all HBM already reserved by the host engine, or a code section in
    which an allocator call could fail or stall the device).  bf16 only; the problem must fit
    ``STATIC_SCRATCH_BYTES`` (raises RpxError RPX_ERR_WORKSPACE otherwise); calls that overlap on
    the GPU race on the shared array.
    """
    lib = load_library()
    if _dtype_code(hidden) != RPX_BF16 or _dtype_code(w_vocab) != RPX_BF16:
        raise TypeError("the allocation-free entry point takes bfloat16 tensors only")
    if hidden.dim() != 2 or hidden.stride(1) != 1 or not w_vocab.is_contiguous():
        raise ValueError("hidden must be [N, H] with contiguous rows and w_vocab contiguous [V, H]")
    n, hdim = hidden.shape
    row_stride = hidden.stride(0) if n > 1 else hdim
    rc = lib.rpx_token_logprobs_static(_ptr(hidden), row_stride, _ptr(w_vocab), _ptr(target_ids), n, hdim,
                                       w_vocab.shape[0], _ptr(logprobs), _ptr(lse), _ptr(device_status),
                                       _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_token_logprobs_static")
    return logprobs


@_in_call_context
def token_logprobs_shard(hidden, w_shard, target_ids, vocab_begin: int, shard_stats=None, workspace=None,
                         device_status=None, stream=None):
    """rpx_token_logprobs_shard: this rank's share of a vocabulary-parallel LM head.

    w_shard holds rows vocab_begin .. vocab_begin + V_local - 1 of W_vocab; target_ids are global ids.
    Returns shard_stats float32 [N, 4] to be gathered over ranks and passed to token_logprobs_merge."""
    torch = _torch()
    lib = load_library()
    code = _dtype_code(hidden)
    if _dtype_code(w_shard) != code:
        raise TypeError("hidden and w_shard must share an element type")
    if hidden.dim() != 2 or hidden.stride(1) != 1 or not w_shard.is_contiguous():
        raise ValueError("hidden must be [N, H] with contiguous rows and w_shard contiguous [V_local, H]")
    n, hdim = hidden.shape
    v_local = w_shard.shape[0]
    if shard_stats is None:
        shard_stats = torch.empty((n, 4), dtype=torch.float32, device=hidden.device)
    ws = _workspace(int(lib.rpx_token_logprobs_workspace_bytes(n, hdim, v_local, code)), hidden.device, workspace)
    rc = lib.rpx_token_logprobs_shard(_ptr(hidden), hidden.stride(0) if n > 1 else hdim, _ptr(w_shard), _ptr(target_ids), n,
                                      hdim, v_local, int(vocab_begin), code, _ptr(shard_stats), _ptr(ws),
                                      ws.numel() * ws.element_size(), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_token_logprobs_shard")
    return shard_stats


@_in_call_context
def token_logprobs_merge(all_stats, target_ids, vocab_total: int, logprobs=None, return_lse: bool = False, entropy=None,
                         device_status=None, stream=None):
    """rpx_token_logprobs_merge: final log-probs from the gathered shard records float32 [R, N, 4]."""
    torch = _torch()
    lib = load_library()
    if all_stats.dim() != 3 or all_stats.shape[2] != 4 or all_stats.dtype != torch.float32 or not all_stats.is_contiguous():
        raise ValueError("all_stats must be a contiguous float32 [shards, N, 4] tensor")
    r, n, _ = all_stats.shape
    if logprobs is None:
        logprobs = torch.empty((n,), dtype=torch.float32, device=all_stats.device)
    lse = torch.empty((n,), dtype=torch.float32, device=all_stats.device) if return_lse else None
    rc = lib.rpx_token_logprobs_merge(_ptr(all_stats), r, _ptr(target_ids), n, int(vocab_total), _ptr(logprobs), _ptr(lse),
                                      _ptr(entropy), _ptr(device_status), _stream_ptr(stream))
    if rc != 0:
        raise RpxError(rc, "rpx_token_logprobs_merge")
    return (logprobs, lse) if return_lse else logprobs
