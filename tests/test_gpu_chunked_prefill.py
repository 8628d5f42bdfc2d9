"""Chunked prefill (rpx_chunk_attn): each prompt is fed in chunks; a chunk attends to the earlier
chunks through the paged cache plus causally to itself and appends its own K/V.  After the last
chunk the outputs and the cache image must equal the oracle's one-pass values, and a suffix pass
on top must still reproduce one-pass attention over prompt + response."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import bf16_bits, to_device

import test_gpu_attention as T

pytestmark = pytest.mark.gpu


def _chunked_prefill(wl, dev, chunk, first_call_is_prefix_attn=False):
    cfg = wl.cfg
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = torch.full((wl.num_blocks, cfg.num_kv_heads, 16, cfg.head_dim), T.SENTINEL, dtype=torch.int16, device=dev)
    k_cache, v_cache = pool.view(torch.bfloat16), pool.clone().view(torch.bfloat16)
    cache = (k_cache, v_cache, to_device(wl.block_table, dev))
    qp, kp, vp = (wl.prefix_pack(t) for t in (wl.q, wl.k, wl.v))
    P = wl.prompt_lens.astype(np.int64)
    n_pre = int(P.sum())
    out = np.zeros((n_pre, cfg.num_q_heads, cfg.head_dim))
    lse = np.zeros((n_pre, cfg.num_q_heads))
    n_calls = 0
    for c in range(int(-(-int(P.max()) // chunk))):
        starts, ends = np.minimum(c * chunk, P), np.minimum((c + 1) * chunk, P)
        lens = ends - starts
        idx = np.concatenate([wl.cu_prefix[s] + np.arange(starts[s], ends[s]) for s in range(cfg.batch)]).astype(np.int64)
        if idx.size == 0:
            continue
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        args = [to_device(np.ascontiguousarray(t[idx]), dev) for t in (qp, kp, vp)]
        if c == 0 and first_call_is_prefix_attn:
            o, l = rpx.prefix_attn(*args, to_device(cu, dev), int(lens.max()), cache=cache, return_lse=True,
                                   device_status=status)
        else:
            # finished prompts have an empty chunk; their cached_lens (not page multiples) must be ignored
            o, l = rpx.chunk_attn(*args, to_device(cu, dev), to_device(starts.astype(np.int32), dev), int(lens.max()),
                                  int(starts.max()), cache, return_lse=True, device_status=status)
        n_calls += 1
        out[idx] = o.double().cpu().numpy()
        lse[idx] = l.double().cpu().numpy()
    torch.cuda.synchronize()
    assert int(status.item()) == 0, rpx.status_string(int(status.item()))
    return out, lse, cache, n_calls


def _check_prefix_rows(wl, out, lse):
    cfg = wl.cfg
    qp, kp, vp = (wl.prefix_pack(t) for t in (wl.q, wl.k, wl.v))
    rows = oracle.all_rows(wl.cu_prefix, cfg.num_q_heads)
    ref_o, ref_l = oracle.attn_rows(qp, kp, vp, wl.cu_prefix, rows)
    tok = wl.cu_prefix[rows[:, 0]].astype(np.int64) + rows[:, 1]
    err = np.abs(out[tok, rows[:, 2]] - ref_o)
    assert (err <= T.out_tolerance(ref_o)).all(), f"max error {err.max():.3e}"
    assert np.abs(lse[tok, rows[:, 2]] - ref_l).max() <= T.LSE_TOL


@pytest.mark.parametrize("head_dim,chunk,first_prefix", [(128, 256, False), (128, 208, True), (64, 128, False), (64, 48, False)])
def test_chunked_prefill_equals_one_pass(cuda_device, head_dim, chunk, first_prefix):
    dev = cuda_device
    plens = [700, 256, 16, 1, 0, 513, 1000] if chunk >= 128 else [300, 48, 0, 97, 1]
    rlens = [40, 0, 130, 5, 9, 257, 1][: len(plens)]
    cfg = wk.Config("chunked", "bf16", len(plens), 4, 2, head_dim, 64, 64, ("list", plens), ("list", rlens))
    wl = wk.make_workload(cfg, seed=31, lm=False)
    out, lse, cache, n_calls = _chunked_prefill(wl, dev, chunk, first_prefix)
    assert n_calls == -(-max(plens) // chunk)
    _check_prefix_rows(wl, out, lse)
    T.check_cache(wl, bf16_bits(cache[0]), bf16_bits(cache[1]))
    # the suffix pass reads the chunk-built cache like any other
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    qs, ks, vs = (to_device(wl.suffix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    o_suf, l_suf = rpx.suffix_attn(qs, ks, vs, to_device(wl.cu_suffix, dev), to_device(wl.prompt_lens, dev),
                                   int(wl.response_lens.max()), int(wl.prompt_lens.max()), cache, return_lse=True,
                                   device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    full_o = np.zeros((wl.n_tokens, cfg.num_q_heads, cfg.head_dim))
    full_l = np.zeros((wl.n_tokens, cfg.num_q_heads))
    full_o[wl.prefix_rows()], full_l[wl.prefix_rows()] = out, lse
    full_o[wl.suffix_rows()], full_l[wl.suffix_rows()] = o_suf.double().cpu().numpy(), l_suf.double().cpu().numpy()
    T.check_rows(wl, full_o, full_l, oracle.all_rows(wl.cu_full, cfg.num_q_heads))


def test_chunk_not_on_a_page_edge_is_reported_and_not_stored(cuda_device):
    dev = cuda_device
    cfg = wk.Config("chunked", "bf16", 2, 2, 1, 128, 64, 64, ("list", [64, 64]), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=32, lm=False)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = torch.full((wl.num_blocks, 1, 16, 128), T.SENTINEL, dtype=torch.int16, device=dev)
    k_cache, v_cache = pool.view(torch.bfloat16), pool.clone().view(torch.bfloat16)
    cache = (k_cache, v_cache, to_device(wl.block_table, dev))
    qp, kp, vp = (wl.prefix_pack(t) for t in (wl.q, wl.k, wl.v))
    # first 24 tokens of sequence 0 / 32 of sequence 1 by the prefix pass ...
    idx = np.concatenate([np.arange(0, 24), 64 + np.arange(0, 32)])
    rpx.prefix_attn(*(to_device(np.ascontiguousarray(t[idx]), dev) for t in (qp, kp, vp)),
                    to_device(np.array([0, 24, 56], np.int32), dev), 32, cache=cache, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    before_k = bf16_bits(k_cache).copy()
    # ... then the rest: sequence 0 would start at token 24 (not a multiple of 16), sequence 1 at 32
    idx = np.concatenate([np.arange(24, 64), 64 + np.arange(32, 64)])
    o = rpx.chunk_attn(*(to_device(np.ascontiguousarray(t[idx]), dev) for t in (qp, kp, vp)),
                       to_device(np.array([0, 40, 72], np.int32), dev), to_device(np.array([24, 32], np.int32), dev),
                       40, 32, cache, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -8  # RPX_ERR_DEVICE_DATA
    assert torch.isfinite(o.float()).all()
    after_k = bf16_bits(k_cache)
    ref_k, _ = oracle.cache_image(kp, vp, wl.cu_prefix, wl.block_table, wl.num_blocks, sentinel=T.SENTINEL)
    blocks0 = wl.block_table[0, : 64 // 16]
    blocks1 = wl.block_table[1, : 64 // 16]
    assert np.array_equal(after_k[blocks0], before_k[blocks0])  # sequence 0: nothing appended
    assert np.array_equal(after_k[blocks1], ref_k[blocks1])     # sequence 1: complete
