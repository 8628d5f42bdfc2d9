"""GPU parity of rpx_token_logprobs_backward (through the C ABI) against the fp64 oracle's gradient.

Tolerance: dhidden is delivered as bf16 (half an ulp is 2^-9 of the value), and dL/dz passes through bf16 once on
its way to the second GEMM (each term carries 2^-9 relative rounding, summed over the vocabulary in random signs).
Both sides read the same bf16 input bits; the bound used is 1 % of the largest gradient magnitude of the row plus
2^-8 relative per element."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import binding as B
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device

pytestmark = pytest.mark.gpu


def _check(dev, n_tokens, hidden, vocab, seed, w_scale=None, bad_target=False):
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=seed, attn=False)
    w_host = wl.w
    if w_scale is not None:  # sharper distributions: scale W up (exactly, by a power of two, in the bf16 bits' value)
        w_host = wk.f32_to_bf16_bits(wk.bf16_bits_to_f32(wl.w) * w_scale).reshape(wl.w.shape)
    ids = wl.ids.copy()
    if bad_target:
        ids[3] = vocab + 5
    h, w, tid = to_device(wl.hidden, dev), to_device(w_host, dev), to_device(ids, dev)
    g = np.random.default_rng(seed + 1).standard_normal(n_tokens).astype(np.float32)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _, lse = rpx.token_logprobs(h, w, tid, return_lse=True, device_status=status)
    status.zero_()
    dh = rpx.token_logprobs_backward(h, w, tid, lse, torch.from_numpy(g).to(dev), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == (-8 if bad_target else 0)
    got = dh.double().cpu().numpy()
    ref = oracle.logprob_backward(wl.hidden, w_host, ids, g.astype(np.float64))
    rows = np.ones(n_tokens, bool)
    if bad_target:
        rows[3] = False  # the oracle has no one-hot term either, but keep the row out of the claim
    err = np.abs(got - ref)[rows]
    bound = 0.01 * np.abs(ref[rows]).max(axis=1, keepdims=True) + np.abs(ref[rows]) * 2.0 ** -8
    assert np.isfinite(got).all()
    assert (err <= bound).all(), f"max excess {(err - bound).max():.3e}, max err {err.max():.3e}, max |ref| {np.abs(ref).max():.3e}"
    return err.max()


@pytest.mark.parametrize("n_tokens,hidden,vocab", [(288, 256, 4096), (130, 72, 1000), (1, 64, 257), (700, 512, 9000),
                                                   (300, 200, 255), (257, 128, 64)])
def test_dhidden_matches_the_oracle(cuda_device, n_tokens, hidden, vocab):
    _check(cuda_device, n_tokens, hidden, vocab, 71)


def test_dhidden_with_peaked_distributions_and_an_invalid_target(cuda_device):
    _check(cuda_device, 200, 256, 3000, 72, w_scale=8.0)      # logits of a few tens: rows dominated by a few tokens
    _check(cuda_device, 150, 128, 2000, 73, bad_target=True)


def test_rows_beyond_one_block_and_strided_hidden_rows(cuda_device):
    dev = cuda_device
    # more rows than one block of 9472: the second block reuses the workspace
    n_tokens, hidden, vocab = 9472 + 300, 64, 320
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=74, attn=False)
    # hidden rows with a stride (a slice of a wider tensor)
    wide = torch.zeros((n_tokens, hidden + 64), dtype=torch.bfloat16, device=dev)
    wide[:, :hidden] = to_device(wl.hidden, dev)
    h = wide[:, :hidden]
    w, tid = to_device(wl.w, dev), to_device(wl.ids, dev)
    g = np.random.default_rng(75).standard_normal(n_tokens).astype(np.float32)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _, lse = rpx.token_logprobs(h, w, tid, return_lse=True, device_status=status)
    assert B.token_logprobs_backward_workspace_bytes(n_tokens, hidden, vocab) == 9472 * 320 * 2
    dh = rpx.token_logprobs_backward(h, w, tid, lse, torch.from_numpy(g).to(dev), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    sample = np.concatenate([np.arange(0, 40), np.arange(9460, 9490), np.arange(n_tokens - 20, n_tokens)])
    ref = oracle.logprob_backward(wl.hidden[sample], wl.w, wl.ids[sample], g[sample].astype(np.float64))
    got = dh.double().cpu().numpy()[sample]
    bound = 0.01 * np.abs(ref).max(axis=1, keepdims=True) + np.abs(ref) * 2.0 ** -8
    assert (np.abs(got - ref) <= bound).all()


def test_backward_rejects_bad_arguments_before_any_launch(cuda_device):
    lib = B.load_library()

    def call(hidden=0x1000, stride=256, w=0x1000, ids=0x1000, lse=0x1000, up=0x1000, n=8, h=256, v=4096, dt=B.RPX_BF16,
             dh=0x1000, ws=0x10000, ws_bytes=1 << 30):
        return lib.rpx_token_logprobs_backward(hidden, stride, w, ids, lse, up, n, h, v, dt, dh, ws, ws_bytes, None, None)

    assert call(dt=B.RPX_F32) == -3
    assert call(lse=None) == -1 and call(up=None) == -1 and call(dh=None) == -1
    assert call(h=100) == -2 and call(stride=128) == -2
    assert call(ws=None) == -5 and call(ws_bytes=64) == -5 and call(ws=0x10010) == -4
    assert call(n=0, hidden=None) == 0


def _dw_close(got, ref):
    got = got.double().cpu().numpy()
    assert np.isfinite(got).all()
    # dL/dz passes through bf16 (2^-9 relative per term) before the products are summed over the rows in fp32
    bound = 0.01 * np.abs(ref).max() + np.abs(ref) * 2.0 ** -7 + 1e-7
    err = np.abs(got - ref)
    assert (err <= bound).all(), f"dW: max err {err.max():.3e} of max |ref| {np.abs(ref).max():.3e}"


@pytest.mark.parametrize("n_tokens,hidden,vocab", [(288, 256, 4096), (130, 72, 1000), (1, 64, 257), (700, 512, 9000),
                                                   (300, 200, 255), (257, 128, 64)])
def test_weight_gradient_matches_the_oracle(cuda_device, n_tokens, hidden, vocab):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=81, attn=False)
    h, w, tid = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    g = np.random.default_rng(82).standard_normal(n_tokens).astype(np.float32)
    tg = torch.from_numpy(g).to(dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _, lse = rpx.token_logprobs(h, w, tid, return_lse=True, device_status=status)
    dh_only = rpx.token_logprobs_backward(h, w, tid, lse, tg, device_status=status)
    dh, dw = rpx.token_logprobs_backward(h, w, tid, lse, tg, want_dw=True, device_status=status)
    none, dw_only = rpx.token_logprobs_backward(h, w, tid, lse, tg, want_dw=True, want_dhidden=False, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert none is None and torch.equal(dh, dh_only) and torch.equal(dw, dw_only)
    _, ref_dw = oracle.logprob_backward(wl.hidden, wl.w, wl.ids, g.astype(np.float64), want_dw=True)
    _dw_close(dw, ref_dw)
    # gradient accumulation: a second call adds its gradient to the buffer
    dw2 = dw.clone()
    rpx.token_logprobs_backward(h, w, tid, lse, tg, dw=dw2, accumulate_dw=True, want_dhidden=False, device_status=status)
    torch.cuda.synchronize()
    _dw_close(dw2, 2.0 * ref_dw)


def test_weight_gradient_over_more_rows_than_one_block(cuda_device):
    dev = cuda_device
    n_tokens, hidden, vocab = 9472 + 300, 64, 320   # the second block of rows adds to the first one's dW
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=83, attn=False)
    h, w, tid = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    g = np.random.default_rng(84).standard_normal(n_tokens).astype(np.float32)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _, lse = rpx.token_logprobs(h, w, tid, return_lse=True, device_status=status)
    _, dw = rpx.token_logprobs_backward(h, w, tid, lse, torch.from_numpy(g).to(dev), want_dw=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    _, ref_dw = oracle.logprob_backward(wl.hidden, wl.w, wl.ids, g.astype(np.float64), want_dw=True)
    _dw_close(dw, ref_dw)
