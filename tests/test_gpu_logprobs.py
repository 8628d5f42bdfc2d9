"""GPU parity of rpx_token_logprobs (through the C ABI) against the fp64 CPU oracle.

Tolerance (stated by the benchmark spec): per-token log-prob abs error <= 2e-2.  With bf16
inputs both sides read the same bits, so the observed error is fp32 accumulation order only
(~1e-5); the tests also assert that much tighter bound so a real bug cannot hide inside 2e-2.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device

pytestmark = pytest.mark.gpu

TOL = 2e-2
TIGHT = 5e-4


def _run(wl, dev, rows=None):
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    lp, lse = rpx.token_logprobs(to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev),
                                 return_lse=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, rpx.status_string(int(status.item()))
    lp, lse = lp.double().cpu().numpy(), lse.double().cpu().numpy()
    if rows is None:
        rows = np.arange(wl.n_tokens, dtype=np.int64)
    ref_lp, ref_lse = oracle.logprob_rows(wl.hidden, wl.w, wl.ids, rows)
    return lp[rows], lse[rows], ref_lp, ref_lse


def test_c1_tiny_fp32_all_rows(cuda_device):
    wl = wk.make_workload(wk.CONFIGS["C1"], seed=0, attn=False)
    lp, lse, ref_lp, ref_lse = _run(wl, cuda_device)
    assert np.abs(lp - ref_lp).max() <= TOL
    assert np.abs(lse - ref_lse).max() <= TOL
    # against the oracle fed the bf16-rounded inputs only accumulation order differs
    hb = wk.f32_to_bf16_bits(wl.hidden).reshape(wl.hidden.shape)
    wb = wk.f32_to_bf16_bits(wl.w).reshape(wl.w.shape)
    ref_b, _ = oracle.logprob_rows(hb, wb, wl.ids)
    assert np.abs(lp - ref_b).max() <= TIGHT


@pytest.mark.parametrize("n_tokens,hidden,vocab", [
    (300, 200, 1000),     # ragged rows, K tail (200 = 3*64 + 8), ragged vocab tile and 32-column chunk
    (128, 64, 256),       # exactly one tile of everything
    (1, 8, 3),            # smallest legal problem
    (257, 512, 5000),     # two vocab chunks (20 tiles of 256), row tail of one
    (640, 1024, 33000),   # nine chunks, more work items than one wave of 4-wide groups
])
def test_ragged_shapes_all_rows(cuda_device, n_tokens, hidden, vocab):
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=3, attn=False)
    lp, lse, ref_lp, ref_lse = _run(wl, cuda_device)
    assert np.abs(lp - ref_lp).max() <= TIGHT
    assert np.abs(lse - ref_lse).max() <= TIGHT


def test_large_logits_need_the_running_max(cuda_device):
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 256, 2048, ("fixed", 200), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=4, attn=False)
    w = wk.bf16_bits_to_f32(wl.w).reshape(wl.w.shape) * 40.0      # logits of a few hundred
    wl.w = wk.f32_to_bf16_bits(w).reshape(w.shape)
    lp, lse, ref_lp, ref_lse = _run(wl, cuda_device)
    assert np.isfinite(lp).all()
    assert np.abs(lse - ref_lse).max() <= 1e-4 * np.abs(ref_lse).max() + 1e-3
    assert np.abs(lp - ref_lp).max() <= 1e-4 * np.abs(ref_lp).max() + 1e-3


def test_strided_hidden_rows_and_invalid_targets(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 128, 700, ("fixed", 150), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=5, attn=False)
    wide = torch.zeros((150, 256), dtype=torch.bfloat16, device=dev)
    wide[:, :128] = to_device(wl.hidden, dev)
    ids = wl.ids.copy()
    ids[7], ids[149] = 700, -3
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    lp = rpx.token_logprobs(wide[:, :128], to_device(wl.w, dev), to_device(ids, dev), device_status=status)
    torch.cuda.synchronize()
    lp = lp.double().cpu().numpy()
    assert int(status.item()) == -8
    assert np.isnan(lp[7]) and np.isnan(lp[149])
    good = np.ones(150, bool)
    good[[7, 149]] = False
    ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids, np.nonzero(good)[0].astype(np.int64))
    assert np.abs(lp[good] - ref).max() <= TIGHT


def test_two_calls_give_identical_bits(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 512, 9000, ("fixed", 700), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=6, attn=False)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    a = rpx.token_logprobs(h, w, ids).clone()
    b = rpx.token_logprobs(h, w, ids)
    torch.cuda.synchronize()
    assert torch.equal(a, b)


@pytest.mark.parametrize("budget", [1, 37, 100, 1000])
def test_sm_budget_changes_no_bit(cuda_device, budget):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 256, 70000, ("fixed", 3000), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=8, attn=False)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    a = rpx.token_logprobs(h, w, ids).clone()
    try:
        rpx.set_sm_budget(budget)
        b = rpx.token_logprobs(h, w, ids)
        torch.cuda.synchronize()
    finally:
        rpx.set_sm_budget(0)
    assert torch.equal(a, b)


def test_c2_full_size_sampled_rows(cuda_device):
    """BASELINE configs[1] at full size (34 816 rows x 152 064 columns, hidden 3584), in the launch
    configuration the benchmark times; the oracle scores 48 sampled rows one by one."""
    wl = wk.make_workload(wk.CONFIGS["C2"], seed=0, attn=False)
    rows = wk.sample_logprob_rows(wl, 48, seed=1)
    lp, lse, ref_lp, ref_lse = _run(wl, cuda_device, rows)
    assert np.abs(lp - ref_lp).max() <= TIGHT
    assert np.abs(lse - ref_lse).max() <= TIGHT
    assert abs(ref_lp.mean() + (np.log(152064) + 0.5 * 3584 * 0.02 ** 2)) < 0.6


@pytest.mark.parametrize("name", ["C3", "C4", "C5"])
def test_other_full_size_configs_sampled_rows(cuda_device, name):
    """The remaining BASELINE configs at full size (32B shape: hidden 5120; C3 has ~226 k rows, C5
    ~135 k), 24 sampled rows each against the oracle."""
    wl = wk.make_workload(wk.CONFIGS[name], seed=0, attn=False)
    rows = wk.sample_logprob_rows(wl, 24, seed=3)
    lp, lse, ref_lp, ref_lse = _run(wl, cuda_device, rows)
    assert np.abs(lp - ref_lp).max() <= TIGHT
    assert np.abs(lse - ref_lse).max() <= TIGHT


@pytest.mark.parametrize("n_tokens,hidden,vocab,scale", [(300, 200, 1000, 1.0), (257, 512, 5000, 1.0), (200, 256, 2048, 40.0)])
def test_entropy_from_the_same_pass(cuda_device, n_tokens, hidden, vocab, scale):
    """rpx_token_logprobs_entropy: H = -sum p ln p per row against the oracle's definition, on ragged
    shapes, several chunks, and peaked distributions (logits of a few hundred, entropy near 0)."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=8, attn=False)
    if scale != 1.0:
        w = wk.bf16_bits_to_f32(wl.w).reshape(wl.w.shape) * scale
        wl.w = wk.f32_to_bf16_bits(w).reshape(w.shape)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    ent = torch.full((n_tokens,), float("nan"), dtype=torch.float32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    lp = rpx.token_logprobs(h, w, ids, entropy=ent, device_status=status)
    lp_plain = rpx.token_logprobs(h, w, ids)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(lp, lp_plain)
    ref = oracle.entropy_rows(wl.hidden, wl.w)
    got = ent.double().cpu().numpy()
    assert np.isfinite(got).all() and (got > -1e-3).all() and (got < np.log(vocab) + 1e-3).all()
    assert np.abs(got - ref).max() <= TIGHT + 1e-5 * np.abs(ref).max() * (scale > 1)


@pytest.mark.parametrize("n_tokens,hidden,vocab", [
    (300, 200, 1000),     # three row tiles: the second 256-row tile is half empty
    (1, 8, 3),
    (129, 72, 257),
    (640, 1024, 33000),
    (5000, 512, 20000),   # more work items than CTA pairs
])
def test_cta_pair_kernel_matches_the_oracle_and_the_single_cta_kernel(cuda_device, n_tokens, hidden, vocab):
    """The cta_group::2 variant of the LM head (two CTAs per 256 x 256 tile): same oracle, same bound, and - since each
    row's products are accumulated in the same order and folded by the same epilogue - the same bits as the
    single-CTA kernel, entropy included."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=5, attn=False)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    assert not rpx.get_lm_head_pairing()
    ent_a = torch.empty(n_tokens, dtype=torch.float32, device=dev)
    lp_a, lse_a = rpx.token_logprobs(h, w, ids, return_lse=True, entropy=ent_a, device_status=status)
    try:
        rpx.set_lm_head_pairing(True)
        assert rpx.get_lm_head_pairing()
        ent_b = torch.empty(n_tokens, dtype=torch.float32, device=dev)
        lp_b, lse_b = rpx.token_logprobs(h, w, ids, return_lse=True, entropy=ent_b, device_status=status)
        torch.cuda.synchronize()
    finally:
        rpx.set_lm_head_pairing(False)
    assert int(status.item()) == 0
    ref_lp, ref_lse = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    assert np.abs(lp_b.double().cpu().numpy() - ref_lp).max() <= TIGHT
    assert np.abs(lse_b.double().cpu().numpy() - ref_lse).max() <= TIGHT
    assert torch.equal(lp_a, lp_b) and torch.equal(lse_a, lse_b) and torch.equal(ent_a, ent_b)


def test_cta_pair_kernel_under_an_sm_budget_and_through_the_other_entry_points(cuda_device):
    """The pair kernel runs whole clusters only: an odd SM budget leaves one SM unused, a budget of one falls back to
    the single-CTA kernel; the shard and static entry points take the same switch."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 256, 3000, ("fixed", 700), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=6, attn=False)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ref = rpx.token_logprobs(h, w, ids, device_status=status)
    try:
        rpx.set_lm_head_pairing(True)
        for budget in (0, 7, 2, 1):
            rpx.set_sm_budget(budget)
            got = rpx.token_logprobs(h, w, ids, device_status=status)
            torch.cuda.synchronize()
            assert torch.equal(got, ref), budget
        rpx.set_sm_budget(0)
        lp = torch.empty(700, dtype=torch.float32, device=dev)
        rpx.token_logprobs_static(h, w, ids, lp, device_status=status)
        stats = rpx.token_logprobs_shard(h, w[:1500], ids, 0, device_status=status)
        torch.cuda.synchronize()
        assert float((lp - ref).abs().max()) <= 2e-5   # the static entry point always uses 16-tile chunks: another merge order
        assert stats.shape == (700, 4) and bool(torch.isfinite(stats).all())
    finally:
        rpx.set_sm_budget(0)
        rpx.set_lm_head_pairing(False)
    assert int(status.item()) == 0
