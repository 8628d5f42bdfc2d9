"""GPU parity of rpx_prefix_attn / rpx_suffix_attn (through the C ABI) against the fp64 oracle.

Tolerances (the benchmark spec): attention output max-abs <= 1e-2 on the delivered tensor
(bf16 outputs carry their own rounding: spacing 2^-7 below 2, 2^-6 below 4); integer work — slot
mapping, the cache image including untouched sentinel slots — bit-exact.  The fp32 LSE output is
compared as well because it is free of output rounding.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import bf16_bits, to_device

pytestmark = pytest.mark.gpu

TOL = 1e-2
LSE_TOL = 2e-3
SENTINEL = 0x7FC1  # a NaN pattern: a stray read of an unwritten slot poisons the output


def run_split(wl, dev, table=None, sentinel=SENTINEL):
    """Prefix pass (writes the cache) then suffix pass (reads it).  Returns host results."""
    cfg = wl.cfg
    table = wl.block_table if table is None else table
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = torch.full((wl.num_blocks, cfg.num_kv_heads, 16, cfg.head_dim), sentinel, dtype=torch.int16, device=dev)
    k_cache = pool.view(torch.bfloat16)
    v_cache = pool.clone().view(torch.bfloat16)
    cache = (k_cache, v_cache, to_device(table, dev))
    qp, kp, vp = (to_device(wl.prefix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    qs, ks, vs = (to_device(wl.suffix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    max_p = int(wl.prompt_lens.max()) if cfg.batch else 0
    max_r = int(wl.response_lens.max()) if cfg.batch else 0
    o_pre, lse_pre = rpx.prefix_attn(qp, kp, vp, to_device(wl.cu_prefix, dev), max_p, cache=cache, return_lse=True,
                                     device_status=status)
    o_suf, lse_suf = rpx.suffix_attn(qs, ks, vs, to_device(wl.cu_suffix, dev), to_device(wl.prompt_lens, dev), max_r,
                                     max_p, cache=cache, return_lse=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, rpx.status_string(int(status.item()))
    out = np.zeros((wl.n_tokens, cfg.num_q_heads, cfg.head_dim))
    lse = np.zeros((wl.n_tokens, cfg.num_q_heads))
    out[wl.prefix_rows()] = o_pre.double().cpu().numpy()
    out[wl.suffix_rows()] = o_suf.double().cpu().numpy()
    lse[wl.prefix_rows()] = lse_pre.double().cpu().numpy()
    lse[wl.suffix_rows()] = lse_suf.double().cpu().numpy()
    return out, lse, bf16_bits(k_cache), bf16_bits(v_cache), (o_pre, o_suf)


def out_tolerance(ref_o):
    """Element-wise bound on |O_kernel - O_oracle|.

    1e-2 wherever |O| < 4.  The output is stored as bf16, whose half-ulp is 2^-6 = 0.0156 on
    [4, 8) and doubles per binade, so no bf16 result can promise 1e-2 there: those elements (a
    handful per million with unit-variance V) get half an ulp plus 2.5e-3 for the kernel's own
    arithmetic.
    """
    a = np.abs(ref_o)
    half_ulp = np.exp2(np.floor(np.log2(np.maximum(a, 1.0))) - 8.0)
    return np.where(a < 4.0, TOL, half_ulp + 2.5e-3)


def check_rows(wl, out, lse, rows, lse_tol=LSE_TOL, inputs=None, o_extra=0.0):
    q, k, v = (wl.q, wl.k, wl.v) if inputs is None else inputs
    ref_o, ref_l = oracle.attn_rows(q, k, v, wl.cu_full, rows)
    tok = wl.cu_full[rows[:, 0]].astype(np.int64) + rows[:, 1]
    got_o, got_l = out[tok, rows[:, 2]], lse[tok, rows[:, 2]]
    assert np.isfinite(got_o).all()
    err = np.abs(got_o - ref_o)
    over = err - (out_tolerance(ref_o) + o_extra)
    err_l = np.abs(got_l - ref_l).max() if rows.shape[0] else 0.0
    if over.size and over.max() > 0:
        i, j = np.unravel_index(over.argmax(), over.shape)
        raise AssertionError(f"attention error {err[i, j]:.3e} at row {rows[i]} col {j}: ref {ref_o[i, j]:.6f} "
                             f"got {got_o[i, j]:.6f}")
    assert err_l <= lse_tol, f"LSE max-abs error {err_l:.3e}"
    return (err.max() if err.size else 0.0), err_l


def check_cache(wl, kc, vc, table=None):
    table = wl.block_table if table is None else table
    ref_k, ref_v = oracle.cache_image(wl.prefix_pack(wl.k), wl.prefix_pack(wl.v), wl.cu_prefix, table, wl.num_blocks,
                                      sentinel=SENTINEL)
    assert np.array_equal(kc, ref_k), "k_cache image differs (slot mapping or sentinel slots)"
    assert np.array_equal(vc, ref_v), "v_cache image differs (slot mapping or sentinel slots)"


@pytest.mark.parametrize("seed", range(10))
def test_c1_tiny_fp32_all_rows(cuda_device, seed):
    """C1 (fp32 tensors) against the unrounded oracle, every row, ten seeds.  The fp32 path keeps q, the response's
    own K/V and all products in fp32; what remains is the rounding of the prompt's K/V in the bf16 cache, which only
    the response rows see (a few 1e-3)."""
    wl = wk.make_workload(wk.CONFIGS["C1"], seed=seed, lm=False)
    out, lse, kc, vc, _ = run_split(wl, cuda_device)
    rows = oracle.all_rows(wl.cu_full, wl.cfg.num_q_heads)
    check_rows(wl, out, lse, rows, lse_tol=1e-2)
    check_cache(wl, kc, vc)
    pre = rows[rows[:, 1] < wl.prompt_lens[rows[:, 0]]]
    ref_o, ref_l = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, pre)
    tok = wl.cu_full[pre[:, 0]].astype(np.int64) + pre[:, 1]
    assert np.abs(out[tok, pre[:, 2]] - ref_o).max() <= 5e-5   # prompt rows: fp32 accuracy
    assert np.abs(lse[tok, pre[:, 2]] - ref_l).max() <= 5e-5


RAGGED = [
    # (head_dim, q heads, kv heads, prompt lengths, response lengths)
    (128, 4, 2, [300, 77, 128, 1, 513], [40, 150, 0, 5, 257]),
    (128, 7, 1, [16, 17, 255, 256, 257], [1, 128, 129, 2, 300]),
    (64, 6, 3, [129, 31, 400], [260, 3, 64]),
    (128, 2, 2, [0, 5, 0], [33, 0, 0]),          # empty prompts, empty responses, an empty sequence
]


@pytest.mark.parametrize("d,hq,hkv,plens,rlens", RAGGED)
def test_ragged_batches_all_rows(cuda_device, d, hq, hkv, plens, rlens):
    cfg = wk.Config("t", "bf16", len(plens), hq, hkv, d, 64, 64, ("list", plens), ("list", rlens))
    wl = wk.make_workload(cfg, seed=11, lm=False)
    out, lse, kc, vc, _ = run_split(wl, cuda_device)
    rows = oracle.all_rows(wl.cu_full, hq)
    check_rows(wl, out, lse, rows)
    check_cache(wl, kc, vc)


def test_block_shuffle_is_invisible_and_runs_repeat_bit_exactly(cuda_device):
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 64, 64, ("list", [200, 333, 48]), ("list", [100, 20, 260]))
    wl = wk.make_workload(cfg, seed=12, lm=False)
    _, _, kc1, _, (p1, s1) = run_split(wl, cuda_device)
    _, _, kc1b, _, (p1b, s1b) = run_split(wl, cuda_device)
    assert torch.equal(p1, p1b) and torch.equal(s1, s1b) and np.array_equal(kc1, kc1b)
    other, _ = wk.make_block_table(wl.prompt_lens, seed=77)
    assert not np.array_equal(other, wl.block_table)
    _, _, kc2, vc2, (p2, s2) = run_split(wl, cuda_device, table=other)
    assert torch.equal(p1, p2) and torch.equal(s1, s2)
    check_cache(wl, kc2, vc2, table=other)


def test_prefix_without_cache_and_explicit_scale(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 2, 4, 4, 128, 64, 64, ("list", [150, 260]), ("list", [0, 0]))
    wl = wk.make_workload(cfg, seed=13, lm=False)
    q, k, v = (to_device(t, dev) for t in (wl.q, wl.k, wl.v))
    o = rpx.prefix_attn(q, k, v, to_device(wl.cu_full, dev), 260, cache=None, softmax_scale=0.05)
    torch.cuda.synchronize()
    rows = oracle.all_rows(wl.cu_full, 4)
    ref, _ = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, rows, scale=0.05)
    err = np.abs(o.double().cpu().numpy().reshape(-1, 128) - ref).max()
    assert err <= TOL


def test_suffix_pass_split_over_the_cached_prefix(cuda_device):
    """Few, long work items: the launcher cuts every item's cached prefix into ranges taken by different
    CTAs and the last to arrive merges the partial rows.  Mixed prefix lengths: 32 tiles (4 ranges), one
    tile (not split), 20 tiles with a ragged last one; ragged response lengths leave warps without rows."""
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 64, 64, ("list", [4000, 100, 2500]), ("list", [200, 300, 64]))
    wl = wk.make_workload(cfg, seed=17, lm=False)
    out, lse, kc, vc, (p1, s1) = run_split(wl, cuda_device)
    rows = oracle.all_rows(wl.cu_full, cfg.num_q_heads)
    suffix_only = rows[rows[:, 1] >= wl.prompt_lens[rows[:, 0]]]
    check_rows(wl, out, lse, suffix_only)
    check_rows(wl, out, lse, sample_prefix_rows(wl, rows))
    # the merge order of the ranges depends on which CTA arrives last, the merged bits do not
    _, _, _, _, (p2, s2) = run_split(wl, cuda_device)
    assert torch.equal(s1, s2)


def test_suffix_pass_split_in_two_with_head_dim_64(cuda_device):
    """Nine cached tiles at most: two ranges; a 3-tile prefix is cut 1 + 2, a sequence without prefix not at all."""
    cfg = wk.Config("t", "bf16", 3, 8, 1, 64, 64, 64, ("list", [1100, 300, 0]), ("list", [130, 256, 40]))
    wl = wk.make_workload(cfg, seed=18, lm=False)
    out, lse, kc, vc, _ = run_split(wl, cuda_device)
    check_rows(wl, out, lse, oracle.all_rows(wl.cu_full, cfg.num_q_heads))
    check_cache(wl, kc, vc)


def sample_prefix_rows(wl, rows, n=400):
    pre = rows[rows[:, 1] < wl.prompt_lens[rows[:, 0]]]
    pick = np.random.default_rng(5).choice(pre.shape[0], size=min(n, pre.shape[0]), replace=False)
    return pre[np.sort(pick)]


def test_sm_budget_changes_no_bit_of_the_attention_outputs(cuda_device):
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 64, 64, ("list", [600, 333, 48]), ("list", [100, 20, 260]))
    wl = wk.make_workload(cfg, seed=15, lm=False)
    _, _, kc1, vc1, (p1, s1) = run_split(wl, cuda_device)
    try:
        for budget in (1, 5, 147):
            rpx.set_sm_budget(budget)
            _, _, kc2, vc2, (p2, s2) = run_split(wl, cuda_device)
            assert torch.equal(p1, p2) and torch.equal(s1, s2)
            assert np.array_equal(kc1, kc2) and np.array_equal(vc1, vc2)
    finally:
        rpx.set_sm_budget(0)


@pytest.mark.parametrize("growth", [40.0, 400.0])
def test_scores_that_keep_growing_force_the_running_maximum_to_move(cuda_device, growth):
    """Key norms grow along the sequence, so every 128-key tile raises the row maximum by tens
    (growth 40) or hundreds (growth 400: the old accumulator underflows to zero) of log2 units:
    the lazy rescale of O and of the row sum has to fire on every step, in the prefix pass, the
    suffix pass over the cached prefix, and across the prefix/suffix boundary."""
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 64, 64, ("list", [1000, 130, 520]), ("list", [300, 140, 0]))
    wl = wk.make_workload(cfg, seed=21, lm=False)
    k = wk.bf16_bits_to_f32(wl.k)
    for s_ in range(cfg.batch):
        lo, hi = int(wl.cu_full[s_]), int(wl.cu_full[s_ + 1])
        ramp = 1.0 + (growth - 1.0) * np.arange(hi - lo, dtype=np.float32) / max(hi - lo - 1, 1)
        k[lo:hi] *= ramp[:, None, None]
    wl.k = wk.f32_to_bf16_bits(k).reshape(wl.k.shape)
    out, lse, kc, vc, _ = run_split(wl, cuda_device)
    rows = oracle.all_rows(wl.cu_full, cfg.num_q_heads)
    # With scores this steep a row's weight sits on two or three keys, so nothing averages out the
    # rounding of the bf16 probabilities (up to 2^-8 relative each): allow 2^-8 * max|v| on top.
    # LSE is hundreds of nats here; fp32 carries it to about 1e-7 relative.
    v_max = float(np.abs(wk.bf16_bits_to_f32(wl.v)).max())
    check_rows(wl, out, lse, rows, lse_tol=1e-3 * growth / 40.0, o_extra=v_max / 256.0)
    check_cache(wl, kc, vc)


def test_gpu_split_equals_gpu_monolithic_through_the_lm_head(cuda_device):
    """Chain attention into the LM head (hidden = O reshaped, H = H_q * d): log-probs from
    prefix+suffix attention must match log-probs from one-pass attention within 1e-3."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 512, 3000, ("list", [700, 130, 257]), ("list", [90, 300, 129]))
    wl = wk.make_workload(cfg, seed=14)
    _, _, _, _, (o_pre, o_suf) = run_split(wl, dev)
    q, k, v = (to_device(t, dev) for t in (wl.q, wl.k, wl.v))
    o_mono = rpx.prefix_attn(q, k, v, to_device(wl.cu_full, dev), int((wl.prompt_lens + wl.response_lens).max()))
    o_split = torch.empty_like(o_mono)
    o_split[torch.from_numpy(wl.prefix_rows()).to(dev)] = o_pre
    o_split[torch.from_numpy(wl.suffix_rows()).to(dev)] = o_suf
    w, ids = to_device(wl.w, dev), to_device(wl.ids, dev)
    lp_mono = rpx.token_logprobs(o_mono.reshape(wl.n_tokens, 512), w, ids)
    lp_split = rpx.token_logprobs(o_split.reshape(wl.n_tokens, 512), w, ids)
    torch.cuda.synchronize()
    diff_o = (o_mono.float() - o_split.float()).abs().max().item()
    diff_lp = (lp_mono - lp_split).abs().max().item()
    assert diff_o <= TOL
    assert diff_lp <= 1e-3, f"split vs monolithic log-prob differs by {diff_lp:.3e}"
    ref, _ = oracle.logprob_rows(bf16_bits(o_mono.reshape(wl.n_tokens, 512)), wl.w, wl.ids)
    assert np.abs(lp_mono.double().cpu().numpy() - ref).max() <= 2e-2


@pytest.mark.parametrize("name,n_rows", [("C2", 256), ("C4", 96), ("C5", 192), ("C3", 192)])
def test_full_size_configs_sampled_rows(cuda_device, name, n_rows):
    """BASELINE configs at full size, launch configuration as benchmarked; the oracle evaluates a
    stratified sample of rows (first rows, tile edges, around the prefix/suffix split, last rows)."""
    wl = wk.make_workload(wk.CONFIGS[name], seed=0, lm=False)
    out, lse, kc, vc, _ = run_split(wl, cuda_device)
    rows = wk.sample_attn_rows(wl, n_rows, seed=2)
    check_rows(wl, out, lse, rows)
    check_cache(wl, kc, vc)
