"""GPU parity of rpx_attn_backward (through the C ABI) against the fp64 oracle's gradients.

The forward pass that supplies out and lse is the library's own (rpx_prefix_attn over the whole sequences), so the
test covers the chain a caller runs.  Both sides read the same bf16 bits of q, k, v and dout.

Tolerance.  The kernel rounds P and dS to bf16 before the tensor-core products (2^-9 relative per term, random
signs), evaluates 2^x with the special-function unit (2^-22), and computes D_i = sum_c dO O from the bf16 output of the
forward pass.  The last one dominates: each O element is off by up to 2^-9 relative, which moves D_i by about
2^-9 * sqrt(d) * |dO| |O| ~ 0.01 for unit-variance data, and dS_ij = P_ij (dP_ij - D_i) by P_ij times that - an ABSOLUTE
error of about scale * 0.01 * |K| ~ 5e-3 in dq (likewise dk), also in rows whose true gradient is small because
dP_ij - D_i nearly cancels (early rows with a few keys).  So the bound is set against the largest magnitude of the
whole gradient tensor (1 % of it) plus 2^-7 relative per element; a wrong term, sign, mask or index moves entries
by the size of the gradient itself."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device

pytestmark = pytest.mark.gpu


def _batch(lens, hq, hkv, d, seed):
    n = int(sum(lens))
    rng = np.random.default_rng(seed)
    q = wk.f32_to_bf16_bits(rng.standard_normal((n, hq, d)).astype(np.float32)).reshape(n, hq, d)
    k = wk.f32_to_bf16_bits(rng.standard_normal((n, hkv, d)).astype(np.float32)).reshape(n, hkv, d)
    v = wk.f32_to_bf16_bits(rng.standard_normal((n, hkv, d)).astype(np.float32)).reshape(n, hkv, d)
    dout = wk.f32_to_bf16_bits(rng.standard_normal((n, hq, d)).astype(np.float32)).reshape(n, hq, d)
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return q, k, v, dout, cu


def _forward(dev, q, k, v, cu, max_len, scale=0.0):
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out, lse = rpx.prefix_attn(q, k, v, cu, max_len, softmax_scale=scale, return_lse=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return out, lse


def _close(got, ref, what):
    got = got.double().cpu().numpy()
    assert np.isfinite(got).all(), what
    bound = 0.01 * np.abs(ref).max() + np.abs(ref) * 2.0 ** -7 + 1e-6
    err = np.abs(got - ref)
    assert (err <= bound).all(), (f"{what}: max excess {(err - bound).max():.3e}, max err {err.max():.3e}, "
                                  f"max |ref| {np.abs(ref).max():.3e} at {np.unravel_index((err - bound).argmax(), err.shape)}")


def _masked_dout(dout_bits, cu, q_begin, q_end):
    """The oracle's way of restricting the query rows: rows outside the range get a zero upstream gradient."""
    dout = wk.bf16_bits_to_f32(dout_bits).reshape(dout_bits.shape).astype(np.float64)
    if q_begin is None and q_end is None:
        return dout
    keep = np.zeros(dout.shape[0], bool)
    for s in range(cu.shape[0] - 1):
        a, n = int(cu[s]), int(cu[s + 1] - cu[s])
        lo = 0 if q_begin is None else max(0, int(q_begin[s]))
        hi = n if q_end is None else min(n, int(q_end[s]))
        keep[a + lo: a + max(lo, hi)] = True
    dout[~keep] = 0.0
    return dout


def _run(dev, lens, hq, hkv, d, seed, q_begin=None, q_end=None, scale=0.0):
    q, k, v, dout, cu = _batch(lens, hq, hkv, d, seed)
    tq, tk, tv, tdo, tcu = (to_device(x, dev) for x in (q, k, v, dout, cu))
    max_len = int(max(lens)) if len(lens) else 0
    out, lse = _forward(dev, tq, tk, tv, tcu, max_len, scale)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    tb = None if q_begin is None else torch.tensor(q_begin, dtype=torch.int32, device=dev)
    te = None if q_end is None else torch.tensor(q_end, dtype=torch.int32, device=dev)
    dq, dk, dv = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max_len, q_begin=tb, q_end=te, softmax_scale=scale,
                                   device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rq, rk, rv = oracle.attn_backward(q, k, v, cu, _masked_dout(dout, cu, q_begin, q_end),
                                      scale=None if scale == 0.0 else scale)
    _close(dq, rq, "dq")
    _close(dk, rk, "dk")
    _close(dv, rv, "dv")
    return (tq, tk, tv, out, tdo, lse, tcu, max_len), (dq, dk, dv)


@pytest.mark.parametrize("lens,hq,hkv,d", [
    ([300, 129, 1, 128, 517], 4, 2, 128),   # several tiles, ragged tails, a one-token sequence
    ([700, 5], 8, 1, 128),                  # one KV head shared by eight query heads
    ([257, 64, 383], 2, 2, 64),             # head_dim 64, no grouping
    ([130], 6, 2, 64),
    ([1], 2, 1, 128),
])
def test_gradients_match_the_oracle(cuda_device, lens, hq, hkv, d):
    _run(cuda_device, lens, hq, hkv, d, 500 + len(lens) + hq)


def test_a_custom_scale_and_empty_sequences(cuda_device):
    _run(cuda_device, [0, 200, 0, 131, 0], 4, 2, 128, 511, scale=0.2)


def test_row_ranges_give_the_suffix_and_the_prefix_pass(cuda_device):
    dev = cuda_device
    lens, prompt = [400, 150, 260, 90], [256, 100, 0, 90]   # a prompt that is a tile multiple, a ragged one, none, all
    # suffix pass: response rows only
    _run(dev, lens, 4, 2, 128, 520, q_begin=prompt)
    # prefix pass: prompt rows only
    _run(dev, lens, 4, 2, 128, 520, q_end=prompt)
    # a window strictly inside, and ranges that reach outside the sequence (clamped)
    _run(dev, lens, 4, 1, 64, 521, q_begin=[130, -5, 300, 10], q_end=[140, 1000, 200, 11])


def test_suffix_call_plus_accumulating_prefix_call_equals_one_call(cuda_device):
    dev = cuda_device
    lens, prompt = [385, 200, 131], [200, 128, 77]
    (tq, tk, tv, out, tdo, lse, tcu, max_len), (dq, dk, dv) = _run(dev, lens, 8, 2, 128, 530)
    tp = torch.tensor(prompt, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    dq_s, dk2, dv2 = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max_len, q_begin=tp, device_status=status)
    dk_suffix_on_prompt = dk2.clone()
    dq_p, dk2, dv2 = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max_len, q_end=tp, dk=dk2, dv=dv2,
                                       accumulate_dkv=True, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # dq: each row is produced by exactly one of the two calls and by the same arithmetic as in the single call
    assert torch.equal(dq_s + dq_p, dq)
    # dk, dv: the same terms in another summation order
    scale = float(dk.abs().max())
    assert float((dk2 - dk).abs().max()) <= 1e-5 * scale
    assert float((dv2 - dv).abs().max()) <= 1e-5 * float(dv.abs().max())
    # the suffix pass alone does reach the prompt's keys (the gradient crosses the boundary) ...
    cu = tcu.cpu().numpy()
    first_prompt_rows = dk_suffix_on_prompt[int(cu[0]): int(cu[0]) + prompt[0]]
    assert float(first_prompt_rows.abs().max()) > 0.0
    # ... and without accumulate the second call would have overwritten it
    _, dk3, _ = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max_len, q_end=tp, device_status=status)
    torch.cuda.synchronize()
    assert float((dk3 - dk).abs().max()) > 1e-3 * scale


def test_strided_qkv_views_of_a_fused_projection(cuda_device):
    dev = cuda_device
    lens, hq, hkv, d = [260, 77], 4, 2, 128
    q, k, v, dout, cu = _batch(lens, hq, hkv, d, 540)
    n = q.shape[0]
    fused = torch.zeros((n, hq + 2 * hkv, d), dtype=torch.bfloat16, device=dev)
    fused[:, :hq] = to_device(q, dev)
    fused[:, hq:hq + hkv] = to_device(k, dev)
    fused[:, hq + hkv:] = to_device(v, dev)
    tq, tk, tv = fused[:, :hq], fused[:, hq:hq + hkv], fused[:, hq + hkv:]
    tcu, tdo = to_device(cu, dev), to_device(dout, dev)
    out, lse = _forward(dev, tq, tk, tv, tcu, max(lens))
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    dq, dk, dv = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max(lens), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rq, rk, rv = oracle.attn_backward(q, k, v, cu, _masked_dout(dout, cu, None, None))
    _close(dq, rq, "dq")
    _close(dk, rk, "dk")
    _close(dv, rv, "dv")


def test_sequence_offsets_that_leave_the_tensors_are_reported(cuda_device):
    dev = cuda_device
    lens, hq, hkv, d = [200, 100], 2, 1, 64
    q, k, v, dout, cu = _batch(lens, hq, hkv, d, 550)
    tq, tk, tv, tdo, tcu = (to_device(x, dev) for x in (q, k, v, dout, cu))
    out, lse = _forward(dev, tq, tk, tv, tcu, 200)
    bad = torch.tensor([0, 200, 100000], dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    dq, dk, dv = rpx.attn_backward(tq, tk, tv, out, tdo, lse, bad, 200, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -8
    # the well-formed sequence is still differentiated; the other one gets zeros
    rq, rk, rv = oracle.attn_backward(q[:200], k[:200], v[:200], cu[:2], _masked_dout(dout[:200], cu[:2], None, None))
    _close(dq[:200], rq, "dq")
    _close(dk[:200], rk, "dk")
    assert float(dq[200:].abs().max()) == 0.0 and float(dk[200:].abs().max()) == 0.0


def test_peaked_rows_and_a_long_sequence(cuda_device):
    dev = cuda_device
    # scores a few tens apart: most rows put their weight on one or two keys, P is 1 or ~0 and dS nearly cancels
    lens, hq, hkv, d = [300, 200], 4, 2, 64
    q, k, v, dout, cu = _batch(lens, hq, hkv, d, 570)
    q = wk.f32_to_bf16_bits(wk.bf16_bits_to_f32(q) * 4.0).reshape(q.shape)   # exact in bf16
    k = wk.f32_to_bf16_bits(wk.bf16_bits_to_f32(k) * 2.0).reshape(k.shape)
    tq, tk, tv, tdo, tcu = (to_device(x, dev) for x in (q, k, v, dout, cu))
    out, lse = _forward(dev, tq, tk, tv, tcu, 300)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    dq, dk, dv = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, 300, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rq, rk, rv = oracle.attn_backward(q, k, v, cu, _masked_dout(dout, cu, None, None))
    _close(dq, rq, "dq")
    _close(dk, rk, "dk")
    _close(dv, rv, "dv")
    # one long sequence: 40 key tiles, every inner-loop length from 1 to 40
    _run(dev, [5000], 2, 1, 64, 571)


EDGE = [1, 2, 63, 64, 65, 127, 128, 129, 191, 192, 193, 255, 256, 257, 383, 385]


@pytest.mark.parametrize("case", range(12))
def test_random_batches_with_random_row_ranges(cuda_device, case):
    rng = np.random.default_rng(3000 + case)
    group, hkv = int(rng.integers(1, 9)), int(rng.integers(1, 4))
    d = 128 if case % 3 else 64
    batch = int(rng.integers(1, 6))
    lens = [int(rng.choice(EDGE)) if rng.random() < 0.6 else int(rng.integers(0, 420)) for _ in range(batch)]
    if sum(lens) == 0:
        lens[0] = 5
    q_begin = q_end = None
    if case % 3 == 1:    # suffix-pass shape: a prompt length per sequence
        q_begin = [int(rng.integers(0, n + 1)) for n in lens]
    elif case % 3 == 2:  # arbitrary windows, some empty, some reaching outside
        q_begin = [int(rng.integers(-3, n + 2)) for n in lens]
        q_end = [int(rng.integers(-3, n + 5)) for n in lens]
    _run(cuda_device, lens, group * hkv, hkv, d, 3100 + case, q_begin=q_begin, q_end=q_end)


def test_a_sequence_longer_than_the_callers_bound_is_reported(cuda_device):
    dev = cuda_device
    lens, hq, hkv, d = [100, 400], 2, 1, 64
    q, k, v, dout, cu = _batch(lens, hq, hkv, d, 560)
    tq, tk, tv, tdo, tcu = (to_device(x, dev) for x in (q, k, v, dout, cu))
    out, lse = _forward(dev, tq, tk, tv, tcu, 400)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, 256, device_status=status)   # 400 > 256
    torch.cuda.synchronize()
    assert int(status.item()) == -8
    status.zero_()
    rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, 300, device_status=status)   # 300 rounds up to 384, still short of 400
    torch.cuda.synchronize()
    assert int(status.item()) == -8
    status.zero_()
    rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, 390, device_status=status)   # 390 rounds up to 512 >= 400
    torch.cuda.synchronize()
    assert int(status.item()) == 0


def test_c2_at_full_size_against_the_oracle_on_one_kv_group(cuda_device):
    """The benchmark's backward workload (C2: 8 whole sequences of 4352 tokens, 28 query / 4 KV heads, head_dim 128)
    through the same call the benchmark times; the oracle differentiates one (sequence, KV head) slice - attention
    and its gradients are independent per sequence and KV group, so the slice is a complete problem."""
    dev = cuda_device
    cfg = wk.CONFIGS["C2"]
    wl = wk.make_workload(cfg, seed=0, lm=False)
    dout = wk.make_workload(cfg, seed=1, lm=False).q
    tq, tk, tv, tdo, tcu = (to_device(x, dev) for x in (wl.q, wl.k, wl.v, dout, wl.cu_full))
    lens = (wl.prompt_lens + wl.response_lens).astype(np.int64)
    max_len = int(lens.max())
    out, lse = _forward(dev, tq, tk, tv, tcu, max_len)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    dq, dk, dv = rpx.attn_backward(tq, tk, tv, out, tdo, lse, tcu, max_len, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    seq, g = 5, 2
    group = cfg.num_q_heads // cfg.num_kv_heads
    a, b = int(wl.cu_full[seq]), int(wl.cu_full[seq + 1])
    hs = slice(g * group, (g + 1) * group)
    cu1 = np.array([0, b - a], dtype=np.int32)
    do64 = wk.bf16_bits_to_f32(dout[a:b, hs]).reshape(b - a, group, cfg.head_dim).astype(np.float64)
    rq, rk, rv = oracle.attn_backward(np.ascontiguousarray(wl.q[a:b, hs]), np.ascontiguousarray(wl.k[a:b, g:g + 1]),
                                      np.ascontiguousarray(wl.v[a:b, g:g + 1]), cu1, do64)
    _close(dq[a:b, hs], rq, "dq")
    _close(dk[a:b, g:g + 1], rk, "dk")
    _close(dv[a:b, g:g + 1], rv, "dv")
