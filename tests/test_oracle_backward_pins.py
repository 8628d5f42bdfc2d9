"""Pins for the backward routines of the fp64 CPU oracle (gradients through the prefix/suffix boundary,
Section 3.2 and Table 4), checked without any GPU.

The paper prints no worked example, so the pins are what the mathematics fixes: central finite differences of the
FORWARD oracle routines (which are pinned on their own), torch's fp64 autograd on a differently structured
evaluation, closed forms, the identity sum_v dL/dz_v = 0, and the paper's invariant that the split evaluation
(prefix queries and suffix queries accumulated separately into the prefix K/V gradients) equals the one-pass sums.
"""
import numpy as np
import pytest
import torch

import oracle


def _grid(shape, seed, scale=1.0):
    """float32 values on a 2^-8 grid, so that x +- 2^-9 is exact in float32 (for finite differences)."""
    x = np.random.default_rng(seed).standard_normal(shape) * scale
    return (np.round(x * 256.0) / 256.0).astype(np.float32)


def _batch(lens, hq, hkv, d, seed):
    n = int(np.sum(lens))
    cu = np.zeros(len(lens) + 1, np.int32)
    cu[1:] = np.cumsum(lens)
    return _grid((n, hq, d), seed), _grid((n, hkv, d), seed + 1), _grid((n, hkv, d), seed + 2), cu


def _attn_loss(q, k, v, cu, dout):
    rows = oracle.all_rows(cu, q.shape[1])
    out, _ = oracle.attn_rows(q, k, v, cu, rows)
    tok = cu[rows[:, 0]].astype(np.int64) + rows[:, 1]
    return float((out * dout[tok, rows[:, 2]]).sum())


# ---------------------------------------------------------------- finite differences of the forward oracle
@pytest.mark.parametrize("lens,hq,hkv,d", [([5, 3], 4, 2, 4), ([6], 3, 1, 2), ([1, 4, 2], 2, 2, 3)])
def test_attention_backward_matches_finite_differences_of_the_forward_oracle(lens, hq, hkv, d):
    q, k, v, cu = _batch(lens, hq, hkv, d, 300)
    dout = np.random.default_rng(9).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(q, k, v, cu, dout)
    eps = 2.0 ** -9
    rng = np.random.default_rng(10)
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(12):
            idx = tuple(int(rng.integers(0, n)) for n in arr.shape)
            saved = arr[idx]
            arr[idx] = saved + eps
            up = _attn_loss(q, k, v, cu, dout)
            arr[idx] = saved - eps
            down = _attn_loss(q, k, v, cu, dout)
            arr[idx] = saved
            fd = (up - down) / (2 * eps)
            assert abs(fd - grad[idx]) <= 2e-5 * max(1.0, abs(fd)), (name, idx, fd, grad[idx])


def test_logprob_backward_matches_finite_differences_of_the_forward_oracle():
    n, hdim, vocab = 4, 6, 9
    hidden, w = _grid((n, hdim), 310), _grid((vocab, hdim), 311, 0.5)
    ids = np.array([3, 0, 8, 5], dtype=np.int32)
    g = np.array([1.0, -0.5, 2.0, 0.25])
    dh, dw = oracle.logprob_backward(hidden, w, ids, g, want_dw=True)

    def loss():
        lp, _ = oracle.logprob_rows(hidden, w, ids)
        return float((lp * g).sum())

    eps = 2.0 ** -9
    for arr, grad in ((hidden, dh), (w, dw)):
        for idx in np.ndindex(arr.shape):
            saved = arr[idx]
            arr[idx] = saved + eps
            up = loss()
            arr[idx] = saved - eps
            down = loss()
            arr[idx] = saved
            fd = (up - down) / (2 * eps)
            assert abs(fd - grad[idx]) <= 2e-5 * max(1.0, abs(fd)), (idx, fd, grad[idx])


# ---------------------------------------------------------------- torch fp64 autograd, other structure
def _torch_attention(q, k, v, cu, scale):
    """Dense masked softmax per sequence with the KV heads replicated explicitly."""
    hq, hkv = q.shape[1], k.shape[1]
    outs = []
    for s in range(len(cu) - 1):
        a, b = int(cu[s]), int(cu[s + 1])
        qq = q[a:b].transpose(0, 1)                                       # [hq, n, d]
        kk = k[a:b].repeat_interleave(hq // hkv, dim=1).transpose(0, 1)   # [hq, n, d]
        vv = v[a:b].repeat_interleave(hq // hkv, dim=1).transpose(0, 1)
        sc = qq @ kk.transpose(1, 2) * scale
        mask = torch.ones(b - a, b - a, dtype=torch.bool).tril()
        sc = sc.masked_fill(~mask, float("-inf"))
        outs.append((torch.softmax(sc, dim=-1) @ vv).transpose(0, 1))
    return torch.cat(outs, dim=0)


@pytest.mark.parametrize("lens,hq,hkv,d", [([9, 4, 1], 6, 2, 8), ([17], 4, 4, 16), ([5, 5], 8, 1, 4)])
def test_attention_backward_matches_torch_autograd(lens, hq, hkv, d):
    q, k, v, cu = _batch(lens, hq, hkv, d, 320)
    dout = np.random.default_rng(11).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(q, k, v, cu, dout)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    out = _torch_attention(tq, tk, tv, cu, 1.0 / np.sqrt(d))
    (out * torch.tensor(dout)).sum().backward()
    assert np.abs(dq - tq.grad.numpy()).max() <= 1e-10
    assert np.abs(dk - tk.grad.numpy()).max() <= 1e-10
    assert np.abs(dv - tv.grad.numpy()).max() <= 1e-10


def test_attention_backward_reads_bf16_bits_and_a_custom_scale():
    from paper_2608_14498_b200 import workloads as wk

    q, k, v, cu = _batch([6, 3], 4, 2, 8, 330)
    qb, kb, vb = (wk.f32_to_bf16_bits(x).reshape(x.shape) for x in (q, k, v))
    dout = np.random.default_rng(12).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(qb, kb, vb, cu, dout, scale=0.3)
    tq, tk, tv = (torch.tensor(wk.bf16_bits_to_f32(x).reshape(x.shape), dtype=torch.float64, requires_grad=True)
                  for x in (qb, kb, vb))
    (_torch_attention(tq, tk, tv, cu, 0.3) * torch.tensor(dout)).sum().backward()
    assert np.abs(dq - tq.grad.numpy()).max() <= 1e-10
    assert np.abs(dk - tk.grad.numpy()).max() <= 1e-10
    assert np.abs(dv - tv.grad.numpy()).max() <= 1e-10


def test_logprob_backward_matches_torch_autograd():
    n, hdim, vocab = 7, 24, 50
    hidden, w = _grid((n, hdim), 340), _grid((vocab, hdim), 341, 0.3)
    ids = np.random.default_rng(13).integers(0, vocab, n).astype(np.int32)
    g = np.random.default_rng(14).standard_normal(n)
    dh, dw = oracle.logprob_backward(hidden, w, ids, g, want_dw=True)
    th = torch.tensor(hidden, dtype=torch.float64, requires_grad=True)
    tw = torch.tensor(w, dtype=torch.float64, requires_grad=True)
    lp = torch.log_softmax(th @ tw.T, dim=-1).gather(1, torch.tensor(ids, dtype=torch.int64)[:, None])[:, 0]
    (lp * torch.tensor(g)).sum().backward()
    assert np.abs(dh - th.grad.numpy()).max() <= 1e-10
    assert np.abs(dw - tw.grad.numpy()).max() <= 1e-10
    assert np.array_equal(dh, oracle.logprob_backward(hidden, w, ids, g))  # dw is optional


# ---------------------------------------------------------------- closed forms and identities
def test_one_key_sequences_pass_the_gradient_straight_to_v():
    # a sequence of one token: P = 1, so dS = 0, dQ = dK = 0, and dV is dO summed over the heads of the group
    q, k, v, cu = _batch([1, 1, 1], 4, 2, 5, 350)
    dout = np.random.default_rng(15).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(q, k, v, cu, dout)
    assert np.abs(dq).max() == 0.0 and np.abs(dk).max() == 0.0
    assert np.abs(dv - dout.reshape(3, 2, 2, 5).sum(axis=2)).max() <= 1e-15


def test_zero_queries_give_running_mean_gradients():
    # Q = 0: every row weighs its keys equally, P_ij = 1 / (i + 1); dK = scale * sum dS * Q = 0 and
    # dV[j] = sum_{i >= j} dO[i] / (i + 1), summed over the heads of the group
    lens, hq, hkv, d = [6], 2, 1, 3
    q, k, v, cu = _batch(lens, hq, hkv, d, 360)
    q[:] = 0
    dout = np.random.default_rng(16).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(q, k, v, cu, dout)
    assert np.abs(dk).max() == 0.0
    want = np.zeros_like(dv)
    for j in range(6):
        for i in range(j, 6):
            want[j, 0] += dout[i].sum(axis=0) / (i + 1)
    assert np.abs(dv - want).max() <= 1e-14
    # dQ[i] = scale * sum_j P_ij (dP_ij - D_i) K_j with dP_ij = dO[i] . V_j: written out independently
    scale = 1.0 / np.sqrt(d)
    for i in range(6):
        for h in range(hq):
            dp = np.array([dout[i, h] @ v[j, 0].astype(np.float64) for j in range(i + 1)])
            ds = (dp - dp.mean()) / (i + 1)
            assert np.abs(dq[i, h] - scale * (ds[:, None] * k[:i + 1, 0].astype(np.float64)).sum(axis=0)).max() <= 1e-14


def test_logit_gradients_sum_to_zero_and_zero_hidden_gives_the_centred_target_row():
    n, hdim, vocab = 5, 8, 13
    hidden = _grid((n, hdim), 370)
    ids = np.array([0, 12, 5, 5, 7], dtype=np.int32)
    g = np.array([1.0, 2.0, -1.0, 0.5, 3.0])
    # every row of W the same vector: dhidden = (sum_v dL/dz_v) * that vector = 0, whatever the softmax is
    w_same = np.tile(_grid((1, hdim), 371), (vocab, 1))
    assert np.abs(oracle.logprob_backward(hidden, w_same, ids, g)).max() <= 1e-15
    # hidden = 0: uniform softmax, so dhidden[n] = g[n] * (W[target] - mean_v W[v]) and dW = 0
    w = _grid((vocab, hdim), 372)
    dh, dw = oracle.logprob_backward(np.zeros_like(hidden), w, ids, g, want_dw=True)
    w64 = w.astype(np.float64)
    assert np.abs(dh - g[:, None] * (w64[ids] - w64.mean(axis=0))).max() <= 1e-14
    assert np.abs(dw).max() == 0.0
    # the gradient is linear in the upstream gradient
    dh1 = oracle.logprob_backward(hidden, w, ids, g)
    dh2 = oracle.logprob_backward(hidden, w, ids, 2.0 * g)
    assert np.abs(dh2 - 2.0 * dh1).max() <= 1e-14


# ---------------------------------------------------------------- split == monolithic (the paper's invariant)
def _split_backward(q, k, v, cu, plens, dout, scale):
    """Independent numpy evaluation in the split form: for every sequence, the prefix pass (prompt queries over prompt
    keys) and the suffix pass (response queries over [prompt keys ; response keys]) each produce dQ for their own rows
    and their own additions to dK / dV; the prompt keys' gradients are the SUM of both passes' additions."""
    hq, hkv = q.shape[1], k.shape[1]
    grp = hq // hkv
    dq, dk, dv = (np.zeros(x.shape) for x in (q, k, v))
    q, k, v = (x.astype(np.float64) for x in (q, k, v))
    for s in range(len(cu) - 1):
        a, b, p = int(cu[s]), int(cu[s + 1]), int(plens[s])
        for rows in (range(0, p), range(p, b - a)):   # the two passes
            for h in range(hq):
                g = h // grp
                for i in rows:
                    sc = (k[a:a + i + 1, g] @ q[a + i, h]) * scale
                    pr = np.exp(sc - sc.max())
                    pr /= pr.sum()
                    dp = v[a:a + i + 1, g] @ dout[a + i, h]
                    ds = pr * (dp - (pr * dp).sum())
                    dq[a + i, h] = scale * ds @ k[a:a + i + 1, g]
                    dk[a:a + i + 1, g] += scale * np.outer(ds, q[a + i, h])
                    dv[a:a + i + 1, g] += np.outer(pr, dout[a + i, h])
    return dq, dk, dv


def test_prefix_plus_suffix_backward_equals_monolithic_backward():
    lens, plens = [11, 6, 4], [7, 6, 0]
    q, k, v, cu = _batch(lens, 4, 2, 8, 380)
    dout = np.random.default_rng(17).standard_normal(q.shape)
    dq, dk, dv = oracle.attn_backward(q, k, v, cu, dout)
    sq, sk, sv = _split_backward(q, k, v, cu, plens, dout, 1.0 / np.sqrt(8))
    assert np.abs(dq - sq).max() <= 1e-12
    assert np.abs(dk - sk).max() <= 1e-12
    assert np.abs(dv - sv).max() <= 1e-12
    # and the prompt keys really do receive gradient from the response queries: dropping the suffix pass changes them
    dout_prefix_only = dout.copy()
    for s in range(3):
        dout_prefix_only[cu[s] + plens[s]:cu[s + 1]] = 0.0
    _, dk_p, dv_p = oracle.attn_backward(q, k, v, cu, dout_prefix_only)
    assert np.abs(dk[:7] - dk_p[:7]).max() > 1e-3 and np.abs(dv[:7] - dv_p[:7]).max() > 1e-3
