"""The training actor's backward schedule end to end on the GPU (Section 3.2): log-probs -> hidden rows -> attention
output -> Q, K, V, with the suffix pass differentiated first and the prefix pass's gradients added on top, against
the oracle's gradients of the same chain.

The chain: hidden = attention output viewed as [tokens, H_q * d]; loss = sum_n g[n] * logprob[n].  Both sides take
the LM head's gradient at the GPU's bf16 attention output (the values the LM head read); the oracle then
differentiates its own fp64 attention with that upstream gradient."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from paper_2608_14498_b200.pipeline import backward_through_boundary
from helpers import bf16_bits, to_device

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lens,prompts,hq,hkv,d,vocab", [
    ([300, 77, 200, 129], [256, 50, 0, 129], 4, 2, 64, 1000),
    ([260, 131], [130, 64], 2, 1, 128, 513),
])
def test_gradients_cross_the_boundary_like_the_oracles(cuda_device, lens, prompts, hq, hkv, d, vocab):
    dev = cuda_device
    n = int(sum(lens))
    rng = np.random.default_rng(77)
    bits = lambda a: wk.f32_to_bf16_bits(a.astype(np.float32)).reshape(a.shape)
    q, k, v = bits(rng.standard_normal((n, hq, d))), bits(rng.standard_normal((n, hkv, d))), bits(rng.standard_normal((n, hkv, d)))
    w = bits(rng.standard_normal((vocab, hq * d)) * 0.05)
    ids = rng.integers(0, vocab, n).astype(np.int32)
    g = rng.standard_normal(n).astype(np.float32)
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    tq, tk, tv, tw, tids, tcu = (to_device(x, dev) for x in (q, k, v, w, ids, cu))
    tp = torch.tensor(prompts, dtype=torch.int32, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out, attn_lse = rpx.prefix_attn(tq, tk, tv, tcu, max(lens), return_lse=True, device_status=status)
    _, lm_lse = rpx.token_logprobs(out.reshape(n, hq * d), tw, tids, return_lse=True, device_status=status)
    dq_s, dq_p, dk, dv = backward_through_boundary(tq, tk, tv, out, attn_lse, tcu, tp, max(lens), tw, tids, lm_lse,
                                                   torch.from_numpy(g).to(dev), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # ---- the oracle's chain
    hidden_bits = bf16_bits(out).reshape(n, hq * d)
    dh = oracle.logprob_backward(hidden_bits, w, ids, g.astype(np.float64))
    rq, rk, rv = oracle.attn_backward(q, k, v, cu, dh.reshape(n, hq, d))
    # the two calls own disjoint rows of dq
    is_prompt = np.zeros(n, bool)
    for s, p in enumerate(prompts):
        is_prompt[cu[s]: cu[s] + p] = True
    got_s, got_p = dq_s.double().cpu().numpy(), dq_p.double().cpu().numpy()
    assert np.abs(got_s[is_prompt]).max(initial=0.0) == 0.0 and np.abs(got_p[~is_prompt]).max(initial=0.0) == 0.0
    got_q = np.where(is_prompt[:, None, None], got_p, got_s)
    for name, got, ref in (("dq", got_q, rq), ("dk", dk.double().cpu().numpy(), rk), ("dv", dv.double().cpu().numpy(), rv)):
        bound = 0.015 * np.abs(ref).max() + np.abs(ref) * 2.0 ** -7
        err = np.abs(got - ref)
        assert np.isfinite(got).all()
        assert (err <= bound).all(), f"{name}: max err {err.max():.3e} of max |ref| {np.abs(ref).max():.3e}"
    # the response rows' gradient does reach the prompt's keys: dk of the prompt rows differs from what the prompt rows
    # alone would give
    dout = to_device(bits(dh.reshape(n, hq, d)), dev)
    _, dk_only_prefix, _ = rpx.attn_backward(tq, tk, tv, out, dout, attn_lse, tcu, max(lens), q_end=tp,
                                             device_status=status)
    torch.cuda.synchronize()
    rows = np.where(is_prompt)[0]
    assert float((dk[rows] - dk_only_prefix[rows]).abs().max()) > 1e-3 * float(dk.abs().max())
