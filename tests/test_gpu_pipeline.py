"""The scoring session: device-resident pass vs the overlapped host-resident pass vs the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_14498_b200 import workloads as wk
from paper_2608_14498_b200.pipeline import Batch, ScoringSession
from helpers import to_device

pytestmark = pytest.mark.gpu


def _host_batch(wl):
    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.pin_memory()

    pre, suf = wl.prefix_rows(), wl.suffix_rows()
    return Batch(t(wl.q[pre]), t(wl.k[pre]), t(wl.v[pre]), t(wl.q[suf]), t(wl.k[suf]), t(wl.v[suf]), t(wl.cu_prefix),
                 t(wl.cu_suffix), t(wl.prompt_lens), t(wl.block_table), t(wl.hidden[pre]), t(wl.ids[pre]),
                 t(wl.hidden[suf]), t(wl.ids[suf]), int(wl.prompt_lens.max()), int(wl.response_lens.max()))


def test_host_pass_equals_device_pass_and_oracle(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 512, 6000, ("list", [700, 130, 257]), ("list", [90, 300, 129]))
    wl = wk.make_workload(cfg, seed=31)
    hb = _host_batch(wl)
    db = Batch(*[x.to(dev) for x in hb.tensors()], hb.max_prefix_len, hb.max_suffix_len)
    sess = ScoringSession(to_device(wl.w, dev), wl.num_blocks, cfg.num_kv_heads, cfg.head_dim)
    lp_p, lp_s, o_p, o_s = sess.score(db)
    lp_p, lp_s, o_p, o_s = lp_p.clone(), lp_s.clone(), o_p.clone(), o_s.clone()
    host_p = torch.empty(wl.n_prefix, dtype=torch.float32).pin_memory()
    host_s = torch.empty(wl.n_suffix, dtype=torch.float32).pin_memory()
    for _ in range(2):  # the second pass reuses the staging buffers while the first may still be in flight
        sess.score_from_host(hb, host_p, host_s, lm_slices=3, min_slice_rows=128)
    torch.cuda.synchronize()
    sess.check_status()
    assert torch.equal(host_p, lp_p.cpu()) and torch.equal(host_s, lp_s.cpu())
    assert torch.equal(sess._out["o_p"], o_p) and torch.equal(sess._out["o_s"], o_s)
    assert sess.kernels_last_host_pass == 2 + 2 * (3 + 1)  # three prompt-row slices, one response-row call
    # against the oracle: concatenated prefix and suffix log-probs are the full-sequence values
    ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    got = np.empty(wl.n_tokens)
    got[wl.prefix_rows()] = host_p.double().numpy()
    got[wl.suffix_rows()] = host_s.double().numpy()
    assert np.abs(got - ref).max() <= 5e-4


def test_host_pass_with_sliced_response_rows(cuda_device):
    """Response-heavy batch (the text-workload shape): the response rows of the LM head are cut into
    slices too and run before the suffix attention; results must not depend on any of that."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 4, 4, 2, 64, 256, 1500, ("list", [40, 64, 17, 100]), ("list", [2500, 3000, 2400, 2100]))
    wl = wk.make_workload(cfg, seed=33)
    hb = _host_batch(wl)
    db = Batch(*[x.to(dev) for x in hb.tensors()], hb.max_prefix_len, hb.max_suffix_len)
    sess = ScoringSession(to_device(wl.w, dev), wl.num_blocks, cfg.num_kv_heads, cfg.head_dim)
    lp_p, lp_s, o_p, o_s = (x.clone() for x in sess.score(db))
    host_p = torch.empty(wl.n_prefix, dtype=torch.float32).pin_memory()
    host_s = torch.empty(wl.n_suffix, dtype=torch.float32).pin_memory()
    for _ in range(3):  # alternates between the two staging sets
        sess.score_from_host(hb, host_p, host_s)
    torch.cuda.synchronize()
    sess.check_status()
    # slices of 5000 rows sweep the vocabulary in shorter chunks than one call over 10000 rows, so the
    # partial sums are merged in another order: equal to fp32 rounding, not bit for bit
    assert torch.equal(host_p, lp_p.cpu()) and (host_s - lp_s.cpu()).abs().max().item() <= 2e-5
    assert torch.equal(sess._out["o_p"], o_p) and torch.equal(sess._out["o_s"], o_s)
    assert sess.kernels_last_host_pass == 2 + 2 * (1 + 2)  # one prompt-row call (221 rows), two response-row slices
    rows = np.sort(np.random.default_rng(0).choice(wl.n_tokens, 200, replace=False))
    ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids, rows=rows)
    got = np.empty(wl.n_tokens)
    got[wl.prefix_rows()] = host_p.double().numpy()
    got[wl.suffix_rows()] = host_s.double().numpy()
    assert np.abs(got[rows] - ref).max() <= 5e-4
