"""Seeded random ragged batches through the whole path (prefix pass, suffix pass over the paged
cache, LM head on both halves) against the oracle, all rows.  Shapes are drawn to hit what the
fixed cases may miss: every GQA group size from 1 to 8, both head dims, both element types,
lengths around every tile and page edge, many short sequences in one batch."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device

import test_gpu_attention as T

pytestmark = pytest.mark.gpu

EDGE = [1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300, 511, 513]


def _draw(rng, case):
    group = int(rng.integers(1, 9))
    hkv = int(rng.integers(1, 4))
    d = 128 if case % 3 else 64
    dtype = "f32" if case % 5 == 4 else "bf16"
    batch = int(rng.integers(1, 7)) if case % 4 else int(rng.integers(12, 25))
    hi = 80 if batch > 8 else 520
    plens = [int(rng.choice(EDGE)) if rng.random() < 0.6 else int(rng.integers(0, hi)) for _ in range(batch)]
    rlens = [int(rng.choice(EDGE)) if rng.random() < 0.4 else int(rng.integers(0, hi // 2)) for _ in range(batch)]
    plens = [min(p, hi) for p in plens]
    rlens = [min(r, hi) for r in rlens]
    hidden = int(rng.choice([64, 72, 200, 256]))
    vocab = int(rng.choice([3, 255, 256, 257, 1000, 4100]))
    return wk.Config(f"rand{case}", dtype, batch, group * hkv, hkv, d, hidden, vocab, ("list", plens), ("list", rlens))


@pytest.mark.parametrize("case", range(24))
def test_random_batch_matches_the_oracle(cuda_device, case):
    dev = cuda_device
    rng = np.random.default_rng(1000 + case)
    cfg = _draw(rng, case)
    wl = wk.make_workload(cfg, seed=2000 + case)
    if wl.n_tokens == 0:
        pytest.skip("empty draw")
    out, lse, kc, vc, _ = T.run_split(wl, dev)
    rows = oracle.all_rows(wl.cu_full, cfg.num_q_heads)
    if cfg.dtype == "bf16":
        T.check_rows(wl, out, lse, rows)
    else:
        # fp32 tensors: against the UNROUNDED oracle.  The only rounding left is that of the prompt's K/V in the
        # bf16 cache the suffix pass reads, so the prompt rows match to fp32 accuracy and the response rows stay
        # inside the bound of the bf16 configs.
        T.check_rows(wl, out, lse, rows, lse_tol=1e-2)
        pre = rows[rows[:, 1] < wl.prompt_lens[rows[:, 0]]]
        if pre.shape[0]:
            ref_o, ref_l = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, pre)
            tok = wl.cu_full[pre[:, 0]].astype(np.int64) + pre[:, 1]
            assert np.abs(out[tok, pre[:, 2]] - ref_o).max() <= 5e-5
            assert np.abs(lse[tok, pre[:, 2]] - ref_l).max() <= 5e-5
    T.check_cache(wl, kc, vc)
    # LM head on the prompt rows and on the response rows, concatenated = the full-sequence values
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    w = to_device(wl.w, dev)
    got = np.empty(wl.n_tokens)
    for idx in (wl.prefix_rows(), wl.suffix_rows()):
        if idx.size:
            lp = rpx.token_logprobs(to_device(wl.hidden[idx], dev), w, to_device(wl.ids[idx], dev), device_status=status)
            got[idx] = lp.double().cpu().numpy()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    if cfg.dtype == "bf16":
        ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
        assert np.abs(got - ref).max() <= 5e-4
    else:
        ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
        assert np.abs(got - ref).max() <= 2e-2
