"""Vocabulary-parallel LM head: ranks' shard records, gathered and merged, must give what the whole
vocabulary gives.  With one GPU the ranks are emulated one after the other on the same device (no
kernel waits on another): each 'rank' runs the shard call on its slice of W_vocab."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import dist as rdist
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device


def test_vocab_shard_bounds_cover_the_vocabulary():
    for vocab, world in [(152064, 8), (1000, 3), (1024, 4), (5000, 2), (257, 2)]:
        spans = [rdist.vocab_shard_bounds(vocab, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == vocab
        for (a, b), (c, d) in zip(spans[:-1], spans[1:]):
            assert b == c and a < b
        assert all(a % 256 == 0 for a, _ in spans)
    assert rdist.vocab_shard_bounds(152064, 8, 3) == (56832, 76032)  # 594 tiles of 256: tiles 222..296


@pytest.mark.gpu
@pytest.mark.parametrize("n_tokens,hidden,vocab,world", [(300, 256, 5000, 4), (257, 128, 1000, 3), (64, 64, 4096, 8)])
def test_sharded_lm_head_equals_the_whole_vocabulary(cuda_device, n_tokens, hidden, vocab, world):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=51, attn=False)
    h, w, ids = to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    ent_full = torch.empty(n_tokens, dtype=torch.float32, device=dev)
    lp_full = rpx.token_logprobs(h, w, ids, entropy=ent_full, device_status=status)
    stats = []
    for r in range(world):
        a, b = rdist.vocab_shard_bounds(vocab, world, r)
        if b > a:
            stats.append(rpx.token_logprobs_shard(h, w[a:b].contiguous(), ids, a, device_status=status))
    gathered = torch.stack(stats).contiguous()
    ent = torch.empty(n_tokens, dtype=torch.float32, device=dev)
    lp, lse = rpx.token_logprobs_merge(gathered, ids, vocab, return_lse=True, entropy=ent, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (lp - lp_full).abs().max().item() <= 2e-5
    assert (ent - ent_full).abs().max().item() <= 2e-5
    ref_lp, ref_lse = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    assert np.abs(lp.double().cpu().numpy() - ref_lp).max() <= 5e-4
    assert np.abs(lse.double().cpu().numpy() - ref_lse).max() <= 5e-4
    # the single-process form of the distributed helper is the one-shard case
    lp_one = rdist.vocab_parallel_token_logprobs(h, w, ids, 0, vocab)
    torch.cuda.synchronize()
    assert (lp_one - lp_full).abs().max().item() <= 2e-5
