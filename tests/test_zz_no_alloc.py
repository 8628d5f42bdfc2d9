"""rpx_token_logprobs_static: the entry point for callers that cannot allocate device memory.

Some callers of this library have no workspace to pass and no way to make one: a scoring hook
running inside an engine that has already given every free byte of HBM to its KV pool, or a code
section where an allocator call could fail or stall the device.  For them the library keeps the
LM-head partial records in a fixed array of its own.  This file checks, through the C ABI, that
the variant returns what the oracle computes and what rpx_token_logprobs returns (the two CUDA entry
points differ only in the order fp32 partial sums are merged), twice in a row (the array is shared
between calls and keeps the previous call's contents), and that it refuses problems larger than the
array.

It is collected last on purpose, so that a run stopping at the first failure has already run every
other test; it must also pass alone in a fresh process.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import binding as B
from paper_2608_14498_b200 import workloads as wk
from helpers import to_device

pytestmark = pytest.mark.gpu

TIGHT = 5e-4  # the bound tests/test_gpu_logprobs.py uses for bf16 inputs


def _case(dev, n_tokens, hidden, vocab, seed, with_workload=False):
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, hidden, vocab, ("fixed", n_tokens), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=seed, attn=False)
    dev_tensors = (to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev))
    return dev_tensors + (wl,) if with_workload else dev_tensors


def test_static_scratch_variant_matches_the_workspace_variant_twice(cuda_device):
    dev = cuda_device
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # two different problems back to back: the second call finds the first call's records in the array
    for n_tokens, hidden, vocab, seed in [(700, 512, 9000, 21), (333, 256, 5000, 22)]:
        h, w, ids, wl = _case(dev, n_tokens, hidden, vocab, seed, with_workload=True)
        ref, ref_lse = rpx.token_logprobs(h, w, ids, return_lse=True, device_status=status)
        oracle_lp, oracle_lse = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
        out = torch.full((n_tokens,), float("nan"), dtype=torch.float32, device=dev)
        lse = torch.full((n_tokens,), float("nan"), dtype=torch.float32, device=dev)
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(dev)
        rpx.token_logprobs_static(h, w, ids, out, lse=lse, device_status=status)
        assert torch.cuda.memory_allocated(dev) == before  # nothing was allocated through torch either
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        assert torch.isfinite(out).all()
        # against the oracle (the definition), on the same bits
        assert np.abs(out.double().cpu().numpy() - oracle_lp).max() <= TIGHT
        assert np.abs(lse.double().cpu().numpy() - oracle_lse).max() <= TIGHT
        # and against the entry point it is a variant of
        assert (out - ref).abs().max().item() <= TIGHT
        assert (lse - ref_lse).abs().max().item() <= TIGHT


def test_static_scratch_variant_rejects_what_does_not_fit(cuda_device):
    dev = cuda_device
    h, w, ids = _case(dev, 64, 64, 300, 23)
    out = torch.empty(64, dtype=torch.float32, device=dev)
    lib = B.load_library()
    # 152064 columns = 38 chunks; 38 * n * 16 bytes must stay within the 8 MiB array
    fits = B.STATIC_SCRATCH_BYTES // (38 * 16)
    assert fits == 13797
    rc = lib.rpx_token_logprobs_static(h.data_ptr(), 64, w.data_ptr(), ids.data_ptr(), fits + 1, 64, 152064,
                                       out.data_ptr(), None, None, None)
    assert rc == -5 and "workspace" in B.status_string(rc)
    with pytest.raises(TypeError):
        rpx.token_logprobs_static(h.float(), w.float(), ids, out)
    # a legal empty call is a no-op
    assert lib.rpx_token_logprobs_static(None, 64, None, None, 0, 64, 300, None, None, None, None) == 0
