"""Edge cases on the GPU: degenerate batches, bad device-side ids, and the bounded wait itself.
Nothing here is expected to fault: bad ids are clamped or skipped by the kernels and reported."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import binding as B
from paper_2608_14498_b200 import workloads as wk
from helpers import bf16_bits, to_device

pytestmark = pytest.mark.gpu
SENTINEL = 0x7FC1


def test_bounded_wait_times_out_and_the_context_survives(cuda_device):
    dev = cuda_device
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rpx.selftest_bounded_wait(2_000_000, status)      # about a millisecond
    torch.cuda.synchronize()
    assert int(status.item()) == -9 and "wait" in rpx.status_string(-9)
    # the context is intact: a real kernel runs and is correct afterwards
    cfg = wk.Config("t", "bf16", 1, 1, 1, 64, 64, 300, ("fixed", 40), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=41, attn=False)
    status.zero_()
    lp = rpx.token_logprobs(to_device(wl.hidden, dev), to_device(wl.w, dev), to_device(wl.ids, dev), device_status=status)
    torch.cuda.synchronize()
    ref, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    assert int(status.item()) == 0 and np.abs(lp.double().cpu().numpy() - ref).max() <= 5e-4
    with pytest.raises(B.RpxError):
        rpx.selftest_bounded_wait(0, status)


def test_empty_batches_are_no_ops_on_the_device(cuda_device):
    dev = cuda_device
    lib = B.load_library()
    desc = B.AttnDesc(4, 2, 128, 0.0, B.RPX_BF16)
    cu = torch.zeros(4, dtype=torch.int32, device=dev)
    out = torch.full((8, 4, 128), 7.0, dtype=torch.bfloat16, device=dev)
    q = torch.zeros((8, 4, 128), dtype=torch.bfloat16, device=dev)
    kv = torch.zeros((8, 2, 128), dtype=torch.bfloat16, device=dev)
    # three sequences of length zero inside a non-empty allocation: every CTA exits at once
    ws = torch.empty(256, dtype=torch.uint8, device=dev)  # the kernel's work-item counter lives here
    rc = lib.rpx_prefix_attn(ctypes.byref(desc), q.data_ptr(), kv.data_ptr(), kv.data_ptr(), 512, 256, 256, cu.data_ptr(),
                             3, 8, 256, None, out.data_ptr(), None, ws.data_ptr(), 256, None, None)
    torch.cuda.synchronize()
    assert rc == 0 and bool((out == 7.0).all())
    assert lib.rpx_prefix_attn(ctypes.byref(desc), None, None, None, 512, 256, 256, None, 0, 0, 0, None, None, None, None,
                               0, None, None) == 0
    assert lib.rpx_token_logprobs(None, 64, None, None, 0, 64, 100, 0, None, None, None, 0, None, None) == 0


def test_out_of_range_block_ids_are_reported_not_followed(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 2, 4, 2, 128, 64, 64, ("list", [200, 40]), ("list", [30, 20]))
    wl = wk.make_workload(cfg, seed=42, lm=False)
    table = wl.block_table.copy()
    table[0, 3] = wl.num_blocks + 5   # past the pool
    table[1, 0] = -2                  # negative
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = torch.full((wl.num_blocks, 2, 16, 128), SENTINEL, dtype=torch.int16, device=dev)
    k_cache, v_cache = pool.view(torch.bfloat16), pool.clone().view(torch.bfloat16)
    qp, kp, vp = (to_device(wl.prefix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    o = rpx.prefix_attn(qp, kp, vp, to_device(wl.cu_prefix, dev), 200, cache=(k_cache, v_cache, to_device(table, dev)),
                        device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -8
    # attention itself does not depend on the table in the prefix pass
    rows = oracle.all_rows(wl.cu_prefix, 4)
    ref, _ = oracle.attn_rows(wl.prefix_pack(wl.q), wl.prefix_pack(wl.k), wl.prefix_pack(wl.v), wl.cu_prefix, rows)
    assert np.abs(o.double().cpu().numpy().reshape(-1, 128) - ref).max() <= 1e-2
    # pages with a bad id are skipped; every other page holds exactly its tokens; nothing else was touched
    good = wl.block_table.copy()
    ref_k, _ = oracle.cache_image(wl.prefix_pack(wl.k), wl.prefix_pack(wl.v), wl.cu_prefix, good, wl.num_blocks,
                                  sentinel=SENTINEL)
    got_k = bf16_bits(k_cache)
    skipped = {int(good[0, 3]), int(good[1, 0])}
    for blk in range(wl.num_blocks):
        if blk in skipped:
            assert (got_k[blk] == SENTINEL).all()
        else:
            assert np.array_equal(got_k[blk], ref_k[blk])
    # the suffix pass clamps a bad id to block 0 and reports it; the call completes
    status.zero_()
    qs, ks, vs = (to_device(wl.suffix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    rpx.suffix_attn(qs, ks, vs, to_device(wl.cu_suffix, dev), to_device(wl.prompt_lens, dev), 30, 200,
                    cache=(k_cache, v_cache, to_device(table, dev)), device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -8


def test_strided_fp32_inputs(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "f32", 2, 4, 2, 64, 64, 64, ("list", [70, 9]), ("list", [0, 0]))
    wl = wk.make_workload(cfg, seed=43, lm=False)
    wide_q = torch.zeros((wl.n_tokens, 6, 64), dtype=torch.float32, device=dev)
    wide_q[:, :4] = to_device(wl.q, dev)
    o, lse = rpx.prefix_attn(wide_q[:, :4], to_device(wl.k, dev), to_device(wl.v, dev), to_device(wl.cu_full, dev), 70,
                             return_lse=True)
    torch.cuda.synchronize()
    assert o.dtype == torch.float32
    rows = oracle.all_rows(wl.cu_full, 4)
    got, got_l = o.double().cpu().numpy().reshape(-1, 64), lse.double().cpu().numpy().reshape(-1)
    # fp32 tensors take the fp32 CUDA-core path: nothing is rounded in a prefix pass, so the unrounded oracle is met
    # to fp32 accuracy (sums of <= 70 products of magnitude <= 20, exp2 to 2^-22)
    ref, ref_l = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, rows)
    assert np.abs(got - ref).max() <= 2e-5
    assert np.abs(got_l - ref_l).max() <= 2e-5


def test_a_sequence_longer_than_the_callers_bound_is_reported(cuda_device):
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 2, 2, 1, 64, 64, 64, ("list", [100, 600]), ("fixed", 0))
    wl = wk.make_workload(cfg, seed=41, lm=False)
    q, k, v = (to_device(t, dev) for t in (wl.q, wl.k, wl.v))
    cu = to_device(wl.cu_full, dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    rpx.prefix_attn(q, k, v, cu, 600, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rpx.prefix_attn(q, k, v, cu, 500, device_status=status)  # rounds up to 512 < 600
    torch.cuda.synchronize()
    assert int(status.item()) == -8
    status.zero_()
    rpx.prefix_attn(q, k, v, cu, 513, device_status=status)  # rounds up to 768: fine
    torch.cuda.synchronize()
    assert int(status.item()) == 0


def test_two_streams_with_their_own_workspaces_do_not_interfere(cuda_device):
    """The library keeps no device state of its own: the attention kernel's work-item counter and the
    LM head's partial records live in the caller's workspace, so calls on different streams with
    different workspaces may overlap freely."""
    dev = cuda_device
    cfgs = [wk.Config("a", "bf16", 3, 4, 2, 128, 256, 3000, ("list", [700, 130, 257]), ("fixed", 0)),
            wk.Config("b", "bf16", 2, 8, 1, 64, 128, 1000, ("list", [512, 300]), ("fixed", 0))]
    wls = [wk.make_workload(c, seed=50 + i) for i, c in enumerate(cfgs)]
    dev_in = [[to_device(x, dev) for x in (w.q, w.k, w.v, w.cu_full, w.hidden, w.w, w.ids)] for w in wls]

    def run(i, stream):
        q, k, v, cu, h, wv, ids = dev_in[i]
        with torch.cuda.stream(stream):
            o = rpx.prefix_attn(q, k, v, cu, int(wls[i].prompt_lens.max()))
            lp = rpx.token_logprobs(h, wv, ids)
        return o, lp

    main = torch.cuda.current_stream()
    ref = [run(i, main) for i in range(2)]
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for _ in range(3):
        got = [run(i, streams[i]) for i in range(2)]
        torch.cuda.synchronize()
        for (ro, rl), (go, gl) in zip(ref, got):
            assert torch.equal(ro, go) and torch.equal(rl, gl)


def test_sequence_offsets_that_leave_the_packed_tensors_are_reported_not_followed(cuda_device):
    """cu_seqlens live on the device, so the host cannot check them: an end beyond total_tokens, or offsets that run
    backwards, must raise RPX_ERR_DEVICE_DATA and must not make the kernel store outside the output tensor."""
    dev = cuda_device
    cfg = wk.Config("t", "bf16", 3, 4, 2, 128, 64, 64, ("list", [150, 70, 40]), ("list", [0, 0, 0]))
    wl = wk.make_workload(cfg, seed=44, lm=False)
    qp, kp, vp = (to_device(wl.prefix_pack(t), dev) for t in (wl.q, wl.k, wl.v))
    total = qp.shape[0]
    ref_out = rpx.prefix_attn(qp, kp, vp, to_device(wl.cu_prefix, dev), 150)
    torch.cuda.synchronize()
    # the output tensor sits in the middle of a guard region filled with a recognisable value
    guard = torch.full((3 * total, 4, 128), 7.0, dtype=torch.bfloat16, device=dev)
    out = guard[total:2 * total]
    for bad in ([0, 150, 220, total + 300],      # the last sequence claims 300 tokens more than exist
                [0, 150, 120, total],            # offsets run backwards: sequence 1 has a negative length
                [0, 150, 220, -5]):              # a negative end
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        guard.fill_(7.0)
        cu = torch.tensor(bad, dtype=torch.int32, device=dev)
        rpx.prefix_attn(qp, kp, vp, cu, 512, out=out, device_status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == -8, bad
        assert bool((guard[:total] == 7.0).all()) and bool((guard[2 * total:] == 7.0).all()), bad
        # sequence 0 is well-formed in every case and is still computed (in the second case the third sequence,
        # tokens 120..259, overlaps its last rows)
        assert torch.equal(out[:120], ref_out[:120]), bad
    # the context is intact and a well-formed call is clean afterwards
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    again = rpx.prefix_attn(qp, kp, vp, to_device(wl.cu_prefix, dev), 150, device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and torch.equal(again, ref_out)
