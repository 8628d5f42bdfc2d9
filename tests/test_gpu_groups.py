"""Prompt groups (the paper's GRPO setting): the prefix pass runs once per prompt, and all sampled
responses of the prompt score against the one cached prefix through aliased block-table rows.
Every member sequence must still match one-pass scoring of (prompt ‖ that response)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2608_14498_b200 as rpx
from paper_2608_14498_b200 import workloads as wk
from helpers import bf16_bits, to_device

SENTINEL = 0x7FC1


def test_group_workload_shares_prompt_bits():
    cfg = wk.Config("g", "bf16", 2, 4, 2, 128, 256, 500, ("list", [150, 33]), ("uniform", 1, 60))
    gw = wk.make_group_workload(cfg, group=3, seed=5)
    mem, pro = gw.members, gw.prompts
    assert mem.cfg.batch == 6 and (mem.prompt_lens == np.repeat(pro.prompt_lens, 3)).all()
    for m in range(6):
        b = m // 3
        a = int(mem.cu_full[m])
        assert np.array_equal(mem.k[a: a + int(pro.prompt_lens[b])], pro.k[int(pro.cu_full[b]): int(pro.cu_full[b + 1])])
    assert np.array_equal(gw.member_table[0], gw.member_table[2]) and not np.array_equal(gw.member_table[0], gw.member_table[3])
    assert len({int(x) for x in mem.response_lens}) > 1


@pytest.mark.gpu
def test_grouped_scoring_matches_one_pass_scoring_of_every_member(cuda_device):
    dev = cuda_device
    cfg = wk.Config("g", "bf16", 3, 4, 2, 128, 512, 3000, ("list", [300, 129, 40]), ("uniform", 1, 200))
    gw = wk.make_group_workload(cfg, group=4, seed=6)
    pro, mem = gw.prompts, gw.members
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    pool = torch.full((pro.num_blocks, 2, 16, 128), SENTINEL, dtype=torch.int16, device=dev)
    k_cache, v_cache = pool.view(torch.bfloat16), pool.clone().view(torch.bfloat16)
    # Phase 1, once per prompt: prefix attention + cache write, prompt log-probs
    o_pre = rpx.prefix_attn(to_device(pro.q, dev), to_device(pro.k, dev), to_device(pro.v, dev), to_device(pro.cu_full, dev),
                            int(pro.prompt_lens.max()), cache=(k_cache, v_cache, to_device(pro.block_table, dev)),
                            device_status=status)
    w = to_device(pro.w, dev)
    lp_pre = rpx.token_logprobs(to_device(pro.hidden, dev), w, to_device(pro.ids, dev), device_status=status)
    # Phase 2, per member: suffix attention through the aliased table rows, response log-probs
    qs, ks, vs = (to_device(mem.suffix_pack(t), dev) for t in (mem.q, mem.k, mem.v))
    o_suf = rpx.suffix_attn(qs, ks, vs, to_device(mem.cu_suffix, dev), to_device(mem.prompt_lens, dev),
                            int(mem.response_lens.max()), int(mem.prompt_lens.max()),
                            cache=(k_cache, v_cache, to_device(gw.member_table, dev)), device_status=status)
    lp_suf = rpx.token_logprobs(to_device(mem.suffix_pack(mem.hidden), dev), w, to_device(mem.suffix_pack(mem.ids), dev),
                                device_status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    # the cache holds each prompt once
    ref_k, ref_v = oracle.cache_image(pro.k, pro.v, pro.cu_full, pro.block_table, pro.num_blocks, sentinel=SENTINEL)
    assert np.array_equal(bf16_bits(k_cache), ref_k) and np.array_equal(bf16_bits(v_cache), ref_v)
    # oracle: every member scored in one pass over its whole sequence
    rows = oracle.all_rows(mem.cu_full, 4)
    ref_o, _ = oracle.attn_rows(mem.q, mem.k, mem.v, mem.cu_full, rows)
    ref_o = ref_o.reshape(mem.n_tokens, 4, 128)
    ref_lp, _ = oracle.logprob_rows(mem.hidden, mem.w, mem.ids)
    got_o = np.empty_like(ref_o)
    got_lp = np.empty_like(ref_lp)
    o_pre_h, lp_pre_h = o_pre.double().cpu().numpy(), lp_pre.double().cpu().numpy()
    for m in range(mem.cfg.batch):  # a member's prompt rows are its prompt's rows
        b = m // gw.group
        src = slice(int(pro.cu_full[b]), int(pro.cu_full[b + 1]))
        dst = slice(int(mem.cu_full[m]), int(mem.cu_full[m]) + int(pro.prompt_lens[b]))
        got_o[dst], got_lp[dst] = o_pre_h[src], lp_pre_h[src]
    got_o[mem.suffix_rows()] = o_suf.double().cpu().numpy()
    got_lp[mem.suffix_rows()] = lp_suf.double().cpu().numpy()
    assert np.abs(got_o - ref_o).max() <= 1e-2
    assert np.abs(got_lp - ref_lp).max() <= 5e-4
