"""World-size-2 checks of the multi-GPU host logic on the gloo backend (no GPU)."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_14498_b200 import dist as rdist
from paper_2608_14498_b200 import workloads as wk


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # rank r scores its own batch (seed r), as bench.py does; lengths differ per rank
        cfg = wk.Config("t", "bf16", 4, 4, 2, 64, 64, 128, ("lognormal", 60, 0.5, 8, 200), ("uniform", 1, 30))
        wl = wk.make_workload(cfg, seed=rank, attn=False, lm=False)
        units, ms = rdist.job_throughput(wl.n_tokens, 10.0 * (rank + 1))
        # the exchange step of the vocabulary-parallel LM head: records stacked in rank order
        import torch
        stats = torch.full((5, 4), float(rank + 1)) + torch.arange(5, dtype=torch.float32)[:, None]
        gathered = rdist.gather_shard_stats(stats)
        ok = tuple(gathered.shape) == (world, 5, 4) and all(
            torch.equal(gathered[r], torch.full((5, 4), float(r + 1)) + torch.arange(5, dtype=torch.float32)[:, None])
            for r in range(world))
        out.put((rank, wl.n_tokens, units, ms, ok))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_job_throughput_sums_units_and_takes_the_slowest_rank():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    local = [r[1] for r in res]
    assert local[0] != local[1]  # different seeds, different batches
    for _, _, units, ms, gathered_ok in res:
        assert units == float(sum(local)) and ms == 20.0 and gathered_ok


def test_single_process_job_throughput_is_local():
    import torch

    assert rdist.job_throughput(123, 4.5) == (123.0, 4.5)
    assert tuple(rdist.gather_shard_stats(torch.zeros(3, 4)).shape) == (1, 3, 4)


def test_partition_covers_every_sequence_once_and_balances():
    wl = wk.make_workload(wk.CONFIGS["C3"], seed=0, attn=False, lm=False)
    cfg = wl.cfg
    costs = [rdist.sequence_cost(int(p), int(r), cfg.head_dim, cfg.num_q_heads, cfg.hidden, cfg.vocab)
             for p, r in zip(wl.prompt_lens, wl.response_lens)]
    for world in (1, 2, 4, 8):
        parts = rdist.partition_sequences(costs, world)
        flat = sorted(i for p in parts for i in p)
        assert flat == list(range(cfg.batch))
        loads = np.array([sum(costs[i] for i in p) for p in parts])
        assert loads.max() <= (4.0 / 3.0) * max(sum(costs) / world, max(costs)) + 1e-6
    assert rdist.partition_sequences([], 3) == [[], [], []]
    # the cost model counts the causal half of attention plus the LM-head rows
    assert rdist.sequence_cost(1, 0, 128, 28, 3584, 152064) == 2.0 * 128 * 28 * 2 + 2.0 * 3584 * 152064


def test_vocab_shard_bounds_never_hand_out_an_empty_shard():
    """An empty shard would make its rank fail in rpx_token_logprobs_shard while the others wait in the all-gather:
    the bounds either give every rank at least one row or refuse the split."""
    import pytest

    from paper_2608_14498_b200 import dist as rdist

    for vocab, world, multiple in [(152064, 8, 256), (1000, 3, 256), (1000, 8, 64), (4096, 16, 256), (257, 2, 256)]:
        spans = [rdist.vocab_shard_bounds(vocab, world, r, multiple) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == vocab
        assert all(a < b for a, b in spans)
        assert all(spans[r][1] == spans[r + 1][0] for r in range(world - 1))
    for vocab, world in [(1000, 8), (256, 2), (1, 2)]:   # fewer 256-row tiles than ranks
        with pytest.raises(ValueError):
            rdist.vocab_shard_bounds(vocab, world, world - 1)
    assert rdist.vocab_shard_bounds(1000, 8, 7, multiple=8) == (872, 1000)  # 125 tiles of 8: tiles 109..124
    with pytest.raises(ValueError):
        rdist.vocab_shard_bounds(1000, 4, 4)
