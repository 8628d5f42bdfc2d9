"""Multi-GPU plumbing for the scoring path: sequence sharding and whole-job timing.

The path shards by sequence: every step (prefix attention, suffix attention, LM-head log-probs) is
independent per sequence, W_vocab is replicated and each GPU owns its KV pool, so ranks never
exchange data on the data path.  What is left for the host is (a) deciding which sequences a rank
scores and (b) reducing per-rank timings and token counts to a job-level throughput.  Both work
on any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def sequence_cost(prompt_len: int, response_len: int, head_dim: int, num_q_heads: int, hidden: int, vocab: int) -> float:
    """Algorithmic FLOPs of scoring one sequence (causal attention halves + LM head rows)."""
    p, r = float(prompt_len), float(response_len)
    attn = 2.0 * head_dim * num_q_heads * p * (p + 1) + 4.0 * head_dim * num_q_heads * (r * p + r * (r + 1) / 2)
    lm = 2.0 * (p + r) * hidden * vocab
    return attn + lm


def partition_sequences(costs: Sequence[float], world_size: int) -> List[List[int]]:
    """Longest-processing-time-first assignment of sequences to ranks.

    Returns, per rank, the sorted indices of the sequences it scores.  Every sequence goes to
    exactly one rank; the heaviest rank carries at most 4/3 of the optimum (the LPT bound)."""
    if world_size <= 0:
        raise ValueError("world_size must be positive")
    load = [0.0] * world_size
    parts: List[List[int]] = [[] for _ in range(world_size)]
    for idx in sorted(range(len(costs)), key=lambda i: (-costs[i], i)):
        r = min(range(world_size), key=lambda k: (load[k], k))
        parts[r].append(idx)
        load[r] += float(costs[idx])
    return [sorted(p) for p in parts]


def job_throughput(local_units: float, local_ms: float, device=None) -> Tuple[float, float]:
    """(units of all ranks, max over ranks of the elapsed milliseconds).

    Collective-free on the data path; this is the only exchange of a run and it carries two
    numbers.  Without an initialised process group it returns the local values."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(local_units), float(local_ms)
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device)
    n = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(n.item()), float(t.item())


def vocab_shard_bounds(vocab: int, world_size: int, rank: int, multiple: int = 256):
    """[begin, end) of the vocabulary rows rank `rank` holds.  The vocabulary is cut into tiles of `multiple`
    rows (one LM-head tile; the last may be partial) and the tiles are dealt out as evenly as they go, in order.

    Every rank must hold at least one row: an empty shard has no work for rpx_token_logprobs_shard
    (it rejects vocab_local == 0) while the other ranks would wait for it in the all-gather.  A vocabulary
    with fewer tiles than ranks therefore raises ValueError; pass a smaller `multiple`."""
    if world_size <= 0 or not 0 <= rank < world_size:
        raise ValueError("rank must lie in [0, world_size)")
    tiles = -(-vocab // multiple)
    if tiles < world_size:
        raise ValueError(f"a vocabulary of {vocab} rows has {tiles} tiles of {multiple} rows: not enough to give "
                         f"each of {world_size} ranks a non-empty shard")
    begin = (tiles * rank // world_size) * multiple
    end = vocab if rank == world_size - 1 else (tiles * (rank + 1) // world_size) * multiple
    return begin, end


def gather_shard_stats(stats, group=None):
    """All ranks' shard records stacked in rank order: [N, 4] per rank -> [world, N, 4].

    This is the one exchange of the vocabulary-parallel LM head (16 bytes per row and rank).
    Without an initialised process group the result has a single shard."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return stats.unsqueeze(0).contiguous()
    chunks = [torch.empty_like(stats) for _ in range(dist.get_world_size(group))]
    dist.all_gather(chunks, stats.contiguous(), group=group)
    return torch.stack(chunks).contiguous()


def vocab_parallel_token_logprobs(hidden, w_shard, target_ids, vocab_begin: int, vocab_total: int, group=None,
                                  entropy=None, device_status=None):
    """LM-head log-probs with W_vocab sharded over the ranks of `group` (hidden rows replicated):
    shard call, one all-gather of the per-row records, merge call."""
    from . import binding as B

    stats = B.token_logprobs_shard(hidden, w_shard, target_ids, vocab_begin, device_status=device_status)
    gathered = gather_shard_stats(stats, group)
    return B.token_logprobs_merge(gathered, target_ids, vocab_total, entropy=entropy, device_status=device_status)
