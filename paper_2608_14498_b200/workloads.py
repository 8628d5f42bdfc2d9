"""Seeded synthetic workloads shaped like the paper's video-RL scoring batches.

This module only draws numbers and indexes arrays; it holds none of the method's arithmetic, so
both the CUDA path's harness and the CPU oracle's harness may use it.  Everything is generated on
the host with numpy (bf16 tensors are carried as ``uint16`` bit patterns) so that both sides read
exactly the same bits.

Length statistics follow the paper's Figure 2 discussion (prompt tokens are 79-98 % of a video
sample, 11-19 % of a text-reasoning sample) and its evaluation budgets (Section 4.1: 8k prompt +
2k response, 32 prompts per batch); the datasets themselves are not used.

Recipe (all configs, seed 0 unless stated):
  * lengths      fixed, or  P = clip(floor(median * exp(sigma * z)), lo, hi), z ~ N(0,1), or
                 uniform inclusive integers; lengths are NOT rounded to tile multiples
  * Q, K, V      N(0, 1)   (rotary assumed already applied)
  * hidden       N(0, 1)
  * W_vocab      N(0, 0.02)  (standard deviation 0.02)
  * target ids   uniform integers in [0, V)
  * block table  16-token blocks; pool = ceil(1.25 * needed) blocks; each sequence's logical
                 blocks take consecutive entries of one random permutation of the pool, so a
                 quarter of the physical blocks stay unused
  * bf16 configs draw fp32 and round to nearest-even; both sides consume the bf16 bits.
Each tensor has its own stream, SeedSequence([seed, tensor id, chunk]), in chunks of 2**22
elements, so the bits do not depend on thread count.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Optional, Tuple

import numpy as np

BLOCK_SIZE = 16
_CHUNK = 1 << 22
_TENSOR_IDS = {"q": 1, "k": 2, "v": 3, "hidden": 4, "w": 5, "ids": 6, "lengths": 7, "blocks": 8}


@dataclass(frozen=True)
class Config:
    """One benchmark / parity configuration (shapes only)."""

    name: str
    dtype: str  # "bf16" or "f32"
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    hidden: int
    vocab: int
    prompt: Tuple  # ("fixed", P) | ("lognormal", median, sigma, lo, hi) | ("uniform", lo, hi)
    response: Tuple
    stands_in_for: str = ""

    def scaled(self, **kw) -> "Config":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "C1": Config("C1-tiny-f32", "f32", 1, 4, 2, 64, 256, 4096, ("fixed", 256), ("fixed", 32),
                 "correctness only"),
    "C2": Config("C2-7B-b8-4096+256", "bf16", 8, 28, 4, 128, 3584, 152064, ("fixed", 4096), ("fixed", 256),
                 "mid-length video prompts, 7B shape"),
    "C3": Config("C3-32B-varlen-b32", "bf16", 32, 40, 8, 128, 5120, 152064,
                 ("lognormal", 6000, 0.5, 1024, 16384), ("lognormal", 400, 0.6, 32, 2048),
                 "the paper's main setup: 32 prompts, 8k/2k budgets, 32B shape"),
    "C4": Config("C4-32B-long-b2-32768+512", "bf16", 2, 40, 8, 128, 5120, 152064, ("fixed", 32768),
                 ("fixed", 512), "long-video QA tail (98 % prompt share)"),
    "C5": Config("C5-7B-text-b64", "bf16", 64, 28, 4, 128, 3584, 152064, ("uniform", 128, 512),
                 ("lognormal", 1500, 0.5, 256, 4096), "text-reasoning control (~15 % prompt share)"),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal(seed: int, tensor: str, n: int, sigma: float, dtype: str) -> np.ndarray:
    """n draws of N(0, sigma) as float32, or as bf16 bits when dtype == 'bf16'."""
    out = np.empty(n, dtype=np.uint16 if dtype == "bf16" else np.float32)
    tid = _TENSOR_IDS[tensor]

    def fill(c: int) -> None:
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, tid, c])))
        x = rng.standard_normal(hi - lo, dtype=np.float32)
        if sigma != 1.0:
            x *= np.float32(sigma)
        out[lo:hi] = f32_to_bf16_bits(x) if dtype == "bf16" else x

    chunks = range((n + _CHUNK - 1) // _CHUNK)
    if len(chunks) > 1:
        with ThreadPoolExecutor(max_workers=8) as ex:
            list(ex.map(fill, chunks))
    else:
        for c in chunks:
            fill(c)
    return out


def draw_lengths(spec: Tuple, batch: int, rng: np.random.Generator) -> np.ndarray:
    kind = spec[0]
    if kind == "fixed":
        return np.full(batch, int(spec[1]), dtype=np.int32)
    if kind == "lognormal":
        _, median, sigma, lo, hi = spec
        z = rng.standard_normal(batch)
        return np.clip(np.floor(median * np.exp(sigma * z)), lo, hi).astype(np.int32)
    if kind == "uniform":
        _, lo, hi = spec
        return rng.integers(lo, hi + 1, size=batch).astype(np.int32)
    if kind == "list":
        assert len(spec[1]) == batch
        return np.asarray(spec[1], dtype=np.int32)
    raise ValueError(kind)


def _cumsum0(x: np.ndarray) -> np.ndarray:
    cu = np.zeros(x.shape[0] + 1, dtype=np.int64)
    np.cumsum(x, out=cu[1:])
    assert cu[-1] < 2**31
    return cu.astype(np.int32)


@dataclass
class Workload:
    cfg: Config
    seed: int
    prompt_lens: np.ndarray  # int32 [B]
    response_lens: np.ndarray  # int32 [B]
    cu_full: np.ndarray  # int32 [B+1], whole sequences (prompt then response)
    cu_prefix: np.ndarray
    cu_suffix: np.ndarray
    block_table: np.ndarray  # int32 [B, max_blocks]
    num_blocks: int
    q: Optional[np.ndarray] = None  # [N, H_q, d] whole sequences
    k: Optional[np.ndarray] = None  # [N, H_kv, d]
    v: Optional[np.ndarray] = None
    hidden: Optional[np.ndarray] = None  # [N, H]
    w: Optional[np.ndarray] = None  # [V, H]
    ids: Optional[np.ndarray] = None  # int32 [N]
    _prefix_index: Optional[np.ndarray] = field(default=None, repr=False)
    _suffix_index: Optional[np.ndarray] = field(default=None, repr=False)

    @property
    def n_prefix(self) -> int:
        return int(self.cu_prefix[-1])

    @property
    def n_suffix(self) -> int:
        return int(self.cu_suffix[-1])

    @property
    def n_tokens(self) -> int:
        return int(self.cu_full[-1])

    def _indices(self):
        if self._prefix_index is None:
            pre, suf = [], []
            for s in range(self.cfg.batch):
                a, p, r = int(self.cu_full[s]), int(self.prompt_lens[s]), int(self.response_lens[s])
                pre.append(np.arange(a, a + p, dtype=np.int64))
                suf.append(np.arange(a + p, a + p + r, dtype=np.int64))
            self._prefix_index = np.concatenate(pre) if pre else np.zeros(0, np.int64)
            self._suffix_index = np.concatenate(suf) if suf else np.zeros(0, np.int64)
        return self._prefix_index, self._suffix_index

    def prefix_rows(self) -> np.ndarray:
        """Whole-sequence token numbers of the prompt tokens, in prefix-packed order."""
        return self._indices()[0]

    def suffix_rows(self) -> np.ndarray:
        return self._indices()[1]

    def prefix_pack(self, x: np.ndarray) -> np.ndarray:
        return np.ascontiguousarray(x[self.prefix_rows()])

    def suffix_pack(self, x: np.ndarray) -> np.ndarray:
        return np.ascontiguousarray(x[self.suffix_rows()])


def make_block_table(prompt_lens: np.ndarray, seed: int, block_size: int = BLOCK_SIZE):
    """Shuffled block table: returns (table int32 [B, max_blocks], num_blocks)."""
    need = (prompt_lens.astype(np.int64) + block_size - 1) // block_size
    total = int(need.sum())
    pool = max(1, int(np.ceil(1.25 * total)))
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, _TENSOR_IDS["blocks"], 0])))
    perm = rng.permutation(pool).astype(np.int32)
    table = np.zeros((prompt_lens.shape[0], max(1, int(need.max()) if need.size else 1)), dtype=np.int32)
    off = 0
    for s, n in enumerate(need):
        table[s, : int(n)] = perm[off: off + int(n)]
        off += int(n)
    return table, pool


def make_workload(cfg: Config, seed: int = 0, attn: bool = True, lm: bool = True) -> Workload:
    """Draw one batch.  ``attn`` / ``lm`` select which tensor families to materialise."""
    lrng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, _TENSOR_IDS["lengths"], 0])))
    p = draw_lengths(cfg.prompt, cfg.batch, lrng)
    r = draw_lengths(cfg.response, cfg.batch, lrng)
    cu_full, cu_p, cu_s = _cumsum0(p + r), _cumsum0(p), _cumsum0(r)
    table, pool = make_block_table(p, seed)
    wl = Workload(cfg, seed, p, r, cu_full, cu_p, cu_s, table, pool)
    n = wl.n_tokens
    if attn:
        wl.q = _normal(seed, "q", n * cfg.num_q_heads * cfg.head_dim, 1.0, cfg.dtype).reshape(
            n, cfg.num_q_heads, cfg.head_dim)
        wl.k = _normal(seed, "k", n * cfg.num_kv_heads * cfg.head_dim, 1.0, cfg.dtype).reshape(
            n, cfg.num_kv_heads, cfg.head_dim)
        wl.v = _normal(seed, "v", n * cfg.num_kv_heads * cfg.head_dim, 1.0, cfg.dtype).reshape(
            n, cfg.num_kv_heads, cfg.head_dim)
    if lm:
        wl.hidden = _normal(seed, "hidden", n * cfg.hidden, 1.0, cfg.dtype).reshape(n, cfg.hidden)
        wl.w = _normal(seed, "w", cfg.vocab * cfg.hidden, 0.02, cfg.dtype).reshape(cfg.vocab, cfg.hidden)
        irng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, _TENSOR_IDS["ids"], 0])))
        wl.ids = irng.integers(0, cfg.vocab, size=n, dtype=np.int32)
    return wl


def sample_attn_rows(wl: Workload, n: int, seed: int = 0) -> np.ndarray:
    """About ``n`` (sequence, whole-sequence position, head) triples, stratified.

    Always holds row 0, positions around 16 / 128 / 256 and around the prefix/suffix split, the
    last row of every sampled sequence, and random rows spread over position deciles.
    """
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 99, 0])))
    cfg = wl.cfg
    rows = []
    for s in range(cfg.batch):
        p, r = int(wl.prompt_lens[s]), int(wl.response_lens[s])
        length = p + r
        if length == 0:
            continue
        fixed = {0, 15, 16, 17, 127, 128, 129, 255, 256, 257, p - 1, p, p + 1, p + 127, p + 128, length - 1}
        for i in sorted(x for x in fixed if 0 <= x < length):
            rows.append((s, i, int(rng.integers(cfg.num_q_heads))))
    want_random = max(0, n - len(rows))
    for t in range(want_random):
        s = int(rng.integers(cfg.batch))
        length = int(wl.prompt_lens[s] + wl.response_lens[s])
        if length == 0:
            continue
        dec = t % 10
        lo, hi = length * dec // 10, max(length * dec // 10 + 1, length * (dec + 1) // 10)
        rows.append((s, int(rng.integers(lo, hi)), int(rng.integers(cfg.num_q_heads))))
    out = np.asarray(rows, dtype=np.int32).reshape(-1, 3)
    if out.shape[0] > n > 0:
        keep = np.sort(rng.choice(out.shape[0], size=n, replace=False))
        out = out[keep]
    return out


def sample_logprob_rows(wl: Workload, n: int, seed: int = 0) -> np.ndarray:
    """``n`` distinct row numbers: first, last, rows around multiples of 128, random others."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 98, 0])))
    total = wl.n_tokens
    if total <= n:
        return np.arange(total, dtype=np.int64)
    fixed = {0, 1, 127, 128, 129, total - 129, total - 128, total - 1}
    fixed = {x for x in fixed if 0 <= x < total}
    rest = rng.choice(total, size=n, replace=False)
    rows = list(fixed) + [int(x) for x in rest if int(x) not in fixed]
    return np.sort(np.asarray(rows[:n], dtype=np.int64))


# ---------------------------------------------------------------------------------------------
# Prompt groups: the paper's GRPO setting scores N sampled responses per prompt and computes the
# prompt prefix once per group (Section 4.1 lists N = 8 and enables prefix sharing in every system).
# ---------------------------------------------------------------------------------------------
@dataclass
class GroupWorkload:
    """B prompts with `group` responses each.

    `prompts` is a Workload whose sequences are the B prompts alone (response length 0): its
    prefix-packed tensors feed the one prefix pass per prompt.  `members` is a Workload of the
    B * group whole sequences (prompt tokens repeated bit for bit in every member, then that
    member's response): the oracle scores those one by one, and their suffix-packed tensors feed
    the suffix pass.  `member_table` is the block table of the suffix pass: member m of prompt b
    uses row b of the prompts' table, so all members of a group read the same cache blocks.
    """

    group: int
    prompts: Workload
    members: Workload
    member_table: np.ndarray


def make_group_workload(cfg: Config, group: int, seed: int = 0) -> GroupWorkload:
    """cfg.batch prompts drawn as in make_workload; each gets `group` responses of its own length."""
    lrng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, _TENSOR_IDS["lengths"], 1])))
    p = draw_lengths(cfg.prompt, cfg.batch, lrng)
    prompt_cfg = cfg.scaled(name=cfg.name + "-prompts", prompt=("list", [int(x) for x in p]),
                            response=("list", [0] * cfg.batch))
    prompts = make_workload(prompt_cfg, seed=seed)
    n_members = cfg.batch * group
    r = draw_lengths(cfg.response, n_members, lrng)
    member_cfg = cfg.scaled(name=cfg.name + f"-x{group}", batch=n_members, prompt=("list", [int(x) for x in np.repeat(p, group)]),
                            response=("list", [int(x) for x in r]))
    members = make_workload(member_cfg, seed=seed + 1000003)
    # overwrite every member's prompt tokens with its prompt's tensors so the prefix really is shared
    for m in range(n_members):
        b = m // group
        src = slice(int(prompts.cu_full[b]), int(prompts.cu_full[b + 1]))
        dst = slice(int(members.cu_full[m]), int(members.cu_full[m]) + int(p[b]))
        for name in ("q", "k", "v", "hidden", "ids"):
            getattr(members, name)[dst] = getattr(prompts, name)[src]
    members.w = prompts.w
    member_table = np.repeat(prompts.block_table, group, axis=0)
    members.block_table = member_table
    members.num_blocks = prompts.num_blocks
    return GroupWorkload(group, prompts, members, member_table)
