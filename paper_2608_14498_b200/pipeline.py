"""One scoring pass over a batch: the four library calls in the order the paper's schedule runs
them (Section 3.1): Phase 1 = prefix attention (+ boundary-KV write) and prefix log-probs,
Phase 2 = suffix attention over the retained KV and suffix log-probs.

Only plumbing lives here (device buffers, host<->device copies, call order); all arithmetic is in
the CUDA library.  ``ScoringSession.score`` takes tensors already on the device;
``ScoringSession.score_from_host`` takes pinned host tensors, copies them in, runs the same calls
and copies the log-probs back — the end-to-end path a caller with host-resident rollouts uses.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Optional

from . import binding as B

KERNELS_PER_SCORE = 6  # prefix attn, suffix attn, 2 x (LM-head partial + combine)


def backward_through_boundary(q, k, v, out, attn_lse, cu_seqlens, prompt_lens, max_seqlen: int, w_vocab, target_ids,
                              lm_lse, upstream, softmax_scale: float = 0.0, device_status=None):
    """Backward of the scoring chain of a training actor whose prefix stays attached (Section 3.2), for the chained
    case in which the LM head reads the attention output (hidden = out viewed as [tokens, H_q * d]).

    Call order, all arithmetic in the library: (1) the LM head's gradient with respect to its hidden rows from the
    saved lse; (2) the SUFFIX pass's attention backward - the response rows only - which leaves its additions on the
    prompt's K/V as well as on the responses' own; (3) the PREFIX pass's attention backward - the prompt rows - added on
    top.  Whole sequences (prompt followed by response) packed by ``cu_seqlens``; ``prompt_lens`` int32 [B] on the
    device.  Returns (dq of the response rows, dq of the prompt rows, dk, dv): float32, the two dq tensors are zero
    outside their own rows."""
    hidden = out.reshape(out.shape[0], out.shape[1] * out.shape[2])
    dh = B.token_logprobs_backward(hidden, w_vocab, target_ids, lm_lse, upstream, device_status=device_status)
    dout = dh.reshape(out.shape)
    dq_s, dk, dv = B.attn_backward(q, k, v, out, dout, attn_lse, cu_seqlens, max_seqlen, q_begin=prompt_lens,
                                   softmax_scale=softmax_scale, device_status=device_status)
    dq_p, dk, dv = B.attn_backward(q, k, v, out, dout, attn_lse, cu_seqlens, max_seqlen, q_end=prompt_lens,
                                   softmax_scale=softmax_scale, dk=dk, dv=dv, accumulate_dkv=True,
                                   device_status=device_status)
    return dq_s, dq_p, dk, dv


@dataclass
class Batch:
    """Tensors of one batch (all on one device, or all pinned host tensors).

    q_p/k_p/v_p: prompt tokens packed by cu_prefix; q_s/k_s/v_s: response tokens packed by
    cu_suffix; hidden_p/ids_p and hidden_s/ids_s: final hidden rows and next-token ids scored in
    the prefix call and in the suffix call; block_table int32 [B, max_blocks].
    """

    q_p: object
    k_p: object
    v_p: object
    q_s: object
    k_s: object
    v_s: object
    cu_prefix: object
    cu_suffix: object
    prefix_lens: object
    block_table: object
    hidden_p: object
    ids_p: object
    hidden_s: object
    ids_s: object
    max_prefix_len: int
    max_suffix_len: int

    def tensors(self):
        return [self.q_p, self.k_p, self.v_p, self.q_s, self.k_s, self.v_s, self.cu_prefix, self.cu_suffix,
                self.prefix_lens, self.block_table, self.hidden_p, self.ids_p, self.hidden_s, self.ids_s]

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in self.tensors())


class ScoringSession:
    """Owns the device-side state that outlives one call: W_vocab, the paged KV pool, the status
    word, workspaces and (for host batches) staging buffers."""

    def __init__(self, w_vocab, num_blocks: int, num_kv_heads: int, head_dim: int):
        import torch

        B.load_library()
        self.torch = torch
        self.device = w_vocab.device
        self.w_vocab = w_vocab
        self.k_cache = torch.zeros((num_blocks, num_kv_heads, B.BLOCK_SIZE, head_dim), dtype=torch.bfloat16,
                                   device=self.device)
        self.v_cache = torch.zeros_like(self.k_cache)
        self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self._ws = {}
        self._staging = [None, None]       # two device staging sets: the next pass uploads while this one computes
        self._staging_free = [None, None]  # event: the pass that used the set has finished reading it
        self._staging_turn = 0
        self._copy_stream = None
        self.kernels_last_host_pass = 0
        self._out = {}

    def _workspace(self, key: str, nbytes: int):
        ws = self._ws.get(key)
        if ws is None or ws.numel() < nbytes:
            ws = self.torch.empty(max(nbytes, 16), dtype=self.torch.uint8, device=self.device)
            self._ws[key] = ws
        return ws

    def _buf(self, key: str, shape, dtype):
        t = self._out.get(key)
        if t is None or tuple(t.shape) != tuple(shape) or t.dtype != dtype:
            t = self.torch.empty(shape, dtype=dtype, device=self.device)
            self._out[key] = t
        return t

    def score(self, b: Batch, events=None):
        """Runs the pass on device tensors; returns (prefix log-probs, suffix log-probs, O_p, O_s).

        ``events``: optional list of five CUDA events recorded before, between and after the four
        library calls (per-kernel timing on the launching stream)."""
        t = self.torch

        def mark(i):
            if events is not None:
                events[i].record()

        cache = (self.k_cache, self.v_cache, b.block_table)
        code = B.RPX_BF16 if b.hidden_p.dtype == t.bfloat16 else B.RPX_F32
        vocab, hdim = self.w_vocab.shape
        o_p = self._buf("o_p", b.q_p.shape, b.q_p.dtype)
        o_s = self._buf("o_s", b.q_s.shape, b.q_s.dtype)
        lp_p = self._buf("lp_p", (b.hidden_p.shape[0],), t.float32)
        lp_s = self._buf("lp_s", (b.hidden_s.shape[0],), t.float32)
        mark(0)
        B.prefix_attn(b.q_p, b.k_p, b.v_p, b.cu_prefix, b.max_prefix_len, cache=cache, out=o_p,
                      workspace=self._workspace("attn", B.prefix_attn_workspace_bytes(
                          b.q_p.shape[1], b.k_p.shape[1], b.q_p.shape[2], B._dtype_code(b.q_p), b.q_p.shape[0])),
                      device_status=self.status)
        mark(1)
        B.token_logprobs(b.hidden_p, self.w_vocab, b.ids_p, logprobs=lp_p, device_status=self.status,
                         workspace=self._workspace("lm", B.token_logprobs_workspace_bytes(
                             b.hidden_p.shape[0], hdim, vocab, code)))
        mark(2)
        B.suffix_attn(b.q_s, b.k_s, b.v_s, b.cu_suffix, b.prefix_lens, b.max_suffix_len, b.max_prefix_len, cache=cache,
                      out=o_s, workspace=self._workspace("attn", B.suffix_attn_workspace_bytes(
                          b.q_s.shape[1], b.k_s.shape[1], b.q_s.shape[2], B._dtype_code(b.q_s), b.q_s.shape[0])),
                      device_status=self.status)
        mark(3)
        B.token_logprobs(b.hidden_s, self.w_vocab, b.ids_s, logprobs=lp_s, device_status=self.status,
                         workspace=self._workspace("lm", B.token_logprobs_workspace_bytes(
                             b.hidden_s.shape[0], hdim, vocab, code)))
        mark(4)
        return lp_p, lp_s, o_p, o_s

    def score_from_host(self, hb: Batch, lp_p_host, lp_s_host, lm_slices: int = 4, min_slice_rows: int = 2048):
        """Pinned host batch in, log-probs out into the pinned ``lp_*_host`` tensors.

        Host->device copies run on a copy stream in the order the kernels need them and each
        kernel waits only for its own inputs: the rows of the LM head (the longest kernels) are cut
        into row slices (``lm_slices`` for the prompt rows, the response rows in proportion) so that
        scoring starts after the first slice has landed and the remaining copies hide behind it.  Kernels and the device->host copy of the
        results are enqueued on the current stream; the caller synchronises.  Two staging sets
        alternate, so back-to-back calls overlap one pass's uploads with the previous pass's kernels."""
        t = self.torch
        turn = self._staging_turn
        self._staging_turn ^= 1
        if self._copy_stream is None:
            self._copy_stream = t.cuda.Stream(device=self.device)
        main = t.cuda.current_stream()
        copy = self._copy_stream
        cur = self._staging[turn]
        if cur is None or any(tuple(a.shape) != tuple(c.shape) or a.dtype != c.dtype
                              for a, c in zip(cur.tensors(), hb.tensors())):
            dev = [t.empty(x.shape, dtype=x.dtype, device=self.device) for x in hb.tensors()]
            self._staging[turn] = Batch(*dev, hb.max_prefix_len, hb.max_suffix_len)
            self._staging_free[turn] = None
        d = self._staging[turn]
        d.max_prefix_len, d.max_suffix_len = hb.max_prefix_len, hb.max_suffix_len
        if self._staging_free[turn] is not None:
            copy.wait_event(self._staging_free[turn])  # the pass before last has finished reading this set
        else:
            copy.wait_stream(main)

        def upload(pairs):
            with t.cuda.stream(copy):
                for dst, src in pairs:
                    dst.copy_(src, non_blocking=True)
                ev = t.cuda.Event()
                ev.record(copy)
            return ev

        n_p, n_s = hb.hidden_p.shape[0], hb.hidden_s.shape[0]

        def cut(n, parts, short_first):
            """Row bounds of ``parts`` slices of n rows; optionally a short first slice (1/16 of the rows,
            a multiple of 128) so the first kernel can start early."""
            if n <= 0:
                return [0, 0]
            first = min(n, -(-(n // 16) // 128) * 128) if (short_first and parts > 1) else 0
            rest = max(parts - (1 if first else 0), 1)
            return sorted(set([0] + [first + (n - first) * i // rest for i in range(rest + 1)]))

        # no slice below min_slice_rows rows; response rows: slices of about the prompt-row slices' size, at most 8
        bounds_p = cut(n_p, max(1, min(lm_slices, n_p // min_slice_rows)), True)
        bounds_s = cut(n_s, max(1, min(8, round(lm_slices * n_s / max(n_p, 1)), n_s // (2 * min_slice_rows))), False)
        cache = (self.k_cache, self.v_cache, d.block_table)
        code = B._dtype_code(d.hidden_p)
        vocab, hdim = self.w_vocab.shape
        lp_p = self._buf("lp_p", (n_p,), t.float32)
        lp_s = self._buf("lp_s", (n_s,), t.float32)
        o_p = self._buf("o_p", d.q_p.shape, d.q_p.dtype)
        o_s = self._buf("o_s", d.q_s.shape, d.q_s.dtype)
        lm_calls = [b - a for a, b in zip(bounds_p[:-1], bounds_p[1:])] + [b - a for a, b in zip(bounds_s[:-1], bounds_s[1:])]
        lm_ws = self._workspace("lm", max(B.token_logprobs_workspace_bytes(n, hdim, vocab, code) for n in lm_calls))
        attn_ws = self._workspace("attn", max(
            B.prefix_attn_workspace_bytes(d.q_p.shape[1], d.k_p.shape[1], d.q_p.shape[2], B._dtype_code(d.q_p), d.q_p.shape[0]),
            B.suffix_attn_workspace_bytes(d.q_s.shape[1], d.k_s.shape[1], d.q_s.shape[2], B._dtype_code(d.q_s), d.q_s.shape[0])))

        def lm(hidden, ids, out, a, b):
            def launch():
                if b > a:
                    B.token_logprobs(hidden[a:b], self.w_vocab, ids[a:b], logprobs=out[a:b], workspace=lm_ws,
                                     device_status=self.status)
                return 1 if b > a else 0
            return launch

        def attn_prefix():
            B.prefix_attn(d.q_p, d.k_p, d.v_p, d.cu_prefix, d.max_prefix_len, cache=cache, out=o_p, workspace=attn_ws,
                          device_status=self.status)
            return 0

        def attn_suffix():
            B.suffix_attn(d.q_s, d.k_s, d.v_s, d.cu_suffix, d.prefix_lens, d.max_suffix_len, d.max_prefix_len,
                          cache=cache, out=o_s, workspace=attn_ws, device_status=self.status)
            return 0

        # Stages = (what to upload, what to launch once it has landed), in the order the kernels run.  Each
        # kernel is enqueued right behind its own upload, so the first one starts as soon as 15 MB have
        # arrived; the copy stream runs the uploads back to back meanwhile.  The response rows of the LM head
        # run before the suffix attention (the two are independent), so that the large q/k/v of the
        # responses, needed last, also arrive last.
        stages = []
        for i, (a, b) in enumerate(zip(bounds_p[:-1], bounds_p[1:])):
            pairs = [(d.hidden_p[a:b], hb.hidden_p[a:b])]
            if i == 0:
                pairs = [(d.ids_p, hb.ids_p), (d.ids_s, hb.ids_s)] + pairs
            stages.append((pairs, lm(d.hidden_p, d.ids_p, lp_p, a, b)))
        stages.append(([(d.q_p, hb.q_p), (d.k_p, hb.k_p), (d.v_p, hb.v_p), (d.cu_prefix, hb.cu_prefix),
                        (d.block_table, hb.block_table)], attn_prefix))
        for a, b in zip(bounds_s[:-1], bounds_s[1:]):
            stages.append(([(d.hidden_s[a:b], hb.hidden_s[a:b])], lm(d.hidden_s, d.ids_s, lp_s, a, b)))
        stages.append(([(d.q_s, hb.q_s), (d.k_s, hb.k_s), (d.v_s, hb.v_s), (d.cu_suffix, hb.cu_suffix),
                        (d.prefix_lens, hb.prefix_lens)], attn_suffix))
        n_lm = 0
        for pairs, launch in stages:
            main.wait_event(upload(pairs))
            n_lm += launch()
        self._staging_free[turn] = t.cuda.Event()
        self._staging_free[turn].record(main)
        lp_p_host.copy_(lp_p, non_blocking=True)
        lp_s_host.copy_(lp_s, non_blocking=True)
        self.kernels_last_host_pass = 2 + 2 * n_lm
        return lp_p_host, lp_s_host

    def check_status(self) -> None:
        code = int(self.status.item())
        if code != 0:
            raise B.RpxError(code, "device status")
