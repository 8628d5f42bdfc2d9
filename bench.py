#!/usr/bin/env python
"""Benchmark of the prefix+suffix scoring hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config C3]
    python bench.py --profile-case lm|lmbwd|lmdw|prefix|suffix|attnbwd [--reps 3]      (small launches for profiler captures)
    python bench.py --attn-alone [--reps 30]                             (attention passes of C2, C3, C4 timed alone)

One step = one pass of the whole path over one synthetic batch: prefix attention (+ paged
boundary-KV write), prefix log-probs, suffix attention over the cached KV, suffix log-probs.
Metric: scored tokens/s (every token of every sequence gets a log-prob) and TFLOP/s.

`value`     inputs already resident in HBM, timed with CUDA events on the launching stream.
`e2e`       the same pass from pinned HOST tensors through ScoringSession.score_from_host:
            host->device copies of the step's inputs and the device->host read of the log-probs
            are inside the timed region (W_vocab is a model weight and stays resident).
`roofline`  the dominant kernel (the fused LM-head kernel on the prompt rows): algorithmic FLOPs
            / its CUDA-event duration, against the measured dense-bf16 peak of this machine.
`cpu_baseline`  the fp64 oracle, as it stands, on a bounded sample of the same workload.
`--impl reference` times that oracle alone (rank 0 only).

The headline workload is C3 (the largest single-GPU config: 32 packed sequences of the 32B shape, the
paper's main setup); with one GPU the line also carries a `configs` record with C2, C4 and C5 measured
the same way in the same invocation (own clock samples each).

N > 1 (torchrun): every rank scores its own batch of the same shape (sequences are independent,
W_vocab replicated, no data-path collective) => weak scaling; time = max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_14498_b200 import workloads as wk  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per launch of the LM-head partial kernel on a config's
# prompt rows, from one-pass ncu captures of this very command on that config.  Configs without a capture: None.
LM_HEAD_TRAFFIC_BYTES = {"C2": 13.291e9 + 43.8e6, "C3": 321.94e9 + 264.6e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def flop_counts(wl):
    cfg = wl.cfg
    p = wl.prompt_lens.astype(np.float64)
    r = wl.response_lens.astype(np.float64)
    d, hq = cfg.head_dim, cfg.num_q_heads
    return {
        "prefix_attn": float((2.0 * d * hq * p * (p + 1)).sum()),
        "suffix_attn": float((4.0 * d * hq * (r * p + r * (r + 1) / 2)).sum()),
        "lm_prefix": 2.0 * wl.n_prefix * cfg.hidden * cfg.vocab,
        "lm_suffix": 2.0 * wl.n_suffix * cfg.hidden * cfg.vocab,
    }


def host_batch(wl, torch, pin=True):
    """Pinned host tensors of one batch, laid out as the library takes them."""
    from paper_2608_14498_b200.pipeline import Batch

    def t(a):
        if a.dtype == np.uint16:
            x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
        else:
            x = torch.from_numpy(a)
        return x.pin_memory() if pin else x

    pre, suf = wl.prefix_rows(), wl.suffix_rows()
    return Batch(
        t(wl.q[pre]), t(wl.k[pre]), t(wl.v[pre]), t(wl.q[suf]), t(wl.k[suf]), t(wl.v[suf]),
        t(wl.cu_prefix), t(wl.cu_suffix), t(wl.prompt_lens), t(wl.block_table),
        t(wl.hidden[pre]), t(wl.ids[pre]), t(wl.hidden[suf]), t(wl.ids[suf]),
        int(wl.prompt_lens.max()), int(wl.response_lens.max()))


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            pass
        self.marks = []

    def mark(self):
        self.tmp.flush()
        self.marks.append(os.path.getsize(self.tmp.name))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
        self.tmp.flush()
        with open(self.tmp.name) as fh:
            data = fh.read()
        os.unlink(self.tmp.name)
        lo = self.marks[0] if self.marks else 0
        hi = self.marks[1] if len(self.marks) > 1 else len(data)
        rows = [ln.split(",") for ln in data[lo:hi].splitlines() if ln.count(",") >= 7]
        all_rows = [ln.split(",") for ln in data.splitlines() if ln.count(",") >= 7]
        rows = rows or all_rows
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm, reasons = [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0]))
            except ValueError:
                continue
            for name, val in zip(names, r[4:8]):
                if val.strip().lower() == "active":
                    reasons.add(name)
        try:
            sm_max = float(rows[0][1])
        except ValueError:
            sm_max = None
        power = [float(r[2]) for r in rows if r[2].strip().replace(".", "", 1).isdigit()]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": sm_max, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


def oracle_sample(wl, n_tokens: int, seed: int):
    """Scores `n_tokens` sampled tokens with the oracle (all query heads + the log-prob row).
    Returns seconds."""
    import oracle

    cfg = wl.cfg
    rng = np.random.default_rng(seed)
    tok = np.sort(rng.choice(wl.n_tokens, size=n_tokens, replace=False)).astype(np.int64)
    seq = np.searchsorted(wl.cu_full, tok, side="right") - 1
    pos = tok - wl.cu_full[seq]
    rows = np.stack([np.repeat(seq, cfg.num_q_heads), np.repeat(pos, cfg.num_q_heads),
                     np.tile(np.arange(cfg.num_q_heads), n_tokens)], axis=1).astype(np.int32)
    t0 = time.perf_counter()
    oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, rows)
    oracle.logprob_rows(wl.hidden, wl.w, wl.ids, tok)
    return time.perf_counter() - t0


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle

    oracle.build()
    cfg = wk.CONFIGS[args.config]
    wl = wk.make_workload(cfg, seed=0)
    n = args.ref_tokens
    for w in range(args.warmup):
        oracle_sample(wl, n, 1000 + w)
    t = 0.0
    for s in range(args.steps):
        t += oracle_sample(wl, n, s)
    value = args.steps * n / t
    cores = oracle.num_threads()
    sample = f"{n} tokens per step drawn uniformly from the batch: {cfg.num_q_heads} attention rows + 1 log-prob row each, fp64"
    line = {
        "impl": "reference", "metric": "scored_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def measure_config(torch, dist, config, steps, warmup, rank, local_rank, world, cpu_tokens=0):
    """Times one config on this rank's GPU: device-resident steps with events around every call, then the
    end-to-end path from pinned host memory (synchronised per step, and with the caller one step behind).
    Rank 0 gets the result record (the others None).  Clocks are sampled while the timed regions run."""
    import paper_2608_14498_b200 as rpx
    from paper_2608_14498_b200.dist import job_throughput
    from paper_2608_14498_b200.pipeline import KERNELS_PER_SCORE, Batch, ScoringSession

    dev = torch.device("cuda", local_rank)

    def barrier():
        if world > 1:
            dist.barrier()

    cfg = wk.CONFIGS[config]
    wl = wk.make_workload(cfg, seed=rank)
    flops = flop_counts(wl)
    hb = host_batch(wl, torch)
    db = Batch(*[x.to(dev) for x in hb.tensors()], hb.max_prefix_len, hb.max_suffix_len)
    w_dev = torch.from_numpy(wl.w.view(np.int16)).view(torch.bfloat16).to(dev) if wl.w.dtype == np.uint16 \
        else torch.from_numpy(wl.w).to(dev)
    sess = ScoringSession(w_dev, wl.num_blocks, cfg.num_kv_heads, cfg.head_dim)
    lp_p_host = torch.empty(wl.n_prefix, dtype=torch.float32).pin_memory()
    lp_s_host = torch.empty(wl.n_suffix, dtype=torch.float32).pin_memory()

    for _ in range(max(warmup, 3)):
        sess.score(db)
    torch.cuda.synchronize()
    sess.check_status()

    try:
        gpu_id = str(torch.cuda.get_device_properties(local_rank).uuid)
        gpu_id = gpu_id if gpu_id.startswith("GPU-") else "GPU-" + gpu_id
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id) if rank == 0 else None
    time.sleep(0.3)

    # ---------------- device-resident timing: events around every call of every step
    names = ["prefix_attn", "lm_prefix", "suffix_attn", "lm_suffix"]
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(steps)]
    barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.mark()
    for s in range(steps):
        sess.score(db, events=ev[s])
    torch.cuda.synchronize()
    if sampler:
        sampler.mark()
    barrier()
    total_ms = ev[0][0].elapsed_time(ev[-1][4])
    per_kernel_ms = {n: sum(ev[s][i].elapsed_time(ev[s][i + 1]) for s in range(steps)) / steps
                     for i, n in enumerate(names)}
    sess.check_status()

    # ---------------- end to end from pinned host memory
    for _ in range(2):
        sess.score_from_host(hb, lp_p_host, lp_s_host)
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        sess.score_from_host(hb, lp_p_host, lp_s_host)
        torch.cuda.current_stream().synchronize()  # the caller consumes the log-probs every step
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    sess.check_status()
    # the same with the caller one step behind: results of step i are read while step i+1 runs (two sets of
    # host result buffers; the session's two device staging sets let step i+1 upload under step i's kernels)
    host_sets = [(lp_p_host, lp_s_host),
                 (torch.empty_like(lp_p_host).pin_memory(), torch.empty_like(lp_s_host).pin_memory())]
    done = [torch.cuda.Event(), torch.cuda.Event()]
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record()
    for i in range(steps):
        if i >= 2:
            done[i & 1].synchronize()  # step i-2's results have landed and been consumed: its buffers are free
        sess.score_from_host(hb, *host_sets[i & 1])
        done[i & 1].record()
    p1.record()
    torch.cuda.synchronize()
    e2e_pipelined_ms = p0.elapsed_time(p1)
    sess.check_status()
    clocks = sampler.stop() if sampler else None

    job_tokens, total_ms = job_throughput(wl.n_tokens, total_ms, dev)
    job_suffix, e2e_ms = job_throughput(wl.n_suffix, e2e_ms, dev)
    _, e2e_pipelined_ms = job_throughput(wl.n_tokens, e2e_pipelined_ms, dev)
    if rank != 0:
        return None

    peaks = load_peaks()
    ms_per_step = total_ms / steps
    total_flops = sum(flops.values())
    step_s = ms_per_step * 1e-3
    # a step is seconds of back-to-back tensor work at the power cap: the sustained peak applies
    peak_tf = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    burst_tf = float(peaks["bf16_tflops"])
    lm_ms = per_kernel_ms["lm_prefix"]
    lm_tf = flops["lm_prefix"] / (lm_ms * 1e-3) / 1e12
    kernels = {}
    for n in names:
        tf = flops[n] / (per_kernel_ms[n] * 1e-3) / 1e12
        kernels[n] = {"ms": round(per_kernel_ms[n], 4), "tflops": round(tf, 1),
                      "frac_of_sustained_peak": round(tf / peak_tf, 4), "frac_of_burst_peak": round(tf / burst_tf, 4),
                      "frac_of_datasheet_dense_bf16": round(tf / 2250.0, 4)}
    gb = lambda n: f"{n / 1e9:.2f} GB"
    rec = {
        "value": job_tokens / step_s, "ms_per_step": ms_per_step,
        "config": {"workload": cfg.name, "batch_per_gpu": cfg.batch, "prompt_tokens": wl.n_prefix,
                   "response_tokens": wl.n_suffix, "scored_tokens_per_gpu": wl.n_tokens, "q_heads": cfg.num_q_heads,
                   "kv_heads": cfg.num_kv_heads, "head_dim": cfg.head_dim, "hidden": cfg.hidden, "vocab": cfg.vocab,
                   "kv_block": 16, "parallelism": f"dp{world} (independent sequences per rank, no collective)",
                   "lm_head_kernel": "CTA pairs (cta_group::2)" if rpx.get_lm_head_pairing() else "one CTA per tile",
                   "l2": f"no flush: per-step inputs (W_vocab {gb(wl.w.nbytes)}, hidden {gb(wl.hidden.nbytes)}, "
                         f"Q/K/V {gb(wl.q.nbytes + wl.k.nbytes + wl.v.nbytes)}) exceed the 126 MB L2",
                   "stands_in_for": cfg.stands_in_for},
        "tflops": total_flops * world / step_s / 1e12,
        "frac_of_sustained_peak": total_flops / step_s / 1e12 / peak_tf,
        "frac_of_burst_peak": total_flops / step_s / 1e12 / burst_tf,
        "response_tokens_per_s": job_suffix / step_s,
        "kernels": kernels,
        "roofline": {"kernel": "lm_head_partial_kernel (prompt rows; event pair spans it and its 0.1 % combine kernel)",
                     "bound": "tensor", "achieved": lm_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": lm_tf / peak_tf,
                     "peak_kind": f"bf16_tflops_sustained of {peaks['source']}",
                     "frac_of_burst_peak": lm_tf / burst_tf,
                     "traffic": LM_HEAD_TRAFFIC_BYTES.get(config),
                     "algorithmic_bytes": (wl.n_prefix * cfg.hidden + cfg.vocab * cfg.hidden) * 2 + 8 * wl.n_prefix},
        "e2e": {"value": job_tokens / (e2e_ms / steps * 1e-3), "unit": "tokens/s",
                "h2d_bytes_per_step": hb.nbytes(), "d2h_bytes_per_step": (wl.n_prefix + wl.n_suffix) * 4,
                "ms_per_step": e2e_ms / steps,
                "note": "the stream is synchronised after every step; with the caller one step behind "
                        "(double-buffered results) a step takes pipelined_ms_per_step.  Only the log-probs come "
                        "back to the host: the attention outputs O_p / O_s stay on the device by design (they "
                        "feed the next layer there), so they are not part of d2h_bytes_per_step",
                "pipelined_ms_per_step": e2e_pipelined_ms / steps},
        "gpu_launches": KERNELS_PER_SCORE * steps,
        "gpu_launches_e2e": sess.kernels_last_host_pass * steps,
        "clocks": clocks,
        "steps": steps,
    }
    if world == 1 and cpu_tokens > 0:
        import oracle

        oracle.build()
        t = oracle_sample(wl, cpu_tokens, 0)
        rec["cpu_baseline"] = {
            "value": cpu_tokens / t, "unit": "tokens/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{cpu_tokens} tokens drawn uniformly from the batch ({cfg.num_q_heads} attention rows + 1 log-prob row each), {t:.1f} s"}
    return rec


def measure_backward(torch, config, local_rank, reps=3):
    """The LM-head backward pass (dL/dz recomputed block by block from the saved lse, then dlogits x W) on the prompt
    rows of one config: milliseconds, TFLOP/s on 4 * N * H * V algorithmic flops (the logits GEMM again plus the
    dhidden GEMM), fractions of the measured peaks, and the clocks sampled meanwhile."""
    import paper_2608_14498_b200 as rpx
    from paper_2608_14498_b200 import binding as B

    dev = torch.device("cuda", local_rank)
    cfg = wk.CONFIGS[config]
    wl = wk.make_workload(cfg, seed=0, attn=False)
    pre = wl.prefix_rows()

    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.to(dev)

    h, w, ids = t(wl.hidden[pre]), t(wl.w), t(wl.ids[pre])
    n = h.shape[0]
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    _, lse = rpx.token_logprobs(h, w, ids, return_lse=True, device_status=status)
    g = torch.ones(n, dtype=torch.float32, device=dev)
    dh = torch.empty_like(h)
    ws = torch.empty(B.token_logprobs_backward_workspace_bytes(n, cfg.hidden, cfg.vocab), dtype=torch.uint8, device=dev)
    rpx.token_logprobs_backward(h, w, ids, lse, g, dhidden=dh, workspace=ws, device_status=status)
    torch.cuda.synchronize()
    try:
        gpu_id = str(torch.cuda.get_device_properties(local_rank).uuid)
        gpu_id = gpu_id if gpu_id.startswith("GPU-") else "GPU-" + gpu_id
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark()
    e0.record()
    for _ in range(reps):
        rpx.token_logprobs_backward(h, w, ids, lse, g, dhidden=dh, workspace=ws, device_status=status)
    e1.record()
    torch.cuda.synchronize()
    sampler.mark()
    clocks = sampler.stop()
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} in the backward pass")
    ms = e0.elapsed_time(e1) / reps
    peaks = load_peaks()
    tf = 4.0 * n * cfg.hidden * cfg.vocab / (ms * 1e-3) / 1e12
    # the same call with the weight gradient as well (a third GEMM over the same block-wise dL/dz)
    dw = torch.empty((cfg.vocab, cfg.hidden), dtype=torch.float32, device=dev)
    rpx.token_logprobs_backward(h, w, ids, lse, g, dhidden=dh, dw=dw, workspace=ws, device_status=status)
    torch.cuda.synchronize()
    sampler = ClockSampler(gpu_id)
    time.sleep(0.3)
    sampler.mark()
    e0.record()
    for _ in range(reps):
        rpx.token_logprobs_backward(h, w, ids, lse, g, dhidden=dh, dw=dw, workspace=ws, device_status=status)
    e1.record()
    torch.cuda.synchronize()
    sampler.mark()
    clocks_dw = sampler.stop()
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} in the backward pass")
    ms_dw = e0.elapsed_time(e1) / reps
    tf_dw = 6.0 * n * cfg.hidden * cfg.vocab / (ms_dw * 1e-3) / 1e12
    sustained = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    return {"what": "rpx_token_logprobs_backward on the prompt rows (dL/dz from the saved lse, then dlogits x W)",
            "workload": cfg.name, "rows": n, "ms": ms, "tflops": tf,
            "frac_of_sustained_peak": tf / sustained,
            "frac_of_burst_peak": tf / float(peaks["bf16_tflops"]), "workspace_bytes": ws.numel(),
            "gpu_launches": 2 * reps * -(-n // 9472), "clocks": clocks,
            "with_weight_gradient": {"what": "rpx_token_logprobs_backward_full: dhidden and dW (6 * N * H * V flops)",
                                     "ms": ms_dw, "tflops": tf_dw, "frac_of_sustained_peak": tf_dw / sustained,
                                     "frac_of_burst_peak": tf_dw / float(peaks["bf16_tflops"]),
                                     "gpu_launches": 3 * reps * -(-n // 9472), "clocks": clocks_dw}}


def measure_attn_backward(torch, config, local_rank, reps=60):
    """rpx_attn_backward over the whole sequences (prompt then response) of one config, with out and lse from the
    library's forward pass: milliseconds; TFLOP/s on the algorithmic flops (five products per causal tile pair: S, dP,
    dV, dK, dQ = 2.5 x the forward pass) and on the executed ones (seven: the dQ kernel recomputes S and dP)."""
    import paper_2608_14498_b200 as rpx
    from paper_2608_14498_b200 import binding as B

    dev = torch.device("cuda", local_rank)
    cfg = wk.CONFIGS[config]
    wl = wk.make_workload(cfg, seed=0, lm=False)

    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.to(dev)

    q, k, v, cu = t(wl.q), t(wl.k), t(wl.v), t(wl.cu_full)
    dout = t(wk.make_workload(cfg, seed=1, lm=False).q)  # an upstream gradient with the same distribution as q
    lens = (wl.prompt_lens + wl.response_lens).astype(np.int64)
    max_len, n = int(lens.max()), int(lens.sum())
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    out, lse = rpx.prefix_attn(q, k, v, cu, max_len, return_lse=True, device_status=status)
    dq = torch.empty(tuple(q.shape), dtype=torch.float32, device=dev)
    dk = torch.empty(tuple(k.shape), dtype=torch.float32, device=dev)
    dvv = torch.empty_like(dk)
    ws = torch.empty(B.attn_backward_workspace_bytes(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, n), dtype=torch.uint8,
                     device=dev)

    def call():
        rpx.attn_backward(q, k, v, out, dout, lse, cu, max_len, dq=dq, dk=dk, dv=dvv, workspace=ws, device_status=status)

    for _ in range(2):
        call()
    torch.cuda.synchronize()
    try:
        gpu_id = str(torch.cuda.get_device_properties(local_rank).uuid)
        gpu_id = gpu_id if gpu_id.startswith("GPU-") else "GPU-" + gpu_id
    except Exception:
        gpu_id = str(local_rank)
    sampler = ClockSampler(gpu_id)
    time.sleep(0.3)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.mark()
    e0.record()
    for _ in range(reps):
        call()
    e1.record()
    torch.cuda.synchronize()
    sampler.mark()
    clocks = sampler.stop()
    if int(status.item()) != 0:
        raise SystemExit(f"device status {int(status.item())} in the attention backward pass")
    ms = e0.elapsed_time(e1) / reps
    peaks = load_peaks()
    fwd = float((4.0 * cfg.head_dim * cfg.num_q_heads * (lens * (lens + 1) / 2)).sum())
    tf, tf_exec = 2.5 * fwd / (ms * 1e-3) / 1e12, 3.5 * fwd / (ms * 1e-3) / 1e12
    sustained = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    return {"what": "rpx_attn_backward over the whole sequences (D, clears, the dK/dV kernel, the dQ kernel)",
            "workload": cfg.name, "tokens": n, "ms": ms, "tflops": tf, "tflops_executed": tf_exec,
            "frac_of_sustained_peak": tf / sustained, "executed_frac_of_sustained_peak": tf_exec / sustained,
            "frac_of_burst_peak": tf / float(peaks["bf16_tflops"]), "workspace_bytes": ws.numel(),
            "gpu_launches": 5 * reps, "clocks": clocks}


def run_ours(args, rank, local_rank, world):
    import torch
    import torch.distributed as dist

    import paper_2608_14498_b200 as rpx

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the scoring path has no CPU fallback")
    rpx.load_library()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    head = measure_config(torch, dist, args.config, args.steps, args.warmup, rank, local_rank, world,
                          cpu_tokens=0 if args.no_cpu_baseline else args.cpu_tokens)
    others = {}
    if world == 1 and not args.no_sub_configs:
        # the other bf16 configs, measured the same way with their own clock samples; C2's steps are short, so it
        # gets four times as many, which keeps every timed loop at two seconds or more (long enough for the power
        # cap to settle and for the clock sampler to see it)
        for name in ("C2", "C4", "C5"):
            if name == args.config:
                continue
            torch.cuda.empty_cache()
            sub = measure_config(torch, dist, name, args.steps * (4 if name == "C2" else 1), args.warmup, rank, local_rank, world)
            others[name] = {k: sub[k] for k in ("value", "ms_per_step", "steps", "tflops", "frac_of_sustained_peak",
                                                "frac_of_burst_peak", "kernels", "e2e", "clocks")}
            others[name]["workload"] = sub["config"]["workload"]
    backward = None
    if world == 1 and not args.no_backward:
        torch.cuda.empty_cache()
        backward = {"lm_head": measure_backward(torch, "C2", local_rank)}
        torch.cuda.empty_cache()
        backward["attention"] = measure_attn_backward(torch, "C2", local_rank)
    if rank == 0:
        line = {
            "metric": "scored_tokens_per_s", "value": head["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        }
        line.update({k: v for k, v in head.items() if k not in ("value", "ms_per_step", "steps")})
        if others:
            line["configs"] = others
        if backward:
            line["backward"] = backward
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_profile_case(args):
    """Small, self-terminating launches of one kernel for profiler captures.  Each case keeps a few hundred MB on
    the device (more than the 126 MB L2, so DRAM counters mean something) and launches the kernel `reps` times
    after one warm-up launch.
      lm      8192 rows x 32768 vocabulary columns, hidden 3584  (7B-shaped slice of the LM head)
      lmbwd   the same slice through rpx_token_logprobs_backward (two kernels per launch: dL/dz, then dhidden)
      lmdw    the same with the weight gradient as well (three kernels per launch: dL/dz, dhidden, dW)
      prefix  4 sequences x 4096 prompt tokens, 28 query / 4 KV heads, head_dim 128, with cache write
      suffix  the same 4 prompts cached, 256 response tokens each
      attnbwd rpx_attn_backward over the same 4 sequences whole (4352 tokens each): D, two clears, the dK/dV kernel,
              the dQ kernel per launch"""
    import torch

    import paper_2608_14498_b200 as rpx

    dev = torch.device("cuda:0")

    def dv(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    case = args.profile_case
    if case == "lm":
        cfg = wk.Config("profile-lm", "bf16", 1, 28, 4, 128, 3584, 32768, ("fixed", 8192), ("fixed", 0))
        wl = wk.make_workload(cfg, seed=0, attn=False)
        h, w, ids = dv(wl.hidden), dv(wl.w), dv(wl.ids)
        for _ in range(1 + args.reps):
            rpx.token_logprobs(h, w, ids, device_status=status)
    elif case in ("lmbwd", "lmdw"):
        cfg = wk.Config("profile-lm", "bf16", 1, 28, 4, 128, 3584, 32768, ("fixed", 8192), ("fixed", 0))
        wl = wk.make_workload(cfg, seed=0, attn=False)
        h, w, ids = dv(wl.hidden), dv(wl.w), dv(wl.ids)
        _, lse = rpx.token_logprobs(h, w, ids, return_lse=True, device_status=status)
        g = torch.ones(h.shape[0], dtype=torch.float32, device=dev)
        dw = torch.empty((w.shape[0], w.shape[1]), dtype=torch.float32, device=dev) if case == "lmdw" else None
        for _ in range(1 + args.reps):
            rpx.token_logprobs_backward(h, w, ids, lse, g, dw=dw, device_status=status)
    elif case == "attnbwd":
        cfg = wk.Config("profile-attn", "bf16", 4, 28, 4, 128, 3584, 1024, ("fixed", 4096), ("fixed", 256))
        wl = wk.make_workload(cfg, seed=0, lm=False)
        q, k, v, cu = dv(wl.q), dv(wl.k), dv(wl.v), dv(wl.cu_full)
        out, lse = rpx.prefix_attn(q, k, v, cu, 4352, return_lse=True, device_status=status)
        dout = dv(wk.make_workload(cfg, seed=1, lm=False).q)
        for _ in range(1 + args.reps):
            rpx.attn_backward(q, k, v, out, dout, lse, cu, 4352, device_status=status)
    else:
        cfg = wk.Config("profile-attn", "bf16", 4, 28, 4, 128, 3584, 1024, ("fixed", 4096), ("fixed", 256))
        wl = wk.make_workload(cfg, seed=0, lm=False)
        kc = torch.zeros((wl.num_blocks, 4, 16, 128), dtype=torch.bfloat16, device=dev)
        cache = (kc, torch.zeros_like(kc), dv(wl.block_table))
        qp, kp, vp = (dv(wl.prefix_pack(t)) for t in (wl.q, wl.k, wl.v))
        qs, ks, vs = (dv(wl.suffix_pack(t)) for t in (wl.q, wl.k, wl.v))
        cu_p, cu_s, pl = dv(wl.cu_prefix), dv(wl.cu_suffix), dv(wl.prompt_lens)
        rpx.prefix_attn(qp, kp, vp, cu_p, 4096, cache=cache, device_status=status)
        for _ in range(args.reps + (1 if case == "suffix" else 0)):
            if case == "prefix":
                rpx.prefix_attn(qp, kp, vp, cu_p, 4096, cache=cache, device_status=status)
            else:
                rpx.suffix_attn(qs, ks, vs, cu_s, pl, 256, 4096, cache=cache, device_status=status)
    torch.cuda.synchronize()
    code = int(status.item())
    if code != 0:
        raise SystemExit(f"device status {code}: {rpx.status_string(code)}")
    print(f"profile case {case}: ok")


def run_attn_alone(args):
    """The attention passes alone, `reps` launches back to back per pass and config, with the clocks sampled during
    each timed region: what the kernels do at the clock they reach when the LM head's power draw is not setting it.
    One JSON line per config (C2, C3, C4): prefix pass (with cache write), suffix pass, TFLOP/s on the algorithmic
    (causal) flops and fractions of the measured peaks."""
    import torch

    import paper_2608_14498_b200 as rpx

    dev = torch.device("cuda", 0)
    peaks = load_peaks()
    try:
        gpu_id = str(torch.cuda.get_device_properties(0).uuid)
        gpu_id = gpu_id if gpu_id.startswith("GPU-") else "GPU-" + gpu_id
    except Exception:
        gpu_id = "0"

    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.to(dev)

    def timed(call):
        for _ in range(3):
            call()
        torch.cuda.synchronize()
        sampler = ClockSampler(gpu_id)
        time.sleep(0.3)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        sampler.mark()
        e0.record()
        for _ in range(args.reps):
            call()
        e1.record()
        torch.cuda.synchronize()
        sampler.mark()
        return e0.elapsed_time(e1) / args.reps, sampler.stop()

    for name in ("C2", "C3", "C4"):
        cfg = wk.CONFIGS[name]
        wl = wk.make_workload(cfg, seed=0, lm=False)
        status = torch.zeros(1, dtype=torch.int32, device=dev)
        kc = torch.zeros((wl.num_blocks, cfg.num_kv_heads, 16, cfg.head_dim), dtype=torch.bfloat16, device=dev)
        cache = (kc, torch.zeros_like(kc), t(wl.block_table))
        qp, kp, vp = (t(wl.prefix_pack(x)) for x in (wl.q, wl.k, wl.v))
        qs, ks, vs = (t(wl.suffix_pack(x)) for x in (wl.q, wl.k, wl.v))
        cu_p, cu_s, pl = t(wl.cu_prefix), t(wl.cu_suffix), t(wl.prompt_lens)
        max_p, max_r = int(wl.prompt_lens.max()), int(wl.response_lens.max())
        op, os_ = torch.empty_like(qp), torch.empty_like(qs)
        ws_p = torch.empty(rpx.prefix_attn_workspace_bytes(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, 0, qp.shape[0]),
                           dtype=torch.uint8, device=dev)
        ws_s = torch.empty(rpx.suffix_attn_workspace_bytes(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim, 0, qs.shape[0]),
                           dtype=torch.uint8, device=dev)
        ms_p, clk_p = timed(lambda: rpx.prefix_attn(qp, kp, vp, cu_p, max_p, cache=cache, out=op, workspace=ws_p,
                                                    device_status=status))
        ms_s, clk_s = timed(lambda: rpx.suffix_attn(qs, ks, vs, cu_s, pl, max_r, max_p, cache=cache, out=os_, workspace=ws_s,
                                                    device_status=status))
        if int(status.item()) != 0:
            raise SystemExit(f"device status {int(status.item())}")
        p64, r64 = wl.prompt_lens.astype(np.float64), wl.response_lens.astype(np.float64)
        fl_p = float((4.0 * cfg.head_dim * cfg.num_q_heads * p64 * (p64 + 1) / 2).sum())
        fl_s = float((4.0 * cfg.head_dim * cfg.num_q_heads * (r64 * p64 + r64 * (r64 + 1) / 2)).sum())
        rec = {"workload": cfg.name, "reps": args.reps}
        for key, ms, fl, clk in (("prefix_attn", ms_p, fl_p, clk_p), ("suffix_attn", ms_s, fl_s, clk_s)):
            tf = fl / (ms * 1e-3) / 1e12
            rec[key] = {"ms": ms, "tflops": tf,
                        "frac_of_sustained_peak": tf / float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])),
                        "frac_of_burst_peak": tf / float(peaks["bf16_tflops"]), "frac_of_datasheet": tf / 2250.0,
                        "clocks": clk}
        print(json.dumps(rec), flush=True)
        del qp, kp, vp, qs, ks, vs, op, os_, kc, cache
        torch.cuda.empty_cache()


def run_group(args):
    """Prompt groups (GRPO: N sampled responses per prompt).  Times one scoring pass with the prompt
    prefix computed once per group (cache rows aliased by the group's members) against the same
    members scored as unrelated sequences, each with its own copy of the prompt."""
    import torch

    import paper_2608_14498_b200 as rpx
    from paper_2608_14498_b200.pipeline import Batch, ScoringSession

    dev = torch.device("cuda", 0)
    cfg = wk.CONFIGS[args.config]
    if args.group_responses:  # e.g. 16:64 = response lengths uniform in [16, 64] (short answers: most of a query tile is padding)
        lo, hi = (int(x) for x in args.group_responses.split(":"))
        cfg = cfg.scaled(name=f"{cfg.name}-r{lo}to{hi}", response=("uniform", lo, hi))
    gw = wk.make_group_workload(cfg, args.group, seed=0)
    pro, mem = gw.prompts, gw.members

    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.to(dev)

    w = t(pro.w)
    sess = ScoringSession(w, pro.num_blocks, cfg.num_kv_heads, cfg.head_dim)
    pre, suf = mem.prefix_rows(), mem.suffix_rows()
    shared = Batch(t(pro.q), t(pro.k), t(pro.v), t(mem.q[suf]), t(mem.k[suf]), t(mem.v[suf]), t(pro.cu_full),
                   t(mem.cu_suffix), t(mem.prompt_lens), t(gw.member_table), t(pro.hidden), t(pro.ids), t(mem.hidden[suf]),
                   t(mem.ids[suf]), int(pro.prompt_lens.max()), int(mem.response_lens.max()))
    own_table, own_blocks = wk.make_block_table(mem.prompt_lens, seed=1)
    sess_own = ScoringSession(w, own_blocks, cfg.num_kv_heads, cfg.head_dim)
    unshared = Batch(t(mem.q[pre]), t(mem.k[pre]), t(mem.v[pre]), shared.q_s, shared.k_s, shared.v_s, t(mem.cu_prefix),
                     shared.cu_suffix, shared.prefix_lens, t(own_table), t(mem.hidden[pre]), t(mem.ids[pre]), shared.hidden_s,
                     shared.ids_s, shared.max_prefix_len, shared.max_suffix_len)

    def timed(session, batch, kernel_ms=None):
        for _ in range(3):
            session.score(batch)
        torch.cuda.synchronize()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
        for s in range(args.steps):
            session.score(batch, events=ev[s])
        torch.cuda.synchronize()
        session.check_status()
        if kernel_ms is not None:
            for i, n in enumerate(["prefix_attn", "lm_prefix", "suffix_attn", "lm_suffix"]):
                kernel_ms[n] = sum(e[i].elapsed_time(e[i + 1]) for e in ev) / args.steps
        return ev[0][0].elapsed_time(ev[-1][4]) / args.steps

    kernel_ms = {}
    ms_shared, ms_unshared = timed(sess, shared, kernel_ms), timed(sess_own, unshared)
    r = mem.response_lens.astype(np.float64)
    pl = mem.prompt_lens.astype(np.float64)
    suffix_flops = float((4.0 * cfg.head_dim * cfg.num_q_heads * (r * pl + r * (r + 1) / 2)).sum())
    lp_a = sess.score(shared)[1].clone()
    lp_b = sess_own.score(unshared)[1]
    torch.cuda.synchronize()
    line = {
        "metric": "scored_tokens_per_s", "value": mem.n_tokens / (ms_shared * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": 3, "ms_per_step": ms_shared, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{cfg.name} as {cfg.batch} prompts x {args.group} responses, prefix scored once per prompt",
                   "member_tokens": mem.n_tokens, "prompt_rows_computed": pro.n_tokens, "response_rows": mem.n_suffix,
                   "response_lens": [int(mem.response_lens.min()), int(mem.response_lens.max())]},
        "kernels_ms": {k: round(v, 4) for k, v in kernel_ms.items()},
        "suffix_attn_tflops": suffix_flops / (kernel_ms["suffix_attn"] * 1e-3) / 1e12,
        "group": {"size": args.group, "ms_shared_prefix": ms_shared, "ms_every_member_own_prefix": ms_unshared,
                  "speedup": ms_unshared / ms_shared,
                  "suffix_logprob_max_abs_diff": float((lp_a - lp_b).abs().max().item())},
        "gpu_launches": 6 * args.steps,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="C3", choices=sorted(wk.CONFIGS), help="headline workload (C3 = the largest single-GPU config)")
    ap.add_argument("--no-sub-configs", action="store_true", help="skip the C2 / C4 / C5 records of the `configs` key")
    ap.add_argument("--no-backward", action="store_true", help="skip the LM-head backward record (key `backward`)")
    ap.add_argument("--profile-case", choices=["lm", "lmbwd", "lmdw", "prefix", "suffix", "attnbwd"], help="launch one kernel a few times on a small case and exit")
    ap.add_argument("--lm-head-pairing", action="store_true",
                    help="run the LM head's CTA-pair (cta_group::2) kernel instead of the single-CTA one")
    ap.add_argument("--attn-alone", action="store_true", help="time the attention passes of C2, C3 and C4 alone (--reps launches each)")
    ap.add_argument("--reps", type=int, default=3, help="launches of --profile-case after its warm-up launch")
    ap.add_argument("--cpu-tokens", type=int, default=256, help="tokens the oracle scores for cpu_baseline (~10-20 s)")
    ap.add_argument("--ref-tokens", type=int, default=8, help="tokens per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--group", type=int, default=0, help="score prompt groups of this size (prefix once per prompt)")
    ap.add_argument("--group-responses", default="", help="with --group: LO:HI = response lengths uniform in [LO, HI]")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.lm_head_pairing and args.impl != "reference":
        import paper_2608_14498_b200 as rpx

        rpx.set_lm_head_pairing(True)
    if args.profile_case:
        if rank == 0:
            run_profile_case(args)
    elif args.attn_alone:
        if rank == 0:
            if args.reps < 10:
                args.reps = 30
            run_attn_alone(args)
    elif args.group > 0:
        if rank == 0:
            run_group(args)
    elif args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
