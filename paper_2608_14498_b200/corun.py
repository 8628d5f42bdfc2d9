"""Co-run micro-benchmark for the paper's overlap model (Eq. 1, Section 3.1).

    python -m paper_2608_14498_b200.corun [--config C2] [--ratios 0.5 1 2] [--reps 5]

Eq. 1:  T = max(T_D + Delta_D, T_P) + T_post,   S = T_D + T_P - max(T_D + Delta_D, T_P)
                                                  = min(T_P - Delta_D, T_D)
with T_D the standalone decode time, T_P the makespan of the prefix work that runs beside it and
Delta_D the decode slowdown the co-running prefixes cause.

What runs here, in ONE process on ONE GPU (no MPS, no second process; the GPU's settings are left
alone): the prefix work is this library's Phase-1 pass (prefix attention + KV write, LM-head
log-probs on the prompt rows) on one stream; beside it, on a second stream, a stand-in for
autoregressive decode: a train of bandwidth-bound matrix-vector products, each streaming a
weight matrix from HBM once (what a decode step does with the model weights; the paper measures
under 19 % active SMs for it).  The stand-in is torch.mv — it is the interfering workload, not
part of the scoring path.  Reported per decode length: T_D, T_P alone, both under co-run, Delta_D,
the measured saving S = T_D + T_P - makespan and Eq. 1's S from the measured Delta_D and the
standalone T_P (the model has no term for the prefix work's own slowdown; the difference shows it).

``--sm-budgets`` repeats the measurement with the persistent LM-head grid capped at that many CTAs
(``rpx_set_sm_budget``; 0 = all SMs), which is how a caller leaves the decode side room: T_P grows
by about SMs/budget, Delta_D shrinks.
"""
from __future__ import annotations

import argparse
import json
import statistics
import subprocess
import threading
import time

import numpy as np


class _Clocks:
    """SM clock and throttle reasons sampled with nvidia-smi (read-only) while a measurement runs."""

    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int = 0, period_s: float = 0.1):
        self.index, self.period_s, self.rows, self._stop = index, period_s, [], threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                self.rows.append([x.strip() for x in out.strip().split(",")])
            except (OSError, subprocess.SubprocessError):
                return
            self._stop.wait(self.period_s)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        mhz = [float(r[0]) for r in self.rows if len(r) >= 6 and r[0].replace(".", "", 1).isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 6 for n, v in zip(names, r[2:6]) if v.lower() == "active"})
        sm_max = next((float(r[1]) for r in self.rows if len(r) >= 6 and r[1].replace(".", "", 1).isdigit()), None)
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": sm_max, "reasons": reasons,
                "samples": len(mhz)}


def run(config: str = "C2", ratios=(0.5, 1.0, 2.0), reps: int = 5, decode_gb: float = 4.0, sm_budgets=(0,), workload=None,
        emit=print):
    """Runs the measurement and returns its records (one per SM budget and decode length); `emit` gets each as a
    JSON line.  `workload` overrides the named config (used by the tests with a tiny one).  Also returns, under
    "check", what the scoring pass produced during the last co-run, so a caller can compare it with the oracle."""
    import torch

    from . import binding as B
    from . import workloads as wk
    from .pipeline import ScoringSession

    class _Args:
        pass

    args = _Args()
    args.ratios, args.reps, args.decode_gb, args.sm_budgets = list(ratios), reps, decode_gb, list(sm_budgets)
    dev = torch.device("cuda", 0)
    B.load_library()

    wl = workload if workload is not None else wk.make_workload(wk.CONFIGS[config], seed=0)
    cfg = wl.cfg
    records = []

    def t(a):
        x = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if a.dtype == np.uint16 else torch.from_numpy(a)
        return x.to(dev)

    pre = wl.prefix_rows()
    q, k, v, hid, ids = (t(x[pre]) for x in (wl.q, wl.k, wl.v, wl.hidden, wl.ids))
    cu, table = t(wl.cu_prefix), t(wl.block_table)
    sess = ScoringSession(t(wl.w), wl.num_blocks, cfg.num_kv_heads, cfg.head_dim)
    out = torch.empty_like(q)
    lp = torch.empty(q.shape[0], dtype=torch.float32, device=dev)
    ws = torch.empty(B.token_logprobs_workspace_bytes(q.shape[0], cfg.hidden, cfg.vocab, B.RPX_BF16), dtype=torch.uint8,
                     device=dev)
    max_p = int(wl.prompt_lens.max())

    def prefix_work():
        B.prefix_attn(q, k, v, cu, max_p, cache=(sess.k_cache, sess.v_cache, table), out=out, device_status=sess.status)
        B.token_logprobs(hid, sess.w_vocab, ids, logprobs=lp, workspace=ws, device_status=sess.status)

    cols = 16384
    rows = int(args.decode_gb * 1e9 / 2 / cols)
    wd = torch.randn(rows, cols, device=dev, dtype=torch.bfloat16)
    xd = torch.randn(cols, device=dev, dtype=torch.bfloat16)
    yd = torch.empty(rows, device=dev, dtype=torch.bfloat16)

    def decode_work(steps: int):
        for _ in range(steps):
            torch.mv(wd, xd, out=yd)

    s_p, s_d = torch.cuda.Stream(), torch.cuda.Stream()

    def timed(run_p: bool, steps: int):
        """Milliseconds from a common start to the end of each stream's work."""
        start = torch.cuda.Event(enable_timing=True)
        end_p, end_d = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        start.record()
        s_p.wait_event(start)
        s_d.wait_event(start)
        if steps > 0:
            with torch.cuda.stream(s_d):
                decode_work(steps)
                end_d.record()
        if run_p:
            with torch.cuda.stream(s_p):
                prefix_work()
                end_p.record()
        torch.cuda.synchronize()
        return (start.elapsed_time(end_p) if run_p else 0.0), (start.elapsed_time(end_d) if steps > 0 else 0.0)

    def median(run_p: bool, steps: int):
        vals = [timed(run_p, steps) for _ in range(args.reps)]
        return statistics.median(x[0] for x in vals), statistics.median(x[1] for x in vals)

    for _ in range(3):
        timed(True, 4)
    _, t_step = median(False, 16)
    t_step /= 16
    for budget in args.sm_budgets:
        B.set_sm_budget(budget)
        t_p, _ = median(True, 0)
        sess.check_status()
        for ratio in args.ratios:
            steps = max(1, round(ratio * t_p / t_step))
            with _Clocks() as clk:
                _, t_d = median(False, steps)
                t_p_co, t_d_co = median(True, steps)
            delta_d = t_d_co - t_d
            makespan = max(t_d_co, t_p_co)
            line = {
                "experiment": "corun_eq1", "workload": cfg.name, "sm_budget": budget, "decode_steps": steps,
                "decode_step_bytes": rows * cols * 2, "T_D_ms": t_d, "T_P_ms": t_p, "T_D_corun_ms": t_d_co,
                "T_P_corun_ms": t_p_co, "Delta_D_ms": delta_d, "Delta_D_pct": 100.0 * delta_d / t_d,
                "prefix_slowdown_pct": 100.0 * (t_p_co - t_p) / t_p,
                "S_measured_ms": t_d + t_p - makespan,
                # Eq. 1 with the measured Delta_D; it charges interference to decode only, so the gap to
                # S_measured is the prefix work's own slowdown under co-run
                "S_eq1_ms": t_d + t_p - max(t_d + delta_d, t_p),
                "serial_ms": t_d + t_p, "overlapped_ms": makespan, "speedup": (t_d + t_p) / makespan,
                "clocks": clk.summary(),
            }
            records.append(line)
            emit(json.dumps(line))
    B.set_sm_budget(0)
    sess.check_status()
    torch.cuda.synchronize()
    return {"records": records, "check": {"out": out, "logprobs": lp, "prefix_rows": pre}}


def main() -> None:
    from . import workloads as wk

    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2", choices=sorted(wk.CONFIGS))
    ap.add_argument("--ratios", type=float, nargs="+", default=[0.5, 1.0, 2.0], help="target T_D / T_P")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--decode-gb", type=float, default=4.0, help="weight bytes one decode step streams")
    ap.add_argument("--sm-budgets", type=int, nargs="+", default=[0], help="LM-head CTA caps to sweep (0 = none)")
    args = ap.parse_args()
    run(args.config, args.ratios, args.reps, args.decode_gb, args.sm_budgets, emit=lambda s: print(s, flush=True))


if __name__ == "__main__":
    main()
