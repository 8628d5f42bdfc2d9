"""The co-run micro-benchmark for the overlap model (Eq. 1, Section 3.1) on a tiny workload: the scoring pass that
ran beside the decode stand-in must still match the oracle, under an SM budget as well, and every record must carry
the quantities of Eq. 1 together with the clocks sampled while it was measured."""
import json

import numpy as np
import pytest

import oracle
from paper_2608_14498_b200 import corun
from paper_2608_14498_b200 import workloads as wk

pytestmark = pytest.mark.gpu

KEYS = {"experiment", "workload", "sm_budget", "decode_steps", "T_D_ms", "T_P_ms", "T_D_corun_ms", "T_P_corun_ms",
        "Delta_D_ms", "Delta_D_pct", "prefix_slowdown_pct", "S_measured_ms", "S_eq1_ms", "serial_ms", "overlapped_ms",
        "speedup", "clocks"}


def test_corun_measurement_keeps_scoring_correct_and_reports_eq1(cuda_device):
    cfg = wk.Config("corun-tiny", "bf16", 3, 8, 2, 128, 256, 4096, ("list", [300, 129, 40]), ("list", [0, 0, 0]))
    wl = wk.make_workload(cfg, seed=61)
    lines = []
    res = corun.run(ratios=(1.0, 2.0), reps=2, decode_gb=0.05, sm_budgets=(0, 40), workload=wl, emit=lines.append)
    assert len(res["records"]) == 4 and len(lines) == 4
    for text, rec in zip(lines, res["records"]):
        assert json.loads(text)["workload"] == "corun-tiny"
        assert KEYS <= set(rec)
        assert rec["T_D_ms"] > 0 and rec["T_P_ms"] > 0 and rec["overlapped_ms"] >= max(rec["T_D_corun_ms"], rec["T_P_corun_ms"]) - 1e-9
        # Eq. 1 with the measured decode slowdown: S = T_D + T_P - max(T_D + Delta_D, T_P) = min(T_P - Delta_D, T_D)
        assert rec["S_eq1_ms"] == pytest.approx(min(rec["T_P_ms"] - rec["Delta_D_ms"], rec["T_D_ms"]), abs=1e-6)
        assert rec["S_measured_ms"] == pytest.approx(rec["serial_ms"] - rec["overlapped_ms"], abs=1e-6)
        assert set(rec["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons", "samples"}
    assert [r["sm_budget"] for r in res["records"]] == [0, 0, 40, 40]
    # what the last co-run (under the 40-SM budget) left behind equals the oracle's prefix attention and log-probs
    out = res["check"]["out"].double().cpu().numpy()
    rows = oracle.all_rows(wl.cu_full, cfg.num_q_heads)
    ref_o, _ = oracle.attn_rows(wl.q, wl.k, wl.v, wl.cu_full, rows)
    tok = wl.cu_full[rows[:, 0]].astype(np.int64) + rows[:, 1]
    assert np.abs(out[tok, rows[:, 2]] - ref_o).max() <= 1e-2
    ref_lp, _ = oracle.logprob_rows(wl.hidden, wl.w, wl.ids)
    assert np.abs(res["check"]["logprobs"].double().cpu().numpy() - ref_lp).max() <= 5e-4
