"""Small, self-terminating launches of each kernel for profiler captures.

    python -m paper_2608_14498_b200.profile_case lm      [--reps 3]
    python -m paper_2608_14498_b200.profile_case prefix  [--reps 3]
    python -m paper_2608_14498_b200.profile_case suffix  [--reps 3]

Each case keeps a few hundred MB on the device (more than the 126 MB L2, so DRAM counters mean
something) and launches the kernel `reps` times after one warm-up launch.
  lm      8192 rows x 32768 vocabulary columns, hidden 3584  (7B-shaped slice of the LM head)
  prefix  4 sequences x 4096 prompt tokens, 28 query / 4 KV heads, head_dim 128, with cache write
  suffix  the same 4 prompts cached, 256 response tokens each
"""
from __future__ import annotations

import argparse

import numpy as np


def main() -> None:
    import torch

    import paper_2608_14498_b200 as rpx
    from paper_2608_14498_b200 import workloads as wk

    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["lm", "prefix", "suffix"])
    ap.add_argument("--reps", type=int, default=3)
    args = ap.parse_args()
    dev = torch.device("cuda:0")

    def dv(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).to(dev).view(torch.bfloat16)
        return torch.from_numpy(a).to(dev)

    status = torch.zeros(1, dtype=torch.int32, device=dev)
    if args.case == "lm":
        cfg = wk.Config("profile-lm", "bf16", 1, 28, 4, 128, 3584, 32768, ("fixed", 8192), ("fixed", 0))
        wl = wk.make_workload(cfg, seed=0, attn=False)
        h, w, ids = dv(wl.hidden), dv(wl.w), dv(wl.ids)
        for _ in range(1 + args.reps):
            rpx.token_logprobs(h, w, ids, device_status=status)
    else:
        cfg = wk.Config("profile-attn", "bf16", 4, 28, 4, 128, 3584, 1024, ("fixed", 4096), ("fixed", 256))
        wl = wk.make_workload(cfg, seed=0, lm=False)
        kc = torch.zeros((wl.num_blocks, 4, 16, 128), dtype=torch.bfloat16, device=dev)
        cache = (kc, torch.zeros_like(kc), dv(wl.block_table))
        qp, kp, vp = (dv(wl.prefix_pack(t)) for t in (wl.q, wl.k, wl.v))
        qs, ks, vs = (dv(wl.suffix_pack(t)) for t in (wl.q, wl.k, wl.v))
        cu_p, cu_s, pl = dv(wl.cu_prefix), dv(wl.cu_suffix), dv(wl.prompt_lens)
        rpx.prefix_attn(qp, kp, vp, cu_p, 4096, cache=cache, device_status=status)
        for _ in range(args.reps):
            if args.case == "prefix":
                rpx.prefix_attn(qp, kp, vp, cu_p, 4096, cache=cache, device_status=status)
            else:
                rpx.suffix_attn(qs, ks, vs, cu_s, pl, 256, 4096, cache=cache, device_status=status)
        if args.case == "suffix":
            rpx.suffix_attn(qs, ks, vs, cu_s, pl, 256, 4096, cache=cache, device_status=status)
    torch.cuda.synchronize()
    code = int(status.item())
    if code != 0:
        raise SystemExit(f"device status {code}: {rpx.status_string(code)}")
    print(f"profile case {args.case}: ok")


if __name__ == "__main__":
    main()
