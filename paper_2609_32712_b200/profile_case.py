"""Runs a few launches of one operator on one synthetic configuration: the small, fixed command that
profiler captures (ncu) are taken on.

  python -m paper_2609_32712_b200.profile_case --op bwd --workload cfg2 --preset R --tau 1e-4 --iters 3
  python -m paper_2609_32712_b200.profile_case --op decode --decode-batch 2 --preset D --tau 1e-4
"""
from __future__ import annotations

import argparse
import dataclasses

import torch

from . import mala, workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", default="fwd", choices=["fwd", "bwd", "decode"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--preset", default="literal")
    ap.add_argument("--tau", type=float, default=1e-4)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--decode-batch", type=int, default=2)
    a = ap.parse_args()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    if a.op == "decode":
        cfg = dataclasses.replace(W.decode_config("cfg5"), B=a.decode_batch)
        w = W.make_decode(cfg, preset=a.preset, device=dev)
        for _ in range(a.iters):
            mala.decode(w["q"], w["kcache"], w["vcache"], w["scale"], a.tau, cfg.num_splits)
    else:
        cfg = W.prefill_config(a.workload)
        w = W.make_prefill(cfg, preset=a.preset, device=dev)
        o, lse, _ = mala.fwd(w["q"], w["k"], w["v"], w["scale"], a.tau)
        for _ in range(a.iters):
            if a.op == "fwd":
                mala.fwd(w["q"], w["k"], w["v"], w["scale"], a.tau, out=o, lse=lse)
            else:
                mala.bwd(w["q"], w["k"], w["v"], o, w["do"], lse, w["scale"], a.tau)
    torch.cuda.synchronize()
    assert mala.device_status() == 0
    print("ok")


if __name__ == "__main__":
    main()
