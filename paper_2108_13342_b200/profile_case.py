"""Runs one workload a few times on cuda:0 -- the command line to put under ncu.

    python -m paper_2108_13342_b200.profile_case --workload masked_softmax --kw batch=64 --iters 3
"""
from __future__ import annotations

import argparse


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", required=True)
    ap.add_argument("--kw", nargs="*", default=[])
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--unfused", action="store_true")
    ap.add_argument("--canon", action="store_true")
    ap.add_argument("--beyond", action="store_true", help="plan with DNNF_PLAN_BEYOND_TABLE3 (single-kernel attention and inverted-residual blocks)")
    ap.add_argument("--plan-flags", type=lambda v: int(v, 0), default=0, help="further dnnf_plan flags, e.g. 0x20000 (DNNF_PLAN_MBCONV_ALWAYS)")
    ap.add_argument("--instances", type=int, default=1, help="independent copies with their own buffers, run round-robin")
    args = ap.parse_args()
    import torch
    from . import binding as B
    from . import workloads as W
    from .runtime import Session
    kw = {k: int(v) for k, v in (x.split("=") for x in args.kw)}
    wl = W.by_name(args.workload, **kw)
    sess = [Session(wl, plan_flags=B.PLAN_UNFUSED if args.unfused else (B.PLAN_FUSED | (B.PLAN_BEYOND_TABLE3 if args.beyond else 0) | args.plan_flags),
                    rewrite_flags=B.REWRITE_CANON_MACRO if args.canon else B.REWRITE_NONE) for _ in range(args.instances)]
    s = sess[0]
    for _ in range(args.iters):
        for x in sess:
            x.run()
    torch.cuda.synchronize()
    st, blk = s.g.status()
    print("status", st, "kernels per run", s.plan_stats.n_kernels)
    for b in s.g.blocks():
        print(b)


if __name__ == "__main__":
    main()
