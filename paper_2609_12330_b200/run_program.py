"""Run one of the fused programs a few times on seeded synthetic inputs (a profiling target).

    python -m paper_2609_12330_b200.run_program qknorm_attn --size full --calls 3
    python -m paper_2609_12330_b200.run_program gated_mlp --size full --set M=8

Allocates the inputs of the named benchmark configuration on the current CUDA device, calls the
program `--calls` times through the C ABI, checks the workspace status word and prints one JSON
line (shape, device time per call from CUDA events, output checksum).  Nothing here computes on
the CPU: without the CUDA library or a GPU it fails.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def main(argv=None):
    import torch

    import paper_2609_12330_b200 as ef
    import workloads as wl

    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("program", choices=wl.PROGRAMS + wl.EXTRA_PROGRAMS)
    ap.add_argument("--size", default="full", choices=["full", "small"])
    ap.add_argument("--calls", type=int, default=3)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--set", action="append", default=[], metavar="NAME=INT", help="override an integer shape parameter")
    args = ap.parse_args(argv)
    if not torch.cuda.is_available():
        raise RuntimeError("run_program needs a CUDA device: the library has no CPU path")
    ef.lib()
    over = {}
    for kv in args.set:
        k, v = kv.split("=")
        over[k] = int(v)
    p, t = wl.make_inputs(args.program, seed=args.seed, size=args.size, **over)
    dev = {k: wl.bf16_bits_to_torch(v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(ef.workspace_bytes(args.program, p))
    out = ef.run(args.program, p, dev, ws)
    ws.check()
    times = []
    for _ in range(args.calls):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        ef.run(args.program, p, dev, ws, out=out)
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b) * 1e3)
    ws.check()
    work = wl.algorithmic_work(args.program, p)
    print(json.dumps({
        "program": args.program, "params": {k: (v if isinstance(v, int) else float(v)) for k, v in p.items()},
        "calls": args.calls, "us_per_call": [round(x, 2) for x in times],
        "algorithmic_flops": work["flops"], "algorithmic_bytes": work["bytes"],
        "out_abs_sum": float(out.float().abs().sum().item()),
    }))


if __name__ == "__main__":
    main()
