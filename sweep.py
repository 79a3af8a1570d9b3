"""Last-scale sweep on the Infinity-2B shape (one GPU): rows kept x batch, against the dense path.

    python sweep.py [--steps K] [--ranks 4096,3072,...] [--batches 2,4,8,16]

Every point is one run of `bench.py --workload infinity2b_last_r<R>_b<B>` in a process of its own (the
KV cache and the workspace are sized by the batch): the 64 x 64 scale, 4096 query tokens per element over a
cache pre-filled with 6425 rows, 32 blocks in 8 groups with cross-attention.  R = 4096 is the unpruned
dense path with both CFG branches; R < 4096 is the method: null-prompt branch only, projection to R rows,
blocks on R rows, restoration.  The method has one knob, the number of rows r that go through the blocks,
so the keep ratios {0.75, 0.5, 0.25} and the ranks {64, 32, 16} of the sweep are all values of R.
Prints one markdown table row per point: ms per step, tokens/s, speed-up over the dense path of the same
batch, the roofline that binds the step (HBM below the ridge, tensor above), the fraction of it reached and the
floor it implies.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.abspath(__file__))


def run_point(R: int, B: int, steps: int):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "infinity2b_last_r%d_b%d" % (R, B),
           "--steps", str(steps), "--warmup", "3", "--no-cpu-baseline"]
    p = subprocess.run(cmd, capture_output=True, text=True)
    lines = [l for l in p.stdout.splitlines() if l.startswith("{")]
    if p.returncode != 0 or not lines:
        raise RuntimeError("bench.py failed for R=%d B=%d:\n%s" % (R, B, p.stderr[-2000:]))
    return json.loads(lines[-1])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--ranks", default="4096,3072,2048,1024,64,32,16")
    ap.add_argument("--batches", default="2,4,8,16", help="batch elements (two per CFG pair)")
    args = ap.parse_args()
    ranks = [int(v) for v in args.ranks.split(",")]
    batches = [int(v) for v in args.batches.split(",")]
    print("| B (pairs) | R | mode | ms / step | tokens/s | vs dense | bound | roofline frac | floor ms | SM MHz, reasons |")
    print("|---|---|---|---|---|---|---|---|---|---|")
    for B in batches:
        dense_ms = None
        for R in ranks:
            d = run_point(R, B, args.steps)
            rf = d["roofline"]
            if R == 4096:
                dense_ms = d["ms_per_step"]
            print("| %d (%d) | %d | %s | %.2f | %.3g | %s | %s | %.2f | %.2f | %s %s |" % (
                B, B // 2, R, "dense, both branches" if R == 4096 else "null branch, RP + RTR", d["ms_per_step"], d["value"],
                "%.1fx" % (dense_ms / d["ms_per_step"]) if dense_ms else "-", rf["bound"], rf["frac"], rf["floor_ms_per_step"],
                d["clocks"]["sm_mhz"], ",".join(d["clocks"]["reasons"]) or "none"), flush=True)


if __name__ == "__main__":
    main()
