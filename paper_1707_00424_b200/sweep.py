"""Update-kernel sweep: time the inner y/z update (Eq. parle_y + parle_z), the fused
x^a update + replica mean (Eq. parle_xa + parle_x) and the stand-alone mean in
isolation on flat parameter vectors, and report achieved HBM GB/s.

    python -m paper_1707_00424_b200.sweep [--d 1048576 16777216 ...] [--n 3 8 16] [--reps 7] [--json out.json]

Every call is timed on its own with CUDA events on the bound stream; between
calls a buffer larger than the L2 cache is overwritten so that small cases are
measured from DRAM too.  State is drawn on the device with a seeded torch
generator (x, y, z ~ N(0,1), gradient ~ N(0, 0.1^2)); values do not matter for
the timing, parity of these kernels is covered by the GPU tests.
"""
from __future__ import annotations

import argparse
import json
import statistics

import torch

from . import Parle

L2_FLUSH_BYTES = 512 << 20


def algorithmic_bytes(kind: str, n: int, d: int) -> int:
    if kind == "inner_update":        # read g, y, x, z; write y, z
        return 24 * n * d
    if kind == "inner_update_first":  # first step of a round: read g, x; write y, z
        return 16 * n * d
    if kind == "outer_step":          # read x^a, z^a, xbar; write x^a, xbar
        return (12 * n + 8) * d
    if kind == "mean":                # read x^a; write xbar
        return (4 * n + 4) * d
    raise ValueError(kind)


def run_case(n: int, d: int, reps: int, device="cuda:0"):
    m = Parle(n, (d,), 0).alloc(device)
    gen = torch.Generator(device=device).manual_seed(1707_00424 + 31 * n + d % 1009)
    for t in (m.x, m.y, m.z):
        t.normal_(generator=gen)
    m.grad.normal_(0.0, 0.1, generator=gen)
    m.mean()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=device)
    times = {k: [] for k in ("inner_update_first", "inner_update", "outer_step", "mean")}

    def timed(kind, fn):
        flush.fill_(1)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); fn(); e1.record()
        torch.cuda.synchronize()
        times[kind].append(e0.elapsed_time(e1))

    for r in range(reps + 2):
        m.round_begin()
        timed("inner_update_first", lambda: m.inner_update(m.grad))
        timed("inner_update", lambda: m.inner_update(m.grad))
        timed("outer_step", m.outer_step)
        timed("mean", m.mean)
    out = []
    for kind, ts in times.items():
        ms = statistics.median(ts[2:])
        b = algorithmic_bytes(kind, n, m.stride)
        out.append({"kernel": kind, "n": n, "d": d, "ms": ms, "bytes": b, "gbs": b / ms / 1e6})
    del m, flush
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--d", type=int, nargs="+", default=[1 << 20, 1 << 24, 1 << 26, 1 << 28])
    ap.add_argument("--n", type=int, nargs="+", default=[3, 8, 16])
    ap.add_argument("--reps", type=int, default=7)
    ap.add_argument("--json", default=None)
    args = ap.parse_args()
    rows = []
    for d in args.d:
        for n in args.n:
            rows += run_case(n, d, args.reps)
    print("| kernel | n | d | ms | algorithmic MB | GB/s |")
    print("|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['kernel']} | {r['n']} | {r['d']} | {r['ms']:.4f} | {r['bytes'] / 1e6:.1f} | {r['gbs']:.0f} |")
    if args.json:
        with open(args.json, "w") as f:
            json.dump(rows, f)


if __name__ == "__main__":
    main()
