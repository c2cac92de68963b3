#!/usr/bin/env python
"""Benchmark of the Parle round (arXiv 1707.00424, Section 3) on B200.

A "step" is one whole Parle round over n replicas: round begin, L inner steps
(forward/backward + Eq. parle_y/parle_z), the outer step (Eq. parle_xa) and the
replica mean (Eq. parle_x).  The metric is replica-inner-steps per second
= n * L * rounds / time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C5] [--impl ours|reference]

Prints ONE JSON line.  The default workload is the largest one that fits a GPU
(C5: 16 replicas of a 243 M-parameter MLP); on one GPU the line also carries
compact records of the CIFAR-100-shaped workload (key "c3") and of the
update-kernel sweep (key "c4_sweep").  With --impl reference the fp64 CPU oracle
is timed on the host cores instead (a bounded sample of the same workload per
step).
Multi-GPU: every rank holds n replicas; the only exchange is the average of the
per-rank means once per round (NCCL all-reduce), so the job has N*n replicas
and scaling is weak.  Under torchrun the ranks come from the environment;
started plainly with --gpus N > 1 the script starts its N ranks itself.
--backend gloo --dry runs the rank logic alone on CPUs (no rounds): start-up,
the exchange, the max-over-ranks timing and the single line.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "parle_replica_inner_steps_per_sec"
UNIT = "replica-inner-steps/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50", "-i", str(self.index)],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------ workloads
def make_round_inputs(cfg, sets: int):
    """`sets` rounds' worth of minibatches: X [sets, L, n, B, d0] fp32, labels [sets, L, n, B] int32."""
    Xs, cs = [], []
    big = cfg.n * cfg.batch * cfg.dims[0] * cfg.L > (1 << 28)      # > 1 GiB of fp32 per round: cycle 4 distinct steps
    for r in range(sets):
        X, c = si.round_batches(cfg, r, pool=4 if big else 0)
        Xs.append(X); cs.append(c)
    return np.stack(Xs), np.stack(cs)


def dense_to_padded(model, cfg, replica_layers):
    out = np.zeros((cfg.n, model.stride), dtype=np.float32)
    for a, layers in enumerate(replica_layers):
        for l, (W, b) in enumerate(layers):
            w_off, b_off = model.layer_offset(l)
            out[a, w_off:w_off + W.size] = W.ravel()
            out[a, b_off:b_off + b.size] = b
    return out


# DRAM bytes per launch of the dominant kernel from the committed ncu capture
# (profiles/ncu_fused_update_and_pair_gemm_C5_one_replica.md), valid only while the kernel source is unchanged.
# The capture ran a one-replica copy of the workload (3.9 GB of state); the kernel's traffic is proportional to the
# number of replicas (every replica's weights are streamed once, nothing is shared between replicas), so the figure
# below is the captured one times 16.
NCU_TRAFFIC = {("C5", "wgrad_gemm_fused_update"): {
    # dram__bytes_read.sum + dram__bytes_write.sum of one launch at n = 1: mean of the two variants that alternate inside
    # a round, "z untouched" (1990.7 + 927.6 MB) and "two-step z" (3008.0 + 1890.7 MB)
    "bytes": 16 * (1990.746880e6 + 927.633920e6 + 3007.953920e6 + 1890.747904e6) / 2,
    "sources": ("paper_1707_00424_b200/csrc/umma_wgrad_update.cuh", "paper_1707_00424_b200/csrc/umma_gemm.cuh",
                "paper_1707_00424_b200/csrc/common.cuh"),
    "sources_sha256_16": "9bb763e99a1edb39"}}


def sources_digest(sources):
    import hashlib
    h = hashlib.sha256()
    for rel in sources:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str, kernel: str):
    rec = NCU_TRAFFIC.get((workload, kernel))
    if not rec or sources_digest(rec["sources"]) != rec["sources_sha256_16"]:
        return None             # no capture, or the kernel changed since the counters were taken
    return rec["bytes"]         # (taken with the default settings: z updated every other step)


def algorithmic_bytes_per_round(cfg, stride, tf32_split=False, paired_z=True, split_y=True):
    """Bytes each kernel class has to move per Parle round (all n replicas), from the data it must
    touch once: parameter-state vectors at 4 B (fp32) or 2 B (bf16 copy) per element, plus GEMM operands.
    tf32_split: the fp32 update also writes the tf32 hi/lo copy of y (8 B per element).
    paired_z: the fused bf16 kernel touches z on every other step only (parle_set_paired_z_update)."""
    n, B, L, dims = cfg.n, cfg.batch, cfg.L, cfg.dims
    nl = len(dims) - 1
    Pw = sum(dims[l] * dims[l + 1] for l in range(nl))
    bf = cfg.gemm_dtype == 1
    act = lambda l: B * dims[l]                          # elements of one replica's activation at level l
    out = {}
    # separate update: read g, y, x, z, write y, z (+2 B bf16 copy); first step of a round reads x for y and z
    # with Eq. (parle_z) applied two steps at a time, half of the later steps leave z alone (8 B less)
    skipped = (L - 1) // 2 if paired_z else 0
    out["inner_update"] = n * stride * ((24 + (2 if bf else 0) + (8 if tf32_split else 0)) * L - 8 - 8 * skipped)
    out["outer_mean"] = stride * (12 * n + 8)
    if bf:
        opnd = sum(2 * (act(l) + act(l + 1)) for l in range(nl))             # dH^T and H^T, bf16
        # fused: read y, x, z (12 B), write y, z, bf16 copy (10 B); first step reads only x (14 B); with Eq. (parle_z)
        # applied two steps at a time the other steps alternate between 14 B (z untouched) and 22 B
        pairs, single = ((L - 1) // 2, (L - 1) % 2) if paired_z else (0, L - 1)
        # y as two 16-bit planes inside a round: every step moves 2 B less (no separate operand copy), the last one
        # stores the fp32 y once more
        ys = 2 if split_y else 0
        out["wgrad_gemm_fused_update"] = n * (Pw * (14 - ys + pairs * (14 + 22 - 2 * ys) + single * (22 - ys) + (4 if split_y else 0)) + opnd * L)
        out["wgrad_gemm"] = n * L * (4 * Pw + opnd)
        out["fwd_gemm"] = n * L * (2 * Pw + sum(2 * act(l) + 4 * act(l + 1) for l in range(nl)))
        out["to_bf16"] = n * Pw * 6                                          # blocked bf16 weight copy from x, once per round
        out["dgrad_gemm"] = n * L * sum(2 * dims[l] * dims[l + 1] + 2 * act(l + 1) + 6 * act(l) for l in range(1, nl))
    return out


def gemm_flops_per_round(cfg):
    """Floating-point operations of the forward / data-gradient / weight-gradient products per round (all replicas)."""
    n, B, L, dims = cfg.n, cfg.batch, cfg.L, cfg.dims
    nl = len(dims) - 1
    Pw = sum(dims[l] * dims[l + 1] for l in range(nl))
    f = {"fwd_gemm": 2 * B * Pw, "dgrad_gemm": 2 * B * (Pw - dims[0] * dims[1]), "wgrad_gemm": 2 * B * Pw,
         "wgrad_gemm_fused_update": 2 * B * Pw}
    return {k: v * n * L for k, v in f.items()}


# ------------------------------------------------------------------ our arm
def build_model(cfg, dev, args):
    """A bound context for `cfg` with its replicas initialised and the bench's settings applied."""
    import torch
    import paper_1707_00424_b200 as pb
    model = pb.Parle(cfg.n, cfg.dims, cfg.batch, cfg.gemm_dtype, gamma=cfg.gamma, rho=cfg.rho,
                     alpha=cfg.alpha, eta=cfg.eta, eta_prime=cfg.eta_prime).alloc(dev)
    if cfg.n_params > 50_000_000:
        # the 243 M-parameter replicas are drawn on the device (seeded torch generator, the same N(0, 1/fan_in)
        # weights and zero biases as the host recipe): sixteen of them from the host generator take minutes
        gen = torch.Generator(device=dev).manual_seed(cfg.seed % (1 << 31))
        for a in range(cfg.n):
            for l in range(cfg.n_layers):
                w_off, _ = model.layer_offset(l)
                model.x[a, w_off:w_off + cfg.dims[l] * cfg.dims[l + 1]].normal_(0.0, cfg.dims[l] ** -0.5, generator=gen)
    else:
        model.x.copy_(torch.from_numpy(dense_to_padded(model, cfg, [si.init_replica(cfg, a) for a in range(cfg.n)])))
    model.mean()
    model.set_round_graphs(bool(args.graphs))
    model.set_paired_z_update(bool(args.paired_z))
    if cfg.gemm_dtype == 1:
        model.set_split_y(bool(args.split_y))
    return model


def class_rooflines(cfg, model, prof, K, args, peaks, clocks):
    """Per kernel class: achieved algorithmic GB/s (or TFLOP/s) over the K profiled rounds against the measured peaks."""
    t3 = cfg.gemm_dtype == 0 and model.fp32_tensor_cores_active
    alg = algorithmic_bytes_per_round(cfg, model.stride, tf32_split=t3, paired_z=bool(args.paired_z), split_y=bool(args.split_y))
    rooflines = {}
    for k, (ms_k, cnt_k) in prof.items():
        if k not in alg:
            continue
        ach = alg[k] * K / (ms_k * 1e-3) / 1e9          # bytes of K rounds / device time of the class over K rounds
        rooflines[k] = {"kernel": k, "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / peaks["hbm_gbs"], "traffic": ncu_traffic(cfg.name, k) if (args.paired_z and args.split_y) else None,
                        "peak_source": peaks["source"], "bytes_per_launch": alg[k] * K / cnt_k,
                        "ms_per_launch": ms_k / cnt_k, "launches_per_round": cnt_k / K}
    flops = gemm_flops_per_round(cfg)
    if cfg.gemm_dtype == 0:
        # fp32 configurations.  Tensor cores: every fp32 product is three tf32 products (hi/lo operand split), so the
        # useful rate can reach a third of the tf32 peak at most; tf32 peak = measured bf16 peak x nominal ratio 1.1 / 2.25.
        # FMA pipes: 148 SMs x 128 lanes x 2 flop x the maximum SM clock.
        sm_max = (clocks or {}).get("sm_max_mhz") or 1965.0
        tf32_peak = peaks["bf16_tflops"] * 1.1 / 2.25
        alu_peak = 148 * 128 * 2 * sm_max * 1e6 / 1e12
        for k, f in flops.items():
            if k not in prof or k == "wgrad_gemm_fused_update":
                continue
            tf = f * K / (prof[k][0] * 1e-3) / 1e12
            rooflines[k] = {"kernel": k, "bound": "tensor" if t3 else "alu", "achieved": tf,
                            "peak": tf32_peak if t3 else alu_peak, "unit": "TFLOP/s", "frac": tf / (tf32_peak if t3 else alu_peak),
                            "traffic": None, "peak_source": (peaks["source"] + " bf16 x 1.1/2.25 (tf32)") if t3 else "148 SMs x 128 FMA lanes x max SM clock",
                            "note": ("useful fp32 flops; the kernel executes 3 tf32 products per fp32 product, so frac <= 1/3" if t3 else
                                     "fp32 FMA pipes"),
                            "ms_per_launch": prof[k][0] / prof[k][1], "launches_per_round": prof[k][1] / K}
        flops = {}
    for k, f in flops.items():
        if k in prof and k in rooflines:
            tf = f * K / (prof[k][0] * 1e-3) / 1e12
            rooflines[k]["tensor_tflops"] = tf
            rooflines[k]["tensor_frac_of_burst_peak"] = tf / peaks["bf16_tflops"]
            rooflines[k]["tensor_frac_of_sustained_peak"] = tf / peaks["bf16_tflops_sustained"]
    return rooflines, t3


def measure(cfg, args, dev, local, world, W, K, full):
    """Time K rounds of `cfg` (after W warm-up rounds) with device-resident inputs, then the per-class device
    times over K more rounds; with `full` also the end-to-end rounds from pinned host buffers and the rounds with
    z and fp32 y touched at every step."""
    import torch
    import torch.distributed as dist
    from paper_1707_00424_b200.parallel import allreduce_mean_

    model = build_model(cfg, dev, args)
    big = cfg.n * cfg.batch * cfg.dims[0] * cfg.L > (1 << 28)
    sets = 1 if big else 2            # one round of inputs is already far larger than L2 there
    Xh, ch = make_round_inputs(cfg, sets)
    Xd, cd = torch.from_numpy(Xh).to(dev), torch.from_numpy(ch).to(dev)
    loss_d = torch.zeros(cfg.L, cfg.n, device=dev)

    def sync_all():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize(dev)

    def exchange():
        if world > 1:       # global mean = mean over ranks of the per-rank means (equal replica counts)
            allreduce_mean_(model.xbar)

    def round_device(r):
        model.round(cfg.L, Xd[r % sets], cd[r % sets], loss_d)
        exchange()

    def timed(fn, warmup, steps, sample_clocks=False):
        for r in range(warmup):
            fn(r)
        sync_all()
        sampler = ClockSampler(local) if sample_clocks else None
        if sampler:
            sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = model.launch_count
        e0.record()
        for r in range(steps):
            fn(warmup + r)
        e1.record()
        sync_all()
        clocks = sampler.stop() if sampler else None
        ms = e0.elapsed_time(e1)
        if world > 1:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, model.launch_count - launches0, clocks

    out = {"cfg": cfg}
    # 1. device-resident inputs: the headline value
    ms, launches, clocks = timed(round_device, W, K, sample_clocks=True)
    out.update(ms=ms, launches=launches, clocks=clocks, flags=model.status(),
               value=world * cfg.n * cfg.L * K / (ms * 1e-3))
    # 2. per-kernel-class device time over the same K rounds (events around every launch)
    model.profile_enable(True)
    for r in range(K):
        round_device(W + r)
    prof, dropped = model.profile_read()
    model.profile_enable(False)
    out.update(prof=prof, dropped=dropped)
    if full:
        # 3. end to end: host (pinned) inputs copied in and per-step losses copied out inside the timed region
        Xp, cp = torch.from_numpy(Xh).pin_memory(), torch.from_numpy(ch).pin_memory()
        loss_p = torch.zeros(cfg.L, cfg.n).pin_memory()

        def round_host(r):
            model.round_host(cfg.L, Xp[r % sets], cp[r % sets], loss_p)
            exchange()

        ms_e2e, _, _ = timed(round_host, min(W, 2), K)
        out["e2e"] = {"value": world * cfg.n * cfg.L * K / (ms_e2e * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": cfg.L * (cfg.n * cfg.batch * cfg.dims[0] * 4 + cfg.n * cfg.batch * 4),
                      "d2h_bytes_per_step": cfg.L * cfg.n * 4, "ms_per_step": ms_e2e / K}
        del Xp, cp
        # 4. for comparison: the same rounds with z read and written at every inner step (Eq. parle_z one step at a time)
        out["every_step"] = None
        if args.paired_z:
            model.set_paired_z_update(False)
            if cfg.gemm_dtype == 1:
                model.set_split_y(False)
            ms_u, _, _ = timed(round_device, min(W, 2), K)
            out["every_step"] = {"value": world * cfg.n * cfg.L * K / (ms_u * 1e-3), "unit": UNIT, "ms_per_step": ms_u / K,
                                 "what": "same rounds with parle_set_paired_z_update(0) and parle_set_split_y(0): z and fp32 y read and written at every inner step"}
    peaks = measured_peaks()
    out["rooflines"], out["t3"] = class_rooflines(cfg, model, prof, K, args, peaks, clocks)
    out["stride"] = model.stride
    del model, Xd, cd
    torch.cuda.empty_cache()
    return out


def compact_c3(args, dev, local):
    """The CIFAR-100-shaped workload in brief: value, time per round and the fractions of the main kernel classes."""
    r = measure(si.CONFIGS["C3"], args, dev, local, 1, 3, 10, full=False)
    total = sum(v[0] for v in r["prof"].values()) or 1.0
    pick = lambda k: ({"frac": r["rooflines"][k]["frac"], "achieved": r["rooflines"][k]["achieved"], "unit": r["rooflines"][k]["unit"],
                       "ms_per_launch": r["rooflines"][k]["ms_per_launch"], "share": r["prof"][k][0] / total,
                       "tensor_tflops": r["rooflines"][k].get("tensor_tflops")} if k in r["rooflines"] else None)
    dom = max(r["prof"], key=lambda k: r["prof"][k][0])
    return {"workload": "C3: n=8, MLP 3072-2048-2048-2048-100, batch 128, L=25, bf16 GEMM operands", "value": r["value"], "unit": UNIT,
            "steps": 10, "warmup": 3, "ms_per_round": r["ms"] / 10, "launches_per_round": r["launches"] / 10,
            "dominant_kernel": dom, "dominant": pick(dom), "fwd_gemm": pick("fwd_gemm"), "dgrad_gemm": pick("dgrad_gemm"),
            "outer_mean": pick("outer_mean"), "device_flags": r["flags"], "clocks": r["clocks"]}


def compact_c4(dev):
    """Corners of the update-kernel sweep: achieved GB/s of the three streaming kernels in isolation, as fractions
    of the measured copy rate and of the nominal 8 TB/s."""
    from paper_1707_00424_b200.sweep import run_case
    peaks = measured_peaks()
    rows = []
    for d in (1 << 24, 1 << 28):
        for n in (3, 16):
            for r in run_case(n, d, reps=5, device=str(dev)):
                rows.append({"kernel": r["kernel"], "n": n, "d": d, "ms": r["ms"], "gbs": r["gbs"],
                             "frac_of_measured": r["gbs"] / peaks["hbm_gbs"], "frac_of_nominal_8tbs": r["gbs"] / 8000.0})
    return {"what": "parle_inner_update (first / later step of a round), parle_outer_step (with its mean), parle_mean on flat fp32 "
                    "vectors, each call timed alone with CUDA events after an L2 flush; algorithmic bytes / time",
            "peak_source": peaks["source"], "rows": rows}


def run_dry(args):
    """The rank logic without a GPU: process group, one exchange per 'round' on a small CPU vector, barrier-bracketed
    timing with the max over ranks, one line from rank 0."""
    import torch
    import torch.distributed as dist
    from paper_1707_00424_b200.parallel import allreduce_mean_
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group(args.backend)
    xbar = torch.full((1024,), float(rank + 1), dtype=torch.float64)     # stands for this rank's replica mean
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        mine = torch.full_like(xbar, float(rank + 1))
        xbar = allreduce_mean_(mine)
    if world > 1:
        dist.barrier()
    ms = (time.perf_counter() - t0) * 1e3
    if world > 1:
        t = torch.tensor([ms], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": None, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                          "ms_per_step": ms / max(args.steps, 1), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                          "dry": True, "backend": args.backend, "exchanged_mean": float(xbar[0]),
                          "config": {"workload": "dry run: no rounds, the exchange of the replica mean only"}}))
    if world > 1:
        dist.destroy_process_group()


def run_ours(args):
    import torch
    import torch.distributed as dist

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the Parle library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        # NCCL's communicator set-up lines go to stderr, so that stdout stays the one JSON line
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")
        dist.init_process_group("nccl", device_id=dev)

    cfg = si.CONFIGS[args.workload]
    if args.replicas:       # a smaller copy of the workload (profiler captures); the line says so
        cfg = cfg.scaled(n=args.replicas)
    if world > 1:           # every rank owns its own n replicas (independent streams per rank)
        cfg = cfg.scaled(seed=cfg.seed + 7919 * rank)
    W, K = max(args.warmup, 0), args.steps
    r = measure(cfg, args, dev, local, world, W, K, full=True)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    prof, clocks = r["prof"], r["clocks"]
    total_ms = sum(v[0] for v in prof.values()) or 1.0
    shares = {k: {"ms_per_round": v[0] / K, "launches_per_round": v[1] / K, "share": v[0] / total_ms} for k, v in prof.items()}
    dom = max(prof, key=lambda k: prof[k][0])
    peaks = measured_peaks()
    rooflines, t3 = r["rooflines"], r["t3"]
    roofline = rooflines.get(dom, {"kernel": dom, "bound": "hbm", "achieved": None, "peak": peaks["hbm_gbs"],
                                   "unit": "GB/s", "frac": None, "traffic": None, "peak_source": peaks["source"]})
    extra = {}
    if world == 1 and args.compact and args.workload == "C5" and not args.replicas:
        extra["c3"] = compact_c3(args, dev, local)
        extra["c4_sweep"] = compact_c4(dev)
    cpu = cpu_baseline(cfg, budget_s=15.0) if args.cpu_baseline else None
    line = {
        "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": r["ms"] / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.gemm_dtype == 1 else "f32", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: n={cfg.n} replicas/GPU, MLP {'-'.join(map(str, cfg.dims))}, batch {cfg.batch}, L={cfg.L}, "
                               f"{'bf16 GEMM operands, fp32 master state' if cfg.gemm_dtype == 1 else ('fp32 (products as 3 x tf32 on the tensor cores)' if t3 else 'fp32 (FMA pipes)')}",
                   "step": "one Parle round (L inner steps + outer step + replica mean)" +
                           ("; z updated every other inner step with the two-step form of Eq. (parle_z)" if args.paired_z else "") +
                           ("; y of the weights kept as bf16 operand copy + lower-half plane inside the round" if cfg.gemm_dtype == 1 and args.split_y else ""),
                   "l2": "state + gradients per round >> 126 MB L2 (no flush needed)" if cfg.n * r["stride"] * 16 > 4e8 else "working set may be L2 resident",
                   "launch": "rounds replayed from CUDA graphs (same kernels, same order)" if args.graphs else "one launch per kernel",
                   "parallelism": f"{world} x {cfg.n} replicas, one all-reduce of xbar per round" if world > 1 else "single GPU"},
        "gpu_launches": r["launches"], "device_flags": r["flags"], "clocks": clocks,
        "e2e": r["e2e"],
        "roofline": roofline, "roofline_other_kernels": {k: v for k, v in rooflines.items() if k != dom},
        "kernel_shares": shares, "profile_dropped": r["dropped"],
        "z_every_step": r["every_step"],
        "cpu_baseline": cpu,
    }
    line.update(extra)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------ oracle timing (CPU)
def _blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_replicas(cfg) -> int:
    """Replicas the oracle sample covers: all of them unless their fp64 state would not fit in ~16 GB of host memory."""
    return max(1, min(cfg.n, int(16e9 // (cfg.n_params * 8 * 4))))


class OracleSampler:
    """The oracle on a bounded sample of a workload: `replicas` replicas (drawn once), some inner steps of one round,
    the outer step and the mean."""

    def __init__(self, cfg, replicas=None):
        from oracle import parle_oracle as po
        self.po = po
        self.cfg = cfg.scaled(n=replicas or oracle_replicas(cfg))
        fast = cfg.n_params > 50_000_000
        self.x0 = np.stack([po.pack(si.init_replica(self.cfg, a, fast=fast)) for a in range(self.cfg.n)])
        self.hp = po.Hyper(cfg.eta, cfg.eta_prime, cfg.alpha, cfg.gamma, cfg.rho)

    def run(self, inner_steps: int, rnd: int = 0) -> float:
        """Seconds the oracle needs for `inner_steps` inner steps of round `rnd` + outer step + mean (inputs drawn outside the clock)."""
        po, cfg = self.po, self.cfg
        X, c = si.round_batches(cfg.scaled(L=inner_steps), rnd)
        t0 = time.perf_counter()
        po.parle_round(self.x0, self.x0.mean(axis=0), po.mlp_grad_fn(cfg.dims, X, c), inner_steps, self.hp)
        return time.perf_counter() - t0


def cpu_baseline(cfg, budget_s: float):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload."""
    smp = OracleSampler(cfg)
    t1 = smp.run(1)
    steps = int(max(1, min(cfg.L, budget_s / max(t1, 1e-3))))
    t = smp.run(steps) if steps > 1 else t1
    nr = smp.cfg.n
    return {"value": nr * steps / t, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle",
            "sample": f"{steps} of {cfg.L} inner steps of one round, {nr} of {cfg.n} replicas, fp64 numpy ({t:.1f} s)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = si.CONFIGS[args.workload]
    runs = max(args.steps + args.warmup, 1)
    smp = OracleSampler(cfg)
    t1 = smp.run(1)
    if t1 * runs > 240.0 and smp.cfg.n > 1:          # keep the whole run to a few minutes: one replica per sample
        smp = OracleSampler(cfg, replicas=1)
        t1 = smp.run(1)
    per_step = int(max(1, min(cfg.L, 20.0 / max(t1, 1e-3) / runs)))
    for r in range(args.warmup):
        smp.run(per_step, r)
    t = 0.0
    for r in range(args.steps):
        t += smp.run(per_step, args.warmup + r)
    nr = smp.cfg.n
    value = nr * per_step * args.steps / t
    sample = f"each step = {per_step} of {cfg.L} inner steps of a round, {nr} of {cfg.n} replicas, + outer step and mean; fp64 numpy"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{cfg.name}: n={cfg.n}, MLP {'-'.join(map(str, cfg.dims))}, batch {cfg.batch}, L={cfg.L}", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": _blas_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C5", choices=sorted(si.CONFIGS))
    ap.add_argument("--graphs", type=int, default=1, help="replay rounds from CUDA graphs (parle_set_round_graphs)")
    ap.add_argument("--split-y", type=int, default=1, help="bf16 workloads: y as bf16 copy + lower-half plane inside a round (parle_set_split_y)")
    ap.add_argument("--paired-z", type=int, default=1, help="Eq. (parle_z) two steps at a time inside a round (parle_set_paired_z_update)")
    ap.add_argument("--compact", type=int, default=1, help="one GPU, workload C5: add the compact C3 and update-sweep records to the line")
    ap.add_argument("--replicas", type=int, default=0, help="override the workload's replica count (small cases for profiler captures)")
    ap.add_argument("--cpu-baseline", type=int, default=1, help="0: skip the oracle timing on the host cores")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"], help="process-group backend (gloo: with --dry, on CPUs)")
    ap.add_argument("--dry", action="store_true", help="rank logic only: no CUDA, no rounds")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.impl == "ours" and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: become the launcher of N ranks of this same command (one process per GPU)
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    elif args.dry:
        if args.backend != "gloo":
            raise SystemExit("bench.py: --dry runs on CPUs and needs --backend gloo")
        run_dry(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
