#!/usr/bin/env python
"""Benchmark of the late-scale step on synthetic VAR-shaped data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole hot path over one batch: the late scale steps of the
workload (restore the pre-filled cache state, then for every late scale: scale step + KV append).
Prints ONE JSON line.  `--impl reference` times the CPU oracle on a bounded sample of the same
workload instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

SEED = 2512

WORKLOADS = {
    # VAR-d16-shaped stack, 16 blocks, batch 16 (8 CFG pairs), late scales 10x10, 13x13, 16x16,
    # null-prompt-only CFG + RP + RTR at keep ratio 0.5 in every block group (one block per group).
    "var_d16_late3_b16": dict(shape="d16", B=16, first_late=7, keep=0.5, null_only=True),
    # the same stack run densely on the same three scales, both CFG branches: the unpruned point
    "var_d16_dense3_b16": dict(shape="d16", B=16, first_late=7, keep=1.0, null_only=False),
    "var_d30_late2_b32": dict(shape="d30", B=32, first_late=8, keep=0.5, null_only=True),
    "var_d30_dense2_b32": dict(shape="d30", B=32, first_late=8, keep=1.0, null_only=False),
}


def make_shape(name):
    return {"d16": si.shape_var_d16, "d30": si.shape_var_d30}[name]()


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        out, _ = self.proc.communicate(timeout=10)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------- the oracle leg

def oracle_leg(wl, steps, warmup, sample_pairs=2):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: `sample_pairs` CFG
    pairs, every block, every late scale.  Returns (tokens/s, seconds per step, description, threads)."""
    from oracle import fvar_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threads = os.cpu_count() or 1
    shp = make_shape(wl["shape"])
    B = 2 * sample_pairs
    Ms = shp.tokens_per_scale()
    k0 = wl["first_late"]
    weights = si.make_weights(SEED, shp)
    o = orc.Oracle(weights, shp.n_heads, shp.blocks_per_group, shp.hw(), shp.ln_eps)
    o.set_cond(si.make_cond(SEED, B, shp.width))
    L0 = sum(Ms[:k0])
    K, V = si.make_kv_prefill(SEED, shp.n_blocks, B, L0, shp.width)
    gc = si.make_group_cache(SEED, shp.n_groups, B, Ms[k0 - 1], shp.width)
    toks = {k: si.make_tokens(SEED, B, Ms[k], shp.width) for k in range(k0, len(Ms))}
    late = wl["keep"] < 1.0
    if late:
        for k in range(k0, len(Ms)):
            r = orc.rank_from_keep_ratio(Ms[k], wl["keep"])
            for g in range(shp.n_groups):
                o.set_projection(k, g, si.make_projection(SEED, k, g, Ms[k], r))
    pol = orc.Policy("lowrank_rtr" if late else "dense", "null_only" if wl["null_only"] else "pair", wl["keep"])
    E = B // 2 if wl["null_only"] else B
    tokens_per_step = E * sum(Ms[k0:])

    def one():
        o.load_kv(K, V)
        o.load_group_cache(k0 - 1, gc)
        for k in range(k0, len(Ms)):
            o.scale_step(toks[k], k, pol)
            o.kv_append(k)

    for _ in range(warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = (time.perf_counter() - t0) / max(steps, 1)
    desc = "%d of the workload's CFG pairs, all %d blocks, all %d late scales, fp64 numpy" % (
        sample_pairs, shp.n_blocks, len(Ms) - k0)
    return tokens_per_step / dt, dt, desc, threads


# ------------------------------------------------------------------------------------------- the GPU leg

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="var_d16_late3_b16", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-run", action="store_true",
                    help="for runs under ncu: skip the host-buffer leg, the event pass and the CPU baseline")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    metric = "tokens/s over the late scale steps (output positions delivered per second)"
    config = {"workload": args.workload, "shape": wl["shape"], "batch": wl["B"],
              "late_scale_sides": list(make_shape(wl["shape"]).scales[wl["first_late"]:]), "keep_ratio": wl["keep"],
              "cfg": "null_only" if wl["null_only"] else "pair",
              "l2": "inputs_exceed_l2 (the stack's weights, streamed every step, are larger than L2)"}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = min(args.steps, 3)
        warm = min(args.warmup, 1)
        tps, dt, desc, threads = oracle_leg(wl, steps, warm)
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": tps, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc},
            "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return

    import torch
    from paper_2512_16483_b200 import binding as fv
    from paper_2512_16483_b200 import schedule

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    shp = make_shape(wl["shape"])
    B, k0 = wl["B"], wl["first_late"]
    Ms = shp.tokens_per_scale()
    late_scales = list(range(k0, len(Ms)))
    late = wl["keep"] < 1.0
    mode = fv.LOWRANK_RTR if late else fv.DENSE
    cfg_mode = fv.CFG_NULL_ONLY if wl["null_only"] else fv.CFG_PAIR
    E = B // 2 if wl["null_only"] else B

    def bf16_cuda(a):
        return torch.from_numpy(si.bf16_bits(a).view(np.int16).reshape(a.shape)).view(torch.bfloat16).cuda()

    seed = SEED + rank
    weights = [{k: bf16_cuda(v) for k, v in blk.items()} for blk in si.make_weights(seed, shp)]
    ctx = fv.Fvar(weights, blocks_per_group=shp.blocks_per_group, n_heads=shp.n_heads, head_dim=shp.head_dim,
                  ffn_dim=shp.ffn_dim, scale_hw=shp.hw(), max_batch=B, ln_eps=shp.ln_eps)
    ctx.set_cond(bf16_cuda(si.make_cond(seed, B, shp.width)))
    L0 = sum(Ms[:k0])
    K, V = si.make_kv_prefill(seed, shp.n_blocks, B, L0, shp.width)
    ctx.load_kv(bf16_cuda(K), bf16_cuda(V))
    ctx.load_group_cache(k0 - 1, torch.from_numpy(si.make_group_cache(seed, shp.n_groups, B, Ms[k0 - 1], shp.width)).cuda())
    del K, V
    if late:
        for k in late_scales:
            r = schedule.rank_from_keep_ratio(Ms[k], wl["keep"])
            for g in range(shp.n_groups):
                ctx.set_projection(k, g, bf16_cuda(np.ascontiguousarray(si.make_projection(seed, k, g, Ms[k], r).T)))
    toks = {k: bf16_cuda(si.make_tokens(seed, B, Ms[k], shp.width)) for k in late_scales}
    outs = {k: torch.empty((E, Ms[k], shp.width), dtype=torch.bfloat16, device="cuda") for k in late_scales}
    toks_host = {k: toks[k].cpu().pin_memory() for k in late_scales}
    outs_host = {k: torch.empty((E, Ms[k], shp.width), dtype=torch.bfloat16).pin_memory() for k in late_scales}
    tokens_per_step = E * sum(Ms[k] for k in late_scales)

    def step_device():
        ctx.restore_loaded()
        for k in late_scales:
            ctx.scale_step(toks[k], k, mode=mode, cfg_mode=cfg_mode, keep_ratio=wl["keep"], out=outs[k])
            ctx.kv_append(k)

    def step_host():
        ctx.restore_loaded()
        for k in late_scales:
            ctx.scale_step_host(toks_host[k], k, outs_host[k], mode=mode, cfg_mode=cfg_mode, keep_ratio=wl["keep"])
            ctx.kv_append(k)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = ctx.launch_count()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        ms = e0.elapsed_time(e1)
        if dist is not None:
            t = torch.tensor([ms], device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        return ms, ctx.launch_count() - n0

    warm = max(args.warmup, 3)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    ms_total, launches = timed(step_device, args.steps, warm)
    clocks = sampler.stop() if sampler else None
    ms_e2e, _ = (ms_total, 0) if args.profile_run else timed(step_host, args.steps, 2)
    assert ctx.poll_status() == fv.OK, "device status word reports an error"

    # per-kernel-class event timing: a separate pass over the same steps, events around every launch
    ctx.profile_enable(True)
    prof_steps = 0 if args.profile_run else max(1, min(args.steps, 10))
    for _ in range(prof_steps):
        step_device()
    classes = {}
    for i, name in enumerate(fv.KCLASSES):
        ms, n, fl, by = ctx.profile_read(i)
        if n:
            classes[name] = {"ms_per_step": ms / prof_steps, "launches_per_step": n / prof_steps,
                             "avg_us": 1e3 * ms / n, "tflops": fl / ms / 1e9 if ms else 0.0,
                             "gbs": by / ms / 1e6 if ms else 0.0}
    ctx.profile_enable(False)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = peaks()
    ms_step = ms_total / args.steps
    value = world * tokens_per_step / (ms_step * 1e-3)
    e2e = world * tokens_per_step / (ms_e2e / args.steps * 1e-3)
    g = classes.get("gemm", {"tflops": 0.0})
    roofline = {"bound": "tensor", "kernel": "gemm_kernel (every tile width and epilogue the step launches)",
                "achieved": g["tflops"], "peak": pk["bf16_sustained"], "unit": "TFLOP/s",
                "frac": g["tflops"] / pk["bf16_sustained"], "peak_source": pk["source"] + ", sustained bf16",
                "traffic": None, "how": "separate pass of %d steps with CUDA events around every launch" % prof_steps,
                "classes": classes}
    line = {
        "metric": metric, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "ms_per_scale_step": ms_step / len(late_scales), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e, "unit": "tokens/s",
                "h2d_bytes_per_step": sum(B * Ms[k] * shp.width * 2 for k in late_scales),
                "d2h_bytes_per_step": sum(E * Ms[k] * shp.width * 2 for k in late_scales)},
        "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline and not args.profile_run:
        tps, dt, desc, threads = oracle_leg(wl, 1, 0)
        line["cpu_baseline"] = {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc,
                                "seconds": dt}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
