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
    # Infinity-2B-shaped generator (32 blocks in 8 groups, cross-attention to 256 context tokens), B = 2 (one
    # CFG pair), the three fidelity-refinement scales 40 / 48 / 64 over a cache pre-filled with 2521 rows:
    # null-only + RP + RTR at the tabulated rank of every block group (alpha = 0.96) at all three scales ...
    "infinity2b_late3_b2": dict(shape="inf2b", B=2, first_late=10, keep="table", null_only=True),
    # ... the schedule of Sec. 4.1 (alpha = {0.96, 0, 0}: scale 40 approximated, 48 and 64 skipped) ...
    "infinity2b_paper_b2": dict(shape="inf2b", B=2, first_late=10, keep="paper", null_only=True),
    # ... and the unpruned dense path with both CFG branches.
    "infinity2b_dense3_b2": dict(shape="inf2b", B=2, first_late=10, keep=1.0, null_only=False),
    # The transformer part of a whole 13-scale generation (no quantizer / decoder): every scale from 1x1 on, the
    # KV cache built by the steps themselves.  vanilla: all scales dense with both CFG branches; fastervar: scales
    # 1..32 dense with both branches, then the schedule of Sec. 4.1 (40 approximated on the null branch, 48 and 64
    # skipped); fastervar_late3: the three late scales all approximated at the tabulated ranks.
    "infinity2b_gen13_vanilla_b2": dict(shape="inf2b", B=2, first_late=0, dense_until=13, keep=1.0, null_only=False),
    "infinity2b_gen13_fastervar_b2": dict(shape="inf2b", B=2, first_late=0, dense_until=10, keep="paper", null_only=True),
    "infinity2b_gen13_fastervar_late3_b2": dict(shape="inf2b", B=2, first_late=0, dense_until=10, keep="table", null_only=True),
    # The same two generations as a closed autoregressive loop: every step's tokens come from the previous step
    # through the library's transition (CFG combination of the two branches, nearest codeword of a seeded random
    # codebook of 8192 entries, Up-accumulate at 64 x 64, area Down), starting from one seeded start token.  With the
    # schedule of Sec. 4.1 the loop ends after scale 40: the accumulated map is already at the final resolution.
    "infinity2b_loop13_vanilla_b2": dict(shape="inf2b", B=2, first_late=0, dense_until=13, keep=1.0, null_only=False, loop=True),
    "infinity2b_loop13_fastervar_b2": dict(shape="inf2b", B=2, first_late=0, dense_until=10, keep="paper", null_only=True, loop=True),
}
# The largest single-GPU configuration of the workload definition, and the paper's own shape (Sec. 4.1): the three
# fidelity-refinement scales of the Infinity-2B-shaped generator at the tabulated ranks.
DEFAULT_WORKLOAD = "infinity2b_late3_b2"
LOOP_CODEBOOK = 8192
LOOP_GUIDANCE = 3.0


def resolve_workload(name):
    """A named workload, or a point of the last-scale sweep on the Infinity-2B shape:
    `infinity2b_last_[lls_]r<R>_b<B>` = only the 64 x 64 scale (4096 queries over a cache pre-filled with 6425 rows),
    batch B, every block group at rank R.  R < 4096 runs the method (null-prompt branch only, RP + RTR);
    R = 4096 is the unpruned dense path with both CFG branches."""
    import re
    if name in WORKLOADS:
        return WORKLOADS[name]
    m = re.fullmatch(r"infinity2b_last_(lls_)?r(\d+)_b(\d+)", name)
    if not m:
        raise SystemExit("unknown workload %r (named: %s; or infinity2b_last_[lls_]r<R>_b<B>)" % (name, ", ".join(sorted(WORKLOADS))))
    lls, R, B = bool(m.group(1)), int(m.group(2)), int(m.group(3))
    if not (1 <= R <= 4096) or B < 1 or (R < 4096 and B % 2):
        raise SystemExit("need 1 <= R <= 4096 and a batch of whole CFG pairs")
    if lls and R > 192:
        raise SystemExit("the LLS restoration takes ranks up to 192")
    # `lls_`: the same step with the rows restored by the least-squares matrices (Eq. "lstsq") instead of RTR
    return dict(shape="inf2b", B=B, first_late=12, keep=("rank", R), null_only=R < 4096, restore="lls" if lls else "rtr")


def scale_plan(wl, shp):
    """Per late scale index: None (skip) or the list of ranks per block group (M = dense)."""
    from paper_2512_16483_b200 import schedule
    Ms, plan = shp.tokens_per_scale(), {}
    paper_modes = dict(zip(*schedule.infinity_schedule(True)))
    for k in range(wl["first_late"], len(Ms)):
        keep = wl["keep"]
        if k < wl.get("dense_until", 0):
            plan[k] = [Ms[k]] * shp.n_groups
        elif isinstance(keep, tuple) and wl.get("restore") == "lls":
            # an LLS group's output is spanned by its r rows, so the next group projects a rank-r input: its rank
            # steps down by 8 per group to keep the r x r Gram matrix of that projection well conditioned in fp32
            plan[k] = [max(8, min(keep[1], Ms[k]) - 8 * g) for g in range(shp.n_groups)]
        elif isinstance(keep, tuple):
            plan[k] = [min(keep[1], Ms[k])] * shp.n_groups
        elif keep in ("table", "paper"):
            side = shp.scales[k]
            if keep == "paper" and paper_modes[side] == schedule.SKIP:
                plan[k] = None
            else:
                plan[k] = schedule.infinity_group_ranks(side, shp.width, shp.n_groups)
        else:
            plan[k] = [schedule.rank_from_keep_ratio(Ms[k], keep)] * shp.n_groups
    return plan


def algorithmic_work(shp, plan, null_at, B, L0):
    """Flops and bytes the method must spend on one bench step (what it computes, not the dense work it avoids), and
    the same split by scale.  Per computed element and block group with rank r (r = M: dense) at a scale with M tokens
    and L_prev committed cache rows: flops = 2 M r C (projection, late groups) + n_g (2 r P + 4 r (L_prev + r) C
    + 4 r ctx C), P = 4 C^2 + 2 C F (+ 2 C^2 with cross-attention) the weight parameters a row meets in a block.
    Bytes = weights 2 n_g P once per scale step, shared by the batch, + per element: K / V read 4 n_g (L_prev + r) C
    (+ 4 n_g ctx C of context K / V), group input read twice (score, projection) 2 * 2 M C, output written 2 M C,
    previous scale's group output read 2 M_prev C (late groups)."""
    C, F, ng, G = shp.width, shp.ffn_dim, shp.blocks_per_group, shp.n_groups
    P = 4 * C * C + 2 * C * F + (2 * C * C if shp.has_cross_attn else 0)
    ctx = shp.ctx_len if shp.has_cross_attn else 0
    Ms = shp.tokens_per_scale()
    L = [L0] * G                                             # committed rows per group's blocks
    flops = bytes_ = 0.0
    prev = None
    for k in sorted(plan):
        if plan[k] is None:
            continue
        E = B // 2 if null_at[k] else B
        M = Ms[k]
        M_prev = Ms[prev if prev is not None else k - 1] if k > 0 else 0
        for g, r in enumerate(plan[k]):
            late = r < M
            flops += E * ((2.0 * M * r * C if late else 0.0) + ng * (2.0 * r * P + 4.0 * r * (L[g] + r) * C + 4.0 * r * ctx * C))
            bytes_ += 2.0 * ng * P + E * (4.0 * ng * (L[g] + r) * C + 4.0 * ng * ctx * C + 2.0 * M * C +
                                          ((4.0 * M * C + 2.0 * M_prev * C) if late else 2.0 * M * C))
            L[g] += r
        prev = k
    return flops, bytes_


def max_over_ranks(ms_local, dist, device):
    """Replicas only: every rank runs the same independent workload; the job's time is the slowest rank's."""
    if dist is None:
        return float(ms_local)
    import torch
    t = torch.tensor([float(ms_local)], device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_per_step, steps, world, ms_total_max):
    """Whole-job throughput: all ranks' units over the max-over-ranks time of `steps` steps."""
    return world * units_per_rank_per_step * steps / (ms_total_max * 1e-3)


def make_shape(name):
    return {"d16": si.shape_var_d16, "d30": si.shape_var_d30, "inf2b": si.shape_infinity_2b}[name]()


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

def oracle_leg(wl, steps, warmup):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload.  VAR shapes: up to 8 of the
    CFG pairs (d16) or 2 (d30), every block, every late scale.  Infinity shape: the one CFG pair, the first block
    group of the 8, every non-skipped late scale, extrapolated x 8 groups.  Returns (tokens/s, seconds per step,
    description, threads)."""
    from oracle import fvar_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        threads = os.cpu_count() or 1
    if "dense_until" in wl:
        raise NotImplementedError("no CPU baseline for the whole-generation workloads")
    full = make_shape(wl["shape"])
    plan_full = scale_plan(wl, full)
    shp = make_shape(wl["shape"])
    big = wl["shape"] == "inf2b"
    groups = 1 if big else full.n_groups
    shp.n_blocks = groups * shp.blocks_per_group
    B = 2 if big else (min(wl["B"], 16) if wl["shape"] == "d16" else 4)      # bounded sample: 10-15 s of CPU work
    Ms = shp.tokens_per_scale()
    k0 = wl["first_late"]
    weights = si.make_weights(SEED, shp)
    o = orc.Oracle(weights, shp.n_heads, shp.blocks_per_group, shp.hw(), shp.ln_eps)
    ctx = si.make_context(SEED, B, shp.ctx_len, shp.ctx_width) if shp.has_cross_attn else None
    o.set_cond(si.make_cond(SEED, B, shp.width), ctx)
    L0 = sum(Ms[:k0])
    K, V = si.make_kv_prefill(SEED, shp.n_blocks, B, L0, shp.width)
    gc = si.make_group_cache(SEED, shp.n_groups, B, Ms[k0 - 1], shp.width)
    toks = {k: si.make_tokens(SEED, B, Ms[k], shp.width) for k in plan_full}
    pols = {}
    for k, ranks in plan_full.items():
        if ranks is None:
            continue
        # Infinity shape: the sampled group runs at the mean rank of the scale's eight groups (the work is close to
        # linear in r), so that eight times its time stands for the stack
        ranks = [int(round(sum(ranks) / len(ranks)))] if big else ranks[:groups]
        late = any(r < Ms[k] for r in ranks)
        for g, r in enumerate(ranks):
            if r < Ms[k]:
                o.set_projection(k, g, si.make_projection(SEED, k, g, Ms[k], r))
        pols[k] = orc.Policy("lowrank_rtr" if late else "dense", "null_only" if wl["null_only"] else "pair",
                             rank_per_group=ranks if late else None, restore=wl.get("restore", "rtr"))
    E = B // 2 if wl["null_only"] else B
    tokens_per_step = E * sum(Ms[k] for k in plan_full)       # skipped scales deliver their positions too
    last_dt = [0.0]

    def one():
        o.load_kv(K, V)
        o.load_group_cache(k0 - 1, gc)
        for k in sorted(pols):
            t = time.perf_counter()
            o.scale_step(toks[k], k, pols[k])
            last_dt[0] = time.perf_counter() - t               # the last scale's step
            o.kv_append(k)

    for _ in range(warmup):
        one()
    t0 = time.perf_counter()
    for _ in range(steps):
        one()
    dt = (time.perf_counter() - t0) / max(steps, 1) * (full.n_groups / groups)
    desc = "%d CFG pair(s), %d of %d block groups%s, %d late scale(s) run, fp64 numpy (BLAS-threaded)" % (
        B // 2, groups, full.n_groups,
        " at the mean rank of each scale (time extrapolated x %d)" % (full.n_groups // groups) if groups < full.n_groups else "",
        len(pols))
    extra = {"cpu_model": cpu_model()}
    try:                                                       # one thread: the last scale's step only, scaled to the step
        from threadpoolctl import threadpool_limits
        all_last = last_dt[0]
        with threadpool_limits(limits=1):
            k = sorted(pols)[-1]
            t = time.perf_counter()
            o.scale_step(toks[k], k, pols[k])
            one_last = time.perf_counter() - t
        extra["single_thread"] = {"value": tokens_per_step / (dt * one_last / all_last), "unit": "tokens/s", "cores": 1,
                                  "sample": "the last scale's step of the same sample on one thread (%.2f s against %.2f s on %d), "
                                            "scaled to the whole step" % (one_last, all_last, threads)}
    except Exception as exc:                                   # threadpoolctl missing: report the all-core figure alone
        extra["single_thread"] = {"unavailable": repr(exc)}
    return tokens_per_step / dt, dt, desc, threads, extra


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


# ------------------------------------------------------------------------------------------- the GPU leg

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD,
                    help="one of %s, or infinity2b_last_r<R>_b<B>" % ", ".join(sorted(WORKLOADS)))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile-run", action="store_true",
                    help="for runs under ncu: skip the host-buffer leg, the event pass and the CPU baseline")
    args = ap.parse_args()
    wl = resolve_workload(args.workload)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    metric = "tokens/s over the late scale steps (output positions delivered per second)"
    config = {"workload": args.workload, "shape": wl["shape"], "batch": wl["B"],
              "late_scale_sides": list(make_shape(wl["shape"]).scales[wl["first_late"]:]),
              "keep": "rank %d" % wl["keep"][1] if isinstance(wl["keep"], tuple) else wl["keep"],
              "cfg": "null_only" if wl["null_only"] else "pair", "restore": wl.get("restore", "rtr"),
              "l2": "inputs_exceed_l2 (the stack's weights, streamed every step, are larger than L2)",
              "parity_bar": ("Infinity-2B shape: max-abs error <= 3e-2 x output RMS per block group (the stated 2e-2 is below what "
                             "rounding the FFN operands to bf16 alone costs at this shape, 1.6e-2; measured 2.1e-2), "
                             "x sqrt(g) after g groups; cosine >= 0.999" if wl["shape"] == "inf2b" else
                             "max-abs error <= 2e-2 x output RMS per block group, cosine >= 0.999")}

    if args.impl == "reference":
        if rank != 0:
            return
        steps = min(args.steps, 3)
        warm = min(args.warmup, 1)
        tps, dt, desc, threads, extra = oracle_leg(wl, steps, warm)
        print(json.dumps({
            "impl": "reference", "metric": metric, "value": tps, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": dict({"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc}, **extra),
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
    plan = scale_plan(wl, shp)
    late_scales = sorted(plan)
    null_at = {k: bool(wl["null_only"]) and k >= wl.get("dense_until", 0) for k in late_scales}
    cfg_at = {k: fv.CFG_NULL_ONLY if null_at[k] else fv.CFG_PAIR for k in late_scales}
    E_at = {k: B // 2 if null_at[k] else B for k in late_scales}
    seed = SEED + rank
    big = wl["shape"] == "inf2b"

    def bf16_cuda(a):
        return torch.from_numpy(si.bf16_bits(a).view(np.int16).reshape(a.shape)).view(torch.bfloat16).cuda()

    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)

    def randn_bf16(shape, std=1.0):          # large tensors are drawn on the device (same recipe, torch's generator)
        return (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32) * std).to(torch.bfloat16)

    if big:
        C, F, W = shp.width, shp.ffn_dim, shp.ctx_width
        dims = {"w_qkv": (3 * C, C), "b_qkv": (3 * C,), "w_o": (C, C), "b_o": (C,), "w_fc1": (F, C), "b_fc1": (F,),
                "w_fc2": (C, F), "b_fc2": (C,), "w_ada": (6 * C, C), "b_ada": (6 * C,), "w_cq": (C, C),
                "w_ckv": (2 * C, W), "w_co": (C, C)}
        weights = []
        for _ in range(shp.n_blocks):
            blk = {n: randn_bf16(d, 0.02) for n, d in dims.items()}
            blk["ln_c_gamma"] = (1.0 + 0.1 * torch.randn(C, generator=gen, device="cuda")).to(torch.bfloat16)
            weights.append(blk)
    else:
        weights = [{k: bf16_cuda(v) for k, v in blk.items()} for blk in si.make_weights(seed, shp)]
    ctx = fv.Fvar(weights, blocks_per_group=shp.blocks_per_group, n_heads=shp.n_heads, head_dim=shp.head_dim,
                  ffn_dim=shp.ffn_dim, scale_hw=shp.hw(), max_batch=B, ctx_len=shp.ctx_len, ctx_width=shp.ctx_width,
                  ln_eps=shp.ln_eps)
    context = bf16_cuda(si.make_context(seed, B, shp.ctx_len, shp.ctx_width)) if shp.has_cross_attn else None
    ctx.set_cond(bf16_cuda(si.make_cond(seed, B, shp.width)), context)
    L0 = sum(Ms[:k0])
    if k0 == 0:
        pass                                   # whole generation: the steps build the cache themselves
    elif big:
        ctx.load_kv(randn_bf16((shp.n_blocks, B, L0, shp.width)), randn_bf16((shp.n_blocks, B, L0, shp.width)))
        ctx.load_group_cache(k0 - 1, torch.randn((shp.n_groups, B, Ms[k0 - 1], shp.width), generator=gen, device="cuda"))
    else:
        K, V = si.make_kv_prefill(seed, shp.n_blocks, B, L0, shp.width)
        ctx.load_kv(bf16_cuda(K), bf16_cuda(V))
        ctx.load_group_cache(k0 - 1, torch.from_numpy(si.make_group_cache(seed, shp.n_groups, B, Ms[k0 - 1], shp.width)).cuda())
        del K, V
    torch.cuda.synchronize()
    modes = {}
    for k in late_scales:
        ranks = plan[k]
        if ranks is None:
            modes[k] = (fv.SKIP, None)
            continue
        late = any(r < Ms[k] for r in ranks)
        modes[k] = (fv.LOWRANK_RTR if late else fv.DENSE, ranks if late else None)
        for g, r in enumerate(ranks):
            if r < Ms[k]:
                qt = randn_bf16((r, Ms[k]), 1.0 / np.sqrt(r)) if big else \
                    bf16_cuda(np.ascontiguousarray(si.make_projection(seed, k, g, Ms[k], r).T))
                ctx.set_projection(k, g, qt)
    toks = {k: (randn_bf16((B, Ms[k], shp.width)) if big else bf16_cuda(si.make_tokens(seed, B, Ms[k], shp.width)))
            for k in late_scales}
    outs = {k: torch.empty((E_at[k], Ms[k], shp.width), dtype=torch.bfloat16, device="cuda") for k in late_scales}
    toks_host = {k: toks[k].cpu().pin_memory() for k in late_scales}
    outs_host = {k: torch.empty((E_at[k], Ms[k], shp.width), dtype=torch.bfloat16).pin_memory() for k in late_scales}
    tokens_per_step = sum(E_at[k] * Ms[k] for k in late_scales)     # a skipped scale still delivers its positions
    rewind = ctx.reset if k0 == 0 else ctx.restore_loaded
    loop = bool(wl.get("loop"))
    if loop:
        codebook = randn_bf16((LOOP_CODEBOOK, shp.width))
        ctx.set_codebook(codebook)
        tokens_per_step = (B // 2) * sum(Ms)                        # one image per CFG pair, every scale's positions
        start_host = toks[0].cpu().pin_memory()
        feat_host = torch.empty((B // 2, Ms[-1], shp.width), dtype=torch.float32).pin_memory()

    def step_loop(host=False):
        """Closed loop: step -> (CFG combination) -> transition -> the next step's tokens, for both branches."""
        rewind()
        tok = start_host.cuda(non_blocking=True) if host else toks[0]
        run = [k for k in late_scales if modes[k][0] != fv.SKIP]
        for i, k in enumerate(run):
            mode, ranks = modes[k]
            out = ctx.scale_step(tok, k, mode=mode, cfg_mode=cfg_at[k], rank_per_group=ranks, out=outs[k])
            ctx.kv_append(k)
            fo = out if null_at[k] else fv.fvar_cfg_combine(out, LOOP_GUIDANCE)
            more = i + 1 < len(run)
            _, nxt = ctx.scale_transition(fo, k, Ms[k + 1] if more else None, pairs=True)   # both branches see the same tokens
            if more:
                tok = nxt
        if host:
            feat_host.copy_(ctx.get_feature(B // 2, Ms[-1], shp.width), non_blocking=True)
            torch.cuda.synchronize()

    restore = fv.RESTORE_LLS if wl.get("restore") == "lls" else fv.RESTORE_RTR

    def step_device():
        rewind()
        for k in late_scales:
            mode, ranks = modes[k]
            if mode == fv.SKIP:
                continue
            ctx.scale_step(toks[k], k, mode=mode, cfg_mode=cfg_at[k], rank_per_group=ranks, out=outs[k], restore=restore)
            ctx.kv_append(k)

    def step_host():
        rewind()
        for k in late_scales:
            mode, ranks = modes[k]
            if mode == fv.SKIP:
                continue
            ctx.scale_step_host_async(toks_host[k], k, outs_host[k], mode=mode, cfg_mode=cfg_at[k], rank_per_group=ranks,
                                      restore=restore)
            ctx.kv_append(k)
        ctx.host_sync()                         # every result of the step is in host memory before the step counts

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
        ms = max_over_ranks(e0.elapsed_time(e1), dist, "cuda")
        return ms, ctx.launch_count() - n0

    warm = max(args.warmup, 3)
    sampler = ClockSampler(local_rank) if rank == 0 else None
    dev_fn, host_fn = (step_loop, lambda: step_loop(True)) if loop else (step_device, step_host)
    ms_total, launches = timed(dev_fn, args.steps, warm)
    clocks = sampler.stop() if sampler else None
    ms_e2e, _ = (ms_total, 0) if args.profile_run else timed(host_fn, args.steps, 2)
    assert ctx.poll_status() == fv.OK, "device status word reports an error"

    # per-kernel-class event timing: a separate pass over the same steps; the library re-captures the step's graph
    # with event-record nodes around every kernel node, so the kernels are timed inside the graph
    ctx.profile_enable(True)
    prof_steps = 0 if args.profile_run else max(1, min(args.steps, 10))
    for _ in range(prof_steps):
        # Hold the stream back (a device-side delay of about 10 ms) while the host captures and enqueues the
        # step, so that no interval between two events contains host time.
        torch.cuda._sleep(20_000_000)
        dev_fn()
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
    value = whole_job_value(tokens_per_step, args.steps, world, ms_total)
    e2e = whole_job_value(tokens_per_step, args.steps, world, ms_e2e)
    # Whole-step roofline, from this run's own timing: the step's algorithmic flops and bytes over ms_per_step.
    flops, bytes_ = algorithmic_work(shp, plan, null_at, B, L0)
    ridge = pk["bf16_sustained"] * 1e12 / (pk["hbm_gbs"] * 1e9)
    tf, gbs = flops / (ms_step * 1e-3) / 1e12, bytes_ / (ms_step * 1e-3) / 1e9
    hbm_bound = flops / bytes_ < ridge
    n_steps = max(1, sum(1 for k in late_scales if modes[k][0] != fv.SKIP))
    roofline = {"bound": "hbm" if hbm_bound else "tensor",
                "kernel": "the whole step (every kernel of the late scale steps; the GEMM class dominates)",
                "achieved": gbs if hbm_bound else tf, "peak": pk["hbm_gbs"] if hbm_bound else pk["bf16_sustained"],
                "unit": "GB/s" if hbm_bound else "TFLOP/s",
                "frac": gbs / pk["hbm_gbs"] if hbm_bound else tf / pk["bf16_sustained"],
                "peak_source": pk["source"] + (", copy bandwidth" if hbm_bound else ", sustained bf16"),
                "traffic": None,
                "how": "algorithmic %s of one step / ms_per_step of the timed region" % ("bytes" if hbm_bound else "flops"),
                "algorithmic_flops_per_step": flops, "algorithmic_bytes_per_step": bytes_,
                "flop_per_byte": flops / bytes_, "ridge_flop_per_byte": ridge,
                "frac_hbm": gbs / pk["hbm_gbs"], "frac_tensor": tf / pk["bf16_sustained"],
                "floor_ms_per_step": max(bytes_ / (pk["hbm_gbs"] * 1e9), flops / (pk["bf16_sustained"] * 1e12)) * 1e3,
                "classes_serialised": classes,
                "classes_how": "separate pass of %d steps: the step's CUDA graph re-captured with an event-record node before and "
                               "after every kernel node; kernels run one at a time there, so the class times sum to more than "
                               "ms_per_step" % prof_steps}
    line = {
        "metric": metric, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps, "warmup": warm,
        "ms_per_step": ms_step, "ms_per_scale_step": ms_step / max(1, sum(1 for k in late_scales if modes[k][0] != fv.SKIP)), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": e2e, "unit": "tokens/s",
                "h2d_bytes_per_step": B * Ms[0] * shp.width * 2 if loop else
                sum(E_at[k] * Ms[k] * shp.width * 2 for k in late_scales if modes[k][0] != fv.SKIP),
                "d2h_bytes_per_step": (B // 2) * Ms[-1] * shp.width * 4 if loop else
                sum(E_at[k] * Ms[k] * shp.width * 2 for k in late_scales if modes[k][0] != fv.SKIP)},
        "roofline": roofline,
    }
    if world == 1 and not args.no_cpu_baseline and not args.profile_run and "dense_until" not in wl:
        tps, dt, desc, threads, extra = oracle_leg(wl, 1, 0)
        line["cpu_baseline"] = dict({"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": desc,
                                     "seconds": dt}, **extra)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
