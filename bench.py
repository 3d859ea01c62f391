#!/usr/bin/env python
"""Benchmark of the LoRDO optimizer hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg4] [--variant global|local] [--mode fast|check]

One *step* is one full round of the workload's schedule over synthetic gradients: H inner steps
(clip, project, moments, back-project + weight/error update), one outer synchronisation and one
subspace refresh, i.e. every piece of the path. The default workload is the 1B-decoder-shaped
layer stack (168 matrices, r = 256, K = 8 replicas, H = 128, bf16 weights/gradients/error buffer,
fp32 states), the largest of the five configurations that fits one GPU together with its inputs.

`value` is parameters (weight-replicas) updated per second over whole rounds with every input
resident in HBM; `e2e` is the same unit for inner steps fed from pinned host memory through
lordo_inner_step_host (host->device copy of the gradients and device->host read of the clip
coefficients inside the timed region). `roofline` describes the kernel that takes the largest share
of the step. `cpu_baseline` times the CPU oracle on a bounded sample of the same workload.

The path does not shard: the K workers are a replica axis on one GPU. With --gpus N > 1 (launched
by torch.distributed.run) every rank runs an independent copy of the workload and the value is the
sum over ranks divided by the slowest rank's time; no data-path collective exists.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "inner low-rank opt-step params/s"
UNIT = "params/s"

# hyper-parameters of the paper's sweep table: QHM beta1 = 0.999; omega = 0.97 (Global, full-rank
# QHM) / 0.94 (Local, low-rank QHM); lr = 0.004; outer Nesterov lr 0.8, momentum 0.9
HYPER = {
    "global": dict(variant=0, form=2, beta1=0.999, omega=0.97),
    "local": dict(variant=1, form=1, beta1=0.999, omega=0.94),
}
LR = 0.004

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in the named
# file under profiles/ (taken on 2 of the 24 layers and scaled by 12: traffic grows with the layers).
# An entry is removed when its kernel changes, until the counters have been taken again.
NCU_TRAFFIC = {
    "cfg4_1B_r256:global:fast:apply": (102849540000, "profiles/ncu_project_tma_apply_tma_cfg4_first2layers.md"),
    "cfg4_1B_r256:global:fast:project": (60545076000, "profiles/ncu_project_tma_apply_tma_cfg4_first2layers.md"),
    "cfg4_1B_r256:local:fast:apply": (102849540000, "profiles/ncu_project_tma_apply_tma_cfg4_first2layers.md"),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--variant", default="global", choices=["global", "local"])
    ap.add_argument("--mode", default="fast", choices=["fast", "check"])
    ap.add_argument("--inner-steps", type=int, default=0, help="override H (non-standard; recorded in config)")
    ap.add_argument("--layers", type=int, default=0, help="keep only the first N decoder layers (profiling; recorded in config)")
    ap.add_argument("--matrices", type=int, default=0, help="keep only the first N matrices (profiling / memory; recorded in config)")
    ap.add_argument("--right-side", action="store_true", help="project the matrices with more rows than columns from the right (not in the paper; recorded in config)")
    ap.add_argument("--oversample", type=int, default=0, help="extra sketch columns of the refresh, Rayleigh-Ritz truncation (non-standard; recorded in config)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-legs", action="store_true", help="skip the short legs on the other configurations")
    return ap.parse_args()


def workload(name: str, H: int = 0, layers: int = 0, matrices: int = 0, right_side: bool = False):
    from paper_2602_04396_b200 import synth
    wl = synth.config(int(name[3:]))
    if right_side:
        wl = synth.scaled(wl, sides=tuple(1 if m > n else 0 for m, n, _ in wl.mats), name=f"{wl.name}_tall_from_right")
    if H > 0:
        wl = synth.scaled(wl, H=H)
    if layers > 0 and len(wl.mats) >= 7 * layers:
        wl = synth.scaled(wl, mats=wl.mats[:7 * layers], name=f"{wl.name}_first{layers}layers",
                          sides=wl.sides[:7 * layers] if wl.sides else None)
    if 0 < matrices < len(wl.mats):
        wl = synth.scaled(wl, mats=wl.mats[:matrices], name=f"{wl.name}_first{matrices}matrices",
                          sides=wl.sides[:matrices] if wl.sides else None)
    return wl


def bytes_of(dt: str) -> int:
    return 2 if dt == "bf16" else 4


def algorithmic_bytes(wl, variant: int, form: int, ef: bool = True, fast: bool = True) -> dict:
    """Bytes each kernel class must move per launch if every tensor it touches crossed HBM exactly
    once (operands shared by the K replicas counted once). In fast mode the moment update is part of
    the projection kernel (u, v read and written, bf16 transposed g^ and U~ written) and the update
    kernel reads those two bf16 operands; in check mode g^ and U~ are fp32 and the moments have a
    kernel of their own."""
    K = wl.K
    bw, bg, be = bytes_of(wl.w_dtype), bytes_of(wl.g_dtype), bytes_of(wl.e_dtype)
    out = dict(clip=0, project=0, moments=0, apply=0, outer_states=0, outer_weights=0)
    for i, (m, n, r) in enumerate(wl.mats):
        pm, ln = (n, m) if (wl.sides and wl.sides[i]) else (m, n)  # rows of P, columns of the low-rank arrays
        mn, rn = m * n, r * ln
        p_copies = K if variant == 1 else 1
        dcol = K * ln * 4 if form == 2 else 0
        out["clip"] += K * mn * bg
        stream_in = K * mn * (bg + (be if ef else 0))
        stream_rw = K * mn * (bg + (2 * be if ef else 0) + 2 * bw)
        if fast:
            out["project"] += stream_in + p_copies * pm * r * 2 + K * rn * (16 + 4) + dcol
            out["apply"] += stream_rw + p_copies * pm * r * 2 + K * rn * 4 + dcol
        else:
            out["project"] += stream_in + p_copies * pm * r * 4 + K * rn * 4
            out["moments"] += K * rn * 4 * 6 + dcol  # read g,u,v; write u,v,U~
            out["apply"] += stream_rw + p_copies * pm * r * 4 + K * rn * 4 * 2 + dcol
        out["outer_states"] += 2 * (2 * K * rn * 4)
        out["outer_weights"] += 2 * K * mn * bw + mn * 4 * 5  # X0 r/w, B r/w, Delta w
    return out


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0: float, t1: float) -> dict:
        sm, smax, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if ts < t0 or ts > t1 + 0.3:
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax = max(smax, float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax or None, "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the CPU oracle on a bounded sample (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_sample(wl, variant_name: str, K: int = 0, H: int = 6):
    """Returns (sample workload, description). One matrix of the most common shape class with all
    K replicas (or the first `K` of them), a round of up to `H` inner steps + outer step + refresh."""
    from paper_2602_04396_b200 import synth
    shapes = {}
    for mat in wl.mats:
        shapes[mat] = shapes.get(mat, 0) + 1
    mat = max(shapes, key=lambda s: (shapes[s], -s[0] * s[1]))
    H = min(wl.H, H)
    Ks = min(wl.K, K) if K > 0 else wl.K
    side = (wl.sides[wl.mats.index(mat)],) if wl.sides else None
    sample = synth.scaled(wl, mats=[mat], H=H, rounds=1, K=Ks, sides=side)
    desc = (f"1 matrix {mat[0]}x{mat[1]} r{mat[2]} of {len(wl.mats)}, {'all ' if Ks == wl.K else ''}K={Ks} replicas"
            f"{'' if Ks == wl.K else f' of {wl.K}'}, one round of {H} inner steps + outer step + refresh, {variant_name} rule")
    return sample, desc


def run_oracle_sample(sample, variant_name: str, seed: int = 0):
    """One pass of the CPU oracle over the sample; returns (seconds, params updated)."""
    import numpy as np
    from oracle import lordo_oracle as lo
    from paper_2602_04396_b200 import synth
    hp = HYPER[variant_name]
    cfg = lo.OracleConfig(mats=sample.mats, K=sample.K, H=sample.H, variant=hp["variant"], error_feedback=True,
                          beta2=float(np.float32(0.999)), eps=float(np.float32(1e-8)), clip_rho=sample.clip_rho,
                          outer=lo.OUTER_NESTEROV, outer_lr=float(np.float32(0.8)), outer_momentum=float(np.float32(0.9)),
                          power_iters=sample.power_iters, seed=seed, w_dtype=sample.w_dtype, e_dtype=sample.e_dtype,
                          state_dtype="f32", sides=sample.sides)
    orc = lo.LordoOracle(cfg, synth.init_weights(sample, seed))
    grads = [synth.gradients(sample, seed, 0, h) for h in range(sample.H)]
    t0 = time.perf_counter()
    lo.run_rounds(orc, lambda rnd, h: grads[h], 1, LR, hp["beta1"], hp["omega"], hp["form"], refresh=True)
    dt = time.perf_counter() - t0
    return dt, sample.weight_replicas * sample.H


def max_over_ranks(value_ms: float, device=None) -> float:
    """Slowest rank's time (every rank runs its own copy of the workload; there is no other
    exchange on this path). Works on any initialised process group (NCCL on GPUs, gloo on CPU)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value_ms)
    t = torch.tensor([value_ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(units_per_rank: int, world: int, ms_max: float) -> float:
    """Whole-job throughput: the units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / (ms_max * 1e-3)


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def reference_main(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    wl = workload(args.workload, args.inner_steps, args.layers, args.matrices, args.right_side)
    # one step = one pass of the oracle over the sample; the sample shrinks with the number of passes asked
    # for, so that the whole run stays within a few minutes
    sample, desc = oracle_sample(wl, args.variant, H=6 if args.steps + args.warmup <= 8 else 2)
    for _ in range(args.warmup):
        run_oracle_sample(sample, args.variant)
    total_t, total_p = 0.0, 0
    for _ in range(args.steps):
        dt, p = run_oracle_sample(sample, args.variant)
        total_t += dt
        total_p += p
    value = total_p / total_t
    cores = cpu_threads()
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "variant": args.variant, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))
    return 0


# ------------------------------------------------------------------------------------------------
# the CUDA path
# ------------------------------------------------------------------------------------------------
def run_leg(wl, variant_name: str, mode: str, steps: int, warmup: int, *, dev, rank: int, world: int, local_rank: int,
            oversample: int = 0, e2e_steps: int = 0, peaks=None):
    """One timed leg: builds the workload on the device, runs `warmup` + `steps` rounds (a round = H inner
    steps, with the Local refresh before the first; the outer step; the Global refresh), and returns the
    figures of that leg: whole-round throughput, per-kernel-class times from the library's CUDA events,
    the dominant kernel's roofline fraction, the clock sample of the timed region."""
    import torch
    import torch.distributed as dist
    from paper_2602_04396_b200 import lordo, synth

    hp = HYPER[variant_name]
    H = wl.H
    seed = 1000 + rank  # every rank runs its own copy of the workload on its own inputs
    torch.cuda.reset_peak_memory_stats(dev)
    W0 = synth.init_weights_device(wl, seed, device=str(dev))
    opt = lordo.Lordo(wl.mats, wl.K, H, W0, device=str(dev), g_dtype=synth.torch_dtype(wl.g_dtype),
                      e_dtype=synth.torch_dtype(wl.e_dtype), variant=hp["variant"], error_feedback=True, beta2=0.999,
                      eps=1e-8, clip_rho=wl.clip_rho, outer=lordo.OUTER_NESTEROV, outer_lr=0.8, outer_momentum=0.9,
                      power_iters=wl.power_iters, seed=seed, check_mode=1 if mode == "check" else 0, oversample=oversample,
                      sides=wl.sides)
    del W0
    # two gradient sets (round-level signal + per-replica noise), used alternately
    pool = [synth.gradients_device(wl, seed, 0, s, device=str(dev)) for s in range(2)]
    torch.cuda.synchronize()

    def one_round(rnd: int):
        for h in range(H):
            G = pool[(rnd * H + h) & 1]
            if hp["variant"] == 1 and h == 0:
                opt.refresh_subspace(G, hp["beta1"])
            opt.inner_step(G, LR, hp["beta1"], hp["omega"], hp["form"])
        opt.outer_step()
        if hp["variant"] == 0:
            opt.refresh_subspace(None, hp["beta1"])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for w in range(warmup):
        one_round(w)
    barrier()
    opt.profile_enable(True)
    opt.profile_read()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    launches0 = opt.launch_count
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    ev0.record()
    for s in range(steps):
        one_round(warmup + s)
    ev1.record()
    barrier()
    t_wall1 = time.time()
    ms_total = ev0.elapsed_time(ev1)
    launches = opt.launch_count - launches0
    classes = opt.profile_read()
    opt.profile_enable(False)
    if rank == 0:
        time.sleep(0.25)
        sampler.stop()
    flags = opt.poll_status()

    ms_total = max_over_ranks(ms_total, dev)
    n_inner = H * steps
    value = aggregate_value(wl.weight_replicas * n_inner, world, ms_total)

    # ---- per-class figures and the roofline of the dominant kernel -----------------------------
    tc_active = (mode == "fast" and wl.w_dtype == wl.g_dtype == wl.e_dtype and
                 max(r for _, _, r in wl.mats) <= (512 if wl.w_dtype == "bf16" else 256))
    abytes = algorithmic_bytes(wl, hp["variant"], hp["form"], True, tc_active)
    per_launch = {"clip": n_inner, "project": n_inner, "moments": n_inner, "apply": n_inner, "outer_states": steps,
                  "outer_weights": steps, "refresh": steps * (H if wl.refresh_every_step else 1)}
    kernels = {}
    for name, ms in classes.items():
        cnt = per_launch[name]
        avg = ms / cnt if cnt else 0.0
        ent = {"ms_per_launch": avg, "share": ms / ms_total if ms_total else 0.0}
        if name in abytes and avg > 0:
            ent["algorithmic_GB"] = abytes[name] / 1e9
            ent["GB_per_s"] = abytes[name] / 1e9 / (avg * 1e-3)
        kernels[name] = ent
    peaks = peaks or {}
    hbm_peak = float(peaks.get("hbm_gbs", 6650.0))
    peak_src = "measured" if "hbm_gbs" in peaks else "fallback"
    dom = max((k for k in kernels if k in abytes), key=lambda k: kernels[k]["share"])
    ent = NCU_TRAFFIC.get(f"{wl.name}:{variant_name}:{mode}:{dom}")
    traffic = ent[0] if ent else None
    roofline = {"bound": "hbm", "kernel": dom, "achieved": kernels[dom].get("GB_per_s"), "peak": hbm_peak, "unit": "GB/s",
                "frac": (kernels[dom].get("GB_per_s") or 0.0) / hbm_peak, "peak_source": peak_src, "traffic": traffic,
                "algorithmic_bytes_per_launch": abytes[dom]}
    inner_ms = sum(classes[k] for k in ("clip", "project", "moments", "apply")) / n_inner
    outer_ms = (classes["outer_states"] + classes["outer_weights"]) / steps
    outer_bytes = abytes["outer_states"] + abytes["outer_weights"]
    # the three tensor-core contractions of an inner step (project, error feedback, back-projection)
    inner_flops = sum(6.0 * r * m * n for m, n, r in wl.mats) * wl.K
    tf_peak = float(peaks.get("bf16_tflops_sustained", 1400.0))

    # ---- end to end: inner steps fed from pinned host memory ------------------------------------
    e2e = None
    if e2e_steps > 0:
        n_e2e = max(1, min(e2e_steps, H))
        G_host = [torch.empty(g.shape, dtype=g.dtype, pin_memory=True).copy_(g) for g in pool[0]]
        clip_host = torch.empty(wl.K, dtype=torch.float32, pin_memory=True)
        h2d = sum(g.numel() * g.element_size() for g in G_host)
        stage = pool[1]
        torch.cuda.synchronize()
        if hp["variant"] == 1:
            opt.refresh_subspace(stage, hp["beta1"])
        opt.inner_step_host(G_host, stage, LR, hp["beta1"], hp["omega"], hp["form"], clip_host)  # warm-up
        barrier()
        n_done = max(1, min(n_e2e, H - 1))  # the round's first step was the warm-up call
        ev0.record()
        for _ in range(n_done):
            opt.inner_step_host(G_host, stage, LR, hp["beta1"], hp["omega"], hp["form"], clip_host)
        ev1.record()
        barrier()
        ms_e2e = ev0.elapsed_time(ev1)
        ms_e2e = max_over_ranks(ms_e2e, dev)
        e2e = {"value": aggregate_value(wl.weight_replicas * n_done, world, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 4 * wl.K, "inner_steps_timed": n_done,
               "note": "inner steps through lordo_inner_step_host; the outer step and the refresh take no host input"}
        del G_host

    leg = {
        "value": value, "ms_per_step": ms_total / steps, "steps": steps, "warmup": warmup,
        "config": {"workload": wl.name, "matrices": len(wl.mats), "weights": wl.weights, "K": wl.K, "H": H,
                   "rank": wl.mats[0][2], "variant": variant_name, "qhm": ["none", "low", "full"][hp["form"]],
                   "outer": "nesterov", "mode": mode, "w_dtype": wl.w_dtype, "g_dtype": wl.g_dtype,
                   "step": "one round = H inner steps + outer step + subspace refresh",
                   "l2": "inputs larger than L2 (no flush)" if wl.weight_replicas * 2 > 4e8 else "inputs fit L2",
                   "parallelism": "replicas only" if world > 1 else "1 gpu",
                   **({"oversample": oversample} if oversample else {}),
                   **({"sides": "matrices with m > n projected from the right"} if wl.sides and any(wl.sides) else {})},
        "clocks": sampler.summary(t_wall0, t_wall1),
        "gpu_launches": launches,
        "inner_step": {"ms": inner_ms, "params_per_s": wl.weight_replicas / (inner_ms * 1e-3) if inner_ms else None,
                       "tensor_TFLOP_per_s": inner_flops / 1e12 / (inner_ms * 1e-3) if inner_ms else None,
                       "frac_of_sustained_bf16_peak": (inner_flops / 1e12 / (inner_ms * 1e-3)) / tf_peak if inner_ms else None},
        "outer_sync": {"ms": outer_ms, "GB_per_s": outer_bytes / 1e9 / (outer_ms * 1e-3) if outer_ms else None,
                       "frac_of_hbm_peak": (outer_bytes / 1e9 / (outer_ms * 1e-3)) / hbm_peak if outer_ms else None},
        "refresh": {"ms": classes["refresh"] / per_launch["refresh"]},
        "kernels": kernels,
        "roofline": roofline,
        "e2e": e2e,
        "device_flags": flags,
        "memory": {"workspace_bytes": int(opt.workspace_bytes), "peak_allocated_bytes": int(torch.cuda.max_memory_allocated(dev))},
    }
    opt.close()
    del opt, pool
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    return leg


# The other configurations the path is specified on, timed briefly after the headline workload in the
# same run: (workload, variant, matrices kept (0 = all), warm-up rounds, timed rounds).
EXTRA_LEGS = [
    ("cfg4", "local", 0, 3, 3),
    ("cfg4:right", "global", 0, 3, 3),  # the down projections (m > n) projected from the right
    ("cfg3", "global", 0, 3, 10),
    ("cfg3", "local", 0, 3, 10),
    ("cfg5", "local", 8, 3, 10),   # the first 8 of 32 matrices: all 32 with K = 16 do not fit beside their inputs
    ("cfg5", "global", 8, 3, 10),
]


def main():
    args = parse_args()
    if args.impl == "reference":
        return reference_main(args)

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = {}
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            peaks = json.load(fh)
    except Exception:
        pass
    where = dict(dev=dev, rank=rank, world=world, local_rank=local_rank, peaks=peaks)

    wl = workload(args.workload, args.inner_steps, args.layers, args.matrices, args.right_side)
    main_leg = run_leg(wl, args.variant, args.mode, args.steps, args.warmup, oversample=args.oversample,
                       e2e_steps=0 if args.no_e2e else args.e2e_steps, **where)

    # ---- the other configurations, briefly (one GPU, default workload only) ----------------------
    legs = []
    default_run = (args.workload == "cfg4" and args.variant == "global" and args.mode == "fast" and not args.inner_steps and
                   not args.layers and not args.matrices and not args.oversample and not args.right_side)
    if world == 1 and default_run and not args.no_legs:
        for name, variant, matrices, wu, st in EXTRA_LEGS:
            lw = workload(name.split(":")[0], 0, 0, matrices, right_side=name.endswith(":right"))
            leg = run_leg(lw, variant, "fast", st, wu, **where)
            for drop in ("e2e", "memory"):
                leg.pop(drop, None)
            legs.append(leg)

    # ---- CPU oracle on a bounded sample ---------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample, desc = oracle_sample(wl, args.variant)
        dt, p = run_oracle_sample(sample, args.variant)
        cpu = {"value": p / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc, "seconds": dt}
        one, desc1 = oracle_sample(wl, args.variant, K=2, H=2)
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                dt1, p1 = run_oracle_sample(one, args.variant)
            cpu["single_thread"] = {"value": p1 / dt1, "unit": UNIT, "cores": 1, "sample": desc1, "seconds": dt1}
        except Exception as exc:  # threadpoolctl missing: say so instead of reporting a wrong core count
            cpu["single_thread"] = {"unavailable": str(exc)}

    if rank == 0:
        out = {
            "metric": METRIC, "value": main_leg["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": main_leg["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if args.mode == "fast" else "f32", "data": "synthetic",
        }
        for key in ("config", "clocks", "gpu_launches", "inner_step", "outer_sync", "refresh", "kernels", "roofline", "e2e"):
            out[key] = main_leg[key]
        out["gpu_launches"] = main_leg["gpu_launches"] + sum(l["gpu_launches"] for l in legs)
        out["cpu_baseline"] = cpu
        out["device_flags"] = main_leg["device_flags"]
        out["memory"] = main_leg["memory"]
        out["legs"] = legs
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
