#!/usr/bin/env python
"""Benchmark of the cluster-retrieval decode path on B200.

A *step* is one pass of the hot path over one batch of synthetic input: for every unit of
the workload, score the query against the centroids, select the top clusters under the
token budget, gather their pages and attend, append the step's new key/value to its
nearest cluster and run the split check.  The index is built first (timed separately and
reported under "build").  Prints one JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4] [--impl ours|reference]

N > 1 is launched with torchrun; every rank runs the same workload on its own GPU (units
are independent, no collective on the data path) and the value is the aggregate.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode steps/s at 32-layer 32K ctx; retrieval-attention HBM GB/s vs peak"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100", "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush(); self.f.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.f.name)
        except OSError:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        return out


def _oracle_sample(cfg, n_units: int, steps: int, lloyd_rounds: int):
    """Time the fp64 oracle, as it stands, on a bounded sample of the workload: `n_units`
    units of the config (index built by the oracle itself with `lloyd_rounds` rounds, untimed),
    then `steps` iterations of decode_step + append + split_check, one thread per unit."""
    from concurrent.futures import ThreadPoolExecutor

    import numpy as np

    import oracle as O
    from gen import UnitStream

    cores = min(n_units, os.cpu_count() or 1)

    def prep(u):
        s = UnitStream(cfg, u)
        K, V = s.prefill()
        o = O.OracleUnit(cfg.d, cfg.G, cfg.max_tokens, cfg.max_clusters, gamma=cfg.split_size_factor,
                         alpha=cfg.split_var_factor, split_min_size=cfg.split_min_size, split_iters=cfg.split_iters)
        o.build(K.double().numpy(), V.double().numpy(), cfg.M0, lloyd_rounds, 1234, unit_index=u,
                init_mode=O.INIT_RANDOM)
        q, k, v = s.decode(steps)
        return o, q.double().numpy(), k.double().numpy(), v.double().numpy()

    def run(item):
        o, q, k, v = item
        for t in range(steps):
            o.decode_step(q[t], cfg.budget)
            o.append(k[t], v[t])
            o.split_check()

    with ThreadPoolExecutor(max_workers=cores) as ex:
        items = list(ex.map(prep, range(n_units)))
        t0 = time.perf_counter()
        list(ex.map(run, items))
        dt = time.perf_counter() - t0
    # one "step" of the metric covers all U units; the sample covered n_units of them
    per_step_all_units = dt / steps * (cfg.U / n_units)
    return 1.0 / per_step_all_units, cores, dt


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_units = min(8, os.cpu_count() or 1)
    per = max(1, min(args.steps, 4))
    vals = []
    total_dt = 0.0
    reps = max(1, min(3, args.steps // per))
    for _ in range(reps):
        v, cores, dt = _oracle_sample(cfg, n_units, per, lloyd_rounds=1)
        vals.append(v); total_dt += dt
    value = statistics.median(vals)
    sample = (f"{n_units} of {cfg.U} units of config {cfg.cfg_id} at full size (index built by the oracle with 1 Lloyd "
              f"round, untimed), {per} decode steps per repeat x {reps} repeats, scaled per unit to all {cfg.U} units")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 / value, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config{cfg.cfg_id}:{cfg.name}", "units": cfg.U, "context": cfg.n_prefill,
                   "budget": cfg.budget},
        "cpu_baseline": {"value": value, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import paper_2511_07427_b200 as P
    from gen import UnitStream, make_decode_chunk, make_prefill

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    # all work (generation, library calls, timing events) runs on one side stream: the decode loop is a captured graph
    side = torch.cuda.Stream(device=dev)
    torch.cuda.set_stream(side)
    peaks = _peaks()
    K_steps, W = args.steps, args.warmup
    n_e2e = min(args.e2e_steps, K_steps)
    n_prof = min(args.profile_steps, K_steps)
    total_steps = W + K_steps + n_e2e + n_prof
    assert total_steps <= cfg.steps, "not enough decode capacity in this config for the requested steps"

    # ---- synthetic inputs, generated on the device (seeded per unit and rank)
    U = cfg.U
    streams = [UnitStream(cfg, rank * U + u, device=str(dev)) for u in range(U)]
    Kp, Vp = make_prefill(streams)
    q_all, k_all, v_all = make_decode_chunk(streams, total_steps)
    del streams
    torch.cuda.synchronize()

    ctx = P.DynaKV(P.DynaKVConfig(
        n_units=U, gqa_group=cfg.G, head_dim=cfg.d, kv_dtype=P.F32 if cfg.kv_dtype == "f32" else P.BF16,
        max_tokens=cfg.max_tokens, max_clusters=cfg.max_clusters, kmeans_iters=cfg.T,
        init_mode=P.INIT_KMEANSPP if cfg.init_mode == "kmeanspp" else P.INIT_RANDOM,
        split_size_factor=cfg.split_size_factor, split_var_factor=cfg.split_var_factor,
        split_min_size=cfg.split_min_size, split_iters=cfg.split_iters, trace=0, assign_mode=args.assign_mode))

    # ---- build (prefill indexing), timed on its own
    ctx.set_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    ctx.build_index(Kp, Vp, cfg.M0, 1234)
    e1.record(); torch.cuda.synchronize()
    build_ms = e0.elapsed_time(e1)
    kt = ctx.get_kernel_times(reset=True)
    ctx.set_timing(False)
    del Kp, Vp
    assign_ms = kt["assign"]["ms"] / max(kt["assign"]["launches"], 1)
    assign_flop = 2.0 * cfg.n_prefill * cfg.M0 * cfg.d * U
    build = {
        "seconds": build_ms / 1e3, "lloyd_rounds": cfg.T,
        "assign_ms_per_round": assign_ms, "update_ms_per_round": kt["update"]["ms"] / max(kt["update"]["launches"], 1),
        "init_ms": kt["init"]["ms"], "finalize_ms": kt["finalize"]["ms"],
        "assign_algorithmic_tflops": assign_flop / (assign_ms * 1e-3) / 1e12 if assign_ms > 0 else None,
        "assign_path": "fp32" if args.assign_mode == 1 else "auto",
    }
    build["roofline"] = {"bound": "tensor", "achieved": build["assign_algorithmic_tflops"], "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": (build["assign_algorithmic_tflops"] or 0) / peaks["bf16_tflops"],
                         "traffic": None, "peak_source": peaks["source"] + " burst bf16"}

    out_all = torch.empty((total_steps, U, cfg.G, cfg.d), dtype=torch.float32, device=dev)

    def loop(a, b):
        ctx.decode_loop(q_all[a:b], k_all[a:b], v_all[a:b], cfg.budget, out_all[a:b])

    # ---- warm-up, then the timed region (CUDA-graph replay, inputs resident in HBM)
    pos = 0
    if W > 0:
        loop(pos, pos + W); pos += W
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    st0 = ctx.get_status()
    launches0 = ctx.launch_count()
    sampler = ClockSampler(local) if rank == 0 else None
    torch.cuda.synchronize()
    e0.record()
    loop(pos, pos + K_steps)
    e1.record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    ms = e0.elapsed_time(e1)
    clocks = sampler.stop() if sampler else None
    pos += K_steps
    st1 = ctx.get_status()
    gpu_launches = ctx.launch_count() - launches0
    if world > 1:
        tmax = torch.tensor([ms], device=dev, dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms = float(tmax.item())
    value = world * K_steps / (ms * 1e-3)

    # ---- per-kernel breakdown with CUDA events around every launch (direct calls, same stream)
    ctx.set_timing(True)
    tok0 = ctx.get_status()["tokens_attended_total"]
    for t in range(pos, pos + n_prof):
        ctx.decode_step(q_all[t], cfg.budget, out=out_all[t])
        ctx.append(k_all[t], v_all[t])
        ctx.split_check()
    kt = ctx.get_kernel_times(reset=True)
    ctx.set_timing(False)
    tok1 = ctx.get_status()["tokens_attended_total"]
    pos += n_prof
    bytes_kv = 4 if cfg.kv_dtype == "f32" else 2
    attn_ms = kt["attn"]["ms"] / max(kt["attn"]["launches"], 1)
    tokens_per_launch = (tok1 - tok0) / max(n_prof, 1)
    attn_bytes = tokens_per_launch * 2 * cfg.d * bytes_kv + U * cfg.G * cfg.d * 4
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9 if attn_ms > 0 else 0.0
    kernels = {k: (v["ms"] / v["launches"] * 1e3 if v["launches"] else None) for k, v in kt.items()
               if k in ("select", "attn", "combine", "append", "split")}
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": args.attn_traffic_bytes,
                "kernel": "gather_attn", "us_per_launch": attn_ms * 1e3, "algorithmic_bytes_per_launch": attn_bytes,
                "tokens_per_launch": tokens_per_launch, "frac_of_8TBs_nominal": achieved / 8000.0,
                "peak_source": peaks["source"] + " copy bandwidth", "per_kernel_us": kernels}

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    e2e = None
    if n_e2e > 0:
        qh = q_all[pos:pos + n_e2e].cpu().pin_memory(); kh = k_all[pos:pos + n_e2e].cpu().pin_memory()
        vh = v_all[pos:pos + n_e2e].cpu().pin_memory()
        oh = torch.empty((U, cfg.G, cfg.d), dtype=torch.float32).pin_memory()
        ctx.step_host(qh[0], kh[0], vh[0], cfg.budget, oh)      # warm
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for t in range(1, n_e2e):
            ctx.step_host(qh[t], kh[t], vh[t], cfg.budget, oh)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        if world > 1:
            tm = torch.tensor([dt], device=dev, dtype=torch.float64)
            dist.all_reduce(tm, op=dist.ReduceOp.MAX)
            dt = float(tm.item())
        e2e = {"value": world * (n_e2e - 1) / dt if n_e2e > 1 else None, "unit": "steps/s",
               "h2d_bytes_per_step": int(qh[0].numel() * 4 + 2 * kh[0].numel() * bytes_kv),
               "d2h_bytes_per_step": int(oh.numel() * 4)}
    status = ctx.get_status()
    ctx.destroy()

    if rank == 0:
        cpu_baseline = None
        if world == 1 and not args.no_cpu_baseline:
            n_units = min(8, os.cpu_count() or 1)
            v, cores, dt = _oracle_sample(cfg, n_units, 4, lloyd_rounds=1)
            cpu_baseline = {"value": v, "unit": "steps/s", "cores": cores, "kind": "oracle",
                            "sample": f"{n_units} of {cfg.U} units of config {cfg.cfg_id} at full size (index built by the "
                                      f"oracle with 1 Lloyd round, untimed), 4 decode steps ({dt:.1f} s), scaled per unit "
                                      f"to all {cfg.U} units"}
        line = {
            "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": K_steps, "warmup": W,
            "ms_per_step": ms / K_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32" if cfg.kv_dtype == "f32" else "bf16 KV / f32 math", "data": "synthetic",
            "config": {"workload": f"config{cfg.cfg_id}:{cfg.name}", "units_per_gpu": U, "layers": cfg.L,
                       "kv_heads": cfg.Hkv, "gqa_group": cfg.G, "head_dim": cfg.d, "context": cfg.n_prefill + W,
                       "clusters": cfg.M0, "budget": cfg.budget, "l2": "inputs_larger_than_l2",
                       "loop": "cuda_graph_replay(decode_step,append,split_check)"},
            "e2e": e2e, "gpu_launches": int(gpu_launches), "clocks": clocks, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "build": build,
            "counters": {"splits_in_timed_region": st1["n_splits"] - st0["n_splits"],
                         "tokens_attended_per_step": (st1["tokens_attended_total"] - st0["tokens_attended_total"]) / K_steps,
                         "clusters_selected_per_step": (st1["clusters_selected_total"] - st0["clusters_selected_total"]) / K_steps,
                         "status_bits": status["error_bits"], "assign_rechecked": status["assign_rechecked"]},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--assign-mode", type=int, default=0)
    ap.add_argument("--e2e-steps", type=int, default=64)
    ap.add_argument("--profile-steps", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--attn-traffic-bytes", type=float, default=None,
                    help="ncu dram bytes per launch of the gather-attention kernel (from profiles/), echoed in roofline.traffic")
    args = ap.parse_args()
    from gen import CONFIGS
    cfg = CONFIGS[args.config]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
