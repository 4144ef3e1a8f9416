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
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "decode steps/s at 32-layer 32K ctx; retrieval-attention HBM GB/s vs peak"

# DRAM traffic of the gather-attention kernel from its ncu capture (profiles/gather_attn_config4_96units.txt):
# dram__bytes_read.sum + dram__bytes_write.sum of one launch, and the tokens that launch attended.  Traffic
# is proportional to the rows attended, so a launch's traffic is scaled by its own token count.  Set
# NCU_ATTN_CAPTURE to None whenever the kernel changes after the capture.
NCU_ATTN_CAPTURE = {"dram_bytes": 100.3451e6 + 3.0842e6, "tokens": 195006.5}
# the same for the kernel on FP8 rows (profiles/gather_attn_fp8_config4_96units.txt)
NCU_ATTN_CAPTURE_FP8 = {"dram_bytes": 52.0032e6 + 0.2890e6, "tokens": 194980.75}


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Reads SM clock, power and clock-event reasons from NVML on a background thread
    (read-only queries, a few hundred per second) between start() and stop()."""

    def __init__(self, torch_device_index: int):
        import threading
        self.samples = []          # (t, sm_mhz, power_w, reasons bitmask)
        self.sm_max = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            h = None
            try:
                uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
                h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self._h, self._nv = h, pynvml
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            self._thread = threading.Thread(target=self._run, daemon=True)
        except Exception:
            self._h = None

    def _run(self):
        nv, h = self._nv, self._h
        while not self._stop.is_set():
            try:
                sm = float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                pw = nv.nvmlDeviceGetPowerUsage(h) / 1000.0
                rs = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
                self.samples.append((time.perf_counter(), sm, pw, rs))
            except Exception:
                pass
            self._stop.wait(0.003)

    def start(self):
        if self._thread is not None:
            self._thread.start()

    def stop(self, windows=None) -> dict:
        """windows: list of (t0, t1) perf_counter intervals; samples inside any of them are summarised."""
        out = {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "samples": 0, "power_w_max": None}
        if self._thread is None:
            return out
        self._stop.set(); self._thread.join(timeout=2)
        nv = self._nv
        rows = [r for r in self.samples if windows is None or any(a <= r[0] <= b for a, b in windows)]
        if not rows:
            rows = self.samples
        if rows:
            names = [("hw_slowdown", nv.nvmlClocksEventReasonHwSlowdown),
                     ("hw_thermal_slowdown", nv.nvmlClocksEventReasonHwThermalSlowdown),
                     ("sw_thermal_slowdown", nv.nvmlClocksEventReasonSwThermalSlowdown),
                     ("sw_power_cap", nv.nvmlClocksEventReasonSwPowerCap)]
            mask = 0
            for r in rows:
                mask |= r[3]
            out.update(sm_mhz=statistics.median(r[1] for r in rows), reasons=[n for n, b in names if mask & b],
                       samples=len(rows), power_w_max=max(r[2] for r in rows))
        return out


class OracleSample:
    """The fp64 oracle, as it stands, on a bounded sample of the workload: `n_units` units of
    the config at full size, one host thread per unit.  The index is built by the oracle
    itself (one Lloyd round, untimed); run(n) then times n iterations of
    decode_step + append + split_check on every sampled unit."""

    def __init__(self, cfg, n_units: int, capacity_steps: int):
        from concurrent.futures import ThreadPoolExecutor

        import oracle as O
        from gen import UnitStream

        self.cfg, self.n_units = cfg, n_units
        self.cores = min(n_units, os.cpu_count() or 1)
        self.ex = ThreadPoolExecutor(max_workers=self.cores)
        max_tokens = cfg.n_prefill + capacity_steps + 1

        def prep(u):
            s = UnitStream(cfg.scaled(steps=max(cfg.steps, capacity_steps)), u)
            K, V = s.prefill()
            o = O.OracleUnit(cfg.d, cfg.G, max_tokens, cfg.max_clusters, gamma=cfg.split_size_factor,
                             alpha=cfg.split_var_factor, split_min_size=cfg.split_min_size, split_iters=cfg.split_iters)
            o.build(K.double().numpy(), V.double().numpy(), cfg.M0, 1, 1234, unit_index=u, init_mode=O.INIT_RANDOM)
            return [o, s]

        self.items = list(self.ex.map(prep, range(n_units)))

    def run(self, steps: int) -> float:
        """Seconds taken by `steps` iterations on all sampled units (input generation untimed)."""
        cfg = self.cfg

        def gen(item):
            q, k, v = item[1].decode(steps)
            return item[0], q.double().numpy(), k.double().numpy(), v.double().numpy()

        def work(a):
            o, q, k, v = a
            for t in range(steps):
                o.decode_step(q[t], cfg.budget)
                o.append(k[t], v[t])
                o.split_check()

        args = list(self.ex.map(gen, self.items))
        t0 = time.perf_counter()
        list(self.ex.map(work, args))
        return time.perf_counter() - t0

    def steps_per_s(self, dt: float, steps: int) -> float:
        # one step of the metric covers all U units; the sample covered n_units of them
        return 1.0 / (dt / steps * (self.cfg.U / self.n_units))

    def describe(self, steps: int, dt: float) -> str:
        cfg = self.cfg
        return (f"{self.n_units} of {cfg.U} units of config {cfg.cfg_id} at full size, {steps} decode steps in {dt:.1f} s on "
                f"{self.cores} threads, scaled per unit to all {cfg.U} units; the index under the timed steps is built by "
                f"the oracle, untimed, with 1 Lloyd round instead of the config's {cfg.T} (a full-size oracle build is "
                f"about a minute per unit and round; the decode steps' cost does not depend on how converged the partition is)")


def _host_info() -> dict:
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"nproc": os.cpu_count(), "cpu_model": model}


def _cpu_baseline(cfg, target_seconds: float = 12.0) -> dict:
    n_units = min(16, os.cpu_count() or 1)
    cap = 4096
    smp = OracleSample(cfg, n_units, cap)
    probe = 8
    dt = smp.run(probe)
    steps = int(max(8, min(cap - probe - 1, target_seconds / max(dt / probe, 1e-6))))
    dt = smp.run(steps)
    out = {"value": smp.steps_per_s(dt, steps), "unit": "steps/s", "cores": smp.cores, "kind": "oracle",
           "sample": smp.describe(steps, dt), "host": _host_info()}
    # the same on ONE host thread (one unit), scaled per unit like the figure above
    one = OracleSample(cfg, 1, cap)
    dt1 = one.run(probe)
    steps1 = int(max(8, min(cap - probe - 1, 4.0 / max(dt1 / probe, 1e-6))))
    dt1 = one.run(steps1)
    out["one_thread"] = {"value": one.steps_per_s(dt1, steps1), "unit": "steps/s", "cores": 1, "sample": one.describe(steps1, dt1)}
    return out


def run_reference(args, cfg):
    """The reference arm: the oracle on the host cores.  Every step is one iteration over the
    bounded sample of units; W warm-up steps, then exactly K timed steps."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_units = min(16, os.cpu_count() or 1)
    smp = OracleSample(cfg, n_units, args.warmup + args.steps)
    if args.warmup > 0:
        smp.run(args.warmup)
    dt = smp.run(args.steps)
    value = smp.steps_per_s(dt, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 / value, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_dict(cfg, args.warmup),
        "cpu_baseline": {"value": value, "unit": "steps/s", "cores": smp.cores, "kind": "oracle",
                         "sample": smp.describe(args.steps, dt), "host": _host_info()},
        "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def config_dict(cfg, warmup: int) -> dict:
    """The `config` object of the JSON line, the same for both arms."""
    return {"workload": f"config{cfg.cfg_id}:{cfg.name}", "units_per_gpu": cfg.U, "layers": cfg.L, "kv_heads": cfg.Hkv,
            "gqa_group": cfg.G, "head_dim": cfg.d, "context": cfg.n_prefill + warmup, "clusters": cfg.M0, "budget": cfg.budget,
            "l2": "inputs_larger_than_l2"}


def rank_units(cfg, rank: int):
    """Global unit ids of one rank.  Units are independent, so the job shards with no exchange step: every rank
    owns one full replica of the configuration's unit grid, seeded by its global unit ids (weak scaling)."""
    return [rank * cfg.U + u for u in range(cfg.U)]


def max_over_ranks(value: float, device=None) -> float:
    """MAX all-reduce of a scalar over the default process group (NCCL on GPUs, gloo in the CPU tests)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_steps_per_s(world: int, steps: int, ms_max: float) -> float:
    """Aggregate over all ranks: every rank advanced its own replica by `steps` in at most `ms_max`."""
    return world * steps / (ms_max * 1e-3)


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
    n_e2e = max(0, min(args.e2e_steps, cfg.steps - W - K_steps - 64))
    n_prof = max(0, min(args.profile_steps, max(K_steps, 16), cfg.steps - W - K_steps - n_e2e))
    # the timed region of K steps is run `repeats` times on consecutive slices of the stream (the median is the
    # value); what is left of the config's decode length, up to 512 steps, goes to one long call
    room = cfg.steps - W - n_e2e - n_prof
    assert room >= K_steps, "not enough decode capacity in this config for the requested steps"
    repeats = max(1, min(args.repeats, room // K_steps))
    n_steady = max(0, min(args.steady_steps, room - repeats * K_steps))
    total_steps = W + repeats * K_steps + n_steady + n_e2e + n_prof

    # ---- synthetic inputs, generated on the device (seeded per unit and rank)
    U = cfg.U
    streams = [UnitStream(cfg, g, device=str(dev)) for g in rank_units(cfg, rank)]
    Kp, Vp = make_prefill(streams)
    q_all, k_all, v_all = make_decode_chunk(streams, total_steps)
    del streams
    torch.cuda.synchronize()

    free_before = torch.cuda.mem_get_info(dev)[0]
    ctx = P.DynaKV(P.DynaKVConfig(
        n_units=U, gqa_group=cfg.G, head_dim=cfg.d, kv_dtype={"f32": P.F32, "bf16": P.BF16, "fp8": P.FP8}[cfg.kv_dtype],
        max_tokens=cfg.max_tokens, max_clusters=cfg.max_clusters, kmeans_iters=cfg.T,
        init_mode=P.INIT_KMEANSPP if cfg.init_mode == "kmeanspp" else P.INIT_RANDOM,
        split_size_factor=cfg.split_size_factor, split_var_factor=cfg.split_var_factor,
        split_min_size=cfg.split_min_size, split_iters=cfg.split_iters, trace=0, assign_mode=args.assign_mode,
        tier=1 if args.tier > 0 else 0, cache_pages=args.tier))

    # device memory the context holds (page pool, index, scratch), from the driver's free-memory figure
    context_gb = (free_before - torch.cuda.mem_get_info(dev)[0]) / 1e9
    # ---- build (prefill indexing), timed on its own
    ctx.set_timing(True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    if args.placed > 0:
        # correlation-aware placement from the first decode queries of the stream (they are used again as decode steps)
        ctx.build_index(Kp, Vp, cfg.M0, 1234, placement_queries=q_all[:args.placed].contiguous(), placement_budget=cfg.budget)
    else:
        ctx.build_index(Kp, Vp, cfg.M0, 1234)
    e1.record(); torch.cuda.synchronize()
    build_ms = e0.elapsed_time(e1)
    kt = ctx.get_kernel_times(reset=True)
    ctx.set_timing(False)
    del Kp, Vp
    assign_ms = kt["assign"]["ms"] / max(kt["assign"]["launches"], 1)
    update_ms = kt["update"]["ms"] / max(kt["update"]["launches"], 1)
    round_ms = assign_ms + update_ms
    assign_flop = 2.0 * cfg.n_prefill * cfg.M0 * cfg.d * U
    build = {
        "context_device_gb": context_gb,
        "seconds": build_ms / 1e3, "lloyd_rounds": cfg.T,
        "assign_ms_per_round": assign_ms, "update_ms_per_round": update_ms,
        "init_ms": kt["init"]["ms"], "finalize_ms": kt["finalize"]["ms"],
        # one Lloyd round = assignment (distance GEMM, filter, exact stages, centroid sums) + centroid division
        "round_algorithmic_tflops": assign_flop / (round_ms * 1e-3) / 1e12 if round_ms > 0 else None,
        "assign_path": "fp32" if args.assign_mode == 1 else "auto",
    }
    build["roofline"] = {"bound": "tensor", "achieved": build["round_algorithmic_tflops"], "peak": peaks["bf16_tflops"],
                         "unit": "TFLOP/s", "frac": (build["round_algorithmic_tflops"] or 0) / peaks["bf16_tflops"],
                         "traffic": None, "peak_source": peaks["source"] + " burst bf16",
                         "what": "2 n M d flop of one Lloyd round / (assignment + centroid update) time of the round",
                         "assign_only_tflops": assign_flop / (assign_ms * 1e-3) / 1e12 if assign_ms > 0 else None,
                         "assign_only_frac": (assign_flop / (assign_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]) if assign_ms > 0 else None}

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
    if st0["error_bits"] & P.ST_INTERNAL:
        raise RuntimeError("a bounded wait ran out inside a kernel during warm-up (status bit INTERNAL); not timing")
    # ---- per-kernel breakdown with CUDA events around every launch (direct calls, same stream), right after the
    # warm-up, i.e. on the same stretch of the stream as a short timed run
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
    # bytes the kernel must read per attended row: K and V rows, in FP8 storage one byte per element and a scale byte each
    row_bytes = {"f32": 8 * cfg.d, "bf16": 4 * cfg.d, "fp8": 2 * cfg.d + 2}[cfg.kv_dtype]
    attn_ms_each = kt["attn"]["ms"] / max(kt["attn"]["launches"], 1)      # an event pair around every launch
    attn_ms, attn_how, tokens_per_launch = attn_ms_each, "CUDA events around every launch of %d direct-call steps" % n_prof, \
        (tok1 - tok0) / max(n_prof, 1)
    if cfg.kv_dtype != "f32" and n_prof > 0:
        # the kernel alone: 50 back-to-back ordinary launches on one selection between two events (the step's rows,
        # 267 MB in config 4, are more than twice the L2, so every launch streams from HBM)
        ctx.decode_step(q_all[pos - 1], cfg.budget, out=out_all[pos - 1])
        _, ntok_sel = ctx.get_selection()
        attn_ms = ctx.time_gather_attention(q_all[pos - 1], out_all[pos - 1], 50)
        tokens_per_launch = float(ntok_sel.sum())
        attn_how = "two CUDA events around 50 back-to-back launches on one step's selection (one untimed launch first)"
    attn_bytes = tokens_per_launch * row_bytes + 2 * U * cfg.G * cfg.d * 4
    achieved = attn_bytes / (attn_ms * 1e-3) / 1e9 if attn_ms > 0 else 0.0
    kernels = {k: (v["ms"] / v["launches"] * 1e3 if v["launches"] else None) for k, v in kt.items()
               if k in ("front", "select", "attn", "combine", "append", "split", "tier")}
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"],
                "traffic": (args.attn_traffic_bytes if args.attn_traffic_bytes is not None else
                            (NCU_ATTN_CAPTURE["dram_bytes"] * tokens_per_launch / NCU_ATTN_CAPTURE["tokens"]
                             if NCU_ATTN_CAPTURE and cfg.kv_dtype == "bf16" and cfg.d == 128 else
                             NCU_ATTN_CAPTURE_FP8["dram_bytes"] * tokens_per_launch / NCU_ATTN_CAPTURE_FP8["tokens"]
                             if NCU_ATTN_CAPTURE_FP8 and cfg.kv_dtype == "fp8" else None)),
                "kernel": "gather_attn", "us_per_launch": attn_ms * 1e3, "timed_how": attn_how,
                "us_per_launch_event_pair_each": attn_ms_each * 1e3, "algorithmic_bytes_per_launch": attn_bytes,
                "tokens_per_launch": tokens_per_launch, "frac_of_8TBs_nominal": achieved / 8000.0,
                "peak_source": peaks["source"] + " copy bandwidth", "per_kernel_us": kernels}

    st0 = ctx.get_status()
    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
    torch.cuda.synchronize()
    t_wall0 = time.perf_counter()
    ms_runs, gpu_launches = [], 0
    for r in range(repeats):
        launches0 = ctx.launch_count()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record()
        loop(pos, pos + K_steps)
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms_runs.append(max_over_ranks(e0.elapsed_time(e1), dev))
        gpu_launches = ctx.launch_count() - launches0
        pos += K_steps
    t_wall1 = time.perf_counter()
    st1 = ctx.get_status()
    ms = statistics.median(ms_runs)
    value = whole_job_steps_per_s(world, K_steps, ms)
    clock_windows = [(t_wall0, t_wall1)]
    timed_steps = repeats * K_steps

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region.  Two calls a user
    # can make: the host-array loop (inputs of all steps known: copies overlap the loop) is the e2e figure; the
    # step-synchronous call (one step per call, result on the host before the next call) is reported beside it.
    e2e = None
    if n_e2e > 1:
        n_sync = max(2, n_e2e // 2)
        n_loop = n_e2e - n_sync
        qh = q_all[pos:pos + n_e2e].cpu().pin_memory(); kh = k_all[pos:pos + n_e2e].cpu().pin_memory()
        vh = v_all[pos:pos + n_e2e].cpu().pin_memory()
        oh = torch.empty((U, cfg.G, cfg.d), dtype=torch.float32).pin_memory()
        ctx.step_host(qh[0], kh[0], vh[0], cfg.budget, oh)      # warm
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for t in range(1, n_sync):
            ctx.step_host(qh[t], kh[t], vh[t], cfg.budget, oh)
        torch.cuda.synchronize()
        dt_sync = max_over_ranks(time.perf_counter() - t0, dev)
        h2d = int(qh[0].numel() * 4 + 2 * kh[0].numel() * kh.element_size())
        d2h = int(oh.numel() * 4)
        e2e = {"value": None, "unit": "steps/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "call": "dynakv_decode_loop_host", "steps": n_loop,
               "step_synchronous": {"value": world * (n_sync - 1) / dt_sync, "unit": "steps/s", "call": "dynakv_step_host",
                                    "steps": n_sync - 1}}
        if n_loop > 0:
            ohl = torch.empty((n_loop, U, cfg.G, cfg.d), dtype=torch.float32).pin_memory()
            a = n_sync
            warm = min(2, n_loop - 1)
            if warm > 0:
                ctx.decode_loop_host(qh[a:a + warm], kh[a:a + warm], vh[a:a + warm], cfg.budget, ohl[:warm])
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            t0 = time.perf_counter()
            ctx.decode_loop_host(qh[a + warm:], kh[a + warm:], vh[a + warm:], cfg.budget, ohl[warm:])
            torch.cuda.synchronize()
            dt = max_over_ranks(time.perf_counter() - t0, dev)
            e2e["value"] = world * (n_loop - warm) / dt
            e2e["steps"] = n_loop - warm
    # ---- one more long call at the end: the iteration time far into the stream, where the drifting keys make the
    # variance rule fire more often (the start-up share of the short timed regions is visible against it too)
    steady_us = None
    if n_steady > 0:
        torch.cuda.synchronize()
        ts0 = time.perf_counter()
        e0.record()
        loop(pos, pos + n_steady)
        e1.record()
        torch.cuda.synchronize()
        clock_windows.append((ts0, time.perf_counter()))
        steady_us = max_over_ranks(e0.elapsed_time(e1), dev) * 1e3 / n_steady
        pos += n_steady
    # clocks sampled while the graph loop ran: the timed repeats and the long call above
    clocks = sampler.stop(clock_windows) if sampler else None
    if clocks is not None:
        clocks["sampled_during"] = "the timed repeats and the steady run of the same loop"
    status = ctx.get_status()
    # access contiguity of the last step's gather list (rows read per run of consecutive pages of the pool)
    from paper_2511_07427_b200.placement import mean_contiguous_rows
    # (two-tier runs: the list names cache frames, whose order says nothing about the pool's)
    contiguous_rows = None if args.tier > 0 else mean_contiguous_rows(*ctx.get_work_list())
    tier = None
    if args.tier > 0:
        tier = ctx.get_tier_stats()
        tier["cache_pages_per_unit"] = args.tier
        tier["pool_pages_per_unit_in_use"] = status["pages_in_use"] / U
        n_decode = max(pos, 1)
        tier["pages_fetched_per_step"] = tier["pages_fetched"] / n_decode
        # K and V rows that travelled (of a page only the rows that hold entries; in FP8 storage also the 64 scale
        # exponents of every page touched)
        row_bytes = 2 * cfg.d * {"f32": 4, "bf16": 2, "fp8": 1}[cfg.kv_dtype]
        moved = tier["rows_fetched"] * row_bytes + (tier["pages_fetched"] * 64 if cfg.kv_dtype == "fp8" else 0)
        tier["host_to_device_mb_per_step"] = moved / n_decode / 1e6
        tier["rows_fetched_per_step"] = tier["rows_fetched"] / n_decode
        looked_up = tier["clusters_hit"] + tier["clusters_refreshed"] + tier["clusters_fetched"]
        tier["cluster_hit_rate"] = (tier["clusters_hit"] + tier["clusters_refreshed"]) / max(looked_up, 1)
    ctx.destroy()

    if rank == 0:
        cpu_baseline = None
        if world == 1 and not args.no_cpu_baseline:
            cpu_baseline = _cpu_baseline(cfg)
        line = {
            "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": K_steps, "warmup": W,
            "ms_per_step": ms / K_steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {"f32": "f32", "bf16": "bf16 KV / f32 math", "fp8": "fp8 (e4m3, scale per row) KV / f32 math"}[cfg.kv_dtype],
            "data": "synthetic",
            "config": config_dict(cfg, W),
            "e2e": e2e, "gpu_launches": int(gpu_launches), "clocks": clocks, "roofline": roofline,
            "cpu_baseline": cpu_baseline, "build": build,
            "timing": {"repeats": repeats, "ms_per_repeat": ms_runs, "value_is": "median of the repeats",
                       "steady_us_per_iteration": steady_us, "steady_steps": n_steady,
                       "loop": "cuda_graph_replay(decode_step,append,split_check)"},
            "counters": {"splits_in_timed_region": st1["n_splits"] - st0["n_splits"],
                         "tokens_attended_per_step": (st1["tokens_attended_total"] - st0["tokens_attended_total"]) / timed_steps,
                         "clusters_selected_per_step": (st1["clusters_selected_total"] - st0["clusters_selected_total"]) / timed_steps,
                         "status_bits": status["error_bits"], "assign_rechecked": status["assign_rechecked"],
                         "mean_contiguous_rows_per_stretch": contiguous_rows, "placement_queries": args.placed},
        }
        if tier is not None:
            line["tier"] = tier
            line["config"]["two_tier_cache_pages"] = args.tier
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--repeats", type=int, default=5, help="timed regions of --steps steps each; the median is reported")
    ap.add_argument("--steady-steps", type=int, default=256, help="one more long call after the repeats (start-up share visible)")
    ap.add_argument("--warmup", type=int, default=16)
    ap.add_argument("--config", type=int, default=4)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--assign-mode", type=int, default=0)
    ap.add_argument("--kv", default="", choices=["", "fp8"], help="fp8: the config's bf16 K/V rows kept in FP8 storage")
    ap.add_argument("--placed", type=int, default=0,
                    help="build with correlation-aware placement from this many reference queries (0: clusters in id order)")
    ap.add_argument("--tier", type=int, default=0,
                    help="two-tier mode: the page pool in pinned host memory and this many 32-token page frames per unit in HBM")
    ap.add_argument("--e2e-steps", type=int, default=272,
                    help="steps of the end-to-end legs: half one step per call, half one host-array loop call (as long as a default timed region)")
    ap.add_argument("--profile-steps", type=int, default=64)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--budget", type=int, default=0, help="override the config's token budget (tuning aid)")
    ap.add_argument("--units", type=int, default=0,
                    help="run only the first N units of the config (profiling aid: smaller device footprint); 0 = all")
    ap.add_argument("--attn-traffic-bytes", type=float, default=None,
                    help="ncu dram bytes per launch of the gather-attention kernel (from profiles/), echoed in roofline.traffic")
    args = ap.parse_args()
    from gen import CONFIGS
    cfg = CONFIGS[args.config]
    if args.units > 0:
        # keep the per-unit shape; B*L*Hkv collapses to N units of one layer
        cfg = cfg.scaled(B=1, L=1, Hkv=args.units, Hq=args.units * cfg.G, name=cfg.name + f"[first {args.units} units]")
    if args.budget > 0:
        cfg = cfg.scaled(budget=args.budget, name=cfg.name + f"[budget {args.budget}]")
    if args.kv == "fp8":
        assert cfg.kv_dtype == "bf16" and cfg.d == 128, "FP8 storage is for the bf16 configurations with d = 128"
        cfg = cfg.scaled(kv_dtype="fp8", name=cfg.name + "[fp8 K/V]")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
