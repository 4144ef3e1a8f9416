"""World-size-2 checks of the multi-rank host logic of bench.py on CPU (gloo): unit sharding with no exchange
step, max-over-ranks timing, whole-job aggregation, and the reference arm's rank-0-only rule."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from gen import CONFIGS, UnitStream
    cfg = CONFIGS[2].scaled(B=1, L=2, Hkv=2, Hq=8, n_prefill=64, steps=4)
    units = bench.rank_units(cfg, rank)
    # every rank's first prefill block, to show that different ranks hold different data
    k0, _ = UnitStream(cfg, units[0]).prefill()
    ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    ms_max = bench.max_over_ranks(ms)
    gathered = [None] * world
    dist.all_gather_object(gathered, {"units": units, "k0": float(k0.float().sum())})
    if rank == 0:
        out.put({"ms_max": ms_max, "gathered": gathered, "value": bench.whole_job_steps_per_s(world, 100, ms_max)})
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_units_and_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    a, b = res["gathered"][0]["units"], res["gathered"][1]["units"]
    assert len(a) == len(b) == 4 and not set(a) & set(b) and sorted(a + b) == list(range(8))   # disjoint, complete
    assert res["gathered"][0]["k0"] != res["gathered"][1]["k0"]
    assert res["ms_max"] == 15.0                                  # the slowest rank sets the time
    assert abs(res["value"] - 2 * 100 / 0.015) < 1e-6             # whole-job aggregate over both ranks


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
                        "--warmup", "1", "--config", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""           # other ranks exit 0 without work
    env["RANK"] = "0"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "2",
                        "--warmup", "1", "--config", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["n_gpus"] == 2
