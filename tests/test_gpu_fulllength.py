"""Configs 2 to 5 over their WHOLE decode length (4096 / 32768 / 2048 / 4096 steps) through the CUDA-graph decode
loop, all units, in the launch configuration the benchmark times.  The stream is fed in chunks; after every chunk

  * a few sampled units are followed by the fp64 oracle step by step with NO hints: the attention output of
    every step is compared (a wrong selection, append target or split shows there at once), and the exported
    membership, sizes, representatives and M2 are compared exactly / within tolerance;
  * for EVERY unit Eq. 3 / Eq. 4 are checked on the exported state (membership counts, member means, M2);
  * the status word must show no capacity or internal bit.

These runs take minutes (the oracle is a scalar fp64 program), so they carry the `slow` marker and run only with
DYNAKV_RUN_SLOW=1.  Each run appends a one-line summary per checkpoint to fulllength.jsonl in the log folder
(parity_harness.LOG_DIR)."""
import json
import os
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import paper_2511_07427_b200 as P
from gen import CONFIGS, UnitStream, make_decode_chunk, make_prefill
from parity_harness import (TOL_OUT_ABS, TOL_OUT_L2, ParityReport, check_every_unit, check_state, make_ctx,
                            make_oracle, rel_l2, stored, fp8_round_rows, LOG_DIR)

pytestmark = [pytest.mark.gpu, pytest.mark.slow]

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _log(rec):
    folder = LOG_DIR
    print(json.dumps(rec), flush=True)
    if os.path.isdir(folder):
        with open(os.path.join(folder, "fulllength.jsonl"), "a") as f:
            f.write(json.dumps(rec) + "\n")


# (the last case is config 4 with its rows in FP8 storage: the oracle is handed the rows as the library keeps them)
@pytest.mark.parametrize("cid,sampled,chunk,kv", [(2, [0, 77, 255], 512, ""), (4, [0, 101, 255], 256, ""), (5, [0, 900, 1791], 512, ""),
                                                  (3, [0, 130, 255], 4096, ""), (4, [3, 128, 250], 256, "fp8")])
def test_whole_decode_length(cid, sampled, chunk, kv):
    cfg = CONFIGS[cid] if not kv else CONFIGS[cid].scaled(kv_dtype=kv)
    rows = lambda x: stored(x.cpu(), cfg)
    as_kept = lambda X: X if kv != "fp8" else torch.cat([fp8_round_rows(X[i:i + 32]).to(X.dtype) for i in range(0, X.shape[0], 32)])
    U, n0 = cfg.U, cfg.n_prefill
    steps_total = int(os.environ.get("DYNAKV_FULL_STEPS", cfg.steps))
    side = torch.cuda.Stream()
    pool = ThreadPoolExecutor(max_workers=len(sampled))
    with torch.cuda.stream(side):
        streams = [UnitStream(cfg, u, device="cuda") for u in range(U)]
        K, V = make_prefill(streams)
        ctx = make_ctx(cfg, U, trace=0, assign_mode=0)
        t_b = time.perf_counter()
        ctx.build_index(K, V, cfg.M0, 1234)
        side.synchronize()
        st = ctx.export_state()
        rep = ParityReport()
        oracles = {}
        for u in sampled:
            o = make_oracle(cfg)
            o.install(rows(K[u]), rows(V[u]), st["tok_cluster"][u, :n0], int(st["n_ids"][u]))
            check_state(o, st, u, rep, f"build unit {u}")
            oracles[u] = o
        K_all = torch.empty((U, n0 + steps_total, cfg.d), dtype=K.dtype, device="cuda")
        K_all[:, :n0] = as_kept(K)
        del K, V
        done, worst_abs, worst_l2 = 0, 0.0, 0.0
        gpu_ms = 0.0
        while done < steps_total:
            nb = min(chunk, steps_total - done)
            q, k, v = make_decode_chunk(streams, nb)
            K_all[:, n0 + done: n0 + done + nb] = as_kept(k.transpose(0, 1).contiguous())
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            outs = ctx.decode_loop(q, k, v, cfg.budget)
            e1.record()
            side.synchronize()
            gpu_ms += e0.elapsed_time(e1)
            st = ctx.export_state()
            status = ctx.get_status()
            outs_s = {u: outs[:, u].cpu().numpy().astype(np.float64) for u in sampled}
            qs = {u: q[:, u].double().cpu().numpy() for u in sampled}
            ks = {u: rows(k[:, u]) for u in sampled}
            vs = {u: rows(v[:, u]) for u in sampled}
            del outs, q, k, v

            def follow(u):
                o = oracles[u]
                wa, wl = 0.0, 0.0
                for t in range(nb):
                    out_o, _, _ = o.decode_step(qs[u][t], cfg.budget)
                    ea, el = float(np.abs(outs_s[u][t] - out_o).max()), rel_l2(outs_s[u][t], out_o)
                    assert ea <= TOL_OUT_ABS and el <= TOL_OUT_L2, \
                        f"config {cid} step {done + t} unit {u}: attention abs {ea:.3e} relL2 {el:.3e}"
                    wa, wl = max(wa, ea), max(wl, el)
                    o.append(ks[u][t], vs[u][t])
                    o.split_check()
                return wa, wl

            t_o = time.perf_counter()
            for wa, wl in pool.map(follow, sampled):
                worst_abs, worst_l2 = max(worst_abs, wa), max(worst_l2, wl)
            t_o = time.perf_counter() - t_o
            done += nb
            for u in sampled:
                check_state(oracles[u], st, u, rep, f"config {cid} after step {done} unit {u}")
            inv = check_every_unit(cfg, st, K_all, n0 + done)
            bits = status["error_bits"]
            assert bits & (P.ST_INTERNAL | P.ST_PAGE_POOL | P.ST_MAX_TOKENS) == 0, f"status bits {bits}"
            _log({"config": cid, "steps_done": done, "of": steps_total, "status_bits": bits, "splits": status["n_splits"],
                  "live_clusters_all_units": inv["live_clusters"], "ids_max": inv["ids_max"], "ids_min": inv["ids_min"],
                  "pages_in_use": status["pages_in_use"], "tokens_selected": status["tokens_selected"],
                  "centroid_rel": inv["centroid_rel"], "M2_rel": inv["M2_rel"], "out_max_abs": worst_abs, "out_max_relL2": worst_l2,
                  "oracle_splits_sampled": [int(oracles[u].n_splits) for u in sampled], "gpu_loop_ms_total": gpu_ms,
                  "oracle_seconds_chunk": t_o, "max_centroid_rel_sampled": rep.max_centroid_rel})
        status = ctx.get_status()
        assert status["n_splits"] > 0
        # every unit has split at least once beyond the ids of the build
        assert inv["ids_min"] > cfg.M0 or steps_total < cfg.steps
        ctx.destroy()
