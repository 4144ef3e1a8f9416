"""Cluster quality of the three update modes on a drifting stream: mean intra-cluster variance and the share of
the dense attention mass that the budgeted retrieval keeps.

    python -m paper_2511_07427_b200.mode_report [--config 3] [--steps 8192] [--units 64] [--every 2048]

For every mode (adaptive = the paper's append + split rule, static = append only, local = new entries clustered
among themselves; arXiv 2511.07427 Section 3.1 and the baselines of Section 8.1; with --buf-max also the delayed split
of Algorithm 1, which defers a triggered cluster's split until a query retrieves it) the same seeded stream is run
through the library's CUDA-graph decode loop.  At every checkpoint the exported state gives

  * the mean over live clusters of sigma_j^2 = M2_j / n_j (the scalar the paper's variance table reports per
    cluster), and the same weighted by cluster size;
  * the number of live clusters per unit;

and one more retrieval with the checkpoint's query gives, against plain softmax attention over ALL tokens of the
unit (computed here with torch, no library code),

  * recall = attention mass of the selected clusters' tokens, averaged over units and query heads;
  * the relative L2 distance between the retrieval's output and the dense output.

Prints one JSON line per (mode, checkpoint) and a table.  Everything runs on the GPU; the oracle is not used."""
from __future__ import annotations

import argparse
import json
import math
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import paper_2511_07427_b200 as P  # noqa: E402
from gen import CONFIGS, UnitStream, make_decode_chunk, make_prefill  # noqa: E402


def run_mode(cfg, mode: str, local_max: int, units: int, steps: int, every: int):
    # (for the delayed-split mode the second argument is buf_max)
    name = f"local(max {local_max})" if mode == "local" else f"delayed(B {local_max})" if mode == "delayed" else mode
    side = torch.cuda.Stream()
    rows = []
    with torch.cuda.stream(side):
        streams = [UnitStream(cfg, u, device="cuda") for u in range(units)]
        K, V = make_prefill(streams)
        n0 = cfg.n_prefill
        ctx = P.DynaKV(P.DynaKVConfig(
            n_units=units, gqa_group=cfg.G, head_dim=cfg.d, kv_dtype=P.BF16, max_tokens=n0 + steps, max_clusters=cfg.max_clusters,
            kmeans_iters=cfg.T, init_mode=P.INIT_RANDOM, split_size_factor=cfg.split_size_factor,
            split_var_factor=cfg.split_var_factor, split_min_size=cfg.split_min_size, split_iters=cfg.split_iters,
            update_mode={"adaptive": P.MODE_ADAPTIVE, "static": P.MODE_STATIC, "local": P.MODE_LOCAL,
                         "delayed": P.MODE_DELAYED}[mode], local_max=local_max, buf_max=local_max))
        ctx.build_index(K, V, cfg.M0, 1234)
        K_all = torch.empty((units, n0 + steps, cfg.d), dtype=K.dtype, device="cuda")
        V_all = torch.empty_like(K_all)
        K_all[:, :n0], V_all[:, :n0] = K, V
        sel = torch.full((units, cfg.max_clusters), -1, dtype=torch.int32, device="cuda")
        done, loop_ms = 0, 0.0
        while done < steps:
            nb = min(every, steps - done)
            q, k, v = make_decode_chunk(streams, nb)
            K_all[:, n0 + done: n0 + done + nb] = k.transpose(0, 1)
            V_all[:, n0 + done: n0 + done + nb] = v.transpose(0, 1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.decode_loop(q, k, v, cfg.budget)
            e1.record()
            side.synchronize()
            loop_ms += e0.elapsed_time(e1)
            done += nb
            nt = n0 + done
            st = ctx.export_state()
            cnt = st["counts"].astype(np.float64)
            live = cnt > 0
            var = np.where(live, st["M2"].astype(np.float64) / np.maximum(cnt, 1), 0.0)
            # one more retrieval on this state with the chunk's last query, against dense attention
            qx = q[-1]
            out = ctx.decode_step(qx, cfg.budget, selected_ids=sel)
            side.synchronize()
            _, ntok = ctx.get_selection()
            tokc = torch.from_numpy(st["tok_cluster"][:, :nt].astype(np.int64)).cuda()
            selmask = torch.zeros((units, cfg.max_clusters + 1), dtype=torch.bool, device="cuda")
            selmask.scatter_(1, torch.where(sel >= 0, sel.long(), torch.full_like(sel, cfg.max_clusters).long()), True)
            recall, rel = [], []
            for u0 in range(0, units, 16):
                u1 = min(units, u0 + 16)
                lg = torch.einsum("ugd,utd->ugt", qx[u0:u1].float(), K_all[u0:u1, :nt].float()) / math.sqrt(cfg.d)
                p = torch.softmax(lg, dim=2)
                tm = selmask[u0:u1, :cfg.max_clusters].gather(1, tokc[u0:u1])                 # token retrieved?
                recall.append((p * tm[:, None, :]).sum(2))
                dense = torch.einsum("ugt,utd->ugd", p, V_all[u0:u1, :nt].float())
                rel.append((out[u0:u1] - dense).flatten(1).norm(dim=1) / dense.flatten(1).norm(dim=1))
            recall, rel = torch.cat(recall), torch.cat(rel)
            row = {"mode": name, "steps": done, "tokens_per_unit": nt, "live_clusters_per_unit": float(live.sum() / units),
                   "mean_cluster_variance": float(var[live].mean()),
                   "size_weighted_variance": float(st["M2"].astype(np.float64)[live].sum() / cnt[live].sum()),
                   "attention_mass_recall": float(recall.mean()), "recall_min_over_units": float(recall.mean(1).min()),
                   "rel_l2_to_dense": float(rel.mean()), "tokens_retrieved_per_unit": float(ntok.mean()),
                   "splits": int(ctx.get_status()["n_splits"]), "status_bits": int(ctx.get_status()["error_bits"]),
                   "loop_us_per_step": loop_ms * 1e3 / done}
            print(json.dumps(row), flush=True)
            rows.append(row)
        ctx.destroy()
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--steps", type=int, default=8192)
    ap.add_argument("--units", type=int, default=64)
    ap.add_argument("--every", type=int, default=2048)
    ap.add_argument("--local-max", type=int, nargs="*", default=[64, 512])
    ap.add_argument("--buf-max", type=int, nargs="*", default=[], help="also run the delayed-split mode with these buffer limits")
    args = ap.parse_args()
    cfg = CONFIGS[args.config]
    runs = [("adaptive", 0), ("static", 0)] + [("local", m) for m in args.local_max] + [("delayed", b) for b in args.buf_max]
    table = []
    for mode, lm in runs:
        table += run_mode(cfg, mode, max(lm, 2), args.units, args.steps, args.every)
    print(f"\n{'mode':16s} {'steps':>6s} {'clusters':>9s} {'variance':>9s} {'wtd var':>9s} {'recall':>7s} {'relL2':>7s} {'us/step':>8s} {'splits':>7s}")
    for r in table:
        print(f"{r['mode']:16s} {r['steps']:6d} {r['live_clusters_per_unit']:9.1f} {r['mean_cluster_variance']:9.2f} "
              f"{r['size_weighted_variance']:9.2f} {r['attention_mass_recall']:7.4f} {r['rel_l2_to_dense']:7.4f} "
              f"{r['loop_us_per_step']:8.1f} {r['splits']:7d}")


if __name__ == "__main__":
    main()
