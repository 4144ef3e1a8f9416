"""Lock-step parity driver: runs the CUDA library and the fp64 oracle on the same seeded
inputs, call by call, and compares them under the tie-follow protocol.

Protocol.  Every discrete decision the GPU takes (initial centres, every Lloyd round's
assignment, the selected cluster list, the append target, the split partition) is read
back and offered to the oracle as a *hint*.  The oracle computes its own answer first;
it follows the hint only if its own fp64 numbers put the two candidates within 1e-5
relative of each other (a logged tie), otherwise it keeps its answer, counts a violation,
and the comparison that follows fails.  Compared after each call: cluster membership and
ids (exact), selected lists (exact), centroids (<= 1e-4 relative per vector), attention
output (max abs <= 2e-3, relative L2 <= 1e-3).
"""
from __future__ import annotations

import os
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle as O
from oracle.cluster_cache import ClusterCacheModel
import paper_2511_07427_b200 as P
from gen import UnitStream, WorkloadConfig, make_decode_chunk, make_prefill

TOL_TIE = 1e-5
TOL_CENTROID = 1e-4
TOL_OUT_ABS = 2e-3
TOL_OUT_L2 = 1e-3


@dataclass
class ParityReport:
    ties: int = 0
    violations: int = 0
    steps: int = 0
    splits: int = 0
    max_out_abs: float = 0.0
    max_out_l2: float = 0.0
    max_centroid_rel: float = 0.0
    tokens_selected: List[int] = field(default_factory=list)
    status_bits: int = 0
    rechecked: int = 0
    gpu_splits: int = 0
    tier_stats: Optional[dict] = None     # two-tier runs: the library's cache counters and the model's
    tier_model: Optional[dict] = None
    decisions: int = 0          # discrete decisions offered to the oracle as hints (assignments, selections, appends, checks)


# where test runs leave their one-line summaries: a folder at the repository root, overridable by the environment
LOG_DIR = os.environ.get("DYNAKV_LOG_DIR",
                         os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "gpurun_out"))


def tie_bound(rep: "ParityReport") -> int:
    """Most followed ties a run may show: two, plus one per 10 000 decisions.  A tie needs two candidates within
    1e-5 relative in the oracle's fp64 numbers; on continuous random data that is rare, so a count above this bound
    means the library leans on the tie rule instead of deciding correctly."""
    return 2 + rep.decisions // 10000


def log_ties(name: str, rep: "ParityReport") -> None:
    """Append one JSON line per parity run to parity_ties.jsonl in the run's log folder (LOG_DIR below, when that
    folder exists), so the tie counts of a test session can be read afterwards."""
    import json
    import os
    folder = LOG_DIR
    if os.path.isdir(folder):
        with open(os.path.join(folder, "parity_ties.jsonl"), "a") as f:
            f.write(json.dumps({"run": name, "ties": rep.ties, "violations": rep.violations, "decisions": rep.decisions,
                                "bound": tie_bound(rep), "steps": rep.steps, "splits": rep.splits}) + "\n")


def make_ctx(cfg: WorkloadConfig, n_units: int, trace: int = 1, assign_mode: int = 0, attn_mode: int = 0,
             det_sums: int = 0, cache_pages: int = 0) -> P.DynaKV:
    return P.DynaKV(P.DynaKVConfig(
        n_units=n_units, gqa_group=cfg.G, head_dim=cfg.d,
        kv_dtype={"f32": P.F32, "bf16": P.BF16, "fp8": P.FP8}[cfg.kv_dtype],
        max_tokens=cfg.max_tokens, max_clusters=cfg.max_clusters, kmeans_iters=cfg.T,
        init_mode=P.INIT_KMEANSPP if cfg.init_mode == "kmeanspp" else P.INIT_RANDOM,
        split_size_factor=cfg.split_size_factor, split_var_factor=cfg.split_var_factor,
        split_min_size=cfg.split_min_size, split_iters=cfg.split_iters, trace=trace, assign_mode=assign_mode, attn_mode=attn_mode,
        update_mode={"adaptive": P.MODE_ADAPTIVE, "static": P.MODE_STATIC, "local": P.MODE_LOCAL,
                     "delayed": P.MODE_DELAYED}[cfg.update_mode],
        local_max=cfg.local_max, det_sums=det_sums, buf_max=cfg.buf_max,
        tier=1 if cache_pages > 0 else 0, cache_pages=cache_pages))


def fp8_round_rows(x: "torch.Tensor") -> "torch.Tensor":
    """Rows of x (last axis) as the FP8 storage mode keeps them: e4m3 elements (round to nearest even, largest finite
    value 448) times one power-of-two scale per row, 2^e with e the smallest integer that brings the row's largest
    magnitude to at most 448 (0 for a zero row).  Returned as float64.  The byte conversion is torch's own
    float8_e4m3fn cast; only the scale rule is written out here."""
    xf = x.to(torch.float64)
    amax = xf.abs().amax(dim=-1, keepdim=True)
    safe = torch.where(amax > 0, amax, torch.ones_like(amax))
    e = torch.floor(torch.log2(safe)) - 8                    # 2^8 <= amax / 2^e < 2^9 up to log2's rounding ...
    e = torch.where(safe / torch.exp2(e) > 448.0, e + 1, e)   # ... settled by testing the bound itself
    e = torch.where(safe / torch.exp2(e - 1) <= 448.0, e - 1, e)
    e = torch.where(amax > 0, e.clamp(-120, 120), torch.zeros_like(e))
    scale = torch.exp2(e)
    return (xf / scale).to(torch.float32).to(torch.float8_e4m3fn).to(torch.float64) * scale


def stored(x: "torch.Tensor", cfg: WorkloadConfig) -> np.ndarray:
    """The values the library keeps for rows x under cfg's storage type, as float64 (what the oracle is given)."""
    return (fp8_round_rows(x) if cfg.kv_dtype == "fp8" else x.double()).numpy()


def make_oracle(cfg: WorkloadConfig) -> O.OracleUnit:
    return O.OracleUnit(cfg.d, cfg.G, cfg.max_tokens, cfg.max_clusters,
                        gamma=float(np.float32(cfg.split_size_factor)), alpha=float(np.float32(cfg.split_var_factor)),
                        split_min_size=cfg.split_min_size, split_iters=cfg.split_iters, tol=TOL_TIE,
                        mode={"adaptive": O.MODE_ADAPTIVE, "static": O.MODE_STATIC, "local": O.MODE_LOCAL,
                              "delayed": O.MODE_DELAYED}[cfg.update_mode],
                        local_max=cfg.local_max, buf_max=cfg.buf_max)


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / den if den > 0 else float(np.linalg.norm(a))


def check_state(o: O.OracleUnit, st: dict, ui: int, rep: ParityReport, where: str) -> None:
    n, M = o.n, o.M
    assert int(st["n_tokens"][ui]) == n, f"{where}: token count {st['n_tokens'][ui]} vs oracle {n}"
    assert int(st["n_ids"][ui]) == M, f"{where}: ids in use {st['n_ids'][ui]} vs oracle {M}"
    a_gpu = st["tok_cluster"][ui, :n]
    a_or = o.assign()
    bad = np.nonzero(a_gpu != a_or)[0]
    assert bad.size == 0, f"{where}: membership differs at tokens {bad[:8]} gpu {a_gpu[bad[:8]]} oracle {a_or[bad[:8]]}"
    cnt = o.counts()
    assert np.array_equal(st["counts"][ui, :M], cnt), f"{where}: cluster sizes differ"
    Cg, Co = st["centroids"][ui, :M].astype(np.float64), o.centroids()
    live = cnt > 0
    if live.any():
        num = np.linalg.norm(Cg[live] - Co[live], axis=1)
        den = np.maximum(np.linalg.norm(Co[live], axis=1), 1e-30)
        r = float((num / den).max())
        rep.max_centroid_rel = max(rep.max_centroid_rel, r)
        assert r <= TOL_CENTROID, f"{where}: centroid relative error {r:.3e}"
        m2g, m2o = st["M2"][ui, :M].astype(np.float64)[live], o.M2()[live]
        # floor: fp32 rounding of the centroid itself leaves about n * |c|^2 * 2^-46 in M2 even when the members coincide
        floor = 1e-6 * cnt[live] * (np.linalg.norm(Co[live], axis=1) ** 2)
        scale = np.maximum(np.maximum(m2o, 1e-3 * float(m2o.max())), np.maximum(floor, 1e-30))
        assert float((np.abs(m2g - m2o) / scale).max()) <= 1e-3, f"{where}: M2 differs"


def run_parity(cfg: WorkloadConfig, units: Sequence[int], steps: int, *, assign_mode: int = 0,
               state_every: int = 1, budget: Optional[int] = None, ctx_units: Optional[Sequence[int]] = None,
               seed: int = 1234, device: str = "cuda", check_every: int = 1, attn_mode: int = 0,
               det_sums: int = 0, placement_queries: int = 0, cache_pages: int = 0) -> ParityReport:
    """Run `steps` decode iterations of `cfg`.  The GPU context holds `ctx_units` (default:
    `units`); the oracle follows the units listed in `units` (a subset of ctx_units).  With check_every > 1 the
    split check is called only after every check_every-th append (on both sides).  With cache_pages > 0 the context
    runs in its two-tier mode with that many page frames per unit, every unit is watched, and the library's cache
    counters must equal those of the oracle's cache model fed with the oracle's own selections, sizes and splits."""
    rep = ParityReport()
    ctx_units = list(ctx_units) if ctx_units is not None else list(units)
    pos = {u: i for i, u in enumerate(ctx_units)}
    watch = [pos[u] for u in units]
    budget = cfg.budget if budget is None else budget
    streams = [UnitStream(cfg, u) for u in ctx_units]
    K, V = make_prefill(streams)
    ctx = make_ctx(cfg, len(ctx_units), trace=1, assign_mode=assign_mode, attn_mode=attn_mode, det_sums=det_sums,
                   cache_pages=cache_pages)
    caches = {}
    if cache_pages > 0:
        assert len(watch) == len(ctx_units), "the cache counters are summed over the context's units: watch them all"
        caches = {ui: ClusterCacheModel(cache_pages) for ui in watch}
    if placement_queries > 0:
        # the build with correlation-aware placement: the pages' order in the pool changes, nothing else may
        g = torch.Generator().manual_seed(99)
        q_ref = torch.randn((placement_queries, len(ctx_units), cfg.G, cfg.d), generator=g).to(device)
        ctx.build_index(K.to(device), V.to(device), cfg.M0, seed, placement_queries=q_ref, placement_budget=budget)
    else:
        ctx.build_index(K.to(device), V.to(device), cfg.M0, seed)
    picks, trace = ctx.get_build_trace()
    st = ctx.export_state()
    oracles = {}
    for ui in watch:
        o = make_oracle(cfg)
        o.build(stored(K[ui], cfg), stored(V[ui], cfg), cfg.M0, cfg.T, seed, unit_index=ui,
                init_mode=O.INIT_KMEANSPP if cfg.init_mode == "kmeanspp" else O.INIT_RANDOM,
                hint_picks=picks[ui] if cfg.init_mode == "kmeanspp" else None, hint_assign=trace[:, ui, :])
        assert o.violations == 0, f"build unit {ui}: {o.violations} decisions differ beyond the tie tolerance"
        check_state(o, st, ui, rep, f"build unit {ui}")
        tau_g, tau_o = float(st["tau"][ui]), o.tau
        assert abs(tau_g - tau_o) <= 1e-4 * abs(tau_o) + 1e-30, f"tau {tau_g} vs {tau_o}"
        oracles[ui] = o
    sel = torch.full((len(ctx_units), cfg.max_clusters), -1, dtype=torch.int32, device=device)
    done = 0
    while done < steps:
        nb = min(64, steps - done)
        q, k, v = make_decode_chunk(streams, nb)
        qd, kd, vd = q.to(device), k.to(device), v.to(device)
        for t in range(nb):
            out = ctx.decode_step(qd[t], budget, selected_ids=sel)
            out_np = out.cpu().numpy().astype(np.float64)
            sel_np = sel.cpu().numpy()
            nsel, ntok = ctx.get_selection()
            for ui in watch:
                o = oracles[ui]
                ids_gpu = sel_np[ui][: nsel[ui]]
                assert np.all(sel_np[ui][nsel[ui]:] == -1)
                v0 = o.violations
                out_o, ids_o, tok_o = o.decode_step(q[t, ui].double().numpy(), budget, hint_ids=ids_gpu)
                assert o.violations == v0 and list(ids_o) == list(ids_gpu), \
                    f"step {done + t} unit {ui}: selection differs: gpu {ids_gpu[:12]} oracle {ids_o[:12]}"
                assert tok_o == int(ntok[ui])
                if caches:
                    caches[ui].retrieve(ids_o, o.counts())
                rep.tokens_selected.append(tok_o)
                ea = float(np.abs(out_np[ui] - out_o).max()); el = rel_l2(out_np[ui], out_o)
                rep.max_out_abs = max(rep.max_out_abs, ea); rep.max_out_l2 = max(rep.max_out_l2, el)
                assert ea <= TOL_OUT_ABS and el <= TOL_OUT_L2, \
                    f"step {done + t} unit {ui}: attention error abs {ea:.3e} relL2 {el:.3e}"
            ctx.append(kd[t], vd[t])
            st = ctx.export_state()
            for ui in watch:
                o = oracles[ui]
                n0 = o.n
                v0 = o.violations
                j = o.append(stored(k[t, ui], cfg), stored(v[t, ui], cfg),
                             hint_cluster=int(st["tok_cluster"][ui, n0]))
                assert o.violations == v0 and j == int(st["tok_cluster"][ui, n0]), \
                    f"step {done + t} unit {ui}: append target gpu {st['tok_cluster'][ui, n0]} oracle {j}"
            if (done + t + 1) % check_every != 0:
                continue
            ctx.split_check()
            st = ctx.export_state()
            for ui in watch:
                o = oracles[ui]
                v0 = o.violations
                sizes_before = o.counts().copy()
                o.split_check(hint_assign_after=st["tok_cluster"][ui, : o.n])
                if caches:
                    for j in np.nonzero(o.counts()[: len(sizes_before)] < sizes_before)[0]:      # a cluster that lost entries was split
                        caches[ui].note_split(int(j))
                assert o.violations == v0, f"step {done + t} unit {ui}: split decisions differ beyond the tie tolerance"
                if (done + t) % state_every == 0 or done + t == steps - 1:
                    check_state(o, st, ui, rep, f"step {done + t} unit {ui}")
                else:
                    assert np.array_equal(st["tok_cluster"][ui, : o.n], o.assign()), f"step {done + t} unit {ui}: membership"
        done += nb
    status = ctx.get_status()
    # (only a library built with its index tests can set this bit; see tests/test_gpu_checked.py)
    assert status["error_bits"] & P.ST_BOUNDS == 0, f"an index test failed inside a kernel, site {status['bounds_site']}"
    rep.steps = steps
    n_checks = steps // check_every
    rep.decisions = len(watch) * (cfg.n_prefill * cfg.T + (cfg.M0 if cfg.init_mode == "kmeanspp" else 0) + 2 * steps + n_checks)
    rep.status_bits = status["error_bits"]
    rep.rechecked = status["assign_rechecked"]
    for ui in watch:
        o = oracles[ui]
        rep.ties += o.ties; rep.violations += o.violations; rep.splits += o.n_splits
    rep.gpu_splits = status["n_splits"]
    if caches:
        rep.tier_stats = ctx.get_tier_stats()
        rep.tier_model = {k: sum(m.c[k] for m in caches.values()) for k in next(iter(caches.values())).c}
        rep.tier_model["frames_in_use"] = sum(m.frames_in_use for m in caches.values())
        for k, v in rep.tier_model.items():
            assert rep.tier_stats[k] == v, f"cache counter {k}: library {rep.tier_stats[k]}, model {v}\n{rep.tier_stats}\n{rep.tier_model}"
    ctx.destroy()
    return rep


def check_every_unit(cfg: WorkloadConfig, st: dict, K_all: "torch.Tensor", nt: int) -> dict:
    """Eq. 3 and Eq. 4 on an exported state, for EVERY unit: every token in exactly one live cluster id below the
    unit's id count, sizes equal to the membership counts, representatives equal to the member means, M2 equal to
    the members' squared distances to their mean.  K_all: [U, >= nt, d] keys in token-id order on the GPU (plain
    torch in fp64; no library code).  Returns the worst relative deviations seen."""
    U, Mx, d = K_all.shape[0], cfg.max_clusters, cfg.d
    assert np.all(st["n_tokens"] == nt), "token counts"
    tokc = torch.from_numpy(st["tok_cluster"][:, :nt].astype(np.int64)).cuda()
    counts = torch.from_numpy(st["counts"].astype(np.int64)).cuda()
    cent = torch.from_numpy(st["centroids"]).cuda()
    M2 = torch.from_numpy(st["M2"]).cuda().double()
    n_ids = torch.from_numpy(st["n_ids"].astype(np.int64)).cuda()
    assert int(tokc.min()) >= 0 and bool((tokc < n_ids[:, None]).all()), "a token outside the unit's ids"
    worst_c, worst_m = 0.0, 0.0
    step = max(1, min(64, (1 << 28) // max(nt * d, 1)))
    for u0 in range(0, U, step):
        u1 = min(U, u0 + step)
        nu = u1 - u0
        gid = (torch.arange(nu, device="cuda")[:, None] * Mx + tokc[u0:u1]).reshape(-1)
        Kd = K_all[u0:u1, :nt].double().reshape(-1, d)
        cnt = torch.zeros(nu * Mx, dtype=torch.int64, device="cuda").index_add_(0, gid, torch.ones_like(gid))
        assert torch.equal(cnt.reshape(nu, Mx), counts[u0:u1]), "sizes differ from the membership counts"
        sums = torch.zeros((nu * Mx, d), dtype=torch.float64, device="cuda").index_add_(0, gid, Kd)
        live = cnt > 0
        mean = sums[live] / cnt[live][:, None]
        cg = cent[u0:u1].reshape(nu * Mx, d)[live].double()
        err = ((cg - mean).norm(dim=1) / mean.norm(dim=1).clamp_min(1e-30)).max()
        worst_c = max(worst_c, float(err))
        m2 = torch.zeros(nu * Mx, dtype=torch.float64, device="cuda").index_add_(0, gid, ((Kd - sums[gid] / cnt[gid][:, None]) ** 2).sum(1))
        mg = M2[u0:u1].reshape(-1)[live]
        # floor: the fp32 rounding of a representative leaves about n |r|^2 2^-46 in M2 even when the members coincide
        scale = torch.maximum(m2[live], 1e-6 * cnt[live] * (mean.norm(dim=1) ** 2)).clamp_min(1e-6)
        worst_m = max(worst_m, float(((mg - m2[live]).abs() / scale).max()))
        del Kd, sums, m2
    assert worst_c <= TOL_CENTROID, f"representatives differ from the member means: {worst_c:.2e}"
    assert worst_m <= 2e-3, f"M2 differs from the members' spread: {worst_m:.2e}"
    return {"centroid_rel": worst_c, "M2_rel": worst_m, "live_clusters": int((counts > 0).sum()),
            "ids_max": int(n_ids.max()), "ids_min": int(n_ids.min())}
