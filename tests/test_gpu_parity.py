"""GPU parity tests: the CUDA library against the fp64 oracle through the C ABI."""
import numpy as np
import pytest
import torch

from gen import CONFIGS

pytestmark = pytest.mark.gpu


def _run(cfg, units, steps, **kw):
    from parity_harness import run_parity
    import inspect
    from parity_harness import log_ties, tie_bound
    rep = run_parity(cfg, units, steps, **kw)
    log_ties(f"{inspect.stack()[1].function}:{cfg.name}", rep)
    assert rep.ties <= tie_bound(rep), f"{rep.ties} ties followed in {rep.decisions} decisions"
    print(f"\n[{cfg.name}] steps={rep.steps} ties={rep.ties} splits={rep.splits} max_abs={rep.max_out_abs:.2e} "
          f"max_relL2={rep.max_out_l2:.2e} centroid_rel={rep.max_centroid_rel:.2e} "
          f"tokens/step={np.mean(rep.tokens_selected):.0f} status={rep.status_bits} rechecked={rep.rechecked}")
    assert rep.violations == 0
    return rep


def test_config1_full():
    """Config 1 in full: 2048-key prefill, 64 clusters, 10 rounds from k-means++, 512 decode steps."""
    rep = _run(CONFIGS[1], [0], CONFIGS[1].steps)
    assert rep.splits > 0


@pytest.mark.parametrize("cid", [2, 3, 4, 5])
def test_scaled_bf16_configs(cid):
    """Configs 2-5 at reduced size (several tiles plus a ragged tail), 3 units, fp32 assign path."""
    base = CONFIGS[cid]
    cfg = base.scaled(n_prefill=1111 if cid != 3 else 333, steps=96, M0=37 if cid != 3 else 13,
                      max_clusters=160, budget=300, T=6, new_every=32 if base.new_every else 0)
    _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1)


@pytest.mark.parametrize("mode", ["static", "local"])
def test_update_modes(mode):
    """The static-update and local-update modes (Section 3.1; the baselines of Section 8.1) against the oracle's: drifting
    keys with new mixture components, so that the adaptive rule would split; static never does, local founds clusters
    for the new entries, keeps the build frozen and splits the new clusters above 24 entries."""
    cfg = CONFIGS[3].scaled(n_prefill=500, steps=200, M0=12, max_clusters=96, budget=300, T=4, new_every=64,
                            update_mode=mode, local_max=24)
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1)
    if mode == "static":
        assert rep.gpu_splits == 0 and rep.splits == 0
    else:
        assert rep.splits >= 3 * 4          # 200 new entries in clusters of at most 24: several splits per unit


@pytest.mark.parametrize("cid", [2, 5])
def test_tensor_core_assign_ragged(cid):
    """Distance GEMM on the tensor cores (assign_mode 0): 1111 keys = 8 full 128-key blocks + 87, 37 centres
    padded to one 256-column accumulator; every Lloyd round's assignment is checked against the oracle."""
    import paper_2511_07427_b200 as P
    base = CONFIGS[cid]
    cfg = base.scaled(B=1, L=1, n_prefill=1111, steps=8, M0=37, max_clusters=160, budget=300, T=6)
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=0)
    assert rep.status_bits & P.ST_INTERNAL == 0


def test_tensor_core_assign_several_centre_tiles():
    """600 centres = 3 accumulator tiles (the two TMEM accumulators and the two centre stages wrap), 4500 keys,
    5 units in the context so that CTAs take items of different units."""
    import paper_2511_07427_b200 as P
    cfg = CONFIGS[4].scaled(n_prefill=4500, steps=4, M0=600, max_clusters=1200, budget=512, T=4)
    rep = _run(cfg, [0, 4], cfg.steps, ctx_units=list(range(5)), assign_mode=0)
    assert rep.status_bits & P.ST_INTERNAL == 0
    assert rep.rechecked < 0.5 * 5 * 4500 * 4      # the filter decides most keys


def test_tensor_core_assign_adversarial_keys():
    """Keys chosen to sit on the filter's weak spots: exact duplicates of other keys (exact ties between the
    centres initialised from them), midpoints of key pairs, one channel of magnitude ~200, values around the fp16
    sub-normal range, and all-zero rows.  Every Lloyd round's assignment must still equal the oracle's
    (ties to the lowest id), i.e. whatever the tensor-core filter cannot prove goes through the exact stage."""
    import oracle as O
    import paper_2511_07427_b200 as P
    from parity_harness import ParityReport, check_state, make_ctx, make_oracle
    rng = np.random.default_rng(3)
    n, d, M, T = 1500, 128, 48, 5
    base = rng.normal(size=(40, d)).astype(np.float32)
    K = base[rng.integers(0, 40, size=n)] + 0.05 * rng.normal(size=(n, d)).astype(np.float32)
    K[:200] = K[200:400]                                   # exact duplicates
    K[400:500] = 0.5 * (K[500:600] + K[600:700])           # midpoints
    K[:, 7] *= 200.0                                       # one huge channel
    K[700:800] *= 1e-6                                     # around and below the fp16 sub-normal range
    K[800:820] = 0.0
    Kb = torch.tensor(K).to(torch.bfloat16)[None].contiguous()
    Vb = torch.tensor(rng.normal(size=(1, n, d)).astype(np.float32)).to(torch.bfloat16)
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=n, steps=2, M0=M, max_clusters=96, T=T)
    ctx = make_ctx(cfg, 1, trace=1, assign_mode=0)
    ctx.build_index(Kb.cuda(), Vb.cuda(), M, 21)
    picks, trace = ctx.get_build_trace()
    o = make_oracle(cfg)
    o.build(Kb[0].double().numpy(), Vb[0].double().numpy(), M, T, 21, unit_index=0, init_mode=O.INIT_RANDOM,
            hint_assign=trace[:, 0, :])
    assert o.violations == 0
    check_state(o, ctx.export_state(), 0, ParityReport(), "adversarial build")
    st = ctx.get_status()
    assert st["error_bits"] & P.ST_INTERNAL == 0 and st["assign_rechecked"] > 0
    print(f"\n[adversarial] ties followed {o.ties}, re-decided exactly {st['assign_rechecked']} of {n * T}")
    ctx.destroy()


@pytest.mark.parametrize("cid,assign_mode,attn_mode", [(2, 1, 0), (3, 1, 0), (2, 0, 0), (3, 1, 1), (5, 1, 0)])
def test_fp8_storage(cid, assign_mode, attn_mode):
    """FP8 storage of the K/V rows (the precision of Section 8.1's runs): the library is handed bf16 rows and keeps them
    as e4m3 bytes with a power-of-two scale per row; the oracle is handed the same rows rounded by the test-side
    quantiser.  Decisions, statistics and attention outputs then agree to the same bounds as in bf16 storage; config 3's
    drifting stream makes clusters split, so rows also move between pages.  attn_mode 0 is the streaming kernel on the
    one-byte rows, 1 the plain one."""
    base = CONFIGS[cid]
    cfg = base.scaled(n_prefill=1111 if cid != 3 else 333, steps=96 if cid != 3 else 200, M0=37 if cid != 3 else 13,
                      max_clusters=160, budget=300, T=6, new_every=32 if base.new_every else 0, kv_dtype="fp8")
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=assign_mode, attn_mode=attn_mode)
    if cid == 3:
        assert rep.splits > 0


def test_fp8_storage_keeps_rows_on_the_grid_and_resumes():
    """The rows an FP8 context exports are the handed-over rows rounded to the storage grid, bit for bit, also after
    appends and splits; a context resumed from that export continues with the same outputs."""
    import paper_2511_07427_b200 as P
    from gen import UnitStream, make_prefill, make_decode_chunk
    from parity_harness import fp8_round_rows, make_ctx
    cfg = CONFIGS[3].scaled(n_prefill=333, steps=160, M0=13, max_clusters=160, budget=300, T=4, new_every=32, kv_dtype="fp8",
                            split_size_factor=1.3)
    U = 4
    streams = [UnitStream(cfg, u) for u in range(U)]
    K, V = make_prefill(streams)
    q, k, v = make_decode_chunk(streams, cfg.steps)
    ctx = make_ctx(cfg, U, trace=0, assign_mode=1)
    ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 7)
    half = 100
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    for t in range(half):
        ctx.decode_step(qd[t], cfg.budget); ctx.append(kd[t], vd[t]); ctx.split_check()
    assert ctx.get_status()["n_splits"] > 0
    n = cfg.n_prefill + half
    Ke, Ve = ctx.export_kv(n)
    K_all = torch.cat([K, k[:half].transpose(0, 1)], dim=1); V_all = torch.cat([V, v[:half].transpose(0, 1)], dim=1)
    assert torch.equal(Ke.cpu().double(), fp8_round_rows(K_all)) and torch.equal(Ve.cpu().double(), fp8_round_rows(V_all))
    st = ctx.export_state()
    ctx2 = make_ctx(cfg, U, trace=0, assign_mode=1)
    ctx2.import_state(Ke, Ve, st["tok_cluster"][:, :n], st["n_ids"], st["tau"], cfg.M0)
    for t in range(half, cfg.steps):
        a = ctx.decode_step(qd[t], cfg.budget).clone(); b = ctx2.decode_step(qd[t], cfg.budget).clone()
        assert (a - b).abs().max().item() <= 2e-3
        for c in (ctx, ctx2):
            c.append(kd[t], vd[t]); c.split_check()
    assert np.array_equal(ctx.export_state()["tok_cluster"], ctx2.export_state()["tok_cluster"])
    ctx.destroy(); ctx2.destroy()


def test_fp8_storage_with_clusters_too_large_to_stage():
    """FP8 storage where the clusters that split hold about 200 rows: more than the shared-memory split path stages, so
    the general path runs -- its 2-means and statistics read keys decoded from the one-byte pages, and its row moves
    copy bytes slot to slot.  Direct calls against the oracle, then the same stream through the graph loop, whose
    helper blocks take that path too."""
    cfg = CONFIGS[2].scaled(n_prefill=600, steps=24, M0=3, max_clusters=40, budget=300, T=3, split_min_size=4,
                            split_size_factor=1.05, kv_dtype="fp8")
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1)
    assert rep.splits > 0
    from test_gpu_edge import _loop_vs_direct
    assert _loop_vs_direct(cfg, [0, 1, 2], 24, modes=("direct", "graph")) > 0


@pytest.mark.parametrize("buf_max,budget", [(1000, 120), (6, 60), (1000, 300)])
def test_delayed_split_mode(buf_max, budget):
    """The delayed split of Algorithm 1 (Section 4.2) against the oracle's: with a small budget most triggered clusters
    are not among the retrieved ones, so their splits wait until a query retrieves them (buf_max 1000) or until the
    buffered entries force them (buf_max 6); with a large budget nearly every trigger is split at once.  Membership,
    ids, statistics and outputs must agree at every step, so every deferral and every forced split happens in the same
    step on both sides."""
    cfg = CONFIGS[3].scaled(n_prefill=500, steps=160, M0=12, max_clusters=256, budget=budget, T=4, new_every=64,
                            split_size_factor=1.3, split_var_factor=1.3, update_mode="delayed", buf_max=buf_max)
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1)
    assert rep.splits > 20 and rep.gpu_splits >= rep.splits


def test_correlation_aware_placement_changes_nothing_but_the_page_order():
    """dynakv_build_index_placed against the oracle: the partition, the statistics and every decode result are those of
    a plain build (the oracle knows nothing of pages); splits and appends work on the re-ordered pool."""
    base = CONFIGS[2]
    cfg = base.scaled(n_prefill=1111, steps=64, M0=37, max_clusters=160, budget=300, T=6, split_size_factor=1.3)
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1, placement_queries=24)
    assert rep.splits > 0


def test_correlation_aware_placement_lengthens_contiguous_access():
    """Queries near the mixture components' means retrieve the same few clusters together again and again; placing the
    clusters by those co-retrieval counts (Section 5.1, Eq. 8) must lengthen the contiguous stretches of the page pool
    that a step reads, measured on queries the placement has not seen, and must leave the outputs alone."""
    from gen import UnitStream, make_decode_chunk, make_prefill
    from parity_harness import make_ctx
    from paper_2511_07427_b200.placement import mean_contiguous_rows
    cfg = CONFIGS[2].scaled(B=1, L=1, n_prefill=4096, steps=128, M0=128, max_clusters=256, budget=512, T=6)
    U = 8
    streams = [UnitStream(cfg, u) for u in range(U)]
    K, V = make_prefill(streams)
    q, _, _ = make_decode_chunk(streams, 128)
    q = q.cuda()
    res = {}
    for placed in (False, True):
        ctx = make_ctx(cfg, U, trace=0, assign_mode=1)
        if placed:
            ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 5, placement_queries=q[:64].contiguous(), placement_budget=cfg.budget)
        else:
            ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 5)
        runs, outs = [], []
        for t in range(64, 128):
            outs.append(ctx.decode_step(q[t], cfg.budget).clone())
            runs.append(mean_contiguous_rows(*ctx.get_work_list()))
        st = ctx.export_state()
        res[placed] = (float(np.mean(runs)), torch.stack(outs), st["tok_cluster"].copy(), ctx.get_status()["error_bits"])
        ctx.destroy()
    print(f"\nmean contiguous rows per stretch: id order {res[False][0]:.1f}, placed {res[True][0]:.1f}")
    assert np.array_equal(res[False][2], res[True][2]) and res[True][3] == res[False][3]
    assert (res[False][1] - res[True][1]).abs().max().item() <= 1e-4
    assert res[True][0] >= 1.15 * res[False][0]


@pytest.mark.parametrize("cid,cache_pages,attn_mode,variant", [(3, 20, 0, ""), (2, 24, 0, ""), (2, 48, 1, ""), (1, 24, 0, ""),
                                                               (30, 96, 0, ""), (30, 96, 0, "fp8"), (2, 24, 1, "fp8"),
                                                               (30, 96, 0, "delayed"), (2, 24, 0, "placed"),
                                                               (3, 20, 0, "static"), (30, 24, 0, "local")])
def test_two_tier_mode(cid, cache_pages, attn_mode, variant):
    """The two-tier mode (Section 6; Section 7 on CPU-GPU platforms): the page pool in pinned host memory, a cache of
    cache_pages frames per unit in device memory, whole clusters brought in and replaced (Section 6.2).  The cache is
    invisible in the results: selections, appends, splits, statistics and attention outputs agree with the oracle as
    they do without it, at cache sizes that force evictions every few steps.  And the library's cache counters (pages
    copied, hits, refreshes, fetches, evictions, copies voided by splits, frames in use) equal those of the oracle's
    cache model, fed with the oracle's own selections, sizes and splits.  Case 30 is config 3 set to split often;
    config 1 stores fp32 rows; attn_mode 1 reads the frames with the plain kernel; variant "fp8" keeps pool and frames in
    the one-byte storage (rows and scale exponents travel together); "delayed" adds Algorithm 1's delayed split, whose
    splits then fall on clusters the step has just brought into the cache; "placed" builds the pool with the
    correlation-aware placement first; "static" and "local" are the two baseline update modes (no splits; new
    entries clustered among themselves)."""
    if cid == 30:
        cfg = CONFIGS[3].scaled(n_prefill=500, steps=160, M0=12, max_clusters=256, budget=300, T=4, new_every=32,
                                split_size_factor=1.3, split_var_factor=1.3)
    elif cid == 1:
        cfg = CONFIGS[1].scaled(n_prefill=700, steps=120, M0=24, max_clusters=128, budget=300, T=4)
    else:
        base = CONFIGS[cid]
        cfg = base.scaled(n_prefill=1111 if cid != 3 else 333, steps=96 if cid != 3 else 200, M0=37 if cid != 3 else 13,
                          max_clusters=160, budget=300, T=6, new_every=32 if base.new_every else 0)
    if variant == "fp8":
        cfg = cfg.scaled(kv_dtype="fp8")
    elif variant == "delayed":
        cfg = cfg.scaled(update_mode="delayed", buf_max=6)
    elif variant in ("static", "local"):
        cfg = cfg.scaled(update_mode=variant, local_max=24)
    rep = _run(cfg, [0] if cid == 1 else [0, 1, 2], cfg.steps, assign_mode=1, attn_mode=attn_mode, cache_pages=cache_pages,
               placement_queries=16 if variant == "placed" else 0)
    ts = rep.tier_stats
    print(f"[two tiers, {cache_pages} frames] {ts}")
    assert rep.status_bits == 0
    assert ts["clusters_hit"] > 0 and ts["clusters_refreshed"] > 0 and ts["clusters_evicted"] > 0
    if cid in (3, 30) and variant != "static":
        assert rep.splits > 0 and ts["copies_dropped_stale"] > 0


def test_two_tier_mode_reports_a_cache_that_is_too_small():
    """A cache that cannot hold one step's clusters: the status word says so, nothing is read out of bounds, and the
    context keeps working (with a larger budget than the cache, every step of that unit is flagged)."""
    import paper_2511_07427_b200 as P
    from gen import UnitStream, make_prefill, make_decode_chunk
    from parity_harness import make_ctx
    cfg = CONFIGS[2].scaled(n_prefill=1111, steps=8, M0=37, max_clusters=160, budget=300, T=3)
    streams = [UnitStream(cfg, u) for u in range(2)]
    K, V = make_prefill(streams)
    q, k, v = make_decode_chunk(streams, cfg.steps)
    ctx = make_ctx(cfg, 2, trace=0, assign_mode=1, cache_pages=4)
    ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 7)
    for t in range(cfg.steps):
        out = ctx.decode_step(q[t].cuda(), cfg.budget)
        assert torch.isfinite(out).all()
        ctx.append(k[t].cuda(), v[t].cuda()); ctx.split_check()
    st = ctx.get_status()
    assert st["error_bits"] & P.ST_TIER_CACHE
    assert st["n_appended"] == 2 * cfg.steps
    ctx.destroy()


def test_two_tier_mode_pool_exports_and_resumes_in_a_single_tier_context():
    """The host-memory pool of a two-tier context holds exactly the rows it was given, also after appends and splits
    (export_kv reads it back through the page tables), and a single-tier context resumed from that export continues
    with the same outputs and the same membership as the two-tier one."""
    from gen import UnitStream, make_prefill, make_decode_chunk
    from parity_harness import make_ctx
    cfg = CONFIGS[3].scaled(n_prefill=500, steps=120, M0=12, max_clusters=256, budget=300, T=4, new_every=32,
                            split_size_factor=1.3, split_var_factor=1.3)
    U = 4
    streams = [UnitStream(cfg, u) for u in range(U)]
    K, V = make_prefill(streams)
    q, k, v = make_decode_chunk(streams, cfg.steps)
    ctx = make_ctx(cfg, U, trace=0, assign_mode=1, cache_pages=96)
    ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 7)
    half = 70
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    for t in range(half):
        ctx.decode_step(qd[t], cfg.budget); ctx.append(kd[t], vd[t]); ctx.split_check()
    assert ctx.get_status()["n_splits"] > 20
    n = cfg.n_prefill + half
    Ke, Ve = ctx.export_kv(n)
    K_all = torch.cat([K, k[:half].transpose(0, 1)], dim=1); V_all = torch.cat([V, v[:half].transpose(0, 1)], dim=1)
    assert torch.equal(Ke.cpu(), K_all) and torch.equal(Ve.cpu(), V_all)
    st = ctx.export_state()
    ctx2 = make_ctx(cfg, U, trace=0, assign_mode=1)
    ctx2.import_state(Ke, Ve, st["tok_cluster"][:, :n], st["n_ids"], st["tau"], cfg.M0)
    for t in range(half, cfg.steps):
        a = ctx.decode_step(qd[t], cfg.budget).clone(); b = ctx2.decode_step(qd[t], cfg.budget).clone()
        assert (a - b).abs().max().item() <= 2e-3
        for c in (ctx, ctx2):
            c.append(kd[t], vd[t]); c.split_check()
    assert np.array_equal(ctx.export_state()["tok_cluster"], ctx2.export_state()["tok_cluster"])
    assert ctx.get_status()["error_bits"] == 0 and ctx.get_tier_stats()["clusters_evicted"] > 0
    ctx.destroy(); ctx2.destroy()


@pytest.mark.parametrize("budget,cache_pages", [(1, 8), (100000, 200)])
def test_two_tier_mode_at_the_ends_of_the_budget_range(budget, cache_pages):
    """Budget 1: every step retrieves its best cluster whole although it alone exceeds the budget, so the cache holds
    one or two clusters at a time.  A budget above the context: every step retrieves every cluster, the cache is as
    large as the pool, nothing is ever evicted, and after the first step only appended pages and the pages of split
    clusters travel.  Outputs, state and cache counters against the oracle and its cache model as in the other runs."""
    cfg = CONFIGS[3].scaled(n_prefill=400, steps=60, M0=10, max_clusters=128, budget=budget, T=3, new_every=32,
                            split_size_factor=1.3, split_var_factor=1.3)
    rep = _run(cfg, [0, 1], cfg.steps, assign_mode=1, cache_pages=cache_pages)
    ts = rep.tier_stats
    print(f"[two tiers, budget {budget}] {ts}")
    assert rep.splits > 0
    if budget == 1:
        assert rep.status_bits & P_ST_BUDGET_EXCEEDED and rep.status_bits & (16 | 32 | 64) == 0 and ts["clusters_evicted"] > 0
    else:
        assert rep.status_bits == 0 and ts["clusters_evicted"] == 0 and ts["clusters_refreshed"] > 0 and ts["copies_dropped_stale"] > 0


P_ST_BUDGET_EXCEEDED = 1
