"""GPU edge cases through the C ABI, each checked against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle as O
import paper_2511_07427_b200 as P
from gen import CONFIGS, UnitStream, make_decode_chunk, make_prefill

pytestmark = pytest.mark.gpu


def _run(cfg, units, steps, **kw):
    from parity_harness import run_parity
    import inspect
    from parity_harness import log_ties, tie_bound
    rep = run_parity(cfg, units, steps, **kw)
    log_ties(f"{inspect.stack()[1].function}:{cfg.name}", rep)
    assert rep.ties <= tie_bound(rep), f"{rep.ties} ties followed in {rep.decisions} decisions"
    assert rep.violations == 0
    return rep


@pytest.mark.parametrize("budget", [0, 1, 40, 10_000])
def test_budget_extremes(budget):
    cfg = CONFIGS[2].scaled(n_prefill=700, steps=12, M0=20, max_clusters=64, T=4)
    rep = _run(cfg, [0, 1], cfg.steps, budget=budget, assign_mode=1)
    if budget == 0:
        assert max(rep.tokens_selected) == 0
    if budget == 1:
        assert rep.status_bits & P.ST_BUDGET_EXCEEDED
    if budget == 10_000:
        assert min(rep.tokens_selected) >= 700


@pytest.mark.parametrize("G,d,dtype", [(1, 128, "bf16"), (2, 64, "bf16"), (7, 128, "bf16"), (8, 128, "bf16"),
                                       (3, 64, "f32"), (5, 128, "f32"), (8, 64, "bf16")])
def test_group_sizes_head_dims_dtypes(G, d, dtype):
    base = CONFIGS[2] if dtype == "bf16" else CONFIGS[1]
    cfg = base.scaled(Hq=G, Hkv=1, L=1, B=1, d=d, n_prefill=515, steps=24, M0=19, max_clusters=64, budget=150, T=4,
                      init_mode="kmeanspp" if G % 2 else "random")
    _run(cfg, [0], cfg.steps, assign_mode=1)


def test_attention_ring_wraps_and_units_cut_by_slices():
    # 96 units x ~190 pages: every persistent attention CTA streams a slice of ~60 pages (ten times its
    # ring depth) and most units are cut by slice boundaries, so the split-K combine runs for them
    cfg = CONFIGS[4].scaled(n_prefill=6000, steps=6, M0=200, max_clusters=512, budget=4096, T=3)
    rep = _run(cfg, [0, 17, 95], cfg.steps, ctx_units=list(range(96)), assign_mode=1)
    assert rep.status_bits & P.ST_INTERNAL == 0 and min(rep.tokens_selected) > 3000


def test_more_than_1024_units_keep_the_work_prefix_in_global_memory():
    # above 1024 units the attention CTAs read the prefix of the work lists from global memory instead of a
    # shared-memory copy, and the per-unit kernels run in several waves
    cfg = CONFIGS[5].scaled(B=1, L=1, n_prefill=96, steps=4, M0=6, max_clusters=16, budget=64, T=2)
    rep = _run(cfg, [0, 555, 1099], cfg.steps, ctx_units=list(range(1100)), assign_mode=0)
    assert rep.status_bits & P.ST_INTERNAL == 0


def test_plain_attention_kernel_on_bf16():
    cfg = CONFIGS[5].scaled(B=1, L=1, n_prefill=600, steps=16, M0=24, max_clusters=64, budget=200, T=3, init_mode="random")
    _run(cfg, [0, 1, 2, 3], cfg.steps, assign_mode=1, attn_mode=1)


def test_every_key_its_own_cluster_and_page_boundaries():
    # n == M: every cluster has one member after the first round; then 31/32/33-row pages via appends
    cfg = CONFIGS[2].scaled(n_prefill=48, steps=80, M0=48, max_clusters=64, budget=64, T=2, split_size_factor=0.0,
                            split_var_factor=0.0)
    _run(cfg, [0], cfg.steps, assign_mode=1)


def test_few_clusters_long_chains_and_capacity_bits():
    # 3 clusters over 200 keys (multi-page chains), splitting until the id cap, then the token cap
    cfg = CONFIGS[2].scaled(n_prefill=200, steps=40, M0=3, max_clusters=6, budget=120, T=3, split_min_size=4,
                            split_size_factor=1.05)
    rep = _run(cfg, [0, 1], cfg.steps, assign_mode=1)
    assert rep.status_bits & P.ST_MAX_CLUSTERS


def test_split_check_owed_for_several_appends():
    # The split check runs only after every third append: clusters that took the earlier appends must still be
    # examined (the oracle examines every cluster at every check).  Few clusters and a size trigger of 1.5 x the
    # mean make "an append pushes its cluster over the threshold, and it is not the last append before the check"
    # happen several times in this run (a library that examines only the last appended cluster fails it).
    cfg = CONFIGS[2].scaled(n_prefill=120, steps=399, M0=6, max_clusters=128, budget=120, T=3, split_min_size=4,
                            split_size_factor=1.5, split_var_factor=0.0)
    rep = _run(cfg, [0, 1, 2, 3], cfg.steps, assign_mode=1, check_every=3, state_every=30)
    assert rep.gpu_splits >= 8


def _single_ctx(cfg, K, V, **kw):
    from parity_harness import make_ctx
    ctx = make_ctx(cfg, K.shape[0], trace=0, **kw)
    ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 99)
    return ctx


def test_token_capacity_sets_status_and_drops_append():
    cfg = CONFIGS[2].scaled(n_prefill=64, steps=4, M0=4, max_clusters=16, budget=64, T=2)
    s = [UnitStream(cfg, 0)]
    K, V = make_prefill(s)
    q, k, v = make_decode_chunk(s, 4)
    ctx = _single_ctx(cfg, K, V, assign_mode=1)
    for t in range(4):
        ctx.append(k[t].cuda(), v[t].cuda())
    assert ctx.get_status()["error_bits"] & P.ST_MAX_TOKENS == 0
    ctx.append(k[0].cuda(), v[0].cuda())
    st = ctx.get_status()
    assert st["error_bits"] & P.ST_MAX_TOKENS and st["n_appended"] == 4
    assert ctx.export_state()["n_tokens"][0] == 68
    ctx.destroy()


def test_zero_query_breaks_score_ties_by_id():
    cfg = CONFIGS[2].scaled(n_prefill=400, steps=4, M0=16, max_clusters=32, budget=100, T=3)
    s = [UnitStream(cfg, 0)]
    K, V = make_prefill(s)
    ctx = _single_ctx(cfg, K, V, assign_mode=1)
    st = ctx.export_state()
    q = torch.zeros((1, cfg.G, cfg.d), dtype=torch.float32, device="cuda")
    sel = torch.full((1, cfg.max_clusters), -1, dtype=torch.int32, device="cuda")
    out = ctx.decode_step(q, 100, selected_ids=sel)
    ids = sel[0].cpu().numpy(); ids = ids[ids >= 0]
    cnt = st["counts"][0]
    exp, cum = [], 0
    for j in range(16):
        if cnt[j] == 0:
            continue
        if cum + cnt[j] > 100:
            break
        exp.append(j); cum += cnt[j]
    assert list(ids) == exp
    # uniform softmax over the selected members
    a = st["tok_cluster"][0, :400]
    ref = V[0].double()[np.isin(a, exp)].mean(0).numpy()
    assert np.abs(out[0].cpu().numpy() - ref[None]).max() < 1e-4
    ctx.destroy()


def test_selection_with_bunched_scores_and_outliers():
    """The selection's short way ranks the few clusters of one histogram bin against each other and leaves the job
    to the general radix version when that bin holds more than 64 clusters.  Queries are crafted so that: all
    scores are equal (every cluster in one bin, ties by id); one cluster scores far above a bunch of nearly equal
    ones (the bunch shares a bin); scores are spread out (the common case); and budgets fall on both sides of the
    boundaries.  Every selection must equal the oracle's."""
    from parity_harness import make_oracle
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=3000, steps=4, M0=150, max_clusters=256, budget=400, T=3)
    s = [UnitStream(cfg, 0)]
    K, V = make_prefill(s)
    ctx = _single_ctx(cfg, K, V, assign_mode=1)
    st = ctx.export_state()
    o = make_oracle(cfg)
    o.install(K[0].double().numpy(), V[0].double().numpy(), st["tok_cluster"][0, :cfg.n_prefill], int(st["n_ids"][0]))
    C = torch.from_numpy(st["centroids"][0, :cfg.M0]).float()
    g = torch.Generator().manual_seed(5)
    # a direction nearly orthogonal to every representative, plus a large multiple of one representative's own direction
    r = torch.randn(cfg.d, generator=g)
    r = r - C.T @ torch.linalg.lstsq(C @ C.T + 1e-3 * torch.eye(cfg.M0), C @ r).solution
    queries = {
        "equal": torch.zeros(cfg.G, cfg.d),
        "bunched": (1e-4 * r + 50.0 * C[7] / C[7].norm() ** 2).repeat(cfg.G, 1),
        "spread": torch.randn(cfg.G, cfg.d, generator=g),
    }
    sel = torch.full((1, cfg.max_clusters), -1, dtype=torch.int32, device="cuda")
    for name, q in queries.items():
        q = q.to(torch.bfloat16).float()
        for budget in (1, 25, 400, 1500, 2999, 3000, 10 ** 6):
            ctx.decode_step(q[None].cuda(), budget, selected_ids=sel)
            nsel, ntok = ctx.get_selection()
            ids = sel[0].cpu().numpy()[: nsel[0]]
            v0 = o.violations
            _, ids_o, tok_o = o.decode_step(q.double().numpy(), budget, hint_ids=ids)
            assert o.violations == v0 and list(ids_o) == list(ids) and tok_o == int(ntok[0]), \
                f"{name}, budget {budget}: gpu {ids[:10]} oracle {ids_o[:10]}"
    ctx.destroy()


def test_duplicate_keys_leave_dead_clusters():
    cfg = CONFIGS[1].scaled(n_prefill=256, steps=16, M0=12, max_clusters=32, budget=80, T=4, init_mode="random")
    from parity_harness import make_ctx, make_oracle, check_state, ParityReport
    rng = np.random.default_rng(0)
    base = rng.normal(size=(6, cfg.d)).astype(np.float32)
    K = torch.tensor(base[rng.integers(0, 6, size=256)])[None].contiguous()     # only 6 distinct keys, 12 centres
    V = torch.tensor(rng.normal(size=(1, 256, cfg.d)).astype(np.float32))
    ctx = make_ctx(cfg, 1, trace=1)
    ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 5)
    picks, trace = ctx.get_build_trace()
    o = make_oracle(cfg)
    o.build(K[0].double().numpy(), V[0].double().numpy(), cfg.M0, cfg.T, 5, unit_index=0, init_mode=O.INIT_RANDOM,
            hint_assign=trace[:, 0, :])
    st = ctx.export_state()
    assert o.violations == 0 and (o.counts() == 0).sum() >= 6
    check_state(o, st, 0, ParityReport(), "dup build")
    q = torch.tensor(rng.normal(size=(1, cfg.G, cfg.d)).astype(np.float32))
    sel = torch.full((1, cfg.max_clusters), -1, dtype=torch.int32, device="cuda")
    out = ctx.decode_step(q.cuda(), 80, selected_ids=sel).cpu().numpy()
    ids = sel[0].cpu().numpy(); ids = ids[ids >= 0]
    out_o, ids_o, _ = o.decode_step(q[0].double().numpy(), 80, hint_ids=ids)
    assert list(ids_o) == list(ids) and np.abs(out[0] - out_o).max() < 2e-3
    ctx.destroy()


@pytest.mark.parametrize("mode", ["adaptive", "local"])
def test_checkpoint_and_resume(mode):
    """export_state + export_kv after some decode steps, import into a fresh context, and both contexts must go on
    identically: same membership and ids after more steps (splits included), outputs equal up to the rounding of
    the recomputed statistics."""
    from parity_harness import make_ctx
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=700, steps=120, M0=20, max_clusters=128, budget=300, T=3,
                            update_mode=mode, local_max=20)
    units = [0, 1, 2]
    s = [UnitStream(cfg, u) for u in units]
    K, V = make_prefill(s)
    q, k, v = make_decode_chunk(s, 120)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    a = make_ctx(cfg, 3, trace=0, assign_mode=1)
    a.build_index(K.cuda(), V.cuda(), cfg.M0, 5)
    for t in range(60):
        a.decode_step(qd[t], cfg.budget); a.append(kd[t], vd[t]); a.split_check()
    st = a.export_state()
    n = int(st["n_tokens"][0])
    assert n == 760 and np.all(st["n_tokens"] == n)
    Kx, Vx = a.export_kv(n)
    Kref = torch.cat([K, k[:60].transpose(0, 1)], dim=1)
    assert torch.equal(Kx.cpu(), Kref)                                      # rows come back in token order
    b = make_ctx(cfg, 3, trace=0, assign_mode=1)
    b.import_state(Kx, Vx, st["tok_cluster"][:, :n], st["n_ids"], st["tau"], cfg.M0)
    sb = b.export_state()
    assert np.array_equal(sb["tok_cluster"], st["tok_cluster"]) and np.array_equal(sb["counts"], st["counts"])
    assert np.array_equal(sb["n_ids"], st["n_ids"]) and np.array_equal(sb["tau"], st["tau"])
    live = st["counts"] > 0
    assert np.abs(sb["centroids"][live] - st["centroids"][live]).max() <= 1e-4 * np.abs(st["centroids"][live]).max()
    worst = 0.0
    for t in range(60, 120):
        oa = a.decode_step(qd[t], cfg.budget); ob = b.decode_step(qd[t], cfg.budget)
        worst = max(worst, float((oa - ob).abs().max()))
        a.append(kd[t], vd[t]); b.append(kd[t], vd[t])
        a.split_check(); b.split_check()
    sa, sb = a.export_state(), b.export_state()
    assert np.array_equal(sa["tok_cluster"], sb["tok_cluster"]) and np.array_equal(sa["counts"], sb["counts"])
    assert a.get_status()["n_splits"] > 0 and worst < 1e-4
    a.destroy(); b.destroy()


def test_host_array_loop_matches_direct_calls():
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=500, steps=70, M0=12, max_clusters=64, budget=200, T=3,
                            split_size_factor=1.3)
    assert _loop_vs_direct(cfg, [0, 1, 2, 3], 70, modes=("direct", "hostloop")) > 0


def test_a_bounded_wait_that_runs_out_raises_the_status_bit_and_returns():
    """A wait on a barrier nobody arrives at gives up after its poll limit: the status word gets INTERNAL, the kernel
    returns, and the context goes on working (no fault, no hang)."""
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=300, steps=4, M0=8, max_clusters=32, budget=100, T=2)
    s_ = [UnitStream(cfg, 0)]
    K, V = make_prefill(s_)
    q, k, v = make_decode_chunk(s_, 2)
    ctx = _single_ctx(cfg, K, V, assign_mode=1)
    out0 = ctx.decode_step(q[0].cuda(), cfg.budget).cpu()
    assert ctx.get_status()["error_bits"] & P.ST_INTERNAL == 0
    assert ctx.selftest_wait_expiry() == 1
    assert ctx.get_status()["error_bits"] & P.ST_INTERNAL
    out1 = ctx.decode_step(q[0].cuda(), cfg.budget).cpu()       # the context is still usable and gives the same answer
    assert torch.equal(out0, out1)
    ctx.append(k[0].cuda(), v[0].cuda()); ctx.split_check()
    assert ctx.export_state()["n_tokens"][0] == cfg.n_prefill + 1
    ctx.destroy()


def test_graph_loop_in_local_update_mode():
    # the captured loop founds a cluster for the first new entry inside the tail kernel (an id beyond the ones the
    # unit's centroid pass covered) and splits decode-born clusters above 20 entries
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1, Hq=4, n_prefill=400, steps=90, M0=10, max_clusters=64, budget=200, T=3,
                            update_mode="local", local_max=20)
    assert _loop_vs_direct(cfg, [0, 1, 2, 3, 4], 90, cut=31) >= 5


def test_graph_loop_in_delayed_split_mode():
    # the tail kernel's unit blocks decide, from the step's retrieved clusters and the flags, which splits happen now,
    # which are owed and whether the buffer limit forces one; the helper blocks split; the host-buffer step does the same
    cfg = CONFIGS[3].scaled(n_prefill=500, steps=96, M0=12, max_clusters=256, budget=120, T=4, new_every=32,
                            split_size_factor=1.3, split_var_factor=1.3, update_mode="delayed", buf_max=8)
    assert _loop_vs_direct(cfg, [0, 1, 2, 3, 4], 96, cut=37) > 50


def test_graph_loop_and_host_steps_in_two_tier_mode():
    # the cache bookkeeping and the page copies are part of the captured iteration and of the host step's graph; a
    # stream that splits often, so copies are voided between steps, and helper blocks split rows that live in host memory
    cfg = CONFIGS[3].scaled(n_prefill=500, steps=96, M0=12, max_clusters=256, budget=300, T=4, new_every=32,
                            split_size_factor=1.3, split_var_factor=1.3)
    assert _loop_vs_direct(cfg, [0, 1, 2, 3, 4], 96, modes=("direct", "graph", "host", "hostloop"), cut=37, cache_pages=96) > 50


def _loop_vs_direct(cfg, units, steps, modes=("direct", "graph", "host"), cut=None, cache_pages=0):
    """The captured loop (and the host-buffer step) must leave the same state and outputs as direct calls."""
    s = [UnitStream(cfg, u) for u in units]
    K, V = make_prefill(s)
    q, k, v = make_decode_chunk(s, steps)
    cut = steps // 2 - 3 if cut is None else cut
    side = torch.cuda.Stream()
    outs = {}
    states = {}
    nsplit = {}
    tier = {}
    for mode in modes:
        with torch.cuda.stream(side):
            from parity_harness import make_ctx
            ctx = make_ctx(cfg, len(units), trace=0, assign_mode=1, cache_pages=cache_pages)
            ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 7)
            qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
            if mode == "direct":
                out = torch.empty((steps, len(units), cfg.G, cfg.d), device="cuda")
                for t in range(steps):
                    ctx.decode_step(qd[t], cfg.budget, out=out[t]); ctx.append(kd[t], vd[t]); ctx.split_check()
            elif mode == "graph":
                # two calls: the second one starts from the state the first one left (and a count that is not a
                # multiple of the long graph's eight iterations)
                out = ctx.decode_loop(qd[:cut], kd[:cut], vd[:cut], cfg.budget)
                out2 = ctx.decode_loop(qd[cut:], kd[cut:], vd[cut:], cfg.budget)
                out = torch.cat([out, out2])
            elif mode == "hostloop":
                # host arrays through the chunked, double-buffered loop (70 steps = two full chunks of 32 and a rest)
                qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
                out = torch.empty((steps, len(units), cfg.G, cfg.d)).pin_memory()
                ctx.decode_loop_host(qh, kh, vh, cfg.budget, out)
            else:
                out = torch.empty((steps, len(units), cfg.G, cfg.d))
                qh, kh, vh = q.pin_memory(), k.pin_memory(), v.pin_memory()
                oh = torch.empty((len(units), cfg.G, cfg.d)).pin_memory()
                for t in range(steps):
                    ctx.step_host(qh[t], kh[t], vh[t], cfg.budget, oh); out[t] = oh
            side.synchronize()
            outs[mode] = out.cpu().numpy()
            states[mode] = ctx.export_state()
            st = ctx.get_status()
            nsplit[mode] = st["n_splits"]
            assert st["error_bits"] & (P.ST_INTERNAL | P.ST_BOUNDS) == 0, f"status {st['error_bits']}, site {st['bounds_site']}"
            if cache_pages:
                assert st["error_bits"] == 0
                tier[mode] = ctx.get_tier_stats()
            ctx.destroy()
    for mode in modes[1:]:
        assert nsplit[mode] == nsplit["direct"]
        if cache_pages:         # the cache sees the same steps whichever way they are launched
            assert tier[mode] == tier["direct"], f"{mode}: {tier[mode]} vs {tier['direct']}" 
        assert np.array_equal(states[mode]["tok_cluster"], states["direct"]["tok_cluster"])
        assert np.array_equal(states[mode]["counts"], states["direct"]["counts"])
        assert np.abs(outs[mode] - outs["direct"]).max() < 1e-4
    return nsplit["direct"]


def test_graph_loop_and_host_step_match_direct_calls():
    cfg = CONFIGS[2].scaled(n_prefill=900, steps=48, M0=30, max_clusters=96, budget=256, T=4)
    assert _loop_vs_direct(cfg, [0, 1, 2, 3, 4], 48, cut=20) > 0


def test_graph_loop_with_clusters_too_large_to_stage():
    # three clusters over 600 keys: the clusters that split hold about 200 rows, more than the shared-memory
    # split path stages, so the loop's helper blocks take the general path and patch the children's rows from
    # global memory; an eager size trigger gives several triggered clusters per unit and step
    cfg = CONFIGS[2].scaled(n_prefill=600, steps=24, M0=3, max_clusters=40, budget=300, T=3, split_min_size=4,
                            split_size_factor=1.05)
    assert _loop_vs_direct(cfg, [0, 1, 2], 24, modes=("direct", "graph")) > 0


def test_graph_loop_fp32_d64_and_more_triggered_units_than_helpers():
    # the other instantiation of the tail kernel (fp32 K/V, d = 64), and 48 units that all split in the same
    # steps: more hand-overs than there are helper blocks
    cfg = CONFIGS[1].scaled(B=1, L=1, Hkv=48, Hq=48 * CONFIGS[1].G, n_prefill=256, steps=20, M0=6, max_clusters=40,
                            budget=96, T=3, split_min_size=4, split_size_factor=1.2)
    # first call of one step only: the loop's single iteration has no next step to prepare
    assert _loop_vs_direct(cfg, list(range(48)), 20, modes=("direct", "graph"), cut=1) > 48


def test_graph_loop_with_more_units_than_block_slots():
    # 1100 units: the tail kernel's unit blocks run in several waves with the helper blocks last, the selection
    # runs with 256-thread blocks and its last block lays out the work lists (more than 1024 units)
    cfg = CONFIGS[2].scaled(B=1, L=1, Hkv=1100, Hq=1100 * CONFIGS[2].G, n_prefill=96, steps=12, M0=6, max_clusters=24,
                            budget=64, T=2, split_min_size=4, split_size_factor=1.3)
    assert _loop_vs_direct(cfg, list(range(1100)), 12, modes=("direct", "graph"), cut=5) > 100


def test_wrong_call_order_and_shapes():
    cfg = P.DynaKVConfig(n_units=1, gqa_group=2, head_dim=64, kv_dtype=P.F32, max_tokens=64, max_clusters=8)
    ctx = P.DynaKV(cfg)
    q = torch.zeros((1, 2, 64), device="cuda")
    with pytest.raises(P.DynaKVError):
        ctx.decode_step(q, 8)                      # before build_index
    with pytest.raises(P.DynaKVError):
        ctx.split_check()
    K = torch.randn((1, 32, 64), device="cuda")
    with pytest.raises(P.DynaKVError):
        ctx.build_index(K, K, 33, 0)               # more clusters than keys
    ctx.build_index(K, K, 4, 0)
    with pytest.raises(P.DynaKVError):
        ctx.build_index(K, K, 4, 0)                # twice
    with pytest.raises(P.DynaKVError):
        ctx.decode_loop(q[None], K[:, 0][None], K[:, 0][None], 8)   # default stream: no graph capture
    ctx.destroy()


def test_order_independent_centroid_sums_reproduce_bit_for_bit_and_match_the_oracle():
    """det_sums = 1: the build's centroid sums (Eq. 4) are accumulated as 64-bit integers in units of 2^-24, so they do
    not depend on the order in which the keys' atomic adds arrive.  Two builds of the same input give the same
    assignment in every Lloyd round and the same centroids bit for bit, and the mode passes the same parity run as
    the default one."""
    from parity_harness import make_ctx
    cfg = CONFIGS[2].scaled(B=1, L=1, n_prefill=3000, steps=24, M0=50, max_clusters=128, budget=300, T=6)
    streams = [UnitStream(cfg, u) for u in range(6)]
    K, V = make_prefill(streams)
    res = []
    for _ in range(2):
        ctx = make_ctx(cfg, 6, trace=1, assign_mode=1, det_sums=1)
        ctx.build_index(K.cuda(), V.cuda(), cfg.M0, 11)
        _, trace = ctx.get_build_trace()
        st = ctx.export_state()
        assert ctx.get_status()["error_bits"] == 0
        res.append((trace.copy(), st["centroids"].copy(), st["counts"].copy()))
        ctx.destroy()
    assert np.array_equal(res[0][0], res[1][0]) and np.array_equal(res[0][2], res[1][2])
    assert np.array_equal(res[0][1].view(np.uint32), res[1][1].view(np.uint32))
    rep = _run(cfg, [0, 1, 2], cfg.steps, assign_mode=1, det_sums=1)
    assert rep.status_bits == 0
    _run(cfg, [0, 1], 8, assign_mode=0, det_sums=1)          # with the tensor-core assignment
