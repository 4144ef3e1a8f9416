"""Pins for the fp64 oracle: closed forms, brute force, library cross-checks, hand-worked
fixtures.  Each check is chosen so that a dropped term, a wrong sign or index, or a
transposed operand in the oracle fails it.  None of them re-types the oracle's formula."""
import math
import os

import numpy as np
import pytest

import oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gold(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


# ------------------------------------------------------------------ counter-based uniforms

def test_uniform_matches_published_splitmix64_vector():
    # splitmix64 seeded with 0 returns 0xE220A8397B1DCDAF first (reference vector of the
    # published generator); (seed=0, unit=0, round=0, i=0) feeds the mixer exactly that state.
    bits = 0xE220A8397B1DCDAF >> 41
    assert O.uniform(0, 0, 0, 0) == (bits + 0.5) / 2 ** 23


def test_uniform_grid_and_spread():
    us = np.array([O.uniform(7, 3, r, i) for r in range(4) for i in range(2000)])
    assert us.min() > 0 and us.max() < 1
    assert np.all((us * 2 ** 23 - 0.5) == np.round(us * 2 ** 23 - 0.5))   # 23-bit grid
    assert abs(us.mean() - 0.5) < 0.02 and abs(us.var() - 1 / 12) < 0.01
    # distinct streams per argument
    assert O.uniform(7, 3, 0, 1) != O.uniform(7, 3, 1, 0)
    assert O.uniform(7, 3, 0, 1) != O.uniform(7, 4, 0, 1)
    assert O.uniform(8, 3, 0, 1) != O.uniform(7, 3, 0, 1)


# ------------------------------------------------------------------ assign / Lloyd

def test_assign_is_bruteforce_argmin():
    rng = np.random.default_rng(0)
    K = rng.normal(size=(300, 7)); Cn = rng.normal(size=(11, 7))
    a, _, _ = O.assign(K, Cn)
    D = ((K[:, None, :] - Cn[None, :, :]) ** 2).sum(-1)      # [n, M]; a transposed operand changes this
    assert np.array_equal(a, D.argmin(1))


def test_assign_ties_go_to_lowest_index_and_live_mask():
    K = np.array([[0.0, 0.0]]); Cn = np.array([[1.0, 0.0], [-1.0, 0.0], [0.0, 1.0]])
    a, _, _ = O.assign(K, Cn)
    assert a[0] == 0
    a, _, _ = O.assign(K, Cn, live=[0, 1, 1])
    assert a[0] == 1


def test_lloyd_hand_worked_fixture():
    g = _gold("lloyd_1d.txt")
    K = g["keys"][:, None]; Cn = g["start"][:, None]
    for r in (1, 2, 3):
        a, _, _ = O.assign(K, Cn)
        Cn, cnt = O.update(K, a, Cn)
        assert np.array_equal(a, g[f"assign_round{r}"].astype(int))
        assert np.allclose(Cn[:, 0], g[f"centres_round{r}"], atol=1e-15)


def test_update_is_member_mean_and_empty_keeps_centre():
    rng = np.random.default_rng(1)
    K = rng.normal(size=(50, 3)); a = rng.integers(0, 3, size=50)   # cluster 3 stays empty
    prev = rng.normal(size=(4, 3))
    Cn, cnt = O.update(K, a, prev)
    for j in range(3):
        assert np.allclose(Cn[j], K[a == j].mean(0), atol=1e-14)
        assert cnt[j] == (a == j).sum()
    assert cnt[3] == 0 and np.array_equal(Cn[3], prev[3])


def test_inertia_never_increases_and_single_cluster_is_mean():
    rng = np.random.default_rng(2)
    K = rng.normal(size=(400, 5)) * rng.uniform(0.5, 3, size=5)
    Cn = K[:9].copy(); last = math.inf
    for _ in range(8):
        a, _, _ = O.assign(K, Cn)
        j1 = O.inertia(K, Cn, a); assert j1 <= last + 1e-9; last = j1
        Cn, _ = O.update(K, a, Cn)
        j2 = O.inertia(K, Cn, a); assert j2 <= last + 1e-9; last = j2
    u = O.OracleUnit(5, 1, 500, 4)
    u.build(K, K, 1, 3, seed=1, init_mode=O.INIT_RANDOM)
    assert np.allclose(u.centroids()[0], K.mean(0), atol=1e-13)
    assert np.isclose(u.M2()[0], ((K - K.mean(0)) ** 2).sum())


def test_blobs_recovered():
    rng = np.random.default_rng(3)
    means = rng.normal(size=(6, 8)) * 20
    comp = np.repeat(np.arange(6), 40); rng.shuffle(comp)
    K = means[comp] + 0.1 * rng.normal(size=(240, 8))
    u = O.OracleUnit(8, 1, 300, 12)
    u.build(K, K, 6, 10, seed=11, init_mode=O.INIT_KMEANSPP)
    a = u.assign()
    # purity 1: each cluster holds one component, each component one cluster
    assert len({(a[i], comp[i]) for i in range(240)}) == 6
    for j in range(6):
        c = comp[a == j][0]
        assert np.allclose(u.centroids()[j], K[comp == c].mean(0), atol=1e-12)


def test_lloyd_matches_scikit_learn_from_same_start():
    from sklearn.cluster import KMeans
    rng = np.random.default_rng(4)
    means = rng.normal(size=(5, 6)) * 3
    K = means[rng.integers(0, 5, 500)] + rng.normal(size=(500, 6))
    u = O.OracleUnit(6, 1, 600, 8)
    T = 7
    u.build(K, K, 8, T, seed=5, init_mode=O.INIT_RANDOM)
    start = K[O.init_random(500, 8, 5, 0)]
    # scikit-learn's Lloyd runs T rounds of (label, recompute centres) from the given start, so its
    # centres after max_iter=T equal the oracle's representatives, index for index.
    km = KMeans(n_clusters=8, init=start, n_init=1, max_iter=T, tol=0.0, algorithm="lloyd").fit(K)
    assert u.counts().min() > 0
    assert np.allclose(km.cluster_centers_, u.centroids(), atol=1e-9)
    # and scipy's kmeans2 from the same start agrees as well
    from scipy.cluster.vq import kmeans2
    c2, lab2 = kmeans2(K, start.copy(), iter=T, minit="matrix")
    assert np.allclose(c2, u.centroids(), atol=1e-9)


def test_build_state_satisfies_eq3_eq4():
    rng = np.random.default_rng(5)
    K = rng.normal(size=(256, 4)); V = rng.normal(size=(256, 4))
    u = O.OracleUnit(4, 2, 300, 40)
    u.build(K, V, 16, 5, seed=3)
    a = u.assign(); cnt = u.counts(); Cn = u.centroids(); M2 = u.M2()
    assert a.min() >= 0 and a.max() < 16 and cnt.sum() == 256        # disjoint cover
    for j in range(16):
        if cnt[j]:
            assert np.allclose(Cn[j], K[a == j].mean(0), atol=1e-13)  # Eq. 4
            assert np.isclose(M2[j], ((K[a == j] - Cn[j]) ** 2).sum(), rtol=1e-12)
    live = u.live()
    var = M2[live] / cnt[live]
    assert np.isclose(u.tau, 2.0 * var.mean(), rtol=1e-12)


# ------------------------------------------------------------------ init

def test_kmeanspp_round_frequencies_follow_d2_sampling():
    # 16 points on a line; after a fixed first pick the second pick must follow D^2 / sum D^2.
    K = np.arange(16, dtype=np.float64)[:, None] ** 1.3
    counts = np.zeros(16); first = np.zeros(16); trials = 4000
    cond = {}
    for s in range(trials):
        p, _, _ = O.init_kmeanspp(K, 2, seed=1000 + s)
        first[p[0]] += 1
        cond.setdefault(p[0], np.zeros(16))[p[1]] += 1
    # first pick uniform
    chi = ((first - trials / 16) ** 2 / (trials / 16)).sum()
    assert chi < 45          # chi2(15) 99.99% ~ 44.3
    # second pick | first pick ~ D^2
    for f, c in cond.items():
        D2 = ((K[:, 0] - K[f, 0]) ** 2); p = D2 / D2.sum(); n = c.sum()
        mask = p > 0
        assert c[~mask].sum() == 0
        chi = ((c[mask] - n * p[mask]) ** 2 / (n * p[mask])).sum()
        assert chi < 50, (f, chi)


def test_kmeanspp_picks_are_distinct_points_far_apart():
    rng = np.random.default_rng(6)
    means = rng.normal(size=(4, 3)) * 50
    K = means[np.repeat(np.arange(4), 25)] + rng.normal(size=(100, 3)) * 0.01
    p, _, _ = O.init_kmeanspp(K, 4, seed=9)
    assert sorted(np.repeat(np.arange(4), 25)[p]) == [0, 1, 2, 3]


def test_init_random_is_sort_of_hashes():
    n, M, seed, unit = 500, 37, 123, 5
    u = np.array([O.uniform(seed, unit, 0, i) for i in range(n)])
    order = sorted(range(n), key=lambda i: (u[i], i))[:M]
    assert np.array_equal(O.init_random(n, M, seed, unit), np.array(sorted(order)))


# ------------------------------------------------------------------ append / Welford

def test_welford_hand_worked_fixture():
    g = _gold("welford_4.txt")
    K = g["members"][:, None]
    u = O.OracleUnit(1, 1, 8, 2, gamma=0, alpha=0)
    u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    assert u.append(g["new"], g["new"]) == 0
    assert u.counts()[0] == int(g["n"][0])
    assert np.isclose(u.centroids()[0, 0], g["r"][0], atol=1e-15)
    assert np.isclose(u.M2()[0], g["M2"][0], atol=1e-15)


def test_append_nearest_and_welford_equals_two_pass():
    rng = np.random.default_rng(7)
    K = rng.normal(size=(200, 6)); V = rng.normal(size=(200, 6))
    u = O.OracleUnit(6, 1, 400, 16, gamma=0, alpha=0)
    u.build(K, V, 8, 4, seed=2)
    allK = [K]
    for t in range(150):
        k = rng.normal(size=6) * 1.5; v = rng.normal(size=6)
        Cn = u.centroids(); live = u.live()
        D = ((Cn - k) ** 2).sum(1); D[~live] = np.inf
        j = u.append(k, v)
        assert j == int(D.argmin())
        allK.append(k[None])
    KK = np.concatenate(allK); a = u.assign(); cnt = u.counts()
    assert len(a) == 350 and cnt.sum() == 350
    for j in range(u.M):
        if cnt[j]:
            mem = KK[a == j]
            assert np.allclose(u.centroids()[j], mem.mean(0), atol=1e-12)
            assert np.isclose(u.M2()[j], ((mem - mem.mean(0)) ** 2).sum(), rtol=1e-10)


def test_append_full_unit_sets_status():
    K = np.eye(4)
    u = O.OracleUnit(4, 1, 4, 2, gamma=0, alpha=0)
    u.build(K, K, 2, 2, seed=0)
    assert u.append(K[0], K[0]) == -1 and (u.status & O.ST_MAX_TOKENS)


# ------------------------------------------------------------------ score / select

def _unit(rng, n=300, d=8, G=3, M=12, **kw):
    K = rng.normal(size=(n, d)); V = rng.normal(size=(n, d))
    u = O.OracleUnit(d, G, n + 64, 4 * M, **kw)
    u.build(K, V, M, 5, seed=int(rng.integers(1 << 30)))
    return u, K, V


def test_scores_are_group_mean_inner_products():
    rng = np.random.default_rng(8)
    u, K, V = _unit(rng)
    q = rng.normal(size=(3, 8))
    s = u.scores(q)
    ref = np.einsum("gd,md->m", q, u.centroids()) / 3.0
    assert np.allclose(s[u.live()], ref[u.live()], rtol=1e-13)
    assert np.all(np.isneginf(s[~u.live()]))


@pytest.mark.parametrize("budget", [0, 1, 17, 60, 150, 299, 300, 10_000])
def test_select_is_bruteforce_prefix(budget):
    rng = np.random.default_rng(9)
    u, K, V = _unit(rng)
    q = rng.normal(size=(3, 8)); s = u.scores(q); cnt = u.counts(); live = u.live()
    ids, tok = u.select(s, budget)
    order = sorted([j for j in range(u.M) if live[j]], key=lambda j: (-s[j], j))
    exp, cum = [], 0
    for j in order:
        if cum + cnt[j] > budget:
            break
        exp.append(j); cum += cnt[j]
    if not exp and budget > 0:
        exp, cum = [order[0]], cnt[order[0]]
        assert u.status & O.ST_BUDGET_EXCEEDED
    assert list(ids) == exp and tok == cum


def test_select_equal_scores_break_by_id():
    K = np.array([[1.0, 0], [1, 0], [0, 1], [0, 1], [-1, 0], [-1, 0]])
    u = O.OracleUnit(2, 1, 8, 4, gamma=0, alpha=0)
    u.build(K, K, 3, 3, seed=1)
    s = np.array([1.0, 1.0, 1.0])
    ids, tok = u.select(s, 4)
    assert list(ids) == [0, 1]


# ------------------------------------------------------------------ attention

def _dense_attention(q, K, V):
    import torch
    qt = torch.tensor(q, dtype=torch.float64)[None]              # [1, G, d]
    out = torch.nn.functional.scaled_dot_product_attention(
        qt.transpose(0, 1), torch.tensor(K)[None].expand(q.shape[0], -1, -1),
        torch.tensor(V)[None].expand(q.shape[0], -1, -1))
    return out[:, 0].numpy()


def test_attention_hand_worked_fixture():
    g = _gold("attention_2tok.txt")
    K = np.stack([g["k0"], g["k1"]]); V = np.stack([g["v0"], g["v1"]])
    u = O.OracleUnit(4, 1, 4, 2, gamma=0, alpha=0)
    u.build(K, V, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    out, ids, tok = u.decode_step(g["q"][None], 10)
    assert list(ids) == [0] and tok == 2
    assert np.allclose(out[0], g["out"], atol=1e-15)


def test_full_budget_retrieval_equals_dense_softmax_attention():
    rng = np.random.default_rng(10)
    u, K, V = _unit(rng, n=257, d=16, G=4, M=9)
    q = rng.normal(size=(4, 16)) * 2
    out, ids, tok = u.decode_step(q, 10_000)
    assert tok == 257 and sorted(ids) == [j for j in range(u.M) if u.live()[j]]
    assert np.allclose(out, _dense_attention(q, K, V), atol=1e-12)


def test_partial_retrieval_is_attention_over_selected_members_only():
    rng = np.random.default_rng(11)
    u, K, V = _unit(rng, n=200, d=8, G=2, M=10)
    q = rng.normal(size=(2, 8))
    out, ids, tok = u.decode_step(q, 70)
    a = u.assign(); mask = np.isin(a, ids)
    assert 0 < mask.sum() == tok <= 70
    assert np.allclose(out, _dense_attention(q, K[mask], V[mask]), atol=1e-12)
    # order of the selected ids does not matter
    assert np.allclose(u.attend(q, ids[::-1]), out, atol=1e-13)


def test_single_token_selection_returns_its_value_and_empty_gives_zero():
    K = np.array([[5.0, 0], [0, 5.0], [0, 5.1]]); V = np.array([[1.0, 2], [3, 4], [5, 6]])
    u = O.OracleUnit(2, 1, 4, 3, gamma=0, alpha=0)
    u.build(K, V, 2, 3, seed=4)
    a = u.assign()
    j0 = a[0]
    assert (a == j0).sum() == 1
    assert np.allclose(u.attend(np.array([[0.3, -2.0]]), [j0]), V[0][None], atol=1e-15)
    out, ids, tok = u.decode_step(np.array([[1.0, 1.0]]), 0)
    assert len(ids) == 0 and np.all(out == 0)


def test_attention_large_logits_do_not_overflow():
    K = np.array([[400.0, 0], [399.0, 0]]); V = np.array([[1.0, 0], [0, 1.0]])
    u = O.OracleUnit(2, 1, 4, 2, gamma=0, alpha=0)
    u.build(K, V, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    out = u.attend(np.array([[10.0, 0]]), [0])
    w = 1 / (1 + math.exp(-10 / math.sqrt(2)))
    assert np.allclose(out[0], [w, 1 - w], atol=1e-14)


# ------------------------------------------------------------------ split

def test_split_separates_two_blobs_and_keeps_invariants():
    rng = np.random.default_rng(12)
    A = rng.normal(size=(30, 5)) * 0.1 + 10; B = rng.normal(size=(20, 5)) * 0.1 - 10
    K = np.concatenate([A, B]); perm = rng.permutation(50); K = K[perm]
    is_a = perm < 30
    u = O.OracleUnit(5, 1, 64, 4, gamma=0, alpha=1.0, split_min_size=2)
    u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    parent_M2 = u.M2()[0]
    u.tau = 1.0
    assert u.split_check() == 1 and u.M == 2
    a = u.assign(); cnt = u.counts()
    assert cnt.sum() == 50 and sorted(cnt) == [20, 30]
    assert len(set(a[is_a])) == 1 and len(set(a[~is_a])) == 1 and a[is_a][0] != a[~is_a][0]
    assert a[0] == 0                                   # child with the smallest token id keeps the id
    for j in (0, 1):
        mem = K[a == j]
        assert np.allclose(u.centroids()[j], mem.mean(0), atol=1e-13)
        assert np.isclose(u.M2()[j], ((mem - mem.mean(0)) ** 2).sum(), rtol=1e-12)
    assert u.M2().sum() <= parent_M2
    # no longer triggered: a second check does nothing
    assert u.split_check() == 0


def test_split_identical_members_is_abandoned_until_next_append():
    K = np.ones((12, 3))
    u = O.OracleUnit(3, 1, 32, 4, gamma=0.5, alpha=0, split_min_size=2)
    u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    assert u.split_check() == 0 and u.M == 1
    assert u.split_check() == 0
    u.append(np.array([9.0, 9, 9]), np.zeros(3))       # lifts the hold; now separable
    assert u.split_check() == 1
    a = u.assign()
    assert list(a[:12]) == [0] * 12 and a[12] == 1


def test_size_trigger_and_ascending_ids_and_cap():
    rng = np.random.default_rng(13)
    big1 = rng.normal(size=(40, 2)) + [100, 0]; big2 = rng.normal(size=(40, 2)) + [-100, 0]
    small = np.array([[0.0, 50 + i] for i in range(6)] + [[0.0, -50 - i] for i in range(6)])
    K = np.concatenate([big1, small, big2])
    u = O.OracleUnit(2, 1, 128, 5, gamma=1.5, alpha=0, split_min_size=8)
    u.build(K, K, 4, 6, seed=3)
    cnt0 = u.counts().copy()
    trig = [j for j in range(4) if cnt0[j] * 4 > 1.5 * 92 and cnt0[j] >= 8]
    assert len(trig) == 2
    assert u.split_check() == 1                         # cap: only one id left (max_clusters = 5)
    assert u.status & O.ST_MAX_CLUSTERS
    a = u.assign(); cnt = u.counts()
    assert u.M == 5 and cnt.sum() == 92
    assert cnt[trig[0]] + cnt[4] == cnt0[trig[0]]       # lowest triggered id was the one split
    assert cnt[trig[1]] == cnt0[trig[1]]


def test_min_size_blocks_split():
    K = np.array([[0.0], [100.0], [0.1], [100.1]])
    u = O.OracleUnit(1, 1, 8, 4, gamma=0.1, alpha=0, split_min_size=8)
    u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    assert u.split_check() == 0


# ------------------------------------------------------------------ hints (tie-follow)

def test_hint_adopted_only_within_tolerance():
    K = np.array([[0.0, 0.0], [0.0, 0.0]])
    Cn = np.array([[1.0, 0.0], [-1.0 - 1e-7, 0.0], [3.0, 0.0]])
    a, ties, viol = O.assign(K, Cn, hint=[1, 2])
    assert list(a) == [1, 0] and ties == 1 and viol == 1
    u = O.OracleUnit(2, 1, 8, 4, gamma=0, alpha=0)
    Kb = np.array([[1.0, 0], [1.0, 0], [-1.0 - 1e-7, 0], [-1.0 - 1e-7, 0]])
    u.build(Kb, Kb, 2, 2, seed=1)
    j_far = u.append(np.array([0.0, 0.0]), np.zeros(2), hint_cluster=int(u.assign()[2]))
    assert j_far == u.assign()[2] and u.ties == 1 and u.violations == 0


def test_select_hint_validation():
    K = np.array([[1.0, 0], [1.0, 0], [0, 1.0], [0, 1.0], [-1.0, 0], [-1.0, 0]])
    u = O.OracleUnit(2, 1, 8, 4, gamma=0, alpha=0)
    u.build(K, K, 3, 3, seed=1)
    s = np.array([1.0, 1.0 + 1e-8, 0.5])
    ids, tok = u.select(s, 2)
    assert list(ids) == [1]
    ids, tok = u.select(s, 2, hint_ids=[0])             # near-tied top: accepted
    assert list(ids) == [0] and u.ties == 1
    ids, tok = u.select(s, 2, hint_ids=[2])             # clearly worse: rejected
    assert list(ids) == [1] and u.violations == 1
    ids, tok = u.select(s, 4, hint_ids=[1])             # stops early though the next one fits: rejected
    assert list(ids) == [1, 0] and u.violations == 2


def _unit_with_sizes(sizes):
    """A unit whose cluster j holds sizes[j] copies of the 1-D key 10 * j (three Lloyd rounds from the first keys
    of a seed that picks one key per value)."""
    K = np.concatenate([np.full(s, 10.0 * j) for j, s in enumerate(sizes)])[:, None]
    M = len(sizes)
    for seed in range(2000):
        picks = O.init_random(len(K), M, seed, 0)
        if len({K[p, 0] for p in picks}) == M:
            break
    else:
        raise AssertionError("no seed found")
    u = O.OracleUnit(1, 1, len(K) + 2, M + 2, gamma=0, alpha=0)
    u.build(K, K, M, 2, seed=seed, init_mode=O.INIT_RANDOM)
    assert sorted(u.counts()) == sorted(sizes)
    # cluster ids follow the picks' order, not the values: map value -> id
    ids = {int(round(u.centroids()[j, 0] / 10.0)): j for j in range(M)}
    return u, ids


def test_select_hint_of_one_over_budget_cluster_is_checked():
    # three clusters of 3 tokens, scores (3, 2, 1), budget 2: nothing fits, the best cluster is taken alone.
    # A hint naming the worst cluster alone is over budget too, but it is not the best: a violation.
    u, ids = _unit_with_sizes([3, 3, 3])
    s = np.zeros(3); s[ids[0]], s[ids[1]], s[ids[2]] = 3.0, 2.0, 1.0
    own, tok = u.select(s, 2)
    assert list(own) == [ids[0]] and tok == 3
    got, _ = u.select(s, 2, hint_ids=[ids[2]])
    assert list(got) == [ids[0]] and u.violations == 1 and u.ties == 0
    # the same over-budget answer with a near-tied score is a tie
    s2 = s.copy(); s2[ids[1]] = 3.0 - 1e-8
    got, _ = u.select(s2, 2, hint_ids=[ids[1]])
    assert list(got) == [ids[1]] and u.violations == 1 and u.ties == 1
    # sizes (2, 9, 2), budget 5: the two small clusters fit (4 tokens); the 9-token, lowest-scoring cluster
    # alone is no valid answer
    u, ids = _unit_with_sizes([2, 9, 2])
    s = np.zeros(3); s[ids[0]], s[ids[1]], s[ids[2]] = 3.0, 1.0, 2.0
    own, tok = u.select(s, 5)
    assert list(own) == [ids[0], ids[2]] and tok == 4
    got, tok = u.select(s, 5, hint_ids=[ids[1]])
    assert list(got) == [ids[0], ids[2]] and tok == 4 and u.violations == 1 and u.ties == 0
    # an over-budget hint of one cluster that DOES tie the best score, while the oracle's own answer is within
    # budget, is not an answer the selection rule can give either
    s3 = s.copy(); s3[ids[1]] = 3.0
    got, _ = u.select(s3, 5, hint_ids=[ids[1]])
    assert u.violations == 2


def test_two_means_round_cap_hand_worked_fixture():
    """The round cap of the split's local clustering: with split_iters = 1 or 2 the partition is the capped one,
    not the converged one (hand-worked in the fixture)."""
    g = _gold("two_means_cap_1d.txt")
    K = g["members"][:, None]
    for cap in (1, 2, 3, 8):
        u = O.OracleUnit(1, 1, 16, 4, gamma=0.5, alpha=0, split_min_size=2, split_iters=cap)
        u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
        assert u.split_check() == 1
        assert list(u.assign()) == list(g[f"assign_cap{cap}"].astype(int)), f"cap {cap}"
        if f"centres_cap{cap}" in g:
            # children's representatives are the member means of the final labels (UpdateStats)
            assert np.allclose(u.centroids()[:2, 0], g[f"centres_cap{cap}"], atol=1e-12)
    assert not np.array_equal(g["assign_cap1"], g["assign_cap2"]) and not np.array_equal(g["assign_cap2"], g["assign_cap8"])


def test_two_means_equidistant_member_goes_to_centre_a():
    # members 0, 10, 5 around r = 5: A = token 0 (first of the two farthest), B = token 1;
    # token 2 is equidistant and must join A, so the moved child is {10} alone.
    K = np.array([[0.0], [10.0], [5.0]])
    u = O.OracleUnit(1, 1, 8, 4, gamma=0.5, alpha=0, split_min_size=2)
    u.build(K, K, 1, 1, seed=0, init_mode=O.INIT_RANDOM)
    assert u.split_check() == 1
    assert list(u.assign()) == [0, 1, 0]


def _unit_with_dead_cluster(**kw):
    K = np.array([[0.0], [0.0], [10.0], [10.5], [0.0], [0.0], [10.2], [10.1], [0.0], [10.3]])
    for seed in range(200):
        picks = O.init_random(len(K), 3, seed, 0)
        if picks[0] == 0 and picks[1] == 1:
            break
    else:
        raise AssertionError("no seed found")
    u = O.OracleUnit(1, 1, 16, 8, **kw)
    u.build(K, K, 3, 3, seed=seed, init_mode=O.INIT_RANDOM)
    return u, K


def test_dead_cluster_is_excluded_everywhere():
    u, K = _unit_with_dead_cluster(gamma=0, alpha=2.0)
    live = u.live(); cnt = u.counts()
    assert list(live) == [True, False, True] and cnt[1] == 0
    var = u.M2()[live] / cnt[live]
    assert np.isclose(u.tau, 2.0 * var.mean(), rtol=1e-12)       # mean over live clusters only
    assert np.isneginf(u.scores(np.array([[1.0]]))[1])
    assert u.append(np.array([0.0]), np.array([0.0])) == 0       # never the dead twin at the same spot


def test_size_trigger_uses_live_cluster_count():
    # 10 tokens, clusters of 5 and 5 plus one dead id.  gamma = 1.2: mean live size is 5, so
    # 5 * 2 live > 1.2 * 10 fails (no split); counting the dead id (5 * 3 > 12) would split.
    u, K = _unit_with_dead_cluster(gamma=1.2, alpha=0, split_min_size=2)
    assert sorted(u.counts()) == [0, 5, 5]
    assert u.split_check() == 0


# ------------------------------------------------------------------ installing a partition

def test_install_reproduces_the_state_of_a_build():
    """A partition installed from outside must give exactly the statistics the oracle's own build ends with
    (same member means, M2, sizes, tau), and decode from there must agree."""
    rng = np.random.default_rng(5)
    K = rng.normal(size=(300, 16)); V = rng.normal(size=(300, 16))
    a = O.OracleUnit(16, 2, 400, 32)
    a.build(K, V, 9, 4, 77, init_mode=O.INIT_RANDOM)
    b = O.OracleUnit(16, 2, 400, 32)
    b.install(K, V, a.assign(), a.M)
    assert np.array_equal(a.counts(), b.counts()) and np.array_equal(a.live(), b.live())
    assert np.allclose(a.centroids(), b.centroids(), rtol=0, atol=1e-13)
    assert np.allclose(a.M2(), b.M2(), rtol=1e-12) and abs(a.tau - b.tau) <= 1e-12 * a.tau
    q = rng.normal(size=(2, 16))
    oa, ia, _ = a.decode_step(q, 120); ob, ib, _ = b.decode_step(q, 120)
    assert list(ia) == list(ib) and np.allclose(oa, ob, atol=1e-13)
    # centroid of an installed cluster is the plain mean of its members
    j = int(np.argmax(b.counts()))
    assert np.allclose(b.centroids()[j], K[a.assign() == j].mean(0), atol=1e-13)


# ------------------------------------------------------------------ update modes (static / local)

def _mode_stream(seed=3, n0=300, d=8, steps=160):
    rng = np.random.default_rng(seed)
    means = rng.normal(size=(6, d)) * 4.0
    K0 = means[rng.integers(0, 6, n0)] + 0.3 * rng.normal(size=(n0, d))
    # decode keys drift away from the prefill mixture
    Kd = means[rng.integers(0, 6, steps)] + 0.3 * rng.normal(size=(steps, d)) + np.linspace(0, 6, steps)[:, None]
    return K0, Kd


def test_static_mode_never_splits_and_appends_to_the_nearest_representative():
    K0, Kd = _mode_stream()
    u = O.OracleUnit(K0.shape[1], 1, 600, 64, gamma=1.2, alpha=1.2, split_min_size=4, mode=O.MODE_STATIC)
    u.build(K0, K0, 8, 3, seed=2, init_mode=O.INIT_RANDOM)
    for k in Kd:
        C, live = u.centroids(), u.live()
        dist = ((C - k[None]) ** 2).sum(1)
        dist[~live] = np.inf
        j = u.append(k, k)
        assert j == int(np.argmin(dist))                       # brute force over the representatives as they were
        assert u.split_check() == 0
    assert u.M == 8 and u.n_splits == 0
    # the same stream with the split rules on does split: the mode is what keeps the partition static
    a = O.OracleUnit(K0.shape[1], 1, 600, 64, gamma=1.2, alpha=1.2, split_min_size=4)
    a.build(K0, K0, 8, 3, seed=2, init_mode=O.INIT_RANDOM)
    for k in Kd:
        a.append(k, k); a.split_check()
    assert a.n_splits > 0


def test_local_mode_keeps_the_build_frozen_and_clusters_new_entries_among_themselves():
    K0, Kd = _mode_stream()
    M0, local_max = 8, 24
    u = O.OracleUnit(K0.shape[1], 1, 600, 64, gamma=1.2, alpha=1.2, split_min_size=4, mode=O.MODE_LOCAL, local_max=local_max)
    u.build(K0, K0, M0, 3, seed=2, init_mode=O.INIT_RANDOM)
    C0, n0, m20, a0 = u.centroids().copy(), u.counts().copy(), u.M2().copy(), u.assign().copy()
    first = u.append(Kd[0], Kd[0])
    assert first == M0 and u.M == M0 + 1                       # the first new entry founds a cluster of its own
    assert np.array_equal(u.centroids()[M0], Kd[0]) and u.M2()[M0] == 0.0 and u.counts()[M0] == 1
    u.split_check()
    for k in Kd[1:]:
        C, live = u.centroids(), u.live()
        dist = ((C - k[None]) ** 2).sum(1)
        dist[~live] = np.inf
        dist[:M0] = np.inf                                      # only decode-born clusters are candidates
        j = u.append(k, k)
        assert j == int(np.argmin(dist)) and j >= M0
        u.split_check()
        assert u.counts()[M0:].max() <= local_max               # a cluster above the limit has just been split
    # the clusters of the build are exactly as the build left them
    assert np.array_equal(u.centroids()[:M0], C0) and np.array_equal(u.counts()[:M0], n0)
    assert np.array_equal(u.M2()[:M0], m20) and np.array_equal(u.assign()[: len(a0)], a0)
    assert np.all(u.assign()[len(a0):] >= M0) and u.n_splits > 0
    # Eq. 3 / Eq. 4 hold for the new clusters too
    A = u.assign(); Kall = np.concatenate([K0, Kd])
    for j in range(M0, u.M):
        mem = Kall[A == j]
        assert len(mem) == u.counts()[j] and np.allclose(mem.mean(0), u.centroids()[j], atol=1e-10)


def test_local_mode_separates_two_new_blobs_when_the_size_limit_is_reached():
    rng = np.random.default_rng(8)
    K0 = rng.normal(size=(100, 4))
    blobs = np.array([[50.0, 0, 0, 0], [0, 50.0, 0, 0]])
    lab = np.arange(41) % 2
    Kd = blobs[lab] + 0.1 * rng.normal(size=(41, 4))
    u = O.OracleUnit(4, 1, 200, 16, split_min_size=4, mode=O.MODE_LOCAL, local_max=40)
    u.build(K0, K0, 4, 2, seed=1, init_mode=O.INIT_RANDOM)
    for k in Kd:
        u.append(k, k); u.split_check()
    A = u.assign()[100:]
    assert u.M == 6 and u.n_splits == 1                          # one founding, one split at 41 entries
    assert len(set(A[lab == 0])) == 1 and len(set(A[lab == 1])) == 1 and A[0] != A[1]


# ---------------------------------------------------------------------------------------------------------------
# Delayed split (Algorithm 1, its last two blocks; Section 4.2): hand-built clusters on a line, so that which cluster a
# query retrieves, which cluster an entry joins and when a variance trigger fires can all be read off the numbers.

def _delayed_unit(buf_max, extra_cluster=False, mode=None):
    """Cluster A: six entries at x = -0.05 .. 0.05; cluster B: six at 9.95 .. 10.05; optionally C: six around 30.
    tau = 0.5: an entry 4 away from B's (or C's) centre lifts that cluster's variance over it."""
    xs = [np.linspace(-0.05, 0.05, 6), 10 + np.linspace(-0.05, 0.05, 6)] + ([30 + np.linspace(-0.05, 0.05, 6)] if extra_cluster else [])
    K = np.stack([np.concatenate(xs), np.zeros(6 * len(xs))], axis=1)
    assign = np.repeat(np.arange(len(xs)), 6).astype(np.int32)
    u = O.OracleUnit(2, 1, 64, 16, gamma=0.0, alpha=1.0, split_min_size=2,
                     mode=O.MODE_DELAYED if mode is None else mode, buf_max=buf_max)
    u.install(K, K, assign, len(xs))
    u.tau = 0.5
    return u


def _retrieve(u, x):
    """A query that scores cluster centres by x * centre: positive x retrieves the cluster farthest right, negative x
    cluster A (score 0 against negative scores); the budget holds one cluster."""
    _, ids, _ = u.decode_step(np.array([[x, 0.0]]), 9)
    return list(ids)


def test_delayed_split_waits_until_the_flagged_cluster_is_retrieved():
    u = _delayed_unit(buf_max=100)
    assert _retrieve(u, -1.0) == [0]                      # the query retrieves A
    assert u.append(np.array([14.0, 0.0]), np.zeros(2)) == 1    # the entry joins B and lifts its variance over tau
    assert u.counts()[1] == 7 and u.M2()[1] / 7 > 0.5
    assert u.split_check() == 0                           # B is not among the retrieved clusters: flagged, not split
    f, b = u.flags()
    assert list(f) == [False, True] and list(b) == [0, 1] and u.M == 2
    assert _retrieve(u, -1.0) == [0]
    assert u.append(np.array([14.5, 0.0]), np.zeros(2)) == 1    # buffered for the flagged cluster
    assert u.split_check() == 0
    f, b = u.flags()
    assert list(b) == [0, 2] and u.M == 2
    assert _retrieve(u, 1.0) == [1]                       # now the query retrieves B (8 entries, budget 9)
    assert u.append(np.array([10.0, 0.1]), np.zeros(2)) == 1
    assert u.split_check() == 1                           # the owed split happens, on the cluster with its buffered entries
    f, b = u.flags()
    assert not f.any() and not b.any() and u.M == 3
    a = u.assign()
    assert list(a[:6]) == [0] * 6 and list(a[6:12]) == [1] * 6 and a[14] == 1      # the entries near 10 stay cluster 1
    assert a[12] == 2 and a[13] == 2                      # the two far entries are the new cluster
    # the same members split by the adaptive rule (no delay) give the same partition
    v = _delayed_unit(buf_max=100, mode=O.MODE_ADAPTIVE)
    for x, y in ((14.0, 0.0), (14.5, 0.0), (10.0, 0.1)):
        v.append(np.array([x, y]), np.zeros(2))
    assert v.split_check() == 1 and np.array_equal(v.assign(), a)


def test_delayed_split_is_immediate_for_a_retrieved_cluster():
    u = _delayed_unit(buf_max=100)
    assert _retrieve(u, 1.0) == [1]
    u.append(np.array([14.0, 0.0]), np.zeros(2))
    assert u.split_check() == 1 and u.M == 3 and not u.flags()[0].any()


def test_buffered_entries_reaching_buf_max_force_the_split_of_the_fullest_flagged_cluster():
    u = _delayed_unit(buf_max=3, extra_cluster=True)
    _retrieve(u, -1.0)
    assert u.append(np.array([14.0, 0.0]), np.zeros(2)) == 1 and u.split_check() == 0       # B flagged, 1 buffered
    _retrieve(u, -1.0)
    assert u.append(np.array([34.0, 0.0]), np.zeros(2)) == 2 and u.split_check() == 0       # C flagged, 1 buffered; total 2 < 3
    f, b = u.flags()
    assert list(f) == [False, True, True] and list(b) == [0, 1, 1]
    _retrieve(u, -1.0)
    assert u.append(np.array([34.5, 0.0]), np.zeros(2)) == 2                                # C: 2 buffered; total 3
    assert u.split_check() == 1                           # nothing flagged is retrieved, but the buffers are full: C goes
    f, b = u.flags()
    assert list(f[:3]) == [False, True, False] and list(b[:3]) == [0, 1, 0] and u.M == 4
    a = u.assign()
    assert a[19] == 3 and a[20] == 3 and list(a[12:18]) == [2] * 6
    # with equal buffers the lower id goes first
    w = _delayed_unit(buf_max=2, extra_cluster=True)
    _retrieve(w, -1.0)
    w.append(np.array([14.0, 0.0]), np.zeros(2)); assert w.split_check() == 0
    _retrieve(w, -1.0)
    w.append(np.array([34.0, 0.0]), np.zeros(2)); assert w.split_check() == 1               # total 2: B (id 1) before C
    f, b = w.flags()
    assert list(f[:3]) == [False, False, True]
