"""Hand-worked sequences for the oracle's model of the cluster cache (Section 6: a cache of whole clusters; Section 6.2:
keep small clusters, retain recently updated ones).  Every expected number below was worked out on paper from the
model's stated rules, not produced by running it."""
import pytest

from oracle.cluster_cache import CacheTooSmall, ClusterCacheModel, pages


def test_pages_of_a_cluster():
    assert [pages(n) for n in (1, 31, 32, 33, 64, 65)] == [1, 1, 1, 2, 2, 3]


def test_first_use_fetches_whole_clusters_and_a_repeat_hits():
    m = ClusterCacheModel(10)
    size = {0: 40, 1: 10, 2: 64}            # 2 + 1 + 2 pages
    m.retrieve([0, 1, 2], size)
    assert m.c["pages_fetched"] == 5 and m.c["clusters_fetched"] == 3 and m.frames_in_use == 5
    assert m.c["rows_fetched"] == 40 + 10 + 64          # only rows that hold entries travel
    m.retrieve([2, 0], size)
    assert m.c["clusters_hit"] == 2 and m.c["pages_fetched"] == 5 and m.c["clusters_evicted"] == 0 and m.c["rows_fetched"] == 114


def test_an_appended_cluster_is_refreshed_from_its_former_last_page_on():
    m = ClusterCacheModel(10)
    size = {0: 40}
    m.retrieve([0], size)                   # 2 pages, the second holds 8 rows
    size[0] = 41                            # one append into the second page: that page again, no new frame
    m.retrieve([0], size)
    assert m.c["clusters_refreshed"] == 1 and m.c["pages_fetched"] == 3 and m.frames_in_use == 2
    size[0] = 64                            # fills the second page
    m.retrieve([0], size)
    assert m.c["pages_fetched"] == 4 and m.frames_in_use == 2
    size[0] = 70                            # the last page was full: only the new page is copied
    m.retrieve([0], size)
    assert m.c["pages_fetched"] == 5 and m.frames_in_use == 3 and m.c["clusters_refreshed"] == 3
    size[0] = 130                           # 70 -> 130: page 3 again (6 of 32 rows then) and pages 4, 5
    m.retrieve([0], size)
    assert m.c["pages_fetched"] == 8 and m.frames_in_use == 5 and m.c["clusters_fetched"] == 1
    assert m.c["rows_fetched"] == 40 + 1 + 23 + 6 + 60        # every entry travelled exactly once


def test_a_split_voids_the_copy_even_when_the_size_comes_back():
    m = ClusterCacheModel(10)
    size = {0: 64, 1: 0}
    m.retrieve([0], size)
    m.note_split(0)
    size[0], size[1] = 30, 34               # the split
    size[0] = 64                            # appends bring the old size back: still not the rows that were copied
    m.retrieve([0, 1], size)
    assert m.c["clusters_hit"] == 0 and m.c["copies_dropped_stale"] == 1 and m.c["clusters_fetched"] == 3
    assert m.c["pages_fetched"] == 2 + 2 + 2 and m.frames_in_use == 4


def test_replacement_takes_large_before_small_and_old_before_new():
    m = ClusterCacheModel(8)
    size = {0: 96, 1: 32, 2: 32, 3: 64, 4: 64}      # 3, 1, 1, 2, 2 pages
    m.retrieve([1], size)                   # turn 1
    m.retrieve([0], size)                   # turn 2
    m.retrieve([2], size)                   # turn 3
    m.retrieve([3], size)                   # turn 4: 7 of 8 frames in use
    assert m.frames_in_use == 7
    m.retrieve([4], size)                   # needs 2, 1 free: the 3-page cluster goes although others are older
    assert sorted(m.copies) == [1, 2, 3, 4] and m.c["clusters_evicted"] == 1 and m.frames_in_use == 6
    size[5] = 96
    m.retrieve([5], size)                   # needs 3, 2 free: among the 2-page clusters 3 (turn 4) is older than 4 (turn 5)
    assert sorted(m.copies) == [1, 2, 4, 5] and m.c["clusters_evicted"] == 2
    size[6] = 32 * 4
    m.retrieve([6], size)                   # needs 4, 1 free: 5 (3 pages) goes first, that suffices
    assert sorted(m.copies) == [1, 2, 4, 6] and m.c["clusters_evicted"] == 3


def test_equal_size_and_age_falls_back_to_the_lower_id():
    m = ClusterCacheModel(2)
    size = {7: 32, 3: 32, 9: 32}
    m.retrieve([7, 3], size)                # both copied in the same turn
    m.retrieve([9], size)
    assert sorted(m.copies) == [7, 9]


def test_updated_clusters_are_retained_and_void_copies_go_first():
    m = ClusterCacheModel(6)
    size = {0: 64, 1: 64, 2: 64}
    m.retrieve([0, 1, 2], size)             # cache full
    size[0] = 65                            # 0 took an append since it was copied: retained
    m.note_split(1)
    size[1], size[3] = 40, 24               # 1 was split: its copy is void
    size[4] = 64
    m.retrieve([4], size)                   # needs 2: the void copy of 1 is what goes
    assert sorted(m.copies) == [0, 2, 4] and m.c["copies_dropped_stale"] == 1 and m.c["clusters_evicted"] == 0
    size[5] = 64
    m.retrieve([5], size)                   # 0 (updated) and 2 (unchanged) are candidates, 4 is newer: 2 goes, not 0
    assert sorted(m.copies) == [0, 4, 5] and m.c["clusters_evicted"] == 1


def test_selected_clusters_are_never_evicted_and_too_small_a_cache_fails():
    m = ClusterCacheModel(4)
    size = {0: 64, 1: 64, 2: 32}
    m.retrieve([0, 1], size)
    m.retrieve([0, 2], size)                # 0 is in use, so 1 makes room
    assert sorted(m.copies) == [0, 2]
    with pytest.raises(CacheTooSmall):
        m.retrieve([0, 1, 2], size)         # 2 + 2 + 1 pages cannot fit 4 frames


def test_small_first_keeps_more_clusters_cached_than_plain_lru_on_a_decode_stream():
    """Section 6.2, principle 1, on a synthetic decode stream followed by the oracle (config 4's recipe at a reduced
    size): evicting large clusters first gives more cluster hits than least-recently-used order at the same cache
    size, for about the same number of pages copied (a large cluster costs more to bring back)."""
    import numpy as np
    import oracle as O
    from gen import CONFIGS, UnitStream, make_decode_chunk, make_prefill
    cfg = CONFIGS[4].scaled(n_prefill=2048, steps=150, M0=64, max_clusters=256, budget=256, T=3)
    s = [UnitStream(cfg, 0)]
    K, V = make_prefill(s)
    q, k, v = make_decode_chunk(s, cfg.steps)
    o = O.OracleUnit(cfg.d, cfg.G, cfg.max_tokens, cfg.max_clusters, gamma=cfg.split_size_factor, alpha=cfg.split_var_factor,
                     split_min_size=cfg.split_min_size, split_iters=cfg.split_iters)
    o.build(K[0].double().numpy(), V[0].double().numpy(), cfg.M0, cfg.T, 1234, unit_index=0, init_mode=O.INIT_RANDOM)
    frames = 40
    models = {order: ClusterCacheModel(frames, order) for order in ("small-first", "lru")}
    for t in range(cfg.steps):
        _, ids, _ = o.decode_step(q[t, 0].double().numpy(), cfg.budget)
        sizes = o.counts()
        for m in models.values():
            m.retrieve(ids, sizes)
        o.append(k[t, 0].double().numpy(), v[t, 0].double().numpy())
        before = o.counts().copy()
        o.split_check()
        for j in np.nonzero(o.counts()[: len(before)] < before)[0]:
            for m in models.values():
                m.note_split(int(j))
    hits = {name: m.c["clusters_hit"] + m.c["clusters_refreshed"] for name, m in models.items()}
    fetched = {name: m.c["pages_fetched"] for name, m in models.items()}
    print(f"\ncluster hits {hits}, pages copied {fetched}, {frames} frames")
    assert min(m.c["clusters_evicted"] for m in models.values()) > 100
    assert hits["small-first"] > 1.1 * hits["lru"]
    assert abs(fetched["small-first"] - fetched["lru"]) < 0.1 * fetched["lru"]
