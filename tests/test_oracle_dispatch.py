"""Pins for the oracle's count + quota dispatch + padded layout (no GPU).

The pins are things the oracle does not define itself: numpy.bincount, numpy's stable
argsort (a counting sort by expert), the exact-quota and bijection invariants that follow
from Eq. 2's constraints, Eq. 3's tile count, and an independent sort-and-cut brute force.
"""
import numpy as np
import pytest

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W


def _dispatch(wl, M_cap=None, **kw):
    return O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max,
                            wl.M_cap if M_cap is None else M_cap, **kw)


def _all_small_and_configs():
    yield W.config1()
    yield W.config2()
    yield W.config2(n_valid=200)
    for c in ("uniform", "token_balanced", "hot_whole"):
        yield W.config3(c, T=512)
    for s in range(12):
        yield W.random_small(100 + s)
    yield W.random_small(7, T=9, n_valid=5)
    yield W.config5_point(4, 129, with_x=False)


def brute_force(ids, n_valid, replica_map, quota, G_max):
    """Sort live pairs by (expert, pair index); cut each expert's list by its quotas in column order.

    Only valid for well-formed tables with sum_r quota[e, r] == n_e (the nominal case).
    Returns {slot: [pairs in order]}.
    """
    T, k = ids.shape
    live = [(int(ids[p // k, p % k]), p) for p in range(n_valid * k)]
    live.sort()
    per_slot = {i: [] for i in range(G_max)}
    E, R = replica_map.shape
    for e in range(E):
        mine = [p for (ee, p) in live if ee == e]
        cut = 0
        for r in range(R):
            s = int(replica_map[e, r])
            if s >= 0:
                per_slot[s] = mine[cut:cut + int(quota[e, r])]
                cut += int(quota[e, r])
    return per_slot


@pytest.mark.parametrize("wl", list(_all_small_and_configs()), ids=lambda w: w.name)
def test_counts_match_bincount_and_sum(wl):
    r = _dispatch(wl)
    live = wl.topk_ids[:wl.n_valid].reshape(-1)
    assert np.array_equal(r["counts"], np.bincount(live, minlength=wl.E))
    assert int(r["counts"].sum()) == wl.n_valid * wl.k          # every live pair counted once
    assert int(r["status"]) == 0


@pytest.mark.parametrize("wl", list(_all_small_and_configs()), ids=lambda w: w.name)
def test_quota_honoured_exactly_and_layout(wl):
    r = _dispatch(wl)
    pair_row, row_pair = r["pair_row"], r["row_pair"]
    inst_off, inst_count = r["inst_off"], r["inst_count"]
    # exact quotas (sum_r x_{e,r} = n_e holds for every generated table)
    for e in range(wl.E):
        local = any(wl.replica_map[e] >= 0)
        if local:
            assert int(wl.quota[e][wl.replica_map[e] >= 0].sum()) == int(r["counts"][e])
        for c in range(wl.R_max):
            s = int(wl.replica_map[e, c])
            if s >= 0:
                assert int(inst_count[s]) == int(wl.quota[e, c])
    # Eq. 3: padded rows = sum over instances of ceil(m/128)*128; offsets are tile multiples
    assert int(r["m_pad"]) == int(sum(-(-int(m) // 128) * 128 for m in inst_count))
    assert all(int(o) % 128 == 0 for o in inst_off)
    # bijection between local live pairs and non-pad rows
    rows = pair_row[pair_row >= 0]
    assert len(set(rows.tolist())) == len(rows)
    for p in np.nonzero(pair_row >= 0)[0]:
        assert row_pair[pair_row[p]] == p
    assert int((row_pair >= 0).sum()) == len(rows) == int(inst_count.sum())
    # inside an instance: live rows first, ascending pair index, correct expert, then pad rows
    for i in range(wl.G_max):
        lo, m = int(inst_off[i]), int(inst_count[i])
        ps = row_pair[lo:lo + m]
        assert np.all(ps >= 0) and np.all(np.diff(ps) > 0)
        assert np.all(wl.topk_ids.reshape(-1)[ps] == wl.slot_expert[i])
        assert np.all(row_pair[lo + m:int(inst_off[i + 1])] == -1)
    assert np.all(row_pair[int(r["m_pad"]):] == -1)
    # dead rows and remote experts are not dispatched
    assert np.all(pair_row[wl.n_valid * wl.k:] == -1)
    remote = ~np.isin(wl.topk_ids.reshape(-1), np.nonzero((wl.replica_map >= 0).any(1))[0])
    assert np.all(pair_row[remote] == -1)
    # tile list
    tiles = int(r["m_pad"]) // 128
    expect = np.concatenate([np.full((int(inst_off[i + 1]) - int(inst_off[i])) // 128, i)
                             for i in range(wl.G_max)] + [np.zeros(0, int)])
    assert np.array_equal(r["tile_inst"][:tiles], expect)
    assert np.all(r["tile_inst"][tiles:] == -1)


@pytest.mark.parametrize("wl", list(_all_small_and_configs()), ids=lambda w: w.name)
def test_matches_sort_and_cut_brute_force(wl):
    r = _dispatch(wl)
    bf = brute_force(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max)
    for i in range(wl.G_max):
        lo, m = int(r["inst_off"][i]), int(r["inst_count"][i])
        assert r["row_pair"][lo:lo + m].tolist() == bf[i]


def test_no_replicas_is_a_stable_counting_sort():
    wl = W.config5_point(8, 37, with_x=False)
    ids = np.random.default_rng(5).integers(0, 8, size=(wl.T, 1)).astype(np.int32)
    quota = np.bincount(ids.reshape(-1), minlength=8).astype(np.int32).reshape(8, 1)
    r = O.count_dispatch(ids, wl.T, wl.replica_map, quota, 8, wl.M_cap)
    order = np.argsort(ids.reshape(-1), kind="stable")
    assert np.array_equal(r["row_pair"][r["row_pair"] >= 0], order)


def test_replica_runs_concatenate_to_the_stable_list():
    wl = W.config3("token_balanced", T=512)
    r = _dispatch(wl)
    flat = wl.topk_ids.reshape(-1)
    for e in np.nonzero((wl.replica_map >= 0).any(1))[0]:
        runs = []
        for c in range(wl.R_max):
            s = int(wl.replica_map[e, c])
            if s >= 0:
                lo, m = int(r["inst_off"][s]), int(r["inst_count"][s])
                runs += r["row_pair"][lo:lo + m].tolist()
        assert runs == np.nonzero(flat[:wl.n_valid * wl.k] == e)[0].tolist()


# ---- degenerate tables (Section 4.4: torn or stale rows must stay safe) -----------------------

def _one_expert(n, slots, quotas, G_max=4, T=None):
    T = n if T is None else T
    ids = np.zeros((T, 1), np.int32)
    rmap = np.array([slots], np.int32)
    q = np.array([quotas], np.int32)
    return O.count_dispatch(ids, n, rmap, q, G_max, 128 * 16)


@pytest.mark.parametrize("nrep", [1, 2, 3])
@pytest.mark.parametrize("n", [0, 1, 7, 300])
def test_zero_sum_row_falls_back_to_uniform(n, nrep):
    slots = list(range(nrep)) + [-1] * (3 - nrep)
    r = _one_expert(n, slots, [0, 0, 0])
    m = r["inst_count"][:nrep]
    assert int(m.sum()) == n and int(m.max() - m.min()) <= 1
    assert int(r["status"]) == 0


@pytest.mark.parametrize("quotas", [(600, 200, 0), (3, 1, 0), (1, 1, 1), (0, 5, 0)])
def test_stale_row_is_renormalised(quotas):
    n = 301
    r = _one_expert(n, [0, 1, 2], list(quotas))
    S = sum(quotas)
    m = r["inst_count"][:3]
    assert int(m.sum()) == n
    for i in range(3):
        assert abs(int(m[i]) - quotas[i] * n / S) < 1
    assert int(r["status"]) == 0


def test_never_routes_to_a_replica_without_the_expert():
    r = _one_expert(50, [0, -1, 2], [10, 25, 15])       # share on a column that holds nothing
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert int(r["inst_count"][1]) == 0 and int(r["inst_count"][3]) == 0
    assert int(r["inst_count"][0] + r["inst_count"][2]) == 50
    assert int(r["inst_count"][0]) == 20 and int(r["inst_count"][2]) == 30   # 10:15 renormalised


def test_bad_entries_are_flagged_and_ignored():
    r = _one_expert(40, [0, 9, 1], [20, 10, 20])        # slot 9 out of range
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert r["inst_count"].tolist() == [20, 20, 0, 0]
    r = _one_expert(40, [0, 1, -1], [-5, 40, 0])        # negative share counts as zero
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert r["inst_count"].tolist() == [0, 40, 0, 0]
    # slot claimed twice: the later (expert, column) loses it
    ids = np.array([[0], [1], [1], [0]], np.int32)
    rmap = np.array([[0], [0]], np.int32)
    q = np.array([[2], [2]], np.int32)
    r = O.count_dispatch(ids, 4, rmap, q, 1, 256)
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert r["pair_row"].tolist() == [0, -1, -1, 1]
    # id out of range on a live row
    ids = np.array([[0], [5], [-1], [0]], np.int32)
    r = O.count_dispatch(ids, 4, np.array([[0]], np.int32), np.array([[2]], np.int32), 1, 256)
    assert int(r["status"]) & O.STATUS_BAD_ID
    assert r["counts"].tolist() == [2] and r["pair_row"].tolist() == [0, -1, -1, 1]


def test_absurd_shares_count_as_zero_and_never_pick_a_wrong_replica():
    big = 2 ** 31 - 1
    r = _one_expert(300, [0, 1, 2], [big, big, 7])      # two torn entries: the third column takes everything
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert r["inst_count"][:3].tolist() == [0, 0, 300]
    r = _one_expert(300, [0, 1, 2], [big, big, big])    # nothing usable left: uniform over the holders
    assert int(r["status"]) & O.STATUS_BAD_TABLE
    assert r["inst_count"][:3].tolist() == [100, 100, 100]
    r = _one_expert(300, [0, 1, 2], [2 ** 30, 2 ** 30, 2 ** 29])   # the largest legal shares, 2:2:1
    assert int(r["status"]) == 0
    assert r["inst_count"][:3].tolist() == [120, 120, 60]


def test_padding_rows_are_masked_and_counter_wraps():
    wl = W.config2(n_valid=200)
    cum = np.full(wl.E, 2 ** 32 - 3, np.uint32)
    r = _dispatch(wl, cum_counts=cum)
    assert int(r["counts"].sum()) == 200 * wl.k
    assert np.array_equal(r["cum_counts"], (cum.astype(np.uint64) + r["counts"]) % 2 ** 32)
    assert np.all(r["pair_row"][200 * wl.k:] == -1)
    r0 = O.count_dispatch(wl.topk_ids, 0, wl.replica_map, wl.quota * 0, wl.G_max, wl.M_cap)
    assert int(r0["m_pad"]) == 0 and np.all(r0["pair_row"] == -1) and int(r0["counts"].sum()) == 0


@pytest.mark.parametrize("m", [127, 128, 129])
def test_tile_boundaries(m):
    r = _one_expert(m, [0, -1, -1], [m, 0, 0])
    assert int(r["m_pad"]) == (128 if m <= 128 else 256)
    assert int((r["tile_inst"] == 0).sum()) == int(r["m_pad"]) // 128


def test_capacity_overflow_drops_rows_beyond_m_cap():
    ids = (np.arange(600, dtype=np.int32) % 2).reshape(600, 1)
    rmap = np.array([[0], [1]], np.int32)
    q = np.array([[300], [300]], np.int32)
    r = O.count_dispatch(ids, 600, rmap, q, 2, 640)     # needs 384 + 384 = 768 rows
    assert int(r["status"]) & O.STATUS_CAPACITY
    assert int(r["m_pad"]) == 640 and r["inst_off"].tolist() == [0, 384, 640]
    assert r["inst_count"].tolist() == [300, 256]
    assert int((r["pair_row"] >= 0).sum()) == 556 and int(r["pair_row"].max()) == 639
