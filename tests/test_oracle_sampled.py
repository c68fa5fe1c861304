"""Pins for the oracle's sampled (probabilistic) dispatch (no GPU): the generator's published known-answer
vectors, replica frequencies against the shares, the zero-sum / invalid-column rules, layout invariants."""
import os

import numpy as np

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W


def test_philox_known_answer_vectors():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    n = 0
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(v, 16) for v in line.split()]
        out = O.philox4x32_10(np.array([w[:4]], np.uint32), np.array([w[4:6]], np.uint32))[0]
        assert [int(v) for v in out] == w[6:]
        n += 1
    assert n == 3


def test_uniforms_are_in_range_reproducible_and_flat():
    u = O.pair_uniform(1234567890123, 7, 200000)
    assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0
    assert np.array_equal(u, O.pair_uniform(1234567890123, 7, 200000))
    assert not np.array_equal(u, O.pair_uniform(1234567890123, 8, 200000))
    hist = np.histogram(u, bins=20, range=(0, 1))[0]
    assert np.all(np.abs(hist - 10000) < 500)             # 5 sigma of a binomial(200000, 1/20) is ~490


def _one_expert(n, slots, shares, seed=3, layer=0, G_max=4):
    ids = np.zeros((n, 1), np.int32)
    return O.count_dispatch_sampled(ids, n, np.array([slots], np.int32), np.array([shares], np.float32), seed, layer,
                                    G_max, 128 * ((n + 127) // 128 + G_max))


def test_frequencies_follow_the_renormalised_shares():
    n = 40000
    r = _one_expert(n, [0, 1, 2], [2.0, 1.0, 5.0])          # row does not sum to one: renormalised at use
    m = r["inst_count"][:3].astype(np.float64)
    assert int(m.sum()) == n
    for got, share in zip(m / n, (0.25, 0.125, 0.625)):
        assert abs(got - share) < 5 * np.sqrt(share * (1 - share) / n)


def test_zero_sum_row_is_uniform_and_missing_columns_never_chosen():
    r = _one_expert(30000, [0, -1, 2], [0.0, 0.0, 0.0])
    m = r["inst_count"]
    assert m[1] == 0 and m[3] == 0 and abs(int(m[0]) - 15000) < 5 * np.sqrt(30000 * 0.25) and int(m.sum()) == 30000
    assert int(r["status"]) == 0
    r = _one_expert(1000, [0, -1, 2], [1.0, 7.0, 1.0])      # share on a column that holds nothing: ignored, flagged
    assert int(r["status"]) & O.STATUS_BAD_TABLE and r["inst_count"][1] == 0 and int(r["inst_count"].sum()) == 1000
    r = _one_expert(1000, [0, 1, 2], [np.nan, -3.0, 0.5])   # bad shares count as zero: everything goes to column 2
    assert int(r["status"]) & O.STATUS_BAD_TABLE and r["inst_count"].tolist() == [0, 0, 1000, 0]


def test_layout_invariants_on_a_routed_batch():
    wl = W.config3("uniform", T=512)
    table = (wl.replica_map >= 0).astype(np.float32) * np.random.default_rng(0).random(wl.replica_map.shape).astype(np.float32)
    r = O.count_dispatch_sampled(wl.topk_ids, wl.n_valid, wl.replica_map, table, 99, 3, wl.G_max, wl.M_cap)
    live = wl.topk_ids[:wl.n_valid].reshape(-1)
    assert np.array_equal(r["counts"], np.bincount(live, minlength=wl.E))
    assert int(r["m_pad"]) == int(sum(-(-int(m) // 128) * 128 for m in r["inst_count"]))
    pair_row, row_pair = r["pair_row"], r["row_pair"]
    for p in np.nonzero(pair_row >= 0)[0]:
        assert row_pair[pair_row[p]] == p
    flat = wl.topk_ids.reshape(-1)
    for i in range(wl.G_max):
        lo, m = int(r["inst_off"][i]), int(r["inst_count"][i])
        ps = row_pair[lo:lo + m]
        assert np.all(ps >= 0) and np.all(np.diff(ps) > 0)                 # ascending pair index inside an instance
        assert np.all(flat[ps] == wl.slot_expert[i])                       # only to a slot that holds the expert
        assert np.all(row_pair[lo + m:int(r["inst_off"][i + 1])] == -1)
    local = np.isin(flat[:wl.n_valid * wl.k], np.nonzero((wl.replica_map >= 0).any(1))[0])
    assert int((pair_row >= 0).sum()) == int(local.sum())                   # every local live pair is placed
