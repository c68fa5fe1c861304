"""Pins of the masked layout in the oracle: fixed row ranges, the same pair -> instance assignment and the
same block output as the grouped layout, tile marks, per-instance capacity."""
import numpy as np

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W


def _instances_of_pairs(disp, max_m=None):
    """Instance of every pair (-1 if none), read back from the layout alone."""
    off = np.asarray(disp["inst_off"])
    out = np.full(len(disp["pair_row"]), -1)
    for p, row in enumerate(disp["pair_row"]):
        if row >= 0:
            out[p] = row // max_m if max_m else np.searchsorted(off, row, side="right") - 1
    return out


def test_masked_layout_places_the_same_pairs_in_fixed_ranges():
    for wl in (W.config1(), W.random_small(440, T=60, E=6, k=2), W.random_small(441, T=60, n_valid=31)):
        M = 256
        g = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, wl.M_cap)
        m = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, wl.G_max * M, max_m=M)
        assert int(m["status"]) == int(g["status"])
        assert np.array_equal(m["inst_off"], np.arange(wl.G_max + 1) * M) and int(m["m_pad"]) == wl.G_max * M
        assert np.array_equal(m["inst_count"], g["inst_count"]) and np.array_equal(m["counts"], g["counts"])
        assert np.array_equal(_instances_of_pairs(m, M), _instances_of_pairs(g))
        # position inside the instance is the same stable rank in both layouts
        live = m["pair_row"] >= 0
        assert np.array_equal(m["pair_row"][live] % M, g["pair_row"][live] - g["inst_off"][_instances_of_pairs(g)[live]])
        # inverse maps, rows in use are the first inst_count rows of each range, tiles marked accordingly
        rows = np.nonzero(m["row_pair"] >= 0)[0]
        assert np.array_equal(m["pair_row"][m["row_pair"][rows]], rows)
        for i in range(wl.G_max):
            used = np.nonzero(m["row_pair"][i * M:(i + 1) * M] >= 0)[0]
            assert np.array_equal(used, np.arange(m["inst_count"][i]))
            tiles = m["tile_inst"][i * M // 128:(i + 1) * M // 128]
            n_used = -(-int(m["inst_count"][i]) // 128)
            assert np.all(tiles[:n_used] == i) and np.all(tiles[n_used:] == -1)


def test_masked_block_output_equals_grouped_block_output():
    wl = W.config1()
    g = O.expert_block(wl)
    m = O.expert_block(wl, M_cap=wl.G_max * 128, max_m=128)
    assert np.array_equal(g["out"], m["out"])
    wl = W.config5_point(2, 200, d=256, f=256)
    g = O.expert_block(wl)
    m = O.expert_block(wl, M_cap=2 * 512, max_m=512)
    assert np.array_equal(g["out"], m["out"])
    assert np.all(m["y"][256:512] == 0) and np.all(m["y"][768:] == 0)      # unused tiles stay zero


def test_masked_layout_drops_what_does_not_fit_an_instance():
    wl = W.config5_point(2, 200, d=256, f=256)
    m = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, 2 * 128, max_m=128)
    assert int(m["status"]) & O.STATUS_CAPACITY
    assert np.array_equal(m["inst_count"], [128, 128])
    dropped = np.nonzero(m["pair_row"] < 0)[0]
    assert len(dropped) == 2 * (200 - 128)
    # the pairs that fit are the first 128 of each instance in pair order
    kept0 = np.nonzero((wl.topk_ids.reshape(-1) == 0) & (m["pair_row"] >= 0))[0]
    assert np.array_equal(kept0, np.nonzero(wl.topk_ids.reshape(-1) == 0)[0][:128])
