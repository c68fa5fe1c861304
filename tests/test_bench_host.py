"""Host logic of bench.py (no GPU): the unit counts it divides by agree with the oracle's dispatch."""
import numpy as np
import pytest

import bench
from oracle import tempo_oracle as O


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg3-uniform", "cfg3-token-balanced", "cfg3-hot-whole", "cfg5-4-129"])
def test_workload_stats_match_the_oracle_layout(name):
    wl = bench.make_workload(name)
    st = bench.workload_stats(wl)
    d = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, wl.M_cap)
    assert st["G_act"] == int((d["inst_count"] > 0).sum())
    assert st["N_local"] == int(d["inst_count"].sum())
    assert st["M_pad"] == int(d["m_pad"])
    assert st["weight_bytes"] == st["G_act"] * 3 * wl.d * wl.f
    assert st["padded_flops"] == st["M_pad"] * 6 * wl.d * wl.f


def test_rank_offsets_give_different_batches():
    a, b = bench.make_workload("cfg1", 0), bench.make_workload("cfg1", 1)
    assert not np.array_equal(a.topk_ids, b.topk_ids)


def test_peaks_file_or_fallback():
    p = bench._peaks()
    assert p["hbm_gbs"] > 1000 and p["bf16_tflops_sustained"] > 100 and p["source"] in ("measured", "fallback")
