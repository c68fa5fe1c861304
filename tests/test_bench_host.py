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


def test_both_arms_print_the_same_config_object():
    wl = bench.make_workload("cfg2")
    st = bench.workload_stats(wl)
    a = bench.workload_config("cfg2", wl, st, 1)
    b = bench.workload_config("cfg2", bench.make_workload("cfg2"), bench.workload_stats(bench.make_workload("cfg2")), 1)
    assert a == b and a["workload"] == "cfg2" and "L2" in a["l2"]
    assert set(a) == {"workload", "T", "top_k", "E", "d", "f", "G_act", "N_local", "M_pad", "layout", "l2", "parallelism"}


def test_weight_pool_is_larger_than_l2():
    for bytes_one in (75 << 20, 377 << 20, 1761 << 20):
        n = bench.n_pools_for(bytes_one)
        assert n >= 2 and n * bytes_one >= min(bench.POOL_BYTES, 2 * bytes_one) and n * bytes_one > 4 * bench.L2_BYTES


def test_traffic_figure_comes_from_the_committed_ncu_summary():
    t = bench.ncu_traffic_bytes("cfg2")
    assert t is not None and 377.5e6 <= t <= 1.2 * 377.5e6          # at least the weights, no wasted re-reads
    assert bench.ncu_traffic_bytes("no-such-workload") is None


def test_tensor_denominators_prefer_the_measured_fp8_rate():
    peaks = dict(hbm_gbs=6550.7, bf16_tflops=1647.5, bf16_tflops_sustained=1388.1, source="measured")
    d = bench.tensor_denominators(peaks, dict(fp8_tflops=3180.0, fp8_tflops_sustained=2611.0, how="x"))
    assert next(iter(d)) == "fp8_measured_sustained" and d["fp8_measured_burst"] == 3180.0
    d = bench.tensor_denominators(peaks, dict(fp8_tflops=None, fp8_tflops_sustained=None, how="unavailable"))
    assert next(iter(d)) == "bf16_sustained_x2" and abs(d["bf16_sustained_x2"] - 2776.2) < 1e-9
    assert d["nominal_dense_fp8"] == 4500.0


def test_percentiles_of_the_timed_regions():
    p = bench._pct([1.0, 2.0, 3.0, 4.0, 5.0])
    assert p["p50"] == 3.0 and p["p10"] < p["p50"] < p["p90"]
