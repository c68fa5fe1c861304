"""Masked layout (instance i at rows [i*max_m, (i+1)*max_m)) through the C ABI against the oracle, and against
the grouped layout (a row's result does not depend on where it sits)."""
import numpy as np
import pytest
import torch

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W
from tests.gpu_util import codes_equal_mod_signed_zero, dispatch_outputs, sf_decode, to_np

pytestmark = pytest.mark.gpu

MAX_TOL, MEAN_TOL = 2e-2, 5e-3


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    from paper_2608_13057_b200 import binding
    return binding


def _run(B, wl, max_m):
    buf = B.RankBuffers.for_workload(wl, M_cap=wl.G_max * max_m)
    buf.a_q.fill_(0x55)                                    # unused tiles must be left alone
    buf.run_block_masked(max_m)
    torch.cuda.synchronize()
    return buf


def _err(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    return (np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30),
            np.abs(got - ref).mean() / max(np.abs(ref).mean(), 1e-30))


def _cases():
    yield W.config1(), 128
    yield W.config1(), 384
    yield W.config5_point(3, 129, d=384, f=640), 256
    yield W.config5_rows([300, 10, 0, 140], d=256, f=384), 384          # an empty instance, a full range, ragged ones
    yield W.random_small(450, T=40, E=6, k=2, d=256, f=384), 128
    yield W.random_small(451, T=40, n_valid=23), 256


@pytest.mark.parametrize("wl,max_m", list(_cases()), ids=lambda v: getattr(v, "name", str(v)))
def test_masked_block_matches_oracle_elementwise(B, wl, max_m):
    buf = _run(B, wl, max_m)
    ref = O.expert_block(wl, M_cap=buf.M_cap, max_m=max_m)
    got = dispatch_outputs(buf)
    for key in ("counts", "inst_count", "inst_off", "pair_row", "row_pair", "tile_inst"):
        assert np.array_equal(got[key], ref[key]), key
    assert got["m_pad"] == int(ref["m_pad"]) and got["status"] == int(ref["status"])
    a_q = to_np(buf.a_q)
    a_s = sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)
    y = to_np(buf.y)
    for tau, inst in enumerate(ref["tile_inst"]):
        rows = slice(tau * 128, (tau + 1) * 128)
        if inst < 0:
            assert np.all(a_q[rows] == 0x55)                # not touched
            continue
        assert codes_equal_mod_signed_zero(a_q[rows], ref["a_q"][rows]).all()
        assert np.array_equal(a_s[rows], ref["a_s"][rows])
    used = np.repeat(ref["tile_inst"] >= 0, 128)
    if used.any():
        mx, mean = _err(y[used], ref["y"][used])
        assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    out = to_np(buf.out)
    mx, mean = _err(out[:wl.n_valid], ref["out"][:wl.n_valid])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert np.all(out[wl.n_valid:] == 0)
    assert int(buf.workspace.max().item()) == 0


def test_masked_layout_with_spare_capacity(B):
    """M_cap above G_max * max_m: the tiles above the last instance's range hold nothing and are left alone."""
    wl = W.random_small(452, T=40, E=6, k=2, d=256, f=384)
    max_m = 128
    M_cap = wl.G_max * max_m + 256
    buf = B.RankBuffers.for_workload(wl, M_cap=M_cap)
    buf.a_q.fill_(0x55)
    buf.run_block_masked(max_m)
    torch.cuda.synchronize()
    ref = O.expert_block(wl, M_cap=M_cap, max_m=max_m)
    got = dispatch_outputs(buf)
    for key in ("counts", "inst_count", "inst_off", "pair_row", "row_pair", "tile_inst"):
        assert np.array_equal(got[key], ref[key]), key
    assert got["m_pad"] == int(ref["m_pad"]) and got["status"] == int(ref["status"]) == 0
    assert torch.all(buf.a_q[wl.G_max * max_m:] == 0x55)
    out = to_np(buf.out)
    mx, mean = _err(out[:wl.n_valid], ref["out"][:wl.n_valid])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)


def test_masked_and_grouped_layouts_give_the_same_output_bitwise(B):
    wl = W.config2()
    grouped = B.RankBuffers.for_workload(wl)
    grouped.run_block()
    masked = _run(B, wl, 256)
    torch.cuda.synchronize()
    assert int(masked.status.item()) == 0
    assert torch.equal(grouped.out, masked.out)
    # and again after the counts change (n_valid): nothing in the layout moves
    masked.n_valid.fill_(200)
    grouped.n_valid.fill_(200)
    masked.run_block_masked(256)
    grouped.run_block()
    torch.cuda.synchronize()
    assert torch.equal(grouped.out, masked.out)
    assert torch.equal(masked.inst_off.cpu(), torch.arange(wl.G_max + 1, dtype=torch.int32) * 256)


def test_masked_layout_capacity_per_instance(B):
    wl = W.config5_point(2, 200, d=256, f=256)
    buf = _run(B, wl, 128)
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap, max_m=128)
    got = dispatch_outputs(buf)
    assert got["status"] & B.STATUS_CAPACITY and got["status"] == int(ref["status"])
    for key in ("inst_count", "pair_row", "row_pair", "tile_inst"):
        assert np.array_equal(got[key], ref[key]), key


def test_masked_entry_points_reject_bad_strides(B):
    wl = W.config1()
    buf = B.RankBuffers.for_workload(wl, with_weights=False)
    for bad in (0, 100, 128 * 1000):
        with pytest.raises(B.TempoError):
            buf.run_block_masked(bad, packed=buf.a_q)
