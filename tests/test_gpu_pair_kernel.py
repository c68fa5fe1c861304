"""The CTA-pair FFN kernel (tcgen05 cta_group::2, tempo_set_ffn_mode(2)) against the default kernel and
against the oracle.  Both kernels add the same products in the same order, so their outputs must agree
bit for bit; the oracle comparison uses the tolerances of the main parity tests."""
import numpy as np
import pytest
import torch

from paper_2608_13057_b200 import workloads as W
from oracle import tempo_oracle as O
from tests.gpu_util import sf_decode, to_np

pytestmark = pytest.mark.gpu

MAX_TOL, MEAN_TOL = 2e-2, 5e-3


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    from paper_2608_13057_b200 import binding
    yield binding
    binding.tempo_set_ffn_mode(0)


def _run(B, wl, mode):
    B.tempo_set_ffn_mode(mode)
    try:
        buf = B.RankBuffers.for_workload(wl)
        buf.run_block()
        torch.cuda.synchronize()
    finally:
        B.tempo_set_ffn_mode(0)
    return buf


def _cases():
    yield W.config1()
    yield W.config5_point(1, 40, d=256, f=256)            # one M-tile: the pair's second half is absent
    yield W.config5_point(3, 129, d=384, f=640)           # two M-tiles per instance: whole pairs
    yield W.config5_point(2, 300, d=512, f=256)           # three M-tiles: one whole pair and one half pair
    yield W.random_small(402, T=40, E=6, k=2, d=256, f=384)
    yield W.config5_skewed(6, 200, d=256, f=384)          # 1, 1, 2, 2, 3, 3 tiles per instance
    yield W.config2()                                     # every instance a single M-tile
    yield W.config5_point(8, 512)                         # several pairs per instance, full-size d and f


@pytest.mark.parametrize("wl", list(_cases()), ids=lambda w: w.name)
def test_pair_kernel_equals_default_kernel_bitwise(B, wl):
    a = _run(B, wl, 1)
    b = _run(B, wl, 2)
    m = int(a.m_pad.item())
    assert int(b.m_pad.item()) == m
    assert int(a.status.item()) == 0 and int(b.status.item()) == 0
    assert torch.equal(a.h_q[:m], b.h_q[:m])
    h_sf_a = sf_decode(to_np(a.h_sf), a.M_cap, a.f)[:m]
    h_sf_b = sf_decode(to_np(b.h_sf), b.M_cap, b.f)[:m]
    assert np.array_equal(h_sf_a, h_sf_b)
    assert torch.equal(a.y[:m], b.y[:m])
    assert torch.equal(a.out, b.out)
    assert int(b.workspace.max().item()) == 0              # the H-ready counters are left clean


def test_pair_kernel_matches_oracle_elementwise(B):
    wl = W.config5_point(2, 300, d=512, f=256)
    buf = _run(B, wl, 2)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    m = int(ref["m_pad"])
    assert int(buf.m_pad.item()) == m
    for name, got, want in (("y", to_np(buf.y)[:m], ref["y"][:m]), ("out", to_np(buf.out), ref["out"])):
        got = np.asarray(got, np.float64)
        want = np.asarray(want, np.float64)
        mx = np.abs(got - want).max() / max(np.abs(want).max(), 1e-30)
        mean = np.abs(got - want).mean() / max(np.abs(want).mean(), 1e-30)
        assert mx <= MAX_TOL and mean <= MEAN_TOL, (name, mx, mean)


def test_pair_kernel_two_halves_equal_fused(B):
    """tempo_ffn_gate_up followed by tempo_ffn_down in pair mode gives what the fused launch gives."""
    wl = W.config5_point(3, 129, d=384, f=640)
    fused = _run(B, wl, 2)
    B.tempo_set_ffn_mode(2)
    try:
        buf = B.RankBuffers.for_workload(wl)
        buf.run_block()                                    # fills the dispatch and permute outputs
        buf.h_q.zero_()
        buf.y.zero_()
        s = buf.shape
        B.tempo_ffn_gate_up(s, buf.a_q, buf.a_sf, buf.packed, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf, buf.status)
        B.tempo_ffn_down(s, buf.h_q, buf.h_sf, buf.packed, buf.inst_off, buf.m_pad, buf.y, buf.status)
        torch.cuda.synchronize()
    finally:
        B.tempo_set_ffn_mode(0)
    m = int(buf.m_pad.item())
    assert int(buf.status.item()) == 0
    assert torch.equal(buf.h_q[:m], fused.h_q[:m]) and torch.equal(buf.y[:m], fused.y[:m])


def test_set_ffn_mode_rejects_unknown_values(B):
    with pytest.raises(B.TempoError):
        B.tempo_set_ffn_mode(3)
    B.tempo_set_ffn_mode(0)
