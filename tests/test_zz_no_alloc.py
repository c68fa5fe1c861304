"""tempo_grouped_ffn_static: the FFN entry point for callers that cannot allocate scratch memory.

Collected last on purpose (file name), so a run that stops at the first failure has already run
everything else.  It calls the entry point through the C ABI twice in a row and checks both results
against the regular entry point's on the same inputs, within the parity tolerances of the FFN tests.
It must pass on its own in a fresh process and after the other GPU tests.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2608_13057_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_TOL, MEAN_TOL = 2e-2, 5e-3


def _err(got, ref):
    got = got.float().cpu().numpy().astype(np.float64)
    ref = ref.float().cpu().numpy().astype(np.float64)
    return (np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30),
            np.abs(got - ref).mean() / max(np.abs(ref).mean(), 1e-30))


@pytest.mark.parametrize("make", [W.config1, lambda: W.config3("token_balanced", T=1024)], ids=["cfg1", "cfg3-1k"])
def test_static_scratch_entry_matches_the_regular_one_twice_in_a_row(make):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_13057_b200 import binding as B
    wl = make()
    buf = B.RankBuffers.for_workload(wl)
    buf.run_block()                                   # regular path: fills a_q, h, y through tempo_grouped_ffn
    torch.cuda.synchronize()
    m_pad = int(buf.m_pad.item())
    y_ref, h_ref = buf.y[:m_pad].clone(), buf.h_q[:m_pad].clone()
    assert int(buf.status.item()) == 0

    for call in range(2):
        y2 = torch.full_like(buf.y, float("nan"))
        h2 = torch.zeros_like(buf.h_q)
        hs2 = torch.zeros_like(buf.h_sf)
        B.tempo_grouped_ffn_static(buf.shape, buf.a_q, buf.a_sf, buf.packed, buf.inst_off, buf.m_pad, h2, hs2, y2,
                                   buf.status)
        torch.cuda.synchronize()
        assert int(buf.status.item()) == 0, f"call {call}: device status {int(buf.status.item())}"
        assert not torch.isnan(y2[:m_pad].float()).any(), f"call {call}: rows left unwritten"
        mx, mean = _err(y2[:m_pad], y_ref)
        assert mx <= MAX_TOL and mean <= MEAN_TOL, (call, mx, mean)
        assert torch.equal(h2[:m_pad], h_ref)           # same kernel, same inputs: same codes


def test_static_scratch_entry_rejects_sizes_beyond_its_array():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_13057_b200 import binding as B
    too_big = B.make_shape(1, 1, 1, 1, 1, 128, 128, 128 * 16385)
    one = ctypes.c_void_p(256)                         # non-NULL dummies: the size check comes first, nothing is launched
    rc = B._lib.tempo_grouped_ffn_static(ctypes.byref(too_big), one, one, one, one, one, one, one, one, one, None)
    assert rc == -3 and b"limit" in B._lib.tempo_status_string(rc)
