"""The gather form of steps 2 and 3 (tempo_quantize_tokens + tempo_grouped_ffn_gather) against the oracle and
against the permuted form (tempo_permute_pad + tempo_grouped_ffn), whose results it must repeat bit for bit."""
import numpy as np
import pytest
import torch

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W
from tests.gpu_util import codes_equal_mod_signed_zero, to_np

pytestmark = pytest.mark.gpu

MAX_TOL, MEAN_TOL = 2e-2, 5e-3


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_13057_b200 import binding
    return binding


def _token_scales(buf, T, d):
    stride = buf.x_sf.numel() // T
    b = to_np(buf.x_sf).reshape(T, stride)[:, :d // 128].astype(np.int32)
    return np.exp2((b - 127).astype(np.float64)).astype(np.float32)


def _cases():
    yield W.config1()
    yield W.config5_point(3, 129, d=384, f=640)           # odd block counts: scale bytes per token not a multiple of 4
    yield W.config5_skewed(6, 200, d=256, f=384)
    yield W.random_small(400, T=40, E=6, k=2, d=256, f=384)
    yield W.random_small(410, T=40, n_valid=23)
    yield W.random_small(411, T=50, E=7, k=3, R_max=3, n_valid=41)   # k not a power of two
    yield W.config5_point(48, 130, d=256, f=512)          # 480 tiles: every CTA takes several, gate/up then down
    yield W.config2()
    yield W.config2(n_valid=200)


@pytest.mark.parametrize("wl", list(_cases()), ids=lambda w: w.name)
def test_gather_form_repeats_the_permuted_form_bitwise(B, wl):
    buf = B.RankBuffers.for_workload(wl)
    buf.run_block()
    torch.cuda.synchronize()
    m_pad = int(buf.m_pad.item())
    want = [t.clone() for t in (buf.h_q[:m_pad], buf.y[:m_pad], buf.out)]
    want_sf = buf.h_sf.clone()
    for t in (buf.h_q, buf.y, buf.out, buf.a_q):
        t.fill_(0x55 if t.dtype == torch.uint8 else 1.0)            # stale contents must not survive
    buf.run_block_gather()
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0
    # the per-token buffers are the quantiser's output for every live token
    q, s = O.quantise_1x128(wl.x[:wl.n_valid])
    assert codes_equal_mod_signed_zero(to_np(buf.x_q)[:wl.n_valid], q).all()
    assert np.array_equal(_token_scales(buf, wl.T, wl.d)[:wl.n_valid], s)
    assert torch.equal(buf.h_q[:m_pad], want[0])
    assert torch.equal(buf.y[:m_pad], want[1])
    assert torch.equal(buf.out, want[2])
    tiles = m_pad // 128
    J = ((wl.f // 128) + 3) // 4
    assert torch.equal(buf.h_sf[:tiles * J * 512], want_sf[:tiles * J * 512])
    assert torch.all(buf.a_q == 0x55)                                # the permuted copy is never written


def test_gather_form_matches_the_oracle_elementwise(B):
    wl = W.config5_rows([500, 500, 130, 130, 60, 60], d=2304, f=1536)
    buf = B.RankBuffers.for_workload(wl)
    buf.run_block_gather()
    torch.cuda.synchronize()
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    m_pad = int(ref["m_pad"])
    assert int(buf.m_pad.item()) == m_pad
    err = np.abs(to_np(buf.y)[:m_pad].astype(np.float64) - ref["y"][:m_pad])
    assert err.max() <= MAX_TOL * np.abs(ref["y"]).max() and err.mean() <= MEAN_TOL * np.abs(ref["y"][:m_pad]).mean()
    err = np.abs(to_np(buf.out).astype(np.float64) - ref["out"])
    assert err.max() <= MAX_TOL * np.abs(ref["out"]).max() and err.mean() <= MEAN_TOL * np.abs(ref["out"]).mean()
    assert int(buf.status.item()) == 0


@pytest.mark.parametrize("case", ["uniform", "hot_whole"])
def test_gather_form_on_the_mixed_config_bitwise_and_in_a_graph(B, case):
    wl = W.config3(case)
    buf = B.RankBuffers.for_workload(wl)
    buf.run_block()
    torch.cuda.synchronize()
    m_pad = int(buf.m_pad.item())
    want_y, want_out = buf.y[:m_pad].clone(), buf.out.clone()
    buf.run_block_gather()                                           # warm the launch path outside capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for _ in range(3):
            buf.run_block_gather()
    for _ in range(2):
        buf.y.zero_()
        buf.out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(buf.y[:m_pad], want_y) and torch.equal(buf.out, want_out)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_gather_form_on_the_prefill_config_bitwise(B):
    wl = W.config4()
    buf = B.RankBuffers.for_workload(wl, with_weights=False)
    buf.pack_weights(*W.slot_weights_cuda(wl))
    buf.run_block()
    torch.cuda.synchronize()
    m_pad = int(buf.m_pad.item())
    want_y, want_out = buf.y[:m_pad].clone(), buf.out.clone()
    buf.y.zero_()
    buf.run_block_gather()
    torch.cuda.synchronize()
    assert torch.equal(buf.y[:m_pad], want_y) and torch.equal(buf.out, want_out)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0
