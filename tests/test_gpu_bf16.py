"""Parity of the bf16 variant of steps 2 and 3 (tempo_permute_pad_bf16, tempo_grouped_ffn_bf16) against
the oracle's expert_block_bf16, through the C ABI.  The gather is exact; H, Y and out carry bf16 roundings
and fp32-vs-fp64 accumulation, so they use the block tolerances (max 2e-2 of max|ref|, mean 5e-3)."""
import numpy as np
import pytest
import torch

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W
from tests.gpu_util import to_np

pytestmark = pytest.mark.gpu

MAX_TOL, MEAN_TOL = 2e-2, 5e-3


@pytest.fixture(scope="module")
def B():
    if not torch.cuda.is_available():
        pytest.skip("needs a GPU")
    from paper_2608_13057_b200 import binding
    return binding


def _run(B, wl):
    buf = B.RankBuffers.for_workload(wl, with_weights=False)
    buf.pack_weights_bf16(*wl.slot_weights_bf16())
    buf.run_block_bf16()
    torch.cuda.synchronize()
    return buf


def _err(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    return (np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30),
            np.abs(got - ref).mean() / max(np.abs(ref).mean(), 1e-30))


def _cases():
    yield W.config1()
    yield W.config5_point(1, 40, d=256, f=256)
    yield W.config5_point(3, 129, d=384, f=640)           # two tiles per instance, K not a multiple of 256
    yield W.random_small(420, T=40, E=6, k=2, d=256, f=384)
    yield W.config5_skewed(6, 200, d=256, f=384)          # cold (1-2 tiles) and hot (3 tiles) instances together
    yield W.random_small(421, T=40, n_valid=23)


@pytest.mark.parametrize("wl", list(_cases()), ids=lambda w: w.name)
def test_bf16_block_matches_oracle_elementwise(B, wl):
    buf = _run(B, wl)
    ref = O.expert_block_bf16(wl, M_cap=buf.M_cap)
    m = int(ref["m_pad"])
    assert int(buf.m_pad.item()) == m and int(buf.status.item()) == 0
    assert np.array_equal(to_np(buf.a_bf16)[:m], ref["a"][:m])          # the gather is exact
    if m:
        mx, mean = _err(to_np(buf.h_bf16)[:m], ref["h"][:m])
        assert mx <= MAX_TOL and mean <= MEAN_TOL, ("H", mx, mean)
        mx, mean = _err(to_np(buf.y)[:m], ref["y"][:m])
        assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    out = to_np(buf.out)
    mx, mean = _err(out[:wl.n_valid], ref["out"][:wl.n_valid])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert np.all(out[wl.n_valid:] == 0)
    assert int(buf.workspace.max().item()) == 0


def test_bf16_flat_decode_config_sampled_rows(B):
    """Full-size d and f (config 2's routed batch): instances one at a time against the oracle, a few rows each."""
    wl = W.config2()
    buf = _run(B, wl)
    assert int(buf.status.item()) == 0
    inst_off = to_np(buf.inst_off)
    inst_count = to_np(buf.inst_count)
    a = to_np(buf.a_bf16)
    y = to_np(buf.y)
    rng = np.random.default_rng(5)
    for i in rng.choice(wl.G_max, 4, replace=False):
        n = int(inst_count[i])
        if n == 0:
            continue
        rows = int(inst_off[i]) + np.sort(rng.choice(n, min(n, 5), replace=False))
        w13, w2 = wl.expert_weights_bf16(int(wl.slot_expert[i]))
        _, y_ref = O.expert_ffn_bf16(a[rows], w13, w2)
        mx, mean = _err(y[rows], y_ref)
        assert mx <= MAX_TOL and mean <= MEAN_TOL, (int(i), mx, mean)


def test_bf16_block_is_reproducible_and_split_invariant(B):
    outs = []
    for case in ("uniform", "token_balanced"):
        wl = W.config3(case, T=512)
        wl.d, wl.f = 512, 384
        wl.x = W.config3("uniform", T=512).x[:, :512].copy()
        buf = _run(B, wl)
        first = buf.out.clone()
        buf.run_block_bf16()
        torch.cuda.synchronize()
        assert torch.equal(first, buf.out)
        outs.append(first)
    assert torch.equal(outs[0], outs[1])
