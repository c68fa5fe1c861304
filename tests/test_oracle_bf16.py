"""Pins of the bf16 variant of the oracle (steps 2-4 without the quantiser): torch's CPU bfloat16 cast,
a torch fp32 dense SwiGLU MLP, an einsum evaluation written from the definition, split invariance."""
import numpy as np
import torch

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W


def test_bf16_round_matches_torch_cast():
    rng = np.random.default_rng(11)
    v = np.concatenate([
        rng.standard_normal(20000).astype(np.float32) * np.float32(3.0),
        np.ldexp(rng.standard_normal(2000), rng.integers(-60, 60, 2000)).astype(np.float32),
        # exact ties: 1 + (2j+1) * 2^-8 sits halfway between two bf16 neighbours
        (1.0 + (2 * np.arange(64) + 1) * 2.0 ** -8).astype(np.float32),
        np.array([0.0, -0.0, 1.0, -1.0, 3.3895314e38], np.float32),
    ])
    want = torch.from_numpy(v).to(torch.bfloat16).to(torch.float32).numpy()
    got = O.bf16_round(v)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(O.bf16_round(got), got)            # idempotent


def test_weights_and_activations_are_bf16_values():
    wl = W.config1()
    w13, w2 = wl.expert_weights_bf16(2)
    assert w13.shape == (2 * wl.f, wl.d) and w2.shape == (wl.d, wl.f)
    for a in (w13, w2, wl.x):
        assert np.array_equal(O.bf16_round(a), a)


def _dense(wl, e, rows):
    w13, w2 = wl.expert_weights_bf16(e)
    x = torch.from_numpy(wl.x[rows])
    GU = x @ torch.from_numpy(w13).T
    H = torch.nn.functional.silu(GU[:, :wl.f]) * GU[:, wl.f:]
    Hb = H.to(torch.bfloat16).to(torch.float32)
    return H.numpy(), (Hb @ torch.from_numpy(w2).T).numpy()


def test_ffn_bf16_reduces_to_a_dense_swiglu_mlp():
    wl = W.config1()
    rows = np.arange(24)
    w13, w2 = wl.expert_weights_bf16(5)
    h, y = O.expert_ffn_bf16(wl.x[rows], w13, w2)
    H, Y = _dense(wl, 5, rows)
    assert np.array_equal(O.bf16_round(h), h)
    assert np.abs(h - H).max() <= 2.0 ** -8 * np.abs(H).max() + 1e-12     # one bf16 rounding of H
    assert np.abs(y - Y).max() <= 2e-3 * np.abs(Y).max()
    assert np.abs(y - Y).mean() <= 1e-3 * np.abs(Y).mean()
    # gate/up order and the transposes, from the definition in fp64 without the bf16 rounding of H
    A = wl.x[rows].astype(np.float64)
    g = np.einsum("md,fd->mf", A, w13[:wl.f].astype(np.float64))
    u = np.einsum("md,fd->mf", A, w13[wl.f:].astype(np.float64))
    Yd = np.einsum("mf,cf->mc", g / (1 + np.exp(-g)) * u, w2.astype(np.float64))
    assert np.abs(y - Yd).max() <= 1e-2 * np.abs(Yd).max()
    assert np.abs(y - Yd).mean() <= 3e-3 * np.abs(Yd).mean()
    Ybad = np.einsum("mf,cf->mc", u / (1 + np.exp(-u)) * g, w2.astype(np.float64))
    assert np.abs(y - Ybad).mean() > 0.2 * np.abs(Yd).mean()


def test_block_bf16_one_expert_is_the_dense_mlp_and_pads_with_zeros():
    wl = W.config5_point(1, 40, d=256, f=256)
    r = O.expert_block_bf16(wl)
    _, Y = _dense(wl, 0, np.arange(40))
    assert np.abs(r["out"] - Y).max() <= 2e-3 * np.abs(Y).max()
    assert int(r["m_pad"]) == 128
    assert np.array_equal(r["a"][:40], wl.x[:40]) and np.all(r["a"][40:] == 0)
    assert np.all(r["h"][40:] == 0) and np.all(r["y"][40:] == 0)


def test_block_bf16_split_invariance():
    base = W.config3("uniform", T=96)
    outs = []
    for case in ("uniform", "token_balanced", "hot_whole"):
        wl = W.config3(case, T=96)
        wl.d, wl.f = 256, 256
        wl.x = base.x[:, :256].copy()
        outs.append(O.expert_block_bf16(wl))
    assert np.array_equal(outs[0]["out"], outs[1]["out"]) and np.array_equal(outs[0]["out"], outs[2]["out"])
    assert not np.array_equal(outs[0]["pair_row"], outs[1]["pair_row"])
