"""Pins for the oracle's quantiser, FFN and combine (no GPU).

Pins: torch's CPU float8_e4m3fn cast and decode (library routines), half-ulp error bounds,
idempotence, the defining inequality of the scale, torch fp32 matmuls for the dense special
case of the FFN, split invariance and exact linearity of the whole block.
"""
import numpy as np
import pytest
import torch

from oracle import tempo_oracle as O
from paper_2608_13057_b200 import workloads as W


def test_decode_matches_torch_for_every_code():
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy()
    ok = ~np.isnan(ref)                                  # 0x7F and 0xFF are NaN in the format
    assert ok.sum() == 254
    assert np.array_equal(O.e4m3_decode(codes)[ok], ref[ok])
    assert np.abs(ref[ok]).max() == 448.0


def test_encode_matches_torch_cast_in_range():
    g = np.random.default_rng(0)
    v = np.concatenate([
        g.standard_normal(20000) * 100, g.standard_normal(20000), g.standard_normal(20000) * 1e-2,
        g.uniform(-2 ** -5, 2 ** -5, 20000),             # subnormal range and below
        O.e4m3_decode(np.arange(0, 127, dtype=np.uint8)),            # exact values
        (O.e4m3_decode(np.arange(0, 126, dtype=np.uint8)) + O.e4m3_decode(np.arange(1, 127, dtype=np.uint8))) / 2,  # ties
        [0.0, -0.0, 448.0, -448.0, 2 ** -10, 3 * 2 ** -10, 2 ** -9, 463.9],
    ]).astype(np.float32)
    v = np.clip(v, -448, 448)                            # the torch cast does not saturate
    ref = torch.from_numpy(v).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = O.e4m3_encode(v)
    assert np.array_equal(got, ref)


def test_encode_saturates():
    assert O.e4m3_encode(np.array([449.0, 464.0, 1e9, -1e9, 3e38])).tolist() == [0x7E, 0x7E, 0x7E, 0xFE, 0x7E]


def test_scale_exponent_is_the_smallest_that_fits():
    g = np.random.default_rng(1)
    amax = np.concatenate([np.exp2(g.uniform(-40, 40, 5000)), [448.0, 448.0001, 447.9999, 1.75, 1.7500001,
                                                                 2.0 ** -20 * 448, 2.0 ** 13 * 448, 1e-45, 3e38]])
    amax = amax.astype(np.float32).astype(np.float64)
    eps = O.pow2_scale_exponent(amax).astype(np.float64)
    inside = (eps > -126) & (eps < 127)
    assert np.all(amax <= 448.0 * np.exp2(eps))
    assert np.all((amax > 448.0 * np.exp2(eps - 1))[inside])
    assert O.pow2_scale_exponent(np.array([0.0]))[0] == 0
    # printed-by-hand cases: 448 -> 2^0, 449 -> 2^1, 1.0 -> 2^-8 (1*256 = 256 <= 448), 1.76 -> 2^-7
    assert O.pow2_scale_exponent(np.array([448.0, 449.0, 1.0, 1.76])).tolist() == [0, 1, -8, -7]


def test_quantiser_error_bound_idempotence_and_range():
    g = np.random.default_rng(2)
    v = (g.standard_normal((64, 512)) * np.exp2(g.integers(-12, 12, (64, 1)))).astype(np.float32)
    v[3, 128:256] = 0.0
    q, s = O.quantise_1x128(v)
    assert np.all(s[3, 1] == 1.0) and np.all(q[3, 128:256] == 0)
    dec = O.e4m3_decode(q).astype(np.float64)
    assert np.abs(dec).max() <= 448.0
    deq = O.dequantise_1x128(q, s)
    scaled = np.abs(v.astype(np.float64).reshape(64, 4, 128) / s[:, :, None].astype(np.float64))
    # half an ulp at the scaled magnitude: 2^(floor(log2 a) - 4), and 2^-10 in the subnormal range
    half_ulp = np.exp2(np.floor(np.log2(np.maximum(scaled, 2.0 ** -6))) - 4.0)
    err = np.abs(v.astype(np.float64) - deq).reshape(64, 4, 128) / s[:, :, None]
    assert np.all(err <= half_ulp + 1e-12)
    # each block uses the top of the range: its largest code is at least 224 = 448/2 in magnitude
    top = np.abs(dec).reshape(64, 4, 128).max(axis=2)
    assert np.all((top >= 224.0) | (np.abs(v).reshape(64, 4, 128).max(axis=2) == 0))
    # idempotent as a map on values (a block whose maximum rounded down to exactly 224 re-quantises
    # with half the scale and doubled codes: same values)
    q2, s2 = O.quantise_1x128(deq.astype(np.float32))
    assert np.array_equal(O.dequantise_1x128(q2, s2), deq)


def _torch_dense_swiglu(wl, e, rows):
    """Dense special case: one expert, plain fp32 library matmuls on the dequantised values."""
    w = wl.expert_weights(e)
    x = torch.from_numpy(wl.x[rows])
    q, s = O.quantise_1x128(x.numpy())
    A = torch.from_numpy(O.dequantise_1x128(q, s)).float()
    W13 = torch.from_numpy(O.dequantise_128x128(w.w13_q, w.w13_s)).float()
    W2 = torch.from_numpy(O.dequantise_128x128(w.w2_q, w.w2_s)).float()
    GU = A @ W13.T
    H = torch.nn.functional.silu(GU[:, :wl.f]) * GU[:, wl.f:]
    hq, hs = O.quantise_1x128(H.numpy())
    Hd = torch.from_numpy(O.dequantise_1x128(hq, hs)).float()
    return GU.numpy(), H.numpy(), (Hd @ W2.T).numpy()


def test_ffn_reduces_to_a_dense_swiglu_mlp():
    wl = W.config1()
    rows = np.arange(20)
    w = wl.expert_weights(3)
    a_q, a_s = O.quantise_1x128(wl.x[rows])
    h_q, h_s, y = O.expert_ffn(a_q, a_s, w.w13_q, w.w13_s, w.w2_q, w.w2_s)
    GU, H, Y = _torch_dense_swiglu(wl, 3, rows)
    Hd = O.dequantise_1x128(h_q, h_s)
    # H: the re-quantised value is within one e4m3 step (6.25 % of the block maximum at most)
    # of the library H; a code may differ where fp32 vs double accumulation crosses a rounding
    # boundary, so compare through the down GEMM, where that washes out.
    assert np.abs(Hd - H).max() <= 0.0625 * np.abs(H).max() + 1e-12
    assert np.abs(y - Y).max() <= 2e-3 * np.abs(Y).max()
    assert np.abs(y - Y).mean() <= 2e-4 * np.abs(Y).mean()
    # gate/up order and the transpose: an un-quantised fp64 evaluation written from the definition
    A = O.dequantise_1x128(a_q, a_s)
    Wg = O.dequantise_128x128(w.w13_q, w.w13_s)[:wl.f]
    Wu = O.dequantise_128x128(w.w13_q, w.w13_s)[wl.f:]
    W2 = O.dequantise_128x128(w.w2_q, w.w2_s)
    g = np.einsum("md,fd->mf", A, Wg)
    u = np.einsum("md,fd->mf", A, Wu)
    Yd = np.einsum("mf,cf->mc", g / (1 + np.exp(-g)) * u, W2)
    assert np.abs(y - Yd).max() <= 6e-2 * np.abs(Yd).max()      # only H's fp8 rounding separates them
    assert np.abs(y - Yd).mean() <= 4e-2 * np.abs(Yd).mean()
    # swapping gate and up must be visible (guards the test itself)
    Ybad = np.einsum("mf,cf->mc", u / (1 + np.exp(-u)) * g, W2)
    assert np.abs(y - Ybad).mean() > 0.2 * np.abs(Yd).mean()


def test_block_with_one_expert_k1_w1_is_the_dense_mlp():
    wl = W.config5_point(1, 40, d=256, f=256)
    r = O.expert_block(wl)
    _, _, Y = _torch_dense_swiglu(wl, 0, np.arange(40))
    assert np.abs(r["out"] - Y).max() <= 2e-3 * np.abs(Y).max()
    assert int(r["m_pad"]) == 128 and np.all(r["a_q"][40:128] == 0) and np.all(r["y"][40:128] == 0)


def test_split_invariance_and_linearity():
    base = W.config3("uniform", T=96)
    outs = []
    for case in ("uniform", "token_balanced", "hot_whole"):
        wl = W.config3(case, T=96)
        wl.d, wl.f = 256, 256                       # shrink the expert, keep the routed batch
        wl.x = base.x[:, :256].copy()
        outs.append(O.expert_block(wl))
    # replicas hold copies of the same weights: any feasible split gives the same output
    assert np.array_equal(outs[0]["out"], outs[1]["out"])
    # hot_whole replicates different experts but the local set is the same
    assert np.array_equal(outs[0]["out"], outs[2]["out"])
    assert not np.array_equal(outs[0]["pair_row"], outs[1]["pair_row"])
    wl = W.config3("uniform", T=96)
    wl.d, wl.f = 256, 256
    wl.x = base.x[:, :256].copy()
    wl.topk_w = wl.topk_w * np.float32(2.0)
    assert np.array_equal(O.expert_block(wl)["out"], 2.0 * outs[0]["out"])


def test_combine_is_a_weighted_gather_sum():
    g = np.random.default_rng(3)
    y = g.standard_normal((10, 8)).astype(np.float32)
    pair_row = np.array([3, -1, 0, 9, -1, -1, 2, 2], np.int32)        # T=4, k=2
    w = g.random((4, 2)).astype(np.float32)
    out = O.combine(y, pair_row, w, 3, 4, 2)
    assert np.allclose(out[0], w[0, 0] * y[3])
    assert np.allclose(out[1], w[1, 0] * y[0] + w[1, 1] * y[9])
    assert np.all(out[2] == 0) and np.all(out[3] == 0)                  # no local pair; dead row


# ---------------------------------------------------------------------------------------------
# The layer as Section 2.1 defines it (router -> dispatch -> expert FFN -> combine), written token
# by token with no layout at all: out[t] = sum over the token's slots s, in slot order, of
# w[t,s] * FFN_{e(t,s)}(x[t]) for the experts this rank holds.  No pair_row, no row_pair, no
# padded buffer: it pins the token-of-pair lookup of permute_pad at k > 1, the dispatch maps and
# the combine together, which the k = 1 dense case and the split-invariance test cannot.
# ---------------------------------------------------------------------------------------------

def _local_experts(wl):
    """Experts with at least one replica column that the dispatch accepts (first claim of a slot wins)."""
    claimed, local = set(), set()
    for e in range(wl.E):
        for r in range(wl.R_max):
            s = int(wl.replica_map[e, r])
            if 0 <= s < wl.G_max and s not in claimed:
                claimed.add(s)
                local.add(e)
    return local


def _per_token_definition(wl, ffn_row):
    """ffn_row(e, x_row[1, d]) -> y[1, d] f32.  Slot order, fp32 accumulation, dead rows zero."""
    local = _local_experts(wl)
    out = np.zeros((wl.T, wl.d), np.float32)
    for t in range(wl.n_valid):
        acc = np.zeros(wl.d, np.float32)
        for s in range(wl.k):
            e = int(wl.topk_ids[t, s])
            if e in local:
                acc = acc + np.float32(wl.topk_w[t, s]) * ffn_row(e, wl.x[t:t + 1])[0]
        out[t] = acc
    return out


def _fp8_ffn_row(wl):
    def ffn_row(e, x_row):
        w = wl.expert_weights(e)
        q, s = O.quantise_1x128(x_row)
        return O.expert_ffn(q, s, w.w13_q, w.w13_s, w.w2_q, w.w2_s)[2]
    return ffn_row


def _moe_cases():
    stale = W.random_small(7, T=40, E=6, k=3, R_max=3, n_valid=33, stale=True)
    return [W.config1(), W.random_small(11, T=48, E=7, k=3, R_max=3, n_valid=41), stale,
            W.random_small(5, T=30, E=5, k=2, R_max=2)]


@pytest.mark.parametrize("idx", range(4))
def test_block_equals_the_per_token_moe_definition(idx):
    wl = _moe_cases()[idx]
    r = O.expert_block(wl)
    ref = _per_token_definition(wl, _fp8_ffn_row(wl))
    assert np.any(ref != 0)
    if idx in (1, 2):
        assert wl.n_valid < wl.T and wl.k == 3
        assert len(_local_experts(wl)) < wl.E                      # some experts live on another rank
        assert np.all(r["out"][wl.n_valid:] == 0)
    assert np.array_equal(r["out"], ref)
    # a wrong token-of-pair lookup must be visible (guards the test): shift every token by one
    bad = np.roll(ref, 1, axis=0)
    assert not np.array_equal(r["out"], bad)


def test_block_equals_a_definition_that_shares_no_ffn_code():
    """The same per-token sum with the expert written out from the definition in float64 torch ops
    (dequantised operands, gate rows first, SwiGLU, the 1x128 quantiser in between)."""
    wl = W.random_small(11, T=48, E=7, k=3, R_max=3, n_valid=41)
    cache = {}

    def ffn_row(e, x_row):
        if e not in cache:
            w = wl.expert_weights(e)
            cache[e] = (torch.from_numpy(O.dequantise_128x128(w.w13_q, w.w13_s)),
                        torch.from_numpy(O.dequantise_128x128(w.w2_q, w.w2_s)))
        W13, W2 = cache[e]
        q, s = O.quantise_1x128(x_row)
        a = torch.from_numpy(O.dequantise_1x128(q, s))
        gu = (a @ W13.T).float()
        g, u = gu[:, :wl.f], gu[:, wl.f:]
        h = (g / (1 + torch.exp(-g))) * u
        hq, hs = O.quantise_1x128(h.numpy())
        return (torch.from_numpy(O.dequantise_1x128(hq, hs)) @ W2.T).float().numpy()

    ref = _per_token_definition(wl, ffn_row)
    out = O.expert_block(wl)["out"]
    scale = np.abs(ref).max()
    assert np.abs(out - ref).max() <= 2e-3 * scale          # a rare H code may flip on exp() rounding
    assert np.abs(out - ref).mean() <= 1e-4 * np.abs(ref).mean()


@pytest.mark.parametrize("idx", [0, 1])
def test_bf16_block_equals_the_per_token_moe_definition(idx):
    wl = _moe_cases()[idx]

    def ffn_row(e, x_row):
        w13, w2 = wl.expert_weights_bf16(e)
        return O.expert_ffn_bf16(x_row, w13, w2)[1]

    r = O.expert_block_bf16(wl)
    ref = _per_token_definition(wl, ffn_row)
    assert np.any(ref != 0)
    assert np.array_equal(r["out"], ref)
