"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same seeded inputs.

Bars: integer / index / byte outputs of count+dispatch and permute+quantise are bit-exact (fp8 codes
modulo the sign of zero); FFN outputs are within max|err| <= 2e-2 * max|ref| and
mean|err| / mean|ref| <= 5e-3 of the oracle evaluated on the same dequantised fp8 values.
"""
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
        pytest.skip("no CUDA device")
    from paper_2608_13057_b200 import binding
    return binding


def _dispatch_only(B, wl, M_cap=None, cum=None):
    """Run step 1 alone with small feature dims (the step does not touch them)."""
    buf = B.RankBuffers(wl.T, wl.k, wl.E, wl.G_max, wl.R_max, 128, 128, M_cap=M_cap)
    buf.topk_ids.copy_(torch.from_numpy(wl.topk_ids))
    buf.n_valid.fill_(int(wl.n_valid))
    buf.replica_map.copy_(torch.from_numpy(wl.replica_map))
    buf.quota.copy_(torch.from_numpy(wl.quota))
    if cum is not None:
        buf.cum_counts.copy_(torch.from_numpy(cum.view(np.int32)))
    B.tempo_count_dispatch(buf.shape, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts,
                           buf.counts, buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair, buf.tile_inst,
                           buf.m_pad, buf.status)
    torch.cuda.synchronize()
    return buf, dispatch_outputs(buf)


def _assert_dispatch_equal(got, ref):
    for key in ("counts", "inst_count", "inst_off", "pair_row", "row_pair", "tile_inst"):
        assert np.array_equal(got[key], ref[key]), key
    assert got["m_pad"] == int(ref["m_pad"])
    assert got["status"] == int(ref["status"])
    if "cum_counts" in ref:
        assert np.array_equal(got["cum_counts"], ref["cum_counts"])


def _table_case(ids, n_valid, rmap, quota, G_max, name="table"):
    ids = np.asarray(ids, np.int32)
    T, k = ids.shape
    rmap = np.asarray(rmap, np.int32)
    E, R = rmap.shape
    return W.Workload(name, T, k, E, G_max, R, 128, 128, n_valid, ids, np.ones((T, k), np.float32), rmap,
                      np.asarray(quota, np.int32), np.full(G_max, -1, np.int32), None, 0, 0)


def _dispatch_cases():
    yield W.config1()
    yield W.config2()
    yield W.config2(n_valid=200)
    for c in ("uniform", "token_balanced", "hot_whole"):
        yield W.config3(c)
    yield W.config4(with_x=False)
    yield W.config5_point(4, 129, with_x=False)
    yield W.config5_point(64, 4096, with_x=False)           # 262144 pairs, the largest sweep point
    yield W.config5_point(1, 1, with_x=False)
    for s in range(8):
        yield W.random_small(200 + s)
    for s in range(4):
        yield W.random_small(300 + s, T=200, E=37, k=3, stale=True)   # stale rows: sum != n_e
    yield W.random_small(17, T=9, n_valid=5)
    yield W.random_small(18, T=9, n_valid=0)
    yield W.random_small(19, T=9, n_valid=1)
    g = np.random.default_rng(9)
    # all pairs to one expert, three replicas, zero-sum row -> uniform fallback
    yield _table_case(np.zeros((301, 1)), 301, [[0, 1, 2]], [[0, 0, 0]], 3, "zero-sum")
    # share on a -1 column, slot out of range, negative share, slot claimed twice, ids out of range
    yield _table_case(np.zeros((50, 1)), 50, [[0, -1, 2]], [[10, 25, 15]], 4, "share-on-missing")
    yield _table_case(np.zeros((40, 1)), 40, [[0, 9, 1]], [[20, 10, 20]], 4, "slot-out-of-range")
    yield _table_case(np.zeros((40, 1)), 40, [[0, 1, -1]], [[-5, 40, 0]], 4, "negative-share")
    yield _table_case([[0], [1], [1], [0]], 4, [[0], [0]], [[2], [2]], 1, "slot-claimed-twice")
    # absurd shares (torn table): beyond 2^30 an entry counts as zero, so the split can never wrap
    big = 2 ** 31 - 1
    yield _table_case(np.zeros((300, 1)), 300, [[0, 1, 2]], [[big, big, 7]], 3, "huge-shares")
    yield _table_case(np.zeros((300, 1)), 300, [[0, 1, 2]], [[big, big, big]], 3, "all-huge-shares")
    yield _table_case(np.zeros((300, 1)), 300, [[0, 1, 2]], [[2 ** 30, 2 ** 30, 2 ** 29]], 3, "largest-legal-shares")
    yield _table_case([[0], [5], [-1], [0]], 4, [[0]], [[2]], 1, "bad-ids")
    # an expert with n_e = 0 but a non-zero share; duplicate expert inside one token; E not a multiple of 32
    ids = g.integers(1, 37, size=(64, 4))
    ids[:, 1] = ids[:, 0]
    rmap = np.full((37, 2), -1)
    rmap[:20, 0] = np.arange(20)
    rmap[:5, 1] = 20 + np.arange(5)
    quota = g.integers(0, 30, size=(37, 2))
    yield _table_case(ids, 64, rmap, quota * (rmap >= 0), 25, "dup-in-token")
    for m in (127, 128, 129):
        yield _table_case(np.zeros((m, 1)), m, [[0]], [[m]], 1, f"tile-{m}")


@pytest.mark.parametrize("wl", list(_dispatch_cases()), ids=lambda w: w.name)
def test_count_dispatch_bit_exact(B, wl):
    cum = np.full(wl.E, 2 ** 32 - 5, np.uint32)
    buf, got = _dispatch_only(B, wl, cum=cum)
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap, cum_counts=cum)
    _assert_dispatch_equal(got, ref)


def _sampled_cases():
    g = np.random.default_rng(11)
    for wl in (W.config1(), W.config2(), W.config2(n_valid=200), W.config3("uniform"), W.config4(with_x=False),
               W.config5_point(64, 1024, with_x=False), W.random_small(500, T=200, E=37, k=3), W.random_small(501, T=9, n_valid=0)):
        table = (g.random(wl.replica_map.shape) * (g.random(wl.replica_map.shape) < 0.8)).astype(np.float32)
        yield wl, table
    wl = W.random_small(502, T=300, E=6, k=2)
    table = g.random(wl.replica_map.shape).astype(np.float32)
    table[0, 0], table[1, 0], table[2, :] = np.nan, -1.0, 0.0          # bad shares, a zero-sum row
    table[wl.replica_map < 0] = 2.0                                    # shares on columns that hold nothing
    yield wl, table


@pytest.mark.parametrize("wl,table", list(_sampled_cases()), ids=lambda v: getattr(v, "name", None))
def test_count_dispatch_sampled_bit_exact(B, wl, table):
    buf = B.RankBuffers(wl.T, wl.k, wl.E, wl.G_max, wl.R_max, 128, 128)
    buf.topk_ids.copy_(torch.from_numpy(wl.topk_ids))
    buf.n_valid.fill_(int(wl.n_valid))
    buf.replica_map.copy_(torch.from_numpy(wl.replica_map))
    cum = np.full(wl.E, 2 ** 32 - 5, np.uint32)
    buf.cum_counts.copy_(torch.from_numpy(cum.view(np.int32)))
    t_dev = torch.from_numpy(table).cuda()
    seed, layer = 0x9E3779B97F4A7C15, 17
    B.tempo_count_dispatch_sampled(buf.shape, buf.topk_ids, buf.n_valid, buf.replica_map, t_dev, seed, layer,
                                   buf.cum_counts, buf.counts, buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair,
                                   buf.tile_inst, buf.m_pad, buf.status)
    torch.cuda.synchronize()
    ref = O.count_dispatch_sampled(wl.topk_ids, wl.n_valid, wl.replica_map, table, seed, layer, wl.G_max, buf.M_cap,
                                   cum_counts=cum)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)


def test_count_dispatch_capacity_overflow(B):
    ids = (np.arange(600, dtype=np.int32) % 2).reshape(600, 1)
    wl = _table_case(ids, 600, [[0], [1]], [[300], [300]], 2, "capacity")
    buf, got = _dispatch_only(B, wl, M_cap=640)
    ref = O.count_dispatch(wl.topk_ids, 600, wl.replica_map, wl.quota, 2, 640)
    _assert_dispatch_equal(got, ref)
    assert got["status"] & B.STATUS_CAPACITY


def test_count_dispatch_is_deterministic_and_accumulates(B):
    wl = W.config3("token_balanced")
    buf, first = _dispatch_only(B, wl)
    for _ in range(20):
        B.tempo_count_dispatch(buf.shape, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts,
                               buf.counts, buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair, buf.tile_inst,
                               buf.m_pad, buf.status)
    torch.cuda.synchronize()
    again = dispatch_outputs(buf)
    for key in ("counts", "pair_row", "row_pair", "inst_off"):
        assert np.array_equal(first[key], again[key])
    assert np.array_equal(again["cum_counts"], (21 * first["counts"].astype(np.uint64) % 2 ** 32).astype(np.uint32))


# ---------------------------------------------------------------------------------------------------

def _run_block(B, wl, M_cap=None):
    buf = B.RankBuffers.for_workload(wl, M_cap=M_cap)
    buf.run_block()
    torch.cuda.synchronize()
    return buf


def _check_permute(buf, ref):
    m_pad = int(ref["m_pad"])
    a_q = to_np(buf.a_q)[:m_pad]
    a_s = sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)[:m_pad]
    assert codes_equal_mod_signed_zero(a_q, ref["a_q"][:m_pad]).all()
    assert np.array_equal(a_s, ref["a_s"][:m_pad])


def _err(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    scale = np.abs(ref).max()
    return np.abs(got - ref).max() / max(scale, 1e-30), np.abs(got - ref).mean() / max(np.abs(ref).mean(), 1e-30)


def _small_block_cases():
    yield W.config1()
    yield W.config5_point(1, 40, d=256, f=256)
    yield W.config5_point(3, 129, d=384, f=640)           # two tiles per instance, odd block counts
    yield W.config5_skewed(6, 200, d=256, f=384)          # 1, 1, 2, 2, 3, 3 tiles: cold and hot instances in one batch
    for s in range(3):
        yield W.random_small(400 + s, T=40, E=6, k=2, d=256, f=384)
    yield W.random_small(410, T=40, n_valid=23)


@pytest.mark.parametrize("wl", list(_small_block_cases()), ids=lambda w: w.name)
def test_block_matches_oracle_elementwise(B, wl):
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    m_pad = int(ref["m_pad"])
    # H: compare dequantised values (a code may differ where fp32 accumulation crosses a rounding boundary)
    h_gpu = O.dequantise_1x128(to_np(buf.h_q)[:m_pad], sf_decode(to_np(buf.h_sf), buf.M_cap, buf.f)[:m_pad])
    h_ref = O.dequantise_1x128(ref["h_q"][:m_pad], ref["h_s"][:m_pad])
    if m_pad:
        mx, mean = _err(h_gpu, h_ref)
        assert mx <= 0.07 and mean <= MEAN_TOL, ("H", mx, mean)
        mx, mean = _err(to_np(buf.y)[:m_pad], ref["y"][:m_pad])
        assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    out = to_np(buf.out)
    mx, mean = _err(out[:wl.n_valid], ref["out"][:wl.n_valid])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert np.all(out[wl.n_valid:] == 0)
    assert np.all(out[(ref["pair_row"].reshape(wl.T, wl.k) < 0).all(1)] == 0)
    assert not (int(buf.status.item()) & B.STATUS_TIMEOUT)


def test_flat_decode_config_full(B):
    wl = W.config2()
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    m_pad = int(ref["m_pad"])
    mx, mean = _err(to_np(buf.y)[:m_pad], ref["y"][:m_pad])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    # masking variant: rows >= n_valid are CUDA-graph padding
    wl2 = W.config2(n_valid=200)
    buf2 = _run_block(B, wl2)
    ref2 = O.expert_block(wl2, M_cap=buf2.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf2), ref2)
    mx, mean = _err(to_np(buf2.out)[:200], ref2["out"][:200])
    assert mx <= MAX_TOL and mean <= MEAN_TOL
    assert torch.all(buf2.out[200:] == 0)


def _sampled_rows_check(B, wl, buf, rows_per_inst=6, n_tokens=48, seed=0):
    """Full-size check on sampled outputs the oracle computes one by one."""
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    g = np.random.default_rng(seed)
    tokens = np.sort(g.choice(wl.n_valid, size=min(n_tokens, wl.n_valid), replace=False))
    need = set()
    pr = ref["pair_row"].reshape(wl.T, wl.k)
    for t in tokens:
        need.update(int(r) for r in pr[t] if r >= 0)
    for i in range(wl.G_max):
        lo, m = int(ref["inst_off"][i]), int(ref["inst_count"][i])
        if m == 0:
            continue
        picks = {lo, lo + m - 1, lo + min(m - 1, 127), lo + min(m - 1, 128)}
        picks.update(int(v) for v in lo + g.integers(0, m, size=rows_per_inst))
        need.update(picks)
    rows = np.array(sorted(need))
    inst_of = np.searchsorted(ref["inst_off"][1:], rows, side="right")
    y_ref = np.zeros((len(rows), wl.d), np.float32)
    a_q_gpu = to_np(buf.a_q[torch.from_numpy(rows).cuda()])
    a_s_gpu = sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)[rows]
    for i in np.unique(inst_of):
        sel = np.nonzero(inst_of == i)[0]
        toks = ref["row_pair"][rows[sel]] // wl.k
        a_q, a_s = O.quantise_1x128(wl.x[toks])
        assert codes_equal_mod_signed_zero(a_q_gpu[sel], a_q).all() and np.array_equal(a_s_gpu[sel], a_s)
        w = wl.expert_weights(int(wl.slot_expert[i]))
        _, _, y_ref[sel] = O.expert_ffn(a_q, a_s, w.w13_q, w.w13_s, w.w2_q, w.w2_s)
    y_gpu = to_np(buf.y[torch.from_numpy(rows).cuda()])
    mx, mean = _err(y_gpu, y_ref)
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y rows", mx, mean)
    # combine on the sampled tokens, from the oracle's own Y rows
    pos = {int(r): n for n, r in enumerate(rows)}
    out_ref = np.zeros((len(tokens), wl.d), np.float32)
    for n, t in enumerate(tokens):
        acc = np.zeros(wl.d, np.float32)
        for s in range(wl.k):
            if pr[t, s] >= 0:
                acc = acc + wl.topk_w[t, s] * y_ref[pos[int(pr[t, s])]]
        out_ref[n] = acc
    out_gpu = to_np(buf.out[torch.from_numpy(tokens).cuda()])
    mx, mean = _err(out_gpu, out_ref)
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out rows", mx, mean)
    assert not (int(buf.status.item()) & B.STATUS_TIMEOUT)


def _full_instance_check(wl, buf, ref, i):
    """Every padded row of instance slot i (all its M-tiles, the true d and f) against the oracle: the
    quantised activations bytewise, H through its dequantised values, Y within the FFN tolerance."""
    lo, hi = int(ref["inst_off"][i]), int(ref["inst_off"][i + 1])
    m = int(ref["inst_count"][i])
    assert hi > lo and m > 0
    rp = ref["row_pair"][lo:hi]
    assert np.all(rp[:m] >= 0) and np.all(rp[m:] < 0)
    a_q = np.zeros((hi - lo, wl.d), np.uint8)
    a_s = np.ones((hi - lo, wl.d // 128), np.float32)
    a_q[:m], a_s[:m] = O.quantise_1x128(wl.x[rp[:m] // wl.k])
    assert codes_equal_mod_signed_zero(to_np(buf.a_q[lo:hi]), a_q).all()
    assert np.array_equal(sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)[lo:hi], a_s)
    w = wl.expert_weights(int(wl.slot_expert[i]))
    h_q, h_s, y_ref = O.expert_ffn(a_q, a_s, w.w13_q, w.w13_s, w.w2_q, w.w2_s)
    h_gpu = O.dequantise_1x128(to_np(buf.h_q[lo:hi]), sf_decode(to_np(buf.h_sf), buf.M_cap, buf.f)[lo:hi])
    mx, mean = _err(h_gpu, O.dequantise_1x128(h_q, h_s))
    assert mx <= 0.07 and mean <= MEAN_TOL, ("H", i, mx, mean)
    mx, mean = _err(to_np(buf.y[lo:hi]), y_ref)
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", i, mx, mean)
    assert np.all(to_np(buf.y[lo + m:hi]) == 0)                      # padding rows give exact zeros
    return (hi - lo) // 128


def test_mixed_config_hot_instance_in_full(B):
    """Config 3 at its true shape (d=4096, f=1536): the hottest instance of the keep-hot-whole split
    (about 30 M-tiles, dealt as a hot instance beside cold ones) compared row by row, not sampled."""
    wl = W.config3("hot_whole")
    buf = _run_block(B, wl)
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    hot = int(np.argmax(ref["inst_count"]))
    tiles = _full_instance_check(wl, buf, ref, hot)
    assert tiles >= 24
    cold = int(np.argmin(np.where(ref["inst_count"] > 0, ref["inst_count"], 1 << 30)))
    _full_instance_check(wl, buf, ref, cold)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_prefill_config_multi_tile_instance_in_full(B):
    """Config 4 at its true shape (d=7168, f=2048): one instance of several M-tiles row by row."""
    wl = W.config4()
    buf = _run_block(B, wl)
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    cnt = ref["inst_count"].astype(np.int64)
    multi = [i for i in range(wl.G_max) if 4 * 128 < cnt[i] <= 12 * 128]     # 5 to 12 tiles: seconds on the host
    assert multi, cnt
    i = multi[len(multi) // 2]
    assert _full_instance_check(wl, buf, ref, i) >= 5
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_mixed_config_three_splits_sampled_and_split_invariant(B):
    outs = []
    for case in ("uniform", "token_balanced", "hot_whole"):
        wl = W.config3(case)
        buf = _run_block(B, wl)
        _sampled_rows_check(B, wl, buf)
        outs.append(buf.out.clone())
        del buf
    # replicas hold copies of the same weights and a row's result does not depend on where it sits
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


def test_prefill_config_sampled(B):
    wl = W.config4()
    buf = _run_block(B, wl)
    _sampled_rows_check(B, wl, buf, rows_per_inst=3, n_tokens=16)


@pytest.mark.parametrize("G,N", [(1, 1), (2, 129), (8, 512), (64, 64)])
def test_sweep_points_sampled(B, G, N):
    wl = W.config5_point(G, N)
    buf = _run_block(B, wl)
    _sampled_rows_check(B, wl, buf, rows_per_inst=2, n_tokens=8)


def test_hot_and_cold_instances_dealt_together_elementwise(B):
    """Two hot instances (4 M-tiles) and eight cold ones (1-2 M-tiles) with enough tiles on both sides of the FFN
    (12 gate/up and 9 down tiles per M-tile) for a whole wave to be dealt from both lists: every row against the oracle."""
    wl = W.config5_rows([500, 500, 130, 130, 130, 130, 60, 60, 60, 60], d=2304, f=1536)
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    m_pad = int(ref["m_pad"])
    assert m_pad == 128 * 20
    mx, mean = _err(to_np(buf.y)[:m_pad], ref["y"][:m_pad])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


@pytest.mark.parametrize("n_valid", [8000, 1, 0])
def test_permute_by_rows_and_by_tokens_agree_bitwise(B, n_valid):
    """tempo_permute_pad without pair_row walks the rows and gathers; with it, and x beyond 48 MB, it walks the
    tokens and quantises each row of x once.  Same bytes, and both equal the oracle (x here is 52 MB)."""
    wl = W.random_small(431, T=8192, E=8, k=2, R_max=2, d=3200, f=128, n_valid=n_valid)
    buf = B.RankBuffers.for_workload(wl, with_weights=False)
    s = buf.shape
    B.tempo_count_dispatch(s, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts, buf.counts,
                           buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair, buf.tile_inst, buf.m_pad, buf.status)
    outs = []
    for pair_row in (None, buf.pair_row):
        buf.a_q.fill_(0x55)
        buf.a_sf.fill_(0x55)
        B.tempo_permute_pad(s, buf.x, buf.row_pair, buf.m_pad, buf.a_q, buf.a_sf, buf.status, pair_row=pair_row)
        torch.cuda.synchronize()
        m = int(buf.m_pad.item())
        outs.append((buf.a_q[:m].clone(), sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)[:m].copy()))
        assert torch.all(buf.a_q[m:] == 0x55)                  # rows >= m_pad are not written
    assert torch.equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    assert m == int(ref["m_pad"]) and (m > 0 or n_valid == 0)
    a_q, a_s = O.permute_pad(wl.x, ref["row_pair"], ref["m_pad"], wl.k)
    assert codes_equal_mod_signed_zero(to_np(outs[1][0]), a_q[:m]).all() and np.array_equal(outs[1][1], a_s[:m])


def _small_permute_cases():
    yield W.config1()
    yield W.config2(n_valid=200)
    yield W.config5_point(3, 129, d=384, f=640)           # d below one 512-column chunk
    yield W.random_small(432, T=40, E=6, k=3, d=640, f=128, n_valid=23)   # k not a power of two, ragged last chunk
    yield W.random_small(433, T=1, E=4, k=2, d=256, f=128)
    yield W.random_small(434, T=16, E=4, k=2, d=256, f=128, n_valid=0)
    yield W.config2(T=1024)                               # three items per warp in the one-wave kernel


@pytest.mark.parametrize("wl", list(_small_permute_cases()), ids=lambda w: w.name)
def test_permute_of_a_decode_sized_batch_agrees_with_the_row_walk_bitwise(B, wl):
    """With pair_row and a batch small enough for one warp per item, tempo_permute_pad runs its one-wave kernel;
    without pair_row it walks the rows.  Same bytes in rows below m_pad, nothing written above, both equal the oracle."""
    buf = B.RankBuffers.for_workload(wl, with_weights=False)
    s = buf.shape
    B.tempo_count_dispatch(s, buf.topk_ids, buf.n_valid, buf.replica_map, buf.quota, buf.cum_counts, buf.counts,
                           buf.inst_count, buf.inst_off, buf.pair_row, buf.row_pair, buf.tile_inst, buf.m_pad, buf.status)
    outs = []
    for pair_row in (None, buf.pair_row):
        buf.a_q.fill_(0x55)
        buf.a_sf.fill_(0x55)
        B.tempo_permute_pad(s, buf.x, buf.row_pair, buf.m_pad, buf.a_q, buf.a_sf, buf.status, pair_row=pair_row)
        torch.cuda.synchronize()
        m = int(buf.m_pad.item())
        outs.append((buf.a_q[:m].clone(), sf_decode(to_np(buf.a_sf), buf.M_cap, buf.d)[:m].copy()))
        assert torch.all(buf.a_q[m:] == 0x55)
    assert torch.equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    assert m == int(ref["m_pad"])
    a_q, a_s = O.permute_pad(wl.x, ref["row_pair"], ref["m_pad"], wl.k)
    assert codes_equal_mod_signed_zero(to_np(outs[1][0]), a_q[:m]).all() and np.array_equal(outs[1][1], a_s[:m])
    assert int(buf.status.item()) == 0


def test_many_instances_elementwise(B):
    """300 instance slots (the prefix scans of the FFN kernel run over ten 32-slot groups): empty, one-tile,
    two-tile and four-tile instances mixed, every row against the oracle."""
    rng = np.random.default_rng(77)
    rows = rng.choice([0, 1, 37, 128, 129, 200, 300, 450], size=300, p=[0.1, 0.1, 0.3, 0.1, 0.1, 0.1, 0.1, 0.1])
    wl = W.config5_rows(rows.tolist(), d=128, f=256)
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    m_pad = int(ref["m_pad"])
    mx, mean = _err(to_np(buf.y)[:m_pad], ref["y"][:m_pad])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_limits_of_the_shape_elementwise(B):
    """The documented maxima at once: 1024 experts, 1024 instance slots (most of them empty or tiny), d = f = 128."""
    rng = np.random.default_rng(78)
    rows = rng.choice([0, 0, 0, 1, 2, 5, 130], size=1024)
    wl = W.config5_rows(rows.tolist(), d=128, f=128)
    assert wl.E == 1024 and wl.G_max == 1024
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    m_pad = int(ref["m_pad"])
    mx, mean = _err(to_np(buf.y)[:m_pad], ref["y"][:m_pad])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("Y", mx, mean)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_top_k_32_elementwise(B):
    """k at its documented maximum: 32 slots per token, 40 experts, every expert local."""
    wl = W.random_small(460, T=24, E=40, k=32, R_max=1, d=128, f=128)
    buf = _run_block(B, wl)
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _check_permute(buf, ref)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL, ("out", mx, mean)


def test_skewed_sweep_point_sampled(B):
    """Same totals as a sweep point, rows spread unevenly over the instances (227 ... 1824 rows)."""
    wl = W.config5_skewed(8, 1024)
    buf = _run_block(B, wl)
    ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
    _assert_dispatch_equal(dispatch_outputs(buf), ref)
    _sampled_rows_check(B, wl, buf, rows_per_inst=2, n_tokens=8)


def test_block_is_reproducible_run_to_run(B):
    wl = W.config2()
    buf = _run_block(B, wl)
    first = (buf.h_q.clone(), buf.y.clone(), buf.out.clone())
    for _ in range(5):
        buf.run_block()
    torch.cuda.synchronize()
    assert torch.equal(first[0], buf.h_q) and torch.equal(first[1], buf.y) and torch.equal(first[2], buf.out)
    assert int(buf.workspace.max().item()) == 0                  # the H-ready counters are left clean


def test_graph_replay_matches_eager_launches(B):
    """The launch configuration bench.py times: the four calls captured in one CUDA graph and replayed,
    with the weights coming from a rotated copy.  Replays must reproduce the eager result bit for bit."""
    wl = W.config2()
    buf = _run_block(B, wl)
    eager = (buf.pair_row.clone(), buf.a_q.clone(), buf.h_q.clone(), buf.y.clone(), buf.out.clone())
    other = buf.packed.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        buf.run_block(packed=other)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        buf.run_block(packed=other)
    for t in (buf.pair_row, buf.a_q, buf.h_q, buf.y, buf.out):
        t.zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (buf.pair_row, buf.a_q, buf.h_q, buf.y, buf.out)):
        assert torch.equal(a, b)
    assert int(buf.status.item()) == 0
    ref = O.expert_block(wl, M_cap=buf.M_cap)
    mx, mean = _err(to_np(buf.out), ref["out"])
    assert mx <= MAX_TOL and mean <= MEAN_TOL
    # bench.py's chains: several consecutive steps in ONE graph, each step's first kernel launched
    # programmatically behind the previous step's last one, n_valid changing between the steps
    nv_a, nv_b = buf.n_valid.clone(), torch.full_like(buf.n_valid, 200)
    chain = torch.cuda.CUDAGraph()
    with torch.cuda.graph(chain):
        for i in range(6):
            buf.n_valid.copy_(nv_b if i % 2 == 0 else nv_a)
            buf.run_block(packed=other if i % 2 else buf.packed)
    for t in (buf.pair_row, buf.a_q, buf.h_q, buf.y, buf.out):
        t.zero_()
    chain.replay()
    chain.replay()
    torch.cuda.synchronize()
    for a, b in zip(eager, (buf.pair_row, buf.a_q, buf.h_q, buf.y, buf.out)):   # the last step ran with all rows live
        assert torch.equal(a, b)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_consecutive_steps_with_different_inputs_do_not_mix(B):
    """The fused FFN hands H from CTA to CTA through counters; a down tile that started before its H block was
    visible would read the previous step's block.  Consecutive steps therefore get different activations and the
    last one is compared bit for bit with an eager run, many times over."""
    wl = W.config2()
    buf = _run_block(B, wl)
    want = (buf.h_q.clone(), buf.y.clone(), buf.out.clone())
    xa = buf.x.clone()
    xb = (buf.x.float() * -1.5 + 0.25).to(torch.bfloat16)
    other = buf.packed.clone()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        for i in range(6):
            buf.x.copy_(xb if i % 2 == 0 else xa)
            buf.run_block(packed=other if i % 2 else buf.packed)
    for _ in range(40):
        buf.h_q.zero_()
        buf.y.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(want[0], buf.h_q) and torch.equal(want[1], buf.y) and torch.equal(want[2], buf.out)
    assert int(buf.status.item()) == 0 and int(buf.workspace.max().item()) == 0


def test_bounded_wait_reports_timeout_and_the_context_stays_usable(B):
    """Failure detection without a fault: the down tiles wait for H-ready counters that nothing will
    complete (the workspace is poisoned on the host), the wait gives up after its limit (20 ms here),
    the kernel sets TEMPO_STATUS_TIMEOUT and returns; after re-zeroing the workspace the same buffers
    produce the right result again."""
    wl = W.config1()
    buf = _run_block(B, wl)
    good = buf.y.clone()
    buf.workspace.view(torch.int32).fill_(-1000000)        # counters can never reach their target
    buf.status.zero_()
    B.tempo_grouped_ffn_bounded(buf.shape, buf.a_q, buf.a_sf, buf.packed, buf.inst_off, buf.m_pad, buf.h_q, buf.h_sf,
                                buf.y, buf.status, buf.workspace, 20_000_000)
    torch.cuda.synchronize()                                # returns after about 20 ms
    assert int(buf.status.item()) & B.STATUS_TIMEOUT
    buf.workspace.zero_()
    buf.status.zero_()
    buf.run_block()
    torch.cuda.synchronize()
    assert int(buf.status.item()) == 0
    assert torch.equal(buf.y[:int(buf.m_pad.item())], good[:int(buf.m_pad.item())])


def test_pack_rejects_non_power_of_two_scales(B):
    wl = W.config1()
    buf = B.RankBuffers(wl.T, wl.k, wl.E, wl.G_max, wl.R_max, wl.d, wl.f)
    w13_q, w13_s, w2_q, w2_s = wl.slot_weights()
    buf.pack_weights(w13_q, w13_s, w2_q, w2_s)
    assert int(buf.status.item()) == 0
    w2_s = w2_s.copy()
    w2_s[0, 0, 0] = 0.3
    buf.pack_weights(w13_q, w13_s, w2_q, w2_s)
    assert int(buf.status.item()) & B.STATUS_BAD_SCALE


def test_solver_table_reaches_the_dispatch_kernel_and_is_honoured_exactly(B):
    """The off-path solver's output is the table the in-graph kernel reads (Section 4.2 -> Section 4.4): every
    policy of the mixed-regime batch, the solver's included, goes through tempo_count_dispatch with status 0,
    bit-exact against the oracle, every instance holding exactly the rows its share says."""
    from paper_2608_13057_b200 import policies as P
    from paper_2608_13057_b200 import solver as S
    params = S.CostParams(a=28.4, b=3.42, c=-190.0, beta=0.0246, b2=2.31)       # a fitted B200 block-scope profile
    for case in P.build_cases(params, with_x=False):
        for wl in [case.rank] + case.gpus:
            buf, got = _dispatch_only(B, wl)
            ref = O.count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, buf.M_cap)
            _assert_dispatch_equal(got, ref)
            assert got["status"] == 0
            if wl is case.rank:
                assert np.array_equal(got["inst_count"], case.rank_rows)       # a stale table is renormalised to this
            if wl is not case.rank or case.name != "tempo_fast_stale1":
                for e in range(wl.E):
                    for r in range(wl.R_max):
                        if wl.replica_map[e, r] >= 0:
                            assert int(got["inst_count"][wl.replica_map[e, r]]) == int(wl.quota[e, r])
