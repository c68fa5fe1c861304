"""CPU oracle for the per-rank MoE expert block (TEST INFRASTRUCTURE, not product code).

Only tests, the smoke check and the benchmark's cpu_baseline / reference arm may import
this file.  It shares no code with the CUDA library and never calls it.  It is written to
be checked against the paper by eye: plain sequential loops for the integer steps, numpy
float64 matrix products for the contractions, no blocking, fusion or reordering.

What it computes, step by step (the paper's objects in brackets):

  count_dispatch   per-expert token counts n_e over live rows, a stable rank of every
                   (token, slot) pair inside its expert, and the replica each pair goes to so
                   that replica r of expert e receives exactly its share x_{e,r}
                   [Eq. 2: shares x_{e,g} >= 0, sum_g x_{e,g} = n_e, supported on R(e);
                   Section 4.4: cumulative per-expert counter, padding rows masked, rows
                   renormalised at use, zero-sum row -> uniform over replicas holding the
                   expert, never a replica that lacks the expert].
                   Rows of an instance are padded to 128-row M-tiles [Eq. 3: T = sum ceil(n/128)].
  quantise_1x128   fp8 e4m3 codes with one power-of-two (UE8M0-representable) scale per
                   128 consecutive values of a row [Appendix G ("Multi-node bring-up notes"): the newer architecture needs
                   UE8M0 scale packing].
  permute_pad      gathers token rows into the padded grouped layout and quantises them
                   [Appendix B: the "scatter/gather, quantization" per-token kernels].
  expert_ffn       gate/up GEMM, SwiGLU, re-quantisation, down GEMM per expert instance
                   [Section 2.1: "gate/up, activation, down"].
  combine          weighted sum over a token's k slots [Section 2.1: combine].

Pins (tests/test_oracle_*.py): numpy.bincount and stable argsort for counts and order, a
separately written sort-and-cut brute force for replica assignment, exact quota and
bijection invariants, torch's CPU float8_e4m3fn cast for the code rounding, half-ulp error
bounds and idempotence for the quantiser, torch fp32 dense SwiGLU MLP for the FFN, split
invariance and linearity for the whole block, and the layer as Section 2.1 defines it written
token by token with no layout (out[t] = sum_s w[t,s] * FFN_e(x[t]) over the experts held here,
k > 1, remote experts, dead rows, stale quota rows); for the bf16 variant torch's CPU bfloat16
cast and the same dense-MLP, per-token and split-invariance checks.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np

TILE_M = 128
QBLOCK = 128

STATUS_BAD_ID = 1        # a live pair names an expert outside [0, E): the pair is ignored
STATUS_BAD_TABLE = 2     # malformed replica/quota entry: the entry is treated as absent / zero
STATUS_CAPACITY = 4      # padded rows exceed M_cap: the rows that do not fit are dropped
STATUS_TIMEOUT = 8       # (GPU only) a bounded device wait expired
STATUS_BAD_SCALE = 16    # (GPU only, weight packing) a weight scale is not a power of two

MAX_SHARE = 1 << 30      # a share x_{e,r} beyond this is a malformed table entry (Section 4.4: a torn or
                         # stale row may cost a stale or uniform split, never a wrong replica)


# ----------------------------------------------------------------------------------------
# step 1: counts + quota dispatch + padded layout
# ----------------------------------------------------------------------------------------

def replica_boundaries(n_e: int, slots, quotas, G_max: int, claimed: set):
    """Rank boundaries B_0 <= B_1 <= ... of one expert's replicas, and the status bits raised.

    slots[r]  : instance slot of replica column r, or -1
    quotas[r] : share x_{e,r}
    claimed   : slots already owned by an earlier (expert, column); a slot may hold one expert.
    Returns (valid[r], B[r]) with B cumulative; pairs of rank j in [B[r-1], B[r]) go to column r.
    """
    status = 0
    R = len(slots)
    valid = [False] * R
    q = [0] * R
    for r in range(R):
        s, x = int(slots[r]), int(quotas[r])
        if s == -1:
            if x != 0:
                status |= STATUS_BAD_TABLE      # share on a replica that does not hold the expert
            continue
        if s < 0 or s >= G_max or s in claimed:
            status |= STATUS_BAD_TABLE
            continue
        claimed.add(s)
        valid[r] = True
        if x < 0 or x > MAX_SHARE:                   # malformed share: counts as zero
            status |= STATUS_BAD_TABLE
            x = 0
        q[r] = x
    S = sum(q)
    if S == 0:                                   # zero-sum row: uniform over replicas holding the expert
        q = [1 if v else 0 for v in valid]
        S = sum(q)
    B = [0] * R
    C = 0
    for r in range(R):
        C += q[r]
        B[r] = (C * n_e) // S if S > 0 else 0    # "renormalise the row at use", made deterministic
    return valid, B, status


def count_dispatch(topk_ids, n_valid, replica_map, quota, G_max, M_cap, cum_counts=None, max_m=None):
    """max_m=None: instances follow each other, each padded to whole 128-row tiles (the grouped layout).
    max_m=M (a multiple of 128): the MASKED layout of the grouped GEMM the paper calibrates ("fp8 masked
    grouped GEMM", Appendix B): instance i owns the fixed row range [i*M, (i+1)*M) and only its first
    inst_count[i] rows are in use; pairs beyond M rows of an instance are dropped (CAPACITY)."""
    ids = np.asarray(topk_ids, dtype=np.int64)
    T, k = ids.shape
    E, R = np.asarray(replica_map).shape
    n_valid = max(0, min(int(n_valid), T))
    status = 0

    # counts and stable ranks, in ascending pair index p = t*k + s over live rows only
    seen = [0] * E
    rank = [-1] * (T * k)
    for p in range(n_valid * k):
        e = int(ids[p // k, p % k])
        if e < 0 or e >= E:
            status |= STATUS_BAD_ID
            continue
        rank[p] = seen[e]
        seen[e] += 1
    counts = np.array(seen, dtype=np.int32)

    # replica boundaries per expert; experts claim slots in ascending (e, r)
    claimed: set = set()
    valid = [None] * E
    B = [None] * E
    m = [0] * G_max                       # rows of each instance slot
    for e in range(E):
        valid[e], B[e], st = replica_boundaries(seen[e], replica_map[e], quota[e], G_max, claimed)
        status |= st
        prev = 0
        for r in range(R):
            if valid[e][r]:
                m[int(replica_map[e][r])] = B[e][r] - prev
            prev = B[e][r]

    # padded offsets in ascending slot id
    off = [0] * (G_max + 1)
    for i in range(G_max):
        if max_m is None:
            off[i + 1] = off[i] + TILE_M * ((m[i] + TILE_M - 1) // TILE_M)
        else:
            off[i + 1] = off[i] + int(max_m)
            if m[i] > max_m:
                status |= STATUS_CAPACITY
    M_pad = off[G_max]
    if M_pad > M_cap:
        status |= STATUS_CAPACITY

    pair_row = np.full(T * k, -1, dtype=np.int32)
    row_pair = np.full(M_cap, -1, dtype=np.int32)
    for p in range(n_valid * k):
        j = rank[p]
        if j < 0:
            continue
        e = int(ids[p // k, p % k])
        prev = 0
        for r in range(R):
            if j < B[e][r]:
                if valid[e][r]:                   # (B only grows on valid columns, so this holds)
                    row = off[int(replica_map[e][r])] + (j - prev)
                    if row < M_cap and (max_m is None or j - prev < max_m):
                        pair_row[p] = row
                        row_pair[row] = p
                break
            prev = B[e][r]

    inst_off = np.minimum(np.array(off, dtype=np.int64), M_cap).astype(np.int32)
    inst_count = np.array([max(0, min(m[i], M_cap - off[i], m[i] if max_m is None else max_m))
                           for i in range(G_max)], dtype=np.int32)
    m_pad = min(M_pad, M_cap)
    tile_inst = np.full(M_cap // TILE_M, -1, dtype=np.int32)
    for i in range(G_max):
        used = inst_off[i + 1] if max_m is None else min(inst_off[i + 1], inst_off[i] + TILE_M * (-(-int(inst_count[i]) // TILE_M)))
        for tau in range(inst_off[i] // TILE_M, used // TILE_M):
            tile_inst[tau] = i

    out = dict(counts=counts, inst_count=inst_count, inst_off=inst_off, pair_row=pair_row,
               row_pair=row_pair, tile_inst=tile_inst, m_pad=np.int32(m_pad), status=np.uint32(status))
    if cum_counts is not None:                    # persistent counter: never zeroed, wraps mod 2^32
        out["cum_counts"] = ((np.asarray(cum_counts, dtype=np.uint64) + counts.astype(np.uint64))
                             % (1 << 32)).astype(np.uint32)
    return out


# ----------------------------------------------------------------------------------------
# fp8 e4m3 ("fn": bias 7, 3 mantissa bits, max 448, min subnormal 2^-9, no inf)
# ----------------------------------------------------------------------------------------

def e4m3_decode(codes):
    c = np.asarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    ex = (c >> 3) & 0xF
    man = c & 0x7
    val = np.where(ex == 0, man * 2.0 ** -9, (1.0 + man / 8.0) * np.exp2(ex.astype(np.float64) - 7.0))
    return (sign * val).astype(np.float32)       # (0x7F / 0xFF are NaN in the format; never produced here)


def e4m3_encode(v):
    """Round-to-nearest-even to e4m3, saturating to +-448.  v: finite float array."""
    v = np.asarray(v, dtype=np.float64)
    a = np.minimum(np.abs(v), 448.0)
    _, L = np.frexp(np.where(a > 0, a, 1.0))      # a = m * 2^L, m in [0.5, 1)  ->  floor(log2 a) = L-1
    e = np.maximum(L - 1, -6)                     # subnormals share the exponent of the smallest normal
    quantum = np.exp2(e.astype(np.float64) - 3.0)
    q = np.rint(a / quantum)                      # numpy rint rounds half to even
    val = q * quantum                             # may land on the next binade; still representable
    _, L2 = np.frexp(np.where(val > 0, val, 1.0))
    e2 = L2 - 1
    normal = val >= 2.0 ** -6
    ex = np.where(normal, e2 + 7, 0).astype(np.int64)
    man = np.where(normal, np.rint((val / np.exp2(e2.astype(np.float64)) - 1.0) * 8.0),
                   np.rint(val * 2.0 ** 9)).astype(np.int64)
    code = (ex << 3) | man
    code = np.where(np.signbit(v), code | 0x80, code)
    return code.astype(np.uint8)


def pow2_scale_exponent(amax):
    """Smallest integer eps with amax <= 448 * 2^eps (0 for amax == 0), clamped to [-126, 127].

    By exponent inspection: amax = m * 2^L with m in [1, 2); 448 = 1.75 * 2^8, so
    eps = L - 8 when m <= 1.75 and L - 7 otherwise.
    """
    amax = np.asarray(amax, dtype=np.float64)
    m, L = np.frexp(np.where(amax > 0, amax, 1.0))   # m in [0.5, 1): m' = 2m, L' = L-1
    eps = np.where(2.0 * m <= 1.75, L - 1 - 8, L - 1 - 7)
    eps = np.clip(eps, -126, 127)
    return np.where(amax > 0, eps, 0).astype(np.int32)


def quantise_1x128(v):
    """v f32 [rows, cols] (cols % 128 == 0) -> (codes uint8 [rows, cols], scales f32 [rows, cols/128])."""
    v = np.asarray(v, dtype=np.float32)
    rows, cols = v.shape
    blk = v.reshape(rows, cols // QBLOCK, QBLOCK).astype(np.float64)
    eps = pow2_scale_exponent(np.abs(blk).max(axis=2))
    scale = np.exp2(eps.astype(np.float64))
    codes = e4m3_encode(blk / scale[:, :, None]).reshape(rows, cols)
    return codes, scale.astype(np.float32)


def dequantise_1x128(codes, scales):
    rows, cols = codes.shape
    return (e4m3_decode(codes).astype(np.float64).reshape(rows, cols // QBLOCK, QBLOCK)
            * np.asarray(scales, dtype=np.float64)[:, :, None]).reshape(rows, cols)


def dequantise_128x128(codes, scales):
    R, C = codes.shape
    return (e4m3_decode(codes).astype(np.float64).reshape(R // 128, 128, C // 128, 128)
            * np.asarray(scales, dtype=np.float64)[:, None, :, None]).reshape(R, C)


# ----------------------------------------------------------------------------------------
# step 2: permute + pad + quantise
# ----------------------------------------------------------------------------------------

def permute_pad(x, row_pair, m_pad, k):
    """x f32 [T, d] (bf16-representable).  Rows >= m_pad are not defined by the method (left zero / scale 1)."""
    x = np.asarray(x, dtype=np.float32)
    M_cap = len(row_pair)
    d = x.shape[1]
    a_q = np.zeros((M_cap, d), dtype=np.uint8)
    a_s = np.ones((M_cap, d // QBLOCK), dtype=np.float32)
    live = np.nonzero(np.asarray(row_pair[:int(m_pad)]) >= 0)[0]
    if len(live):
        q, s = quantise_1x128(x[np.asarray(row_pair)[live] // k])
        a_q[live], a_s[live] = q, s
    return a_q, a_s


# ----------------------------------------------------------------------------------------
# steps 3+4: expert FFN on the rows of one instance
# ----------------------------------------------------------------------------------------

def silu_f32(g):
    g = np.asarray(g, dtype=np.float32)
    return (g / (np.float32(1.0) + np.exp(-g, dtype=np.float32))).astype(np.float32)


def expert_ffn(a_q, a_s, w13_q, w13_s, w2_q, w2_s):
    """Rows of one expert instance.  Returns (h_q, h_s, y f32).  W13 rows [0,f) gate, [f,2f) up."""
    f = w2_q.shape[1]
    A = dequantise_1x128(a_q, a_s)                         # exact in float64
    GU = (A @ dequantise_128x128(w13_q, w13_s).T).astype(np.float32)   # double accumulation, fp32 result
    H = (silu_f32(GU[:, :f]) * GU[:, f:]).astype(np.float32)
    h_q, h_s = quantise_1x128(H)
    Y = (dequantise_1x128(h_q, h_s) @ dequantise_128x128(w2_q, w2_s).T).astype(np.float32)
    return h_q, h_s, Y


def grouped_ffn(a_q, a_s, inst_off, inst_count, slot_weights, rows_only=None, masked=False):
    """slot_weights(i) -> (w13_q, w13_s, w2_q, w2_s) of instance slot i.

    Computes every padded row of every activated instance (pad rows are zero rows and give zeros).
    """
    M_cap, d = a_q.shape
    G = len(inst_count)
    w0 = None
    h_q = h_s = y = None
    for i in range(G):
        lo, hi = int(inst_off[i]), int(inst_off[i + 1])
        if masked:                                         # only the tiles that hold rows are computed
            hi = min(hi, lo + TILE_M * (-(-int(inst_count[i]) // TILE_M)))
        if hi <= lo:
            continue
        w = slot_weights(i)
        if h_q is None:
            f = w[2].shape[1]
            h_q = np.zeros((M_cap, f), np.uint8)
            h_s = np.ones((M_cap, f // QBLOCK), np.float32)
            y = np.zeros((M_cap, d), np.float32)
        h_q[lo:hi], h_s[lo:hi], y[lo:hi] = expert_ffn(a_q[lo:hi], a_s[lo:hi], *w)
    return h_q, h_s, y


# ----------------------------------------------------------------------------------------
# step 5: weighted un-permute / combine
# ----------------------------------------------------------------------------------------

def combine(y, pair_row, topk_w, n_valid, T, k):
    y = np.asarray(y, dtype=np.float32)
    out = np.zeros((T, y.shape[1]), dtype=np.float32)
    w = np.asarray(topk_w, dtype=np.float32).reshape(T, k)
    pr = np.asarray(pair_row).reshape(T, k)
    for t in range(min(int(n_valid), T)):
        acc = np.zeros(y.shape[1], dtype=np.float32)
        for s in range(k):                                 # slot order, fp32 accumulation
            if pr[t, s] >= 0:
                acc = acc + w[t, s] * y[pr[t, s]]
        out[t] = acc
    return out


# ----------------------------------------------------------------------------------------
# whole block
# ----------------------------------------------------------------------------------------

def expert_block(wl, M_cap=None, cum_counts=None, max_m=None):
    """Runs all five steps on a workload object (fields as in the seeded generators).
    max_m: the masked layout (see count_dispatch); rows outside the tiles in use are left zero."""
    M_cap = wl.M_cap if M_cap is None else M_cap
    disp = count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, M_cap, cum_counts, max_m)
    a_q, a_s = permute_pad(wl.x, disp["row_pair"], disp["m_pad"], wl.k)

    def slot_weights(i):
        w = wl.expert_weights(int(wl.slot_expert[i]))
        return w.w13_q, w.w13_s, w.w2_q, w.w2_s

    h_q, h_s, y = grouped_ffn(a_q, a_s, disp["inst_off"], disp["inst_count"], slot_weights, masked=max_m is not None)
    if y is None:
        y = np.zeros((M_cap, wl.d), np.float32)
        h_q = np.zeros((M_cap, wl.f), np.uint8)
        h_s = np.ones((M_cap, wl.f // QBLOCK), np.float32)
    out = combine(y, disp["pair_row"], wl.topk_w, wl.n_valid, wl.T, wl.k)
    return dict(disp, a_q=a_q, a_s=a_s, h_q=h_q, h_s=h_s, y=y, out=out)


# ----------------------------------------------------------------------------------------
# bf16 variant of steps 2-4 (the paper calibrates a bf16 grouped GEMM next to the fp8 one:
# Section 2.1 and Table "Fitted cost parameters", row "DSv3 (bf16)")
# ----------------------------------------------------------------------------------------
# No quantiser: the gathered rows stay bf16, both GEMMs multiply bf16 values and accumulate wide,
# and H is rounded to bf16 (round to nearest even) before the down GEMM, as a bf16 grouped-GEMM
# pipeline stores it.  Pins: bf16_round against torch's CPU cast; the one-expert case against a
# torch fp32 dense SwiGLU MLP; split invariance of the block.

def bf16_round(v):
    """f32 -> nearest bf16 (ties to even), returned as f32.  Finite inputs."""
    b = np.ascontiguousarray(v, dtype=np.float32).view(np.uint32).astype(np.uint64)
    b = b + np.uint64(0x7FFF) + ((b >> np.uint64(16)) & np.uint64(1))
    return ((b >> np.uint64(16)) << np.uint64(16)).astype(np.uint32).view(np.float32)


def permute_pad_bf16(x, row_pair, m_pad, k):
    """a f32 [M_cap, d] holding bf16 values: live rows are the token's row, every other row zero."""
    x = np.asarray(x, dtype=np.float32)
    a = np.zeros((len(row_pair), x.shape[1]), dtype=np.float32)
    live = np.nonzero(np.asarray(row_pair[:int(m_pad)]) >= 0)[0]
    if len(live):
        a[live] = x[np.asarray(row_pair)[live] // k]
    return a


def expert_ffn_bf16(a, w13, w2):
    """Rows of one expert instance, all inputs f32 arrays of bf16 values.  Returns (h bf16-valued f32, y f32)."""
    f = w2.shape[1]
    GU = (a.astype(np.float64) @ w13.astype(np.float64).T).astype(np.float32)
    h = bf16_round(silu_f32(GU[:, :f]) * GU[:, f:])
    y = (h.astype(np.float64) @ w2.astype(np.float64).T).astype(np.float32)
    return h, y


def expert_block_bf16(wl, M_cap=None):
    """The block with the bf16 steps 2-4; dispatch and combine are those of expert_block."""
    M_cap = wl.M_cap if M_cap is None else M_cap
    disp = count_dispatch(wl.topk_ids, wl.n_valid, wl.replica_map, wl.quota, wl.G_max, M_cap)
    a = permute_pad_bf16(wl.x, disp["row_pair"], disp["m_pad"], wl.k)
    h = np.zeros((M_cap, wl.f), np.float32)
    y = np.zeros((M_cap, wl.d), np.float32)
    for i in range(wl.G_max):
        lo, hi = int(disp["inst_off"][i]), int(disp["inst_off"][i + 1])
        if hi > lo:
            w13, w2 = wl.expert_weights_bf16(int(wl.slot_expert[i]))
            h[lo:hi], y[lo:hi] = expert_ffn_bf16(a[lo:hi], w13, w2)
    out = combine(y, disp["pair_row"], wl.topk_w, wl.n_valid, wl.T, wl.k)
    return dict(disp, a=a, h=h, y=y, out=out)


# ----------------------------------------------------------------------------------------
# variant of step 1: probabilistic dispatch through a float share table (Section 4.4)
# ----------------------------------------------------------------------------------------
# The deployed kernel of the paper samples a replica per (token, slot) from a row of float shares,
# renormalising the row at use and falling back to uniform over the replicas holding the expert when
# the row sums to zero.  To make that reproducible both sides draw from the same counter-based
# generator, Philox-4x32-10 (Salmon et al., "Parallel random numbers: as easy as 1, 2, 3", SC'11),
# keyed by the seed and indexed by (pair index, layer): u = (word0 >> 8) * 2^-24.
# Pins: the generator's published known-answer vectors; empirical replica frequencies against the
# shares; the zero-sum and invalid-column rules; everything else as for the quota dispatch.

_PHILOX_M0, _PHILOX_M1 = np.uint64(0xD2511F53), np.uint64(0xCD9E8D57)
_PHILOX_W0, _PHILOX_W1 = 0x9E3779B9, 0xBB67AE85


def philox4x32_10(counter, key):
    """counter: uint32 [..., 4], key: uint32 [..., 2] -> uint32 [..., 4]."""
    c = [np.asarray(counter)[..., i].astype(np.uint64) for i in range(4)]
    k = [np.asarray(key)[..., i].astype(np.uint64) for i in range(2)]
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        p0 = _PHILOX_M0 * c[0]
        p1 = _PHILOX_M1 * c[2]
        hi0, lo0 = p0 >> np.uint64(32), p0 & mask
        hi1, lo1 = p1 >> np.uint64(32), p1 & mask
        c = [(hi1 ^ c[1] ^ k[0]) & mask, lo1, (hi0 ^ c[3] ^ k[1]) & mask, lo0]
        k = [(k[0] + np.uint64(_PHILOX_W0)) & mask, (k[1] + np.uint64(_PHILOX_W1)) & mask]
    return np.stack([v.astype(np.uint32) for v in c], axis=-1)


def pair_uniform(seed, layer, n_pairs):
    """u in [0,1) for pairs 0..n_pairs-1, fp32 with 24 random bits."""
    ctr = np.zeros((n_pairs, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(n_pairs, dtype=np.uint64).astype(np.uint32)
    ctr[:, 2] = np.uint32(layer)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    w0 = philox4x32_10(ctr, np.broadcast_to(key, (n_pairs, 2)))[:, 0]
    return ((w0 >> np.uint32(8)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


def count_dispatch_sampled(topk_ids, n_valid, replica_map, table, seed, layer, G_max, M_cap, cum_counts=None):
    """Like count_dispatch, but the replica of each pair is sampled from table[e, :] (float shares)."""
    ids = np.asarray(topk_ids, dtype=np.int64)
    T, k = ids.shape
    rmap = np.asarray(replica_map)
    tab = np.asarray(table, dtype=np.float32)
    E, R = rmap.shape
    n_valid = max(0, min(int(n_valid), T))
    status = 0

    # which columns hold the expert (same ownership rule as the quota variant), cleaned shares
    claimed: set = set()
    valid = np.zeros((E, R), dtype=bool)
    q = np.zeros((E, R), dtype=np.float32)
    for e in range(E):
        for r in range(R):
            s, x = int(rmap[e, r]), tab[e, r]
            if s == -1:
                if x != 0 or np.isnan(x):
                    status |= STATUS_BAD_TABLE
                continue
            if s < 0 or s >= G_max or s in claimed:
                status |= STATUS_BAD_TABLE
                continue
            claimed.add(s)
            valid[e, r] = True
            if not np.isfinite(x) or x < 0:
                status |= STATUS_BAD_TABLE
                x = np.float32(0.0)
            q[e, r] = x

    u = pair_uniform(seed, layer, T * k)
    seen = [0] * E
    slot_of = [-1] * (T * k)
    m = [0] * G_max
    pos = [0] * (T * k)
    for p in range(n_valid * k):
        e = int(ids[p // k, p % k])
        if e < 0 or e >= E:
            status |= STATUS_BAD_ID
            continue
        seen[e] += 1
        cols = [r for r in range(R) if valid[e, r]]
        if not cols:
            continue                                      # expert not on this rank
        S = np.float32(0.0)
        for r in cols:
            S = np.float32(S + q[e, r])                   # fp32 running sum in column order
        w = q[e] if S > 0 else valid[e].astype(np.float32)   # zero-sum row: uniform over holders
        if not S > 0:
            S = np.float32(len(cols))
        thr = np.float32(u[p] * S)                        # one fp32 multiply, compared with fp32 running sums
        C = np.float32(0.0)
        pick = cols[-1]
        for r in cols:
            C = np.float32(C + w[r])
            if thr < C:
                pick = r
                break
        i = int(rmap[e, pick])
        slot_of[p] = i
        pos[p] = m[i]
        m[i] += 1
    counts = np.array(seen, dtype=np.int32)

    off = [0] * (G_max + 1)
    for i in range(G_max):
        off[i + 1] = off[i] + TILE_M * ((m[i] + TILE_M - 1) // TILE_M)
    M_pad = off[G_max]
    if M_pad > M_cap:
        status |= STATUS_CAPACITY
    pair_row = np.full(T * k, -1, dtype=np.int32)
    row_pair = np.full(M_cap, -1, dtype=np.int32)
    for p in range(n_valid * k):
        if slot_of[p] >= 0:
            row = off[slot_of[p]] + pos[p]
            if row < M_cap:
                pair_row[p] = row
                row_pair[row] = p
    inst_off = np.minimum(np.array(off, dtype=np.int64), M_cap).astype(np.int32)
    inst_count = np.array([max(0, min(m[i], M_cap - off[i])) for i in range(G_max)], dtype=np.int32)
    m_pad = min(M_pad, M_cap)
    tile_inst = np.full(M_cap // TILE_M, -1, dtype=np.int32)
    for i in range(G_max):
        for tau in range(inst_off[i] // TILE_M, inst_off[i + 1] // TILE_M):
            tile_inst[tau] = i
    out = dict(counts=counts, inst_count=inst_count, inst_off=inst_off, pair_row=pair_row, row_pair=row_pair,
               tile_inst=tile_inst, m_pad=np.int32(m_pad), status=np.uint32(status), slot_of=np.array(slot_of))
    if cum_counts is not None:
        out["cum_counts"] = ((np.asarray(cum_counts, dtype=np.uint64) + counts.astype(np.uint64))
                             % (1 << 32)).astype(np.uint32)
    return out
