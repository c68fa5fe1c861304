"""Seeded synthetic workloads for the per-rank MoE expert block.

This module only *draws inputs*: router ids and weights, activations, expert
weights already in fp8 e4m3 with 128x128 power-of-two block scales, replica
maps and quota tables.  It contains none of the arithmetic of the hot path
(no counting, no dispatch, no activation quantiser, no GEMM), so both the CPU
oracle's tests and the CUDA path's tests may import it without sharing any
of the method's code.

Shapes and skews follow the paper's workloads (Section 2.2 expert shapes,
Section 5 serving set-ups: Qwen3-235B with 128 experts / top-8 / 16 experts per
rank, DeepSeek-V3 with hidden 7168 / 256 experts / top-8 / 32 experts per rank,
Zipf-skewed routing as in Section 3.2); the paper's recorded routing traces are
not available, these stand in for them.

Every tensor has its own child stream of ``numpy.random.default_rng([seed, tag])``
so the draw order never matters.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional

import numpy as np
import torch

_TAG_ROUTER, _TAG_X, _TAG_W, _TAG_QUOTA = 11, 12, 13, 14


def _rng(seed: int, tag: int, sub: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tag), int(sub)])


@dataclasses.dataclass
class ExpertWeights:
    """One logical expert: fp8 codes (uint8 view of e4m3fn) and fp32 pow2 block scales."""

    w13_q: np.ndarray  # uint8 [2f, d]   rows [0,f) gate, [f,2f) up
    w13_s: np.ndarray  # f32   [2f/128, d/128]
    w2_q: np.ndarray   # uint8 [d, f]
    w2_s: np.ndarray   # f32   [d/128, f/128]


@dataclasses.dataclass
class Workload:
    name: str
    T: int
    k: int
    E: int
    G_max: int
    R_max: int
    d: int
    f: int
    n_valid: int
    topk_ids: np.ndarray      # int32 [T, k]
    topk_w: np.ndarray        # f32   [T, k]
    replica_map: np.ndarray   # int32 [E, R_max]  instance slot id or -1
    quota: np.ndarray         # int32 [E, R_max]
    slot_expert: np.ndarray   # int32 [G_max]     logical expert held by each slot, -1 = empty
    x: Optional[np.ndarray]   # f32 [T, d], every value exactly bf16-representable
    seed: int
    weight_seed: int
    _wcache: Dict[int, ExpertWeights] = dataclasses.field(default_factory=dict, repr=False)

    @property
    def M_cap(self) -> int:
        # same bound the library documents: round128(T*k) + 128*G_max
        return ((self.T * self.k + 127) // 128) * 128 + 128 * self.G_max

    def expert_weights(self, e: int) -> ExpertWeights:
        if e not in self._wcache:
            self._wcache[e] = draw_expert_weights(self.weight_seed, e, self.d, self.f)
        return self._wcache[e]

    def drop_weight_cache(self) -> None:
        self._wcache.clear()

    def expert_weights_bf16(self, e: int):
        """(w13 f32 [2f, d], w2 f32 [d, f]) of the bf16 variant, not cached."""
        return draw_expert_weights_bf16(self.weight_seed, e, self.d, self.f)

    def slot_weights_bf16(self):
        """Per-slot copies for the bf16 variant: (w13 f32 [G_max, 2f, d], w2 f32 [G_max, d, f])."""
        w13 = np.zeros((self.G_max, 2 * self.f, self.d), np.float32)
        w2 = np.zeros((self.G_max, self.d, self.f), np.float32)
        for i in range(self.G_max):
            e = int(self.slot_expert[i])
            if e >= 0:
                w13[i], w2[i] = self.expert_weights_bf16(e)
        return w13, w2

    def slot_weights(self, slots: Optional[List[int]] = None):
        """Stack per-slot copies: every replica slot owns a copy of its expert's weights."""
        slots = list(range(self.G_max)) if slots is None else slots
        d, f = self.d, self.f
        w13_q = np.zeros((len(slots), 2 * f, d), np.uint8)
        w13_s = np.ones((len(slots), 2 * f // 128, d // 128), np.float32)
        w2_q = np.zeros((len(slots), d, f), np.uint8)
        w2_s = np.ones((len(slots), d // 128, f // 128), np.float32)
        for n, i in enumerate(slots):
            e = int(self.slot_expert[i])
            if e < 0:
                continue
            w = self.expert_weights(e)
            w13_q[n], w13_s[n], w2_q[n], w2_s[n] = w.w13_q, w.w13_s, w.w2_q, w.w2_s
        return w13_q, w13_s, w2_q, w2_s


# --------------------------------------------------------------------------------------
# tensors
# --------------------------------------------------------------------------------------

def _pow2_block_scale(amax: torch.Tensor) -> torch.Tensor:
    """Smallest power of two s with amax <= 448*s (1.0 for an all-zero block)."""
    m, L = torch.frexp(amax)  # amax = m * 2**L, m in [0.5, 1)
    eps = torch.where(m <= 0.875, L - 9, L - 8).clamp(-126, 127)
    s = torch.ldexp(torch.ones_like(amax), eps)
    return torch.where(amax > 0, s, torch.ones_like(amax))


def _quantise_weight(w: torch.Tensor):
    """fp32 [R, C] -> (uint8 e4m3fn codes [R, C], fp32 pow2 scales [R/128, C/128])."""
    R, C = w.shape
    blk = w.reshape(R // 128, 128, C // 128, 128)
    s = _pow2_block_scale(blk.abs().amax(dim=(1, 3)))
    q = (blk / s[:, None, :, None]).to(torch.float8_e4m3fn)  # |v| <= 448: the cast never overflows
    return q.reshape(R, C).view(torch.uint8).numpy().copy(), s.numpy().astype(np.float32)


def draw_expert_weights(weight_seed: int, e: int, d: int, f: int, std: float = 0.02) -> ExpertWeights:
    g = _rng(weight_seed, _TAG_W, e)
    w13 = torch.from_numpy(g.standard_normal((2 * f, d), dtype=np.float32)) * std
    w2 = torch.from_numpy(g.standard_normal((d, f), dtype=np.float32)) * std
    w13_q, w13_s = _quantise_weight(w13)
    w2_q, w2_s = _quantise_weight(w2)
    return ExpertWeights(w13_q, w13_s, w2_q, w2_s)


def draw_expert_weights_bf16(weight_seed: int, e: int, d: int, f: int, std: float = 0.02):
    """The same draws as draw_expert_weights, rounded to bf16 instead (torch's CPU cast), as f32 arrays:
    (w13 [2f, d], w2 [d, f]), every value exactly bf16-representable."""
    g = _rng(weight_seed, _TAG_W, e)
    w13 = torch.from_numpy(g.standard_normal((2 * f, d), dtype=np.float32)) * std
    w2 = torch.from_numpy(g.standard_normal((d, f), dtype=np.float32)) * std
    return (w13.to(torch.bfloat16).to(torch.float32).numpy(), w2.to(torch.bfloat16).to(torch.float32).numpy())


def slot_weights_cuda(wl: "Workload", device="cuda", std: float = 0.02):
    """Per-slot weights drawn and quantised ON THE DEVICE, for timing-only runs of the large shapes (the numpy
    draws above take minutes for config 4 and the sweep): same distribution, layout and scale rule as
    draw_expert_weights, other random numbers, so results made with them are not comparable with the oracle's.
    Replica slots of one expert get identical copies.  Returns torch tensors (w13_q u8 [G,2f,d], w13_s f32
    [G,2f/128,d/128], w2_q u8 [G,d,f], w2_s f32 [G,d/128,f/128])."""
    dev = torch.device(device)
    G, d, f = wl.G_max, wl.d, wl.f
    w13_q = torch.zeros(G, 2 * f, d, dtype=torch.uint8, device=dev)
    w13_s = torch.ones(G, 2 * f // 128, d // 128, dtype=torch.float32, device=dev)
    w2_q = torch.zeros(G, d, f, dtype=torch.uint8, device=dev)
    w2_s = torch.ones(G, d // 128, f // 128, dtype=torch.float32, device=dev)

    def quant(w):
        R, C = w.shape
        blk = w.reshape(R // 128, 128, C // 128, 128)
        s = _pow2_block_scale(blk.abs().amax(dim=(1, 3)))
        q = (blk / s[:, None, :, None]).to(torch.float8_e4m3fn)
        return q.reshape(R, C).view(torch.uint8), s

    for i in range(G):
        e = int(wl.slot_expert[i])
        if e < 0:
            continue
        gen = torch.Generator(device=dev).manual_seed(int(wl.weight_seed) * 1000003 + e)
        w13_q[i], w13_s[i] = quant(torch.randn(2 * f, d, generator=gen, device=dev) * std)
        w2_q[i], w2_s[i] = quant(torch.randn(d, f, generator=gen, device=dev) * std)
    return w13_q, w13_s, w2_q, w2_s


def draw_activations(seed: int, T: int, d: int) -> np.ndarray:
    x = _rng(seed, _TAG_X).standard_normal((T, d), dtype=np.float32)
    return torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()


def route_softmax_topk(seed: int, T: int, E: int, k: int):
    """Config-1 router: logits N(0,1), softmax over E, top-k (ties to the lower id), renormalised."""
    logits = _rng(seed, _TAG_ROUTER).standard_normal((T, E), dtype=np.float32)
    p = np.exp(logits - logits.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    ids = np.argsort(-p, axis=1, kind="stable")[:, :k].astype(np.int32)
    w = np.take_along_axis(p, ids, 1)
    w = (w / w.sum(1, keepdims=True)).astype(np.float32)
    return ids, w


def route_zipf_topk(seed: int, T: int, E: int, k: int, s: float):
    """Zipf(s) popularity, k experts per token without replacement (Gumbel top-k).

    Expert 0 is the most popular.  The routing weights are the softmax of the chosen
    experts' perturbed log-popularities.
    """
    g = _rng(seed, _TAG_ROUTER)
    logp = -s * np.log(np.arange(1, E + 1, dtype=np.float64))
    z = logp[None, :] + g.gumbel(size=(T, E))
    ids = np.argsort(-z, axis=1, kind="stable")[:, :k].astype(np.int32)
    zc = np.take_along_axis(z, ids, 1)
    w = np.exp(zc - zc.max(1, keepdims=True))
    w = (w / w.sum(1, keepdims=True)).astype(np.float32)
    return ids, w


def _expert_counts(ids: np.ndarray, n_valid: int, E: int) -> np.ndarray:
    # plain tally of the router output, needed to size the quota rows (sum_r x_{e,r} = n_e)
    return np.bincount(ids[:n_valid].reshape(-1), minlength=E).astype(np.int64)


def _tables(E: int, R_max: int):
    return np.full((E, R_max), -1, np.int32), np.zeros((E, R_max), np.int32)


# --------------------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------------------

def _assemble(name, seed, T, k, E, d, f, ids, w, local_experts, replicated, split, n_valid=None,
              with_x=True, weight_seed=None) -> Workload:
    """local_experts[i] sits in slot i; replicated[j] gets an extra slot len(local)+j.

    split(e, n_e) -> (x_{e,0}, x_{e,1}) for replicated experts.
    """
    n_valid = T if n_valid is None else n_valid
    counts = _expert_counts(ids, n_valid, E)
    R_max = 2 if len(replicated) else 1
    G_max = len(local_experts) + len(replicated)
    rmap, quota = _tables(E, R_max)
    slot_expert = np.full(G_max, -1, np.int32)
    for i, e in enumerate(local_experts):
        rmap[e, 0] = i
        quota[e, 0] = counts[e]
        slot_expert[i] = e
    for j, e in enumerate(replicated):
        i = len(local_experts) + j
        rmap[e, 1] = i
        slot_expert[i] = e
        a, b = split(e, int(counts[e]))
        assert a + b == counts[e] and a >= 0 and b >= 0
        quota[e, 0], quota[e, 1] = a, b
    x = draw_activations(seed, T, d) if with_x else None
    return Workload(name, T, k, E, G_max, R_max, d, f, n_valid, ids, w, rmap, quota, slot_expert, x,
                    seed, seed if weight_seed is None else weight_seed)


def _half(e, n):
    return (n + 1) // 2, n // 2


def _hottest(counts, candidates, n):
    # largest n_e first, ties to the lower id
    return sorted(candidates, key=lambda e: (-int(counts[e]), e))[:n]


def config1(seed: int = 0) -> Workload:
    T, E, k, d, f = 64, 8, 2, 256, 512
    ids, w = route_softmax_topk(seed, T, E, k)
    return _assemble("cfg1-tiny", seed, T, k, E, d, f, ids, w, list(range(8)), [0, 1], _half)


def config2(seed: int = 1, n_valid: Optional[int] = None, T: int = 256) -> Workload:
    E, k, d, f = 128, 8, 4096, 1536
    ids, w = route_zipf_topk(seed, T, E, k, 0.8)
    nv = T if n_valid is None else n_valid
    counts = _expert_counts(ids, nv, E)
    local = list(range(16))
    return _assemble("cfg2-flat-decode", seed, T, k, E, d, f, ids, w, local, _hottest(counts, local, 4),
                     _half, n_valid=n_valid)


def config3(case: str = "uniform", seed: int = 2, T: int = 4096) -> Workload:
    """case in {"uniform", "token_balanced", "hot_whole"} (three fixed splits of one routed batch)."""
    E, k, d, f = 128, 8, 4096, 1536
    ids, w = route_zipf_topk(seed, T, E, k, 1.2)
    counts = _expert_counts(ids, T, E)
    local = list(range(0, 128, 8))
    hot = _hottest(counts, local, 4)
    if case == "uniform":
        rep, split = hot, _half
    elif case == "token_balanced":
        n_local = int(sum(counts[e] for e in local))
        phi = min(1.0, (n_local / 2) / max(1, int(sum(counts[e] for e in hot))))
        rep = hot

        def split(e, n):
            b = int(np.floor(phi * n))
            return n - b, b
    elif case == "hot_whole":
        cold = [e for e in sorted(local, key=lambda e: (int(counts[e]), e)) if counts[e] >= 2][:4]
        rep, split = cold, _half
    else:
        raise ValueError(case)
    return _assemble(f"cfg3-mixed-{case}", seed, T, k, E, d, f, ids, w, local, rep, split)


def config4(seed: int = 3, T: int = 8192, with_x: bool = True) -> Workload:
    E, k, d, f = 256, 8, 7168, 2048
    ids, w = route_zipf_topk(seed, T, E, k, 1.0)
    counts = _expert_counts(ids, T, E)
    local = list(range(32))
    u = _rng(seed, _TAG_QUOTA).random(E)

    def split(e, n):
        a = int(np.floor(u[e] * (n + 1)))
        return a, n - a
    return _assemble("cfg4-dsv3-prefill", seed, T, k, E, d, f, ids, w, local, _hottest(counts, local, 8),
                     split, with_x=with_x)


SWEEP_G = (1, 2, 4, 8, 16, 32, 64)
SWEEP_N = (1, 8, 32, 64, 128, 129, 160, 192, 256, 512, 1024, 2048, 4096)


def config5_point(G: int, N: int, seed: int = 4, d: int = 4096, f: int = 1536, with_x: bool = True) -> Workload:
    """One (G, N) point of the cost-profile sweep: G instances, N rows each, k=1, w=1."""
    T = G * N
    ids = (np.arange(T, dtype=np.int32) % G).reshape(T, 1)
    w = np.ones((T, 1), np.float32)
    rmap = np.arange(G, dtype=np.int32).reshape(G, 1)
    quota = np.full((G, 1), N, np.int32)
    x = draw_activations(seed * 1000003 + G * 8191 + N, T, d) if with_x else None
    return Workload(f"cfg5-sweep-G{G}-N{N}", T, 1, G, G, 1, d, f, T, ids, w, rmap, quota,
                    np.arange(G, dtype=np.int32), x, seed, seed)


def config5_rows(rows, seed: int = 4, d: int = 4096, f: int = 1536, with_x: bool = True, name: str = "") -> Workload:
    """One instance per entry of `rows`, that many rows each, k=1, w=1 (tokens of an instance are contiguous)."""
    m = np.asarray(rows, dtype=np.int64)
    G, T = len(m), int(m.sum())
    ids = np.repeat(np.arange(G, dtype=np.int32), m).reshape(T, 1)
    w = np.ones((T, 1), np.float32)
    rmap = np.arange(G, dtype=np.int32).reshape(G, 1)
    quota = m.astype(np.int32).reshape(G, 1)
    x = draw_activations(seed * 1000003 + G * 8191 + T + 7, T, d) if with_x else None
    return Workload(name or f"cfg5-rows-G{G}-T{T}", T, 1, G, G, 1, d, f, T, ids, w, rmap, quota,
                    np.arange(G, dtype=np.int32), x, seed, seed)


def config5_skewed(G: int, N: int, seed: int = 4, d: int = 4096, f: int = 1536, with_x: bool = True) -> Workload:
    """The (G, N) point with the same total rows G*N spread unevenly: instance i gets about
    2*N*(i+1)/(G+1) rows (a linear ramp, mean N), k=1, w=1.  For the paper's remark that a grouped GEMM can
    run faster under uniform per-slot loads at equal (G, N) (Section "Limitations", L5)."""
    m = np.floor(2.0 * N * (np.arange(G) + 1) / (G + 1)).astype(np.int64)
    m[-1] += G * N - int(m.sum())
    return config5_rows(m, seed, d, f, with_x, name=f"cfg5-skewed-G{G}-N{N}")


def random_small(seed: int, T: int = 24, E: int = 6, k: int = 2, R_max: int = 3, d: int = 256, f: int = 256,
                 n_valid: Optional[int] = None, stale: bool = False) -> Workload:
    """Small random case with up to R_max replicas per expert, some experts remote, for edge-case tests."""
    g = _rng(seed, _TAG_ROUTER)
    ids = np.stack([g.permutation(E)[:k] for _ in range(T)]).astype(np.int32)
    w = g.random((T, k), dtype=np.float32) + 0.1
    w = (w / w.sum(1, keepdims=True)).astype(np.float32)
    nv = T if n_valid is None else n_valid
    counts = _expert_counts(ids, nv, E)
    rmap, quota = _tables(E, R_max)
    slot = 0
    slot_expert: List[int] = []
    for e in range(E):
        if g.random() < 0.2:
            continue  # expert lives on another rank
        nrep = int(g.integers(1, R_max + 1))
        cols = sorted(g.permutation(R_max)[:nrep].tolist())
        cuts = np.sort(g.integers(0, counts[e] + 1, size=nrep - 1)) if nrep > 1 else np.zeros(0, np.int64)
        parts = np.diff(np.concatenate([[0], cuts, [counts[e]]]))
        for c, q in zip(cols, parts):
            rmap[e, c] = slot
            quota[e, c] = int(q) if not stale else int(g.integers(0, 2 * counts[e] + 2))
            slot_expert.append(e)
            slot += 1
    G_max = max(slot, 1)
    se = np.full(G_max, -1, np.int32)
    se[:len(slot_expert)] = slot_expert
    return Workload(f"small-{seed}", T, k, E, G_max, R_max, d, f, nv, ids, w, rmap, quota, se,
                    draw_activations(seed, T, d), seed, seed)
