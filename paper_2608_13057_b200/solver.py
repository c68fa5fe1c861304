"""Off-path host solver for the fixed-charge makespan dispatch problem (never on the timed path).

Problem (Eq. 2): per-expert counts n_e, replica sets R(e) (GPUs holding a copy of expert e), integer shares
x[e][g] >= 0 with sum_g x[e][g] = n_e supported on R(e); minimise max_g t_g with the calibrated cost
t_g = max(a + b*G_g + b2*(Tiles_g - G_g), c + beta*N_g)  (Eq. 1 / Eq. 3), G_g = activated experts on g.

`tempo_fast` follows the four stages of Section 4.2:
  1. cost-aware greedy seeding: experts in descending count, each whole on its cheapest replica;
  2. activation rebalancing by 1- and 2-step augmenting chains of whole-expert moves;
  3. bottleneck local search: whole moves and integer ternary-search partial splits off the bottleneck GPU
     (at most 300 rounds; with a tile term the split is also tried at 128-row boundaries).  A split is also
     tried after first pulling one whole expert of the destination back onto the bottleneck: without that
     compound move the search stalls on the paper's own toy batch (Figure 1b), where splitting the hot
     expert only pays once the destination has shed an activation;
  4. ensemble with a switching tolerance tau: the token-balanced LP split and, under full replication, the
     round-robin placement A3 of Theorem 2 are scored under the same model and adopted only if better by
     more than tau (1 %).
The result is the quota table the GPU path consumes (one column per replica of each expert).
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np

TILE = 128


@dataclasses.dataclass(frozen=True)
class CostParams:
    a: float = 0.0
    b: float = 1.0
    c: float = 0.0
    beta: float = 0.0
    b2: float = 0.0

    def gpu_time(self, rows: Sequence[int]) -> float:
        act = [int(m) for m in rows if m > 0]
        G, N = len(act), sum(act)
        flat = self.a + self.b * G
        if self.b2:
            flat += self.b2 * (sum(-(-m // TILE) for m in act) - G)
        return max(flat, self.c + self.beta * N)


def makespan(x: np.ndarray, p: CostParams) -> float:
    """x[e, g] integer shares -> max over GPUs of the modelled time."""
    return max(p.gpu_time(x[:, g]) for g in range(x.shape[1]))


def lower_bound(counts: Sequence[int], n_gpus: int, p: CostParams) -> float:
    """LB = max(a + b*ceil(E_live/g), c + beta*N/g) <= OPT (Theorem 2's discussion)."""
    live = sum(1 for n in counts if n > 0)
    return max(p.a + p.b * -(-live // n_gpus), p.c + p.beta * sum(counts) / n_gpus)


def _check(counts, replicas, n_gpus):
    for e, n in enumerate(counts):
        if n > 0 and not replicas[e]:
            raise ValueError(f"expert {e} has tokens but no replica")
        if any(g < 0 or g >= n_gpus for g in replicas[e]):
            raise ValueError(f"expert {e}: replica outside [0, {n_gpus})")


def round_robin_a3(counts: Sequence[int], n_gpus: int) -> np.ndarray:
    """Theorem 2's A3 (full replication): whole experts, descending count, GPU i takes ranks i, i+g, ..."""
    x = np.zeros((len(counts), n_gpus), dtype=np.int64)
    order = sorted(range(len(counts)), key=lambda e: (-counts[e], e))
    for rank, e in enumerate(order):
        x[e, rank % n_gpus] = counts[e]
    return x


def uniform_split(counts, replicas, n_gpus) -> np.ndarray:
    x = np.zeros((len(counts), n_gpus), dtype=np.int64)
    for e, n in enumerate(counts):
        r = sorted(replicas[e])
        for j, g in enumerate(r):
            x[e, g] = n // len(r) + (1 if j < n % len(r) else 0)
    return x


def token_lp(counts, replicas, n_gpus) -> np.ndarray:
    """Token balancing: minimise max_g N_g over real splits (an LP), rounded to integers that keep the row sums."""
    from scipy.optimize import linprog
    pairs = [(e, g) for e in range(len(counts)) for g in sorted(replicas[e]) if counts[e] > 0]
    x = np.zeros((len(counts), n_gpus), dtype=np.int64)
    if not pairs:
        return x
    nv = len(pairs) + 1                                   # last variable: the makespan in tokens
    cost = np.zeros(nv)
    cost[-1] = 1.0
    A_ub = np.zeros((n_gpus, nv))
    for j, (e, g) in enumerate(pairs):
        A_ub[g, j] = 1.0
    A_ub[:, -1] = -1.0
    live = [e for e in range(len(counts)) if counts[e] > 0]
    A_eq = np.zeros((len(live), nv))
    for j, (e, g) in enumerate(pairs):
        A_eq[live.index(e), j] = 1.0
    res = linprog(cost, A_ub=A_ub, b_ub=np.zeros(n_gpus), A_eq=A_eq, b_eq=[counts[e] for e in live],
                  bounds=[(0, None)] * nv, method="highs")
    if not res.success:
        return uniform_split(counts, replicas, n_gpus)
    frac = np.zeros((len(counts), n_gpus))
    for j, (e, g) in enumerate(pairs):
        frac[e, g] = res.x[j]
    for e in live:                                        # largest-remainder rounding per expert
        fl = np.floor(frac[e]).astype(np.int64)
        rem = counts[e] - int(fl.sum())
        order = sorted(replicas[e], key=lambda g: -(frac[e, g] - fl[g]))
        for g in order[:rem]:
            fl[g] += 1
        x[e] = fl
    return x


def _best_split(x, e, src, dst, p: CostParams):
    """Best integer amount of expert e to move src -> dst for the pair's max time (unimodal: ternary search)."""
    have = int(x[e, src])

    def pair_time(m):
        xs, xd = x[:, src].copy(), x[:, dst].copy()
        xs[e] -= m
        xd[e] += m
        return max(p.gpu_time(xs), p.gpu_time(xd))

    lo, hi = 0, have
    while hi - lo > 2:
        m1, m2 = lo + (hi - lo) // 3, hi - (hi - lo) // 3
        if pair_time(m1) <= pair_time(m2):
            hi = m2
        else:
            lo = m1
    cands = set(range(lo, hi + 1)) | {0, have}
    if p.b2:                                              # tile-aware: also try splits on 128-row boundaries
        for m in list(cands):
            for snap in ((m // TILE) * TILE, -(-m // TILE) * TILE):
                if 0 <= snap <= have:
                    cands.add(snap)
            rest = have - m
            for snap in ((rest // TILE) * TILE, -(-rest // TILE) * TILE):
                if 0 <= have - snap <= have:
                    cands.add(have - snap)
    best = min(cands, key=lambda m: (pair_time(m), m))
    return best, pair_time(best)


def tempo_fast(counts: Sequence[int], replicas: Sequence[Sequence[int]], n_gpus: int, p: CostParams,
               tau: float = 0.01, max_rounds: int = 300, stages=(1, 2, 3, 4)) -> np.ndarray:
    counts = [int(n) for n in counts]
    replicas = [sorted(set(int(g) for g in r)) for r in replicas]
    _check(counts, replicas, n_gpus)
    E = len(counts)
    x = np.zeros((E, n_gpus), dtype=np.int64)

    # 1. greedy seeding: descending tokens, whole expert on the replica with the lowest resulting time
    for e in sorted(range(E), key=lambda e: (-counts[e], e)):
        if counts[e] == 0:
            continue
        def after(g):
            col = x[:, g].copy()
            col[e] = counts[e]
            return (p.gpu_time(col), int(col.sum()), g)
        g = min(replicas[e], key=after)
        x[e, g] = counts[e]
    if 1 not in stages:
        x = uniform_split(counts, replicas, n_gpus)

    def times():
        return [p.gpu_time(x[:, g]) for g in range(n_gpus)]

    # 2. augmenting chains: whole-expert moves off the bottleneck, directly or through one relay GPU
    if 2 in stages:
        for _ in range(max_rounds):
            t = times()
            bott = int(np.argmax(t))
            best = None
            for e in np.nonzero(x[:, bott])[0]:
                n = int(x[e, bott])
                for g1 in replicas[e]:
                    if g1 == bott:
                        continue
                    xs = x.copy()
                    xs[e, bott] -= n
                    xs[e, g1] += n
                    m1 = makespan(xs, p)
                    if m1 < t[bott] - 1e-12 and (best is None or m1 < best[0]):
                        best = (m1, xs)
                    # 2-step chain: relieve g1 by passing one of its experts on
                    for e2 in np.nonzero(x[:, g1])[0]:
                        if e2 == e:
                            continue
                        n2 = int(x[e2, g1])
                        for g2 in replicas[e2]:
                            if g2 in (g1, bott):
                                continue
                            xt = xs.copy()
                            xt[e2, g1] -= n2
                            xt[e2, g2] += n2
                            m2 = makespan(xt, p)
                            if m2 < t[bott] - 1e-12 and (best is None or m2 < best[0]):
                                best = (m2, xt)
            if best is None:
                break
            x = best[1]

    # 3. bottleneck local search with partial migrations
    if 3 in stages:
        for _ in range(max_rounds):
            t = times()
            bott = int(np.argmax(t))
            cur = t[bott]
            best = None
            for e in np.nonzero(x[:, bott])[0]:
                for g in replicas[e]:
                    if g == bott:
                        continue
                    # plain migration of part (or all) of e, or the same after first taking one whole
                    # expert of g back onto the bottleneck (splitting a hot expert only pays once the
                    # destination has shed an activation)
                    swaps = [None] + [e2 for e2 in np.nonzero(x[:, g])[0] if e2 != e and bott in replicas[e2]]
                    for e2 in swaps:
                        base = x
                        if e2 is not None:
                            base = x.copy()
                            base[e2, bott] += base[e2, g]
                            base[e2, g] = 0
                        m, _ = _best_split(base, e, bott, g, p)
                        if m == 0:
                            continue
                        xs = base.copy()
                        xs[e, bott] -= m
                        xs[e, g] += m
                        ms = makespan(xs, p)
                        if ms < cur - 1e-12 and (best is None or ms < best[0]):
                            best = (ms, xs)
            if best is None:
                break
            x = best[1]

    # 4. ensemble with switching tolerance
    if 4 in stages:
        cands = [token_lp(counts, replicas, n_gpus)]
        if all(len(replicas[e]) == n_gpus for e in range(E) if counts[e] > 0):
            cands.append(round_robin_a3(counts, n_gpus))
        cur = makespan(x, p)
        for cand in cands:
            mc = makespan(cand, p)
            if mc < (1.0 - tau) * cur:
                x, cur = cand, mc
    return x


def quota_table(x: np.ndarray, replica_gpus: Sequence[Sequence[int]], R_max: int) -> np.ndarray:
    """x[e, g] -> quota[e, r] in the column order of replica_gpus[e] (the layout tempo_count_dispatch reads)."""
    q = np.zeros((x.shape[0], R_max), dtype=np.int32)
    for e, gpus in enumerate(replica_gpus):
        for r, g in enumerate(gpus):
            q[e, r] = x[e, g]
    return q
