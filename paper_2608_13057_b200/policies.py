"""Dispatch policies for one routed batch, as quota tables and as per-GPU routed batches (host side, off the
timed path).

The paper's dispatcher decides, per batch, how many tokens of each replicated expert go to which replica so
that the slowest GPU of the expert-parallel group finishes as early as possible under the calibrated cost
t_g = max(a + b*G_g + b2*(Tiles_g - G_g), c + beta*N_g) (Eq. 1 - Eq. 3; solver: Section 4.2), and compares that
against proxy policies that balance tokens or activations instead of time (Figure 1(b), Table "feasible").
This module closes that loop for the mixed-regime configuration: the routed batch of config 3 is spread over
two virtual GPUs - A holds the rank's 16 primary experts, B holds replicas of its four hottest - and every
policy yields
  * the quota table x_{e,r} for the rank that holds all 20 slots (what tempo_count_dispatch consumes), and
  * the routed batch each virtual GPU would see after the dispatch all-to-all (pairs sent to the other GPU
    become ids of an expert that is not local), so each GPU's block can be timed on its own and the
    makespan taken as the maximum, as the paper's microbenchmark does.
Nothing here computes any step of the hot path; it only builds inputs.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Sequence

import numpy as np

from . import costmodel as C
from . import solver as S
from . import workloads as W

# tempo_fast_stale1 is the deployment the paper describes (Section 4.4, "Pricing staleness"): the table is solved on
# the PREVIOUS window's counts, recovered from the cumulative counter, and the kernel renormalises its rows at use.
POLICIES = ("uniform", "token_balanced", "hot_whole", "tempo_fast", "tempo_fast_stale1")


@dataclasses.dataclass
class PolicyCase:
    name: str
    x: np.ndarray                 # [n_local, 2] rows of each local expert on virtual GPU A / B
    rank: W.Workload              # the rank holding all 20 slots, its quota table = the policy's (possibly stale) table
    gpus: List[W.Workload]        # [A, B]: the routed batch each virtual GPU sees, its own slots only
    rank_rows: np.ndarray         # [20] rows every instance slot of the rank must end up with (x in slot order)


def _local_counts(wl: W.Workload, local: Sequence[int]) -> List[int]:
    live = wl.topk_ids[:wl.n_valid].reshape(-1)
    c = np.bincount(live, minlength=wl.E)
    return [int(c[e]) for e in local]


def renormalised(quota_row: Sequence[int], n_e: int) -> List[int]:
    """Rows each replica column receives when a (possibly stale) share row meets n_e pairs: column r takes the
    ranks [floor(C_{r-1} n_e / S), floor(C_r n_e / S)) with C the running sum of the shares, uniform if S = 0."""
    q = [max(int(v), 0) for v in quota_row]
    if sum(q) == 0:
        q = [1] * len(q)
    S_, out, C_, prev = sum(q), [], 0, 0
    for v in q:
        C_ += v
        b = (C_ * int(n_e)) // S_
        out.append(b - prev)
        prev = b
    return out


def shares(policy: str, counts: Sequence[int], hot: Sequence[int], params: S.CostParams) -> np.ndarray:
    """x[i, g]: rows of local expert i on virtual GPU g (0 = A, primaries; 1 = B, replicas of `hot`)."""
    n = len(counts)
    replicas = [[0, 1] if i in hot else [0] for i in range(n)]
    x = np.zeros((n, 2), np.int64)
    if policy == "uniform":                                  # replicas split their expert in halves
        for i, c in enumerate(counts):
            x[i] = ((c + 1) // 2, c // 2) if i in hot else (c, 0)
    elif policy == "token_balanced":                         # equalise tokens per GPU (a token-balancing LP's optimum)
        total, hot_total = sum(counts), sum(counts[i] for i in hot)
        phi = min(1.0, (total / 2) / max(1, hot_total))
        for i, c in enumerate(counts):
            b = int(np.floor(phi * c)) if i in hot else 0
            x[i] = (c - b, b)
    elif policy == "hot_whole":                              # never split: every expert whole on its primary
        for i, c in enumerate(counts):
            x[i] = (c, 0)
    elif policy == "tempo_fast":
        x = S.tempo_fast(list(counts), replicas, 2, params)
    else:
        raise ValueError(policy)
    assert np.array_equal(x.sum(1), np.asarray(counts)) and np.all(x >= 0)
    return x


def modeled(x: np.ndarray, params: S.CostParams) -> Dict[str, float]:
    """The cost model's view of a policy: per virtual GPU, their maximum, and the rank holding all slots."""
    t = [params.gpu_time(x[:, g]) for g in range(x.shape[1])]
    return dict(gpu_us=t, makespan_us=max(t), rank_us=params.gpu_time(x.reshape(-1)))


def previous_window_counts(seed: int, T: int, local: Sequence[int]) -> List[int]:
    """Counts of the window before the batch, the way the off-path thread sees them: another routed batch of
    the same popularity (seed + 1000) has gone through the cumulative counter, which wrapped on the way."""
    prev = W.config3("uniform", seed=seed + 1000, T=T)
    live = prev.topk_ids[:prev.n_valid].reshape(-1)
    counts = np.bincount(live, minlength=prev.E).astype(np.uint64)
    snap0 = np.full(prev.E, 2 ** 32 - 7, np.uint64)                       # the counter just before it wraps
    snap1 = ((snap0 + counts) % (1 << 32)).astype(np.uint32)             # what tempo_count_dispatch leaves behind
    window = C.window_counts(snap1, snap0.astype(np.uint32))
    assert np.array_equal(window.astype(np.uint64), counts)
    return [int(window[e]) for e in local]


def build_cases(params: S.CostParams, seed: int = 2, T: int = 4096, policies: Sequence[str] = POLICIES,
                with_x: bool = True) -> List[PolicyCase]:
    """Config 3's routed batch under each policy."""
    base = W.config3("uniform", seed=seed, T=T)
    if not with_x:
        base.x = None
    local = [int(e) for e in base.slot_expert[:16]]
    hot_experts = [int(e) for e in base.slot_expert[16:20]]
    hot = [local.index(e) for e in hot_experts]
    counts = _local_counts(base, local)
    remote = next(e for e in range(base.E) if e not in local)          # an expert this rank does not hold
    ids = base.topk_ids
    flat = ids.reshape(-1)
    cases = []
    for name in policies:
        if name == "tempo_fast_stale1":
            # solved on last window's counts; the published table is stale, the kernel renormalises each row
            table = shares("tempo_fast", previous_window_counts(seed, T, local), hot, params)
            x = np.array([renormalised(table[i], counts[i]) if i in hot else [counts[i], 0] for i in range(len(local))],
                         np.int64)
        else:
            table = x = shares(name, counts, hot, params)
        # the rank that holds all 20 slots: column 0 = primary slot, column 1 = replica slot
        rmap, quota = base.replica_map.copy(), np.zeros_like(base.quota)
        for i, e in enumerate(local):
            quota[e, 0] = table[i, 0]
            if i in hot:
                quota[e, 1] = table[i, 1]
        rank = dataclasses.replace(base, name=f"cfg3-policy-{name}", replica_map=rmap, quota=quota, _wcache={})
        # what each virtual GPU sees after the all-to-all: of expert e's pairs in ascending pair index, the first
        # x[i, 0] stay on A and the rest go to B (the contiguous rank runs of the dispatch rule)
        ids_a, ids_b = flat.copy(), np.full_like(flat, remote)
        live = base.n_valid * base.k
        for i, e in enumerate(local):
            pairs = np.nonzero(flat[:live] == e)[0]
            to_b = pairs[x[i, 0]:]
            ids_a[to_b] = remote
            ids_b[to_b] = e
        gpus = []
        for g, (gid, slots) in enumerate(((ids_a, local), (ids_b, hot_experts))):
            rm = np.full((base.E, 1), -1, np.int32)
            q = np.zeros((base.E, 1), np.int32)
            for s, e in enumerate(slots):
                rm[e, 0] = s
                q[e, 0] = x[local.index(e), g]
            gpus.append(W.Workload(f"cfg3-policy-{name}-gpu{'AB'[g]}", base.T, base.k, base.E, len(slots), 1, base.d,
                                   base.f, base.n_valid, gid.reshape(ids.shape).astype(np.int32), base.topk_w, rm, q,
                                   np.asarray(slots, np.int32), base.x, base.seed, base.weight_seed))
        rank_rows = np.array([x[i, 0] for i in range(len(local))] + [x[i, 1] for i in hot], np.int64)
        cases.append(PolicyCase(name, x, rank, gpus, rank_rows))
    return cases
