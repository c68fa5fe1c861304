"""Host-side cost profile of the expert block: evaluation and fitting (never on the timed path).

The per-rank time is modelled as the two-piece max-affine profile of Eq. 1,
    t = max(a + b*G, c + beta*N),
with G the number of activated (expert, replica) instances and N the rows they hold, and its
tile-aware form of Eq. 3,
    t = max(a + b*G + b2*(Tiles - G), c + beta*N),   Tiles = sum_i ceil(m_i / 128).
The inflection is n* = b / beta (Table "Fitted cost parameters").  Fitting follows the
calibration appendix: alternating assignment of points to the two pieces, least squares per
piece, at most 50 rounds.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np


def window_counts(cum_now, cum_prev) -> np.ndarray:
    """Per-expert counts of the window between two snapshots of the cumulative u32 counter that
    tempo_count_dispatch keeps (Section 4.4: cumulative counting needs no zeroing kernel in the graph; the
    background thread recovers windows by wrap-safe differencing).  Exact as long as fewer than 2^32 pairs of
    one expert fall into a window."""
    now = np.asarray(cum_now).astype(np.uint32, copy=False)
    prev = np.asarray(cum_prev).astype(np.uint32, copy=False)
    return (now - prev).astype(np.uint32)          # unsigned subtraction wraps mod 2^32


def tiles_of(rows: Sequence[int], tile: int = 128) -> int:
    return int(sum(-(-int(m) // tile) for m in rows if m > 0))


def block_time(a: float, b: float, c: float, beta: float, G, N, b2: float = 0.0, tiles=None):
    """Eq. 1 (b2 == 0) or Eq. 3."""
    G = np.asarray(G, dtype=np.float64)
    N = np.asarray(N, dtype=np.float64)
    flat = a + b * G
    if b2 != 0.0:
        flat = flat + b2 * (np.asarray(tiles, dtype=np.float64) - G)
    return np.maximum(flat, c + beta * N)


def makespan(a, b, c, beta, per_gpu_rows: Sequence[Sequence[int]], b2: float = 0.0) -> float:
    """Eq. 2's objective for a given dispatch: per_gpu_rows[g] lists the rows of each instance on GPU g."""
    worst = 0.0
    for rows in per_gpu_rows:
        act = [m for m in rows if m > 0]
        worst = max(worst, float(block_time(a, b, c, beta, len(act), sum(act), b2, tiles_of(act))))
    return worst


def n_star(b: float, beta: float) -> float:
    return b / beta


def _lstsq(cols, t):
    A = np.stack(cols, axis=1)
    coef, *_ = np.linalg.lstsq(A, t, rcond=None)
    return coef


def fit_max_affine(G, N, t, tiles=None, iters: int = 50, tile_aware: bool = False) -> Dict[str, float]:
    """Alternating-assignment fit of Eq. 1 (or Eq. 3 when tile_aware) to measured (G, N, t).

    Start: points with N/G <= 128 belong to the flat piece.  Each round: least squares per
    piece on its points, then every point moves to the piece that predicts the larger time.
    Stops after `iters` rounds or when no point moves.  Error = mean |pred - t| / t.
    """
    G = np.asarray(G, dtype=np.float64)
    N = np.asarray(N, dtype=np.float64)
    t = np.asarray(t, dtype=np.float64)
    one = np.ones_like(t)
    extra = (np.asarray(tiles, dtype=np.float64) - G) if tile_aware else None
    flat = (N / np.maximum(G, 1)) <= 128
    a = b = c = beta = b2 = 0.0
    for _ in range(iters):
        if flat.sum() >= (3 if tile_aware else 2):
            cols = [one[flat], G[flat]] + ([extra[flat]] if tile_aware else [])
            co = _lstsq(cols, t[flat])
            a, b = float(co[0]), float(co[1])
            b2 = float(co[2]) if tile_aware else 0.0
        if (~flat).sum() >= 2:
            co = _lstsq([one[~flat], N[~flat]], t[~flat])
            c, beta = float(co[0]), float(co[1])
        pf = a + b * G + (b2 * extra if tile_aware else 0.0)
        pl = c + beta * N
        new = pf >= pl
        if np.array_equal(new, flat):
            break
        flat = new
    pred = block_time(a, b, c, beta, G, N, b2, tiles if tile_aware else None)
    err = float(np.mean(np.abs(pred - t) / t))
    return dict(a=a, b=b, c=c, beta=beta, b2=b2, n_star=(b / beta if beta > 0 else float("inf")),
                fit_err=err, n_flat=int(flat.sum()), n_linear=int((~flat).sum()))
