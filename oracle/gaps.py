"""Selection-boundary gaps of a synthetic input, and their repair.

TEST INFRASTRUCTURE ONLY (uses the oracle's FD; never imported by the product).

Index-set parity between the CUDA path (fp32 accumulation) and the oracle
(double) is only claimed on inputs where every decision of Step 2 is separated
by a margin: (i) for every A node, second-lowest FD minus lowest FD; (ii) per
window with 0 < r < |A|, the (r+1)-th lowest best-FD minus the r-th.  This file
measures those margins with the oracle's arithmetic and nudges offending rows
(x_a += step * ||x_a|| * unit(x_b*), which raises only the winning cosine;
for the Euclidean scores x_a moves a step towards x_b*) until every margin is
at least `gap`.  For the Euclidean scores the margin is relative to the
window's mean squared norm (their values scale with the rows).  The repaired
tensor is an INPUT: both sides then read the same bytes.
"""
from __future__ import annotations

from typing import Callable, Dict, Sequence, Tuple

import numpy as np

from . import lightkv_oracle as O


def window_members(pos: np.ndarray, tiles, w: int):
    win = O.window_of(pos, tiles, w)
    for wid in np.unique(win):
        members = np.nonzero(win == wid)[0]
        yield members[np.argsort(pos[members], kind="stable")]


def _sets(members, direction):
    ia, ib = O.bipartition(members)
    return (ib, ia) if direction == "b2a" else (ia, ib)


def _scores(x, ia, ib, metric):
    """Pair scores in units in which `gap` is meant: FD as it is; squared distances divided by the mean squared
    norm of the rows involved; plain distances by its root."""
    fd = O.divergence(x[ia], x[ib], metric)
    if metric == "cosine":
        return fd
    scale = float(np.mean((x[np.concatenate([ia, ib])] ** 2).sum(axis=1)))
    return fd / (scale if metric == "l2sq" else np.sqrt(scale))


def selection_gaps(x: np.ndarray, pos: np.ndarray, tiles, w: int, keep: float, metric: str = "cosine",
                   direction: str = "a2b") -> Dict[str, object]:
    """Smallest margins over all windows; also the offending (a, b*) pairs below
    `gap` are found by enforce_gaps, this only reports the minima."""
    x = np.asarray(x, dtype=np.float64)
    g_partner, g_boundary = np.inf, np.inf
    for members in window_members(np.asarray(pos), tiles, w):
        ia, ib = _sets(members, direction)
        if len(ib) == 0 or len(ia) == 0:
            continue
        fd = _scores(x, ia, ib, metric)
        srt = np.sort(fd, axis=1)
        if fd.shape[1] > 1:
            g_partner = min(g_partner, float((srt[:, 1] - srt[:, 0]).min()))
        r = min(O.removal_count(len(members), keep), len(ia))
        if 0 < r < len(ia):
            f = np.sort(srt[:, 0])
            g_boundary = min(g_boundary, float(f[r] - f[r - 1]))
    return {"partner_gap": g_partner, "boundary_gap": g_boundary}


def enforce_gaps(x: np.ndarray, pos: np.ndarray, tiles, w: int, keep: float, gap: float = 1e-3,
                 rounder: Callable[[np.ndarray], np.ndarray] = lambda a: a,
                 step: float = 0.05, max_sweeps: int = 40, metric: str = "cosine",
                 direction: str = "a2b") -> Tuple[np.ndarray, Dict[str, object]]:
    """Returns (repaired copy of x in the storage type's value set, report)."""
    x = np.array(x, dtype=np.float64, copy=True)
    pos = np.asarray(pos)
    target = gap * 1.25                                   # head-room for the re-rounding
    nudges = 0
    windows = list(window_members(pos, tiles, w))
    for sweep in range(max_sweeps):
        dirty = False
        for members in windows:
            ia, ib = _sets(members, direction)
            if len(ib) == 0 or len(ia) == 0:
                continue
            for _ in range(200):
                fd = _scores(x, ia, ib, metric)
                best = np.argmin(fd, axis=1)
                bad = np.zeros(len(ia), dtype=bool)
                if fd.shape[1] > 1:
                    srt = np.sort(fd, axis=1)
                    bad |= (srt[:, 1] - srt[:, 0]) < target
                r = min(O.removal_count(len(members), keep), len(ia))
                if 0 < r < len(ia):
                    f = fd[np.arange(len(ia)), best]
                    order = np.lexsort((np.arange(len(ia)), f))
                    if f[order[r]] - f[order[r - 1]] < target:
                        bad[order[r - 1]] = True
                if not bad.any():
                    break
                dirty = True
                for a in np.nonzero(bad)[0]:
                    xb = x[ib[best[a]]]
                    if metric == "cosine":
                        na = np.linalg.norm(x[ia[a]])
                        x[ia[a]] = rounder(x[ia[a]] + step * na * xb / np.linalg.norm(xb))
                    else:
                        x[ia[a]] = rounder(x[ia[a]] + step * (xb - x[ia[a]]))
                    nudges += 1
        if not dirty:
            break
    rep = selection_gaps(x, pos, tiles, w, keep, metric, direction)
    rep["nudges"] = nudges
    rep["ok"] = bool(min(rep["partner_gap"], rep["boundary_gap"]) >= gap)
    return x, rep
