"""Selection-boundary gaps of a synthetic input, and their repair.

TEST INFRASTRUCTURE ONLY (uses the oracle's FD; never imported by the product).

Index-set parity between the CUDA path (fp32 accumulation) and the oracle
(double) is only claimed on inputs where every decision of Step 2 is separated
by a margin: (i) for every A node, second-lowest FD minus lowest FD; (ii) per
window with 0 < r < |A|, the (r+1)-th lowest best-FD minus the r-th.  This file
measures those margins with the oracle's arithmetic and nudges offending rows
(x_a += step * ||x_a|| * unit(x_b*), which raises only the winning cosine)
until every margin is at least `gap`.  The repaired tensor is an INPUT: both
sides then read the same bytes.
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


def selection_gaps(x: np.ndarray, pos: np.ndarray, tiles, w: int, keep: float) -> Dict[str, object]:
    """Smallest margins over all windows; also the offending (a, b*) pairs below
    `gap` are found by enforce_gaps, this only reports the minima."""
    x = np.asarray(x, dtype=np.float64)
    g_partner, g_boundary = np.inf, np.inf
    for members in window_members(np.asarray(pos), tiles, w):
        ia, ib = O.bipartition(members)
        if len(ib) == 0:
            continue
        fd = O.feature_divergence(x[ia], x[ib])
        srt = np.sort(fd, axis=1)
        if fd.shape[1] > 1:
            g_partner = min(g_partner, float((srt[:, 1] - srt[:, 0]).min()))
        r = O.removal_count(len(members), keep)
        if 0 < r < len(ia):
            f = np.sort(srt[:, 0])
            g_boundary = min(g_boundary, float(f[r] - f[r - 1]))
    return {"partner_gap": g_partner, "boundary_gap": g_boundary}


def enforce_gaps(x: np.ndarray, pos: np.ndarray, tiles, w: int, keep: float, gap: float = 1e-3,
                 rounder: Callable[[np.ndarray], np.ndarray] = lambda a: a,
                 step: float = 0.05, max_sweeps: int = 40) -> Tuple[np.ndarray, Dict[str, object]]:
    """Returns (repaired copy of x in the storage type's value set, report)."""
    x = np.array(x, dtype=np.float64, copy=True)
    pos = np.asarray(pos)
    target = gap * 1.25                                   # head-room for the re-rounding
    nudges = 0
    windows = list(window_members(pos, tiles, w))
    for sweep in range(max_sweeps):
        dirty = False
        for members in windows:
            ia, ib = O.bipartition(members)
            if len(ib) == 0:
                continue
            for _ in range(200):
                fd = O.feature_divergence(x[ia], x[ib])
                best = np.argmin(fd, axis=1)
                bad = np.zeros(len(ia), dtype=bool)
                if fd.shape[1] > 1:
                    srt = np.sort(fd, axis=1)
                    bad |= (srt[:, 1] - srt[:, 0]) < target
                r = O.removal_count(len(members), keep)
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
                    na = np.linalg.norm(x[ia[a]])
                    x[ia[a]] = rounder(x[ia[a]] + step * na * xb / np.linalg.norm(xb))
                    nudges += 1
        if not dirty:
            break
    rep = selection_gaps(x, pos, tiles, w, keep)
    rep["nudges"] = nudges
    rep["ok"] = bool(min(rep["partner_gap"], rep["boundary_gap"]) >= gap)
    return x, rep
