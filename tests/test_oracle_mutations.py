"""Do the pins bite?  Plausible mistakes are planted in the CPU oracle, one at a time, and the pin suite
(tests/test_oracle_pins.py) must fail for each of them.

Everything here runs on the CPU and touches only `oracle/`: a mutation replaces one function of the oracle
module by a subtly wrong version (a wrong sign, a dropped term, a transposed operand, a swapped set, an
off-by-one), the pins are called as plain functions, and at least one of them has to raise.
"""
import inspect
import math

import numpy as np
import pytest

from oracle import lightkv_oracle as O
from tests import test_oracle_pins as P

F64 = np.float64


def _pin_calls():
    """Every pin as a zero-argument callable (parametrised pins with a few of their cases)."""
    calls = []
    for name, fn in sorted(vars(P).items()):
        if not name.startswith("test_") or not callable(fn):
            continue
        params = list(inspect.signature(fn).parameters)
        if not params:
            calls.append((name, fn))
        elif params == ["n", "keep"]:
            for n, keep in ((8, 0.55), (11, 0.7), (12, 0.5)):
                calls.append((f"{name}[{n},{keep}]", lambda fn=fn, n=n, keep=keep: fn(n, keep)))
        # pins that need pytest's own fixtures are left out here
    return calls


def _first_failure():
    for name, fn in _pin_calls():
        try:
            fn()
        except Exception:                      # noqa: BLE001  (an assertion or a crash both count)
            return name
    return None


def test_unmutated_oracle_passes_the_pins_called_this_way():
    assert len(_pin_calls()) >= 20
    assert _first_failure() is None


# ---- the planted mistakes ------------------------------------------------------------------------------

def _fd_wrong_sign(xa, xb):
    return 2.0 - O_feature_divergence(xa, xb)                   # 1 + cos


def _fd_not_normalised_by_b(xa, xb):
    xa, xb = np.asarray(xa, dtype=F64), np.asarray(xb, dtype=F64)
    na = np.sqrt((xa * xa).sum(axis=1))
    g = xa @ xb.T
    den = na[:, None] * np.ones(len(xb))[None, :]
    return 1.0 - np.divide(g, den, out=np.zeros_like(g), where=den > 0)


def _fd_norms_swapped(xa, xb):
    # row norms of B used for the rows and of A for the columns (only visible when |A| = |B|)
    fd = O_feature_divergence(xa, xb)
    if len(xa) != len(xb):
        return fd
    xa, xb = np.asarray(xa, dtype=F64), np.asarray(xb, dtype=F64)
    na, nb = np.sqrt((xa * xa).sum(axis=1)), np.sqrt((xb * xb).sum(axis=1))
    den = nb[:, None] * na[None, :]
    g = xa @ xb.T
    return 1.0 - np.divide(g, den, out=np.zeros_like(g), where=den > 0)


def _bipartition_swapped(order):
    return order[1::2], order[0::2]


def _removal_count_halved(n_window, keep):
    # the printed floor(rho v / 2)
    if n_window < 2:
        return 0
    return max(0, min(int(math.floor((1.0 - keep) * n_window / 2 + 1e-9)), (n_window + 1) // 2))


def _removal_count_off_by_one(n_window, keep):
    r = O_removal_count(n_window, keep)
    return max(0, r - 1) if n_window >= 4 else r


def _select_highest(fd, r):
    n_a, n_b = fd.shape
    m = np.zeros((n_a, n_b), dtype=np.int64)
    if r <= 0 or n_b == 0:
        return m
    best = np.argmin(fd, axis=1)
    f = fd[np.arange(n_a), best]
    for a in np.lexsort((np.arange(n_a), -f))[:r]:
        m[a, best[a]] = 1
    return m


def _select_farthest_partner(fd, r):
    n_a, n_b = fd.shape
    m = np.zeros((n_a, n_b), dtype=np.int64)
    if r <= 0 or n_b == 0:
        return m
    best = np.argmax(fd, axis=1)
    f = fd[np.arange(n_a), best]
    for a in np.lexsort((np.arange(n_a), f))[:r]:
        m[a, best[a]] = 1
    return m


def _xi_mean_over_heads(q, k, vis_begin, n_vis, text_begin, text_end, causal=True, text_ranges=None):
    return O_xi_from_attention(q, k, vis_begin, n_vis, text_begin, text_end, causal, text_ranges) / q.shape[0]


def _xi_prompt_range_shifted(q, k, vis_begin, n_vis, text_begin, text_end, causal=True, text_ranges=None):
    return O_xi_from_attention(q, k, vis_begin, n_vis, text_begin + 1, text_end, causal, text_ranges)


def _attention_without_causal_mask(q, k, vis_begin, n_vis, causal=True):
    return O_attention_rows(q, k, vis_begin, n_vis, False)


def _attention_without_scale(q, k, vis_begin, n_vis, causal=True):
    return O_attention_rows(np.asarray(q, dtype=F64) * math.sqrt(np.asarray(k).shape[1]), k, vis_begin, n_vis, causal)


def _message_passing_plain_mean(xa, xb, xi_a, xi_b, m):
    return O_message_passing(xa, xb, np.ones_like(np.asarray(xi_a, dtype=F64)), np.ones_like(np.asarray(xi_b, dtype=F64)), m)


def _message_passing_transposed_weights(xa, xb, xi_a, xi_b, m):
    # the A-side weights applied in reversed order (a transposed / mis-indexed operand)
    return O_message_passing(xa, xb, np.asarray(xi_a, dtype=F64)[::-1].copy(), xi_b, m)


def _message_passing_without_the_zero_sum_fallback(xa, xb, xi_a, xi_b, m):
    # the vanishing-denominator branch dropped: the division runs on whatever the sums are
    xa, xb = np.asarray(xa, dtype=F64), np.asarray(xb, dtype=F64)
    xi_a, xi_b = np.asarray(xi_a, dtype=F64), np.asarray(xi_b, dtype=F64)
    mt = m.T.astype(F64)
    den = xi_b + mt @ xi_a
    with np.errstate(all="ignore"):
        num = xb * xi_b[:, None] + mt @ (xa * xi_a[:, None])
        return num / den[:, None], (m.astype(F64) @ (1.0 / den)) * xi_a, xi_b / den


def _message_passing_fallback_hits_every_group(xa, xb, xi_a, xi_b, m):
    # one vanishing sum switches ALL groups to the plain mean
    xi_a, xi_b = np.asarray(xi_a, dtype=F64), np.asarray(xi_b, dtype=F64)
    den = xi_b + m.T.astype(F64) @ xi_a
    if (den < 1e-30).any():
        return O_message_passing(xa, xb, np.ones_like(xi_a), np.ones_like(xi_b), m)
    return O_message_passing(xa, xb, xi_a, xi_b, m)


def _row_logsumexp_without_the_scale(q, k, vis_begin, n_vis, causal=True):
    return O_row_logsumexp(np.asarray(q, dtype=F64) * math.sqrt(np.asarray(k).shape[1]), k, vis_begin, n_vis, causal)


def _xi_first_range_only(q, k, vis_begin, n_vis, text_begin, text_end, causal=True, text_ranges=None):
    return O_xi_from_attention(q, k, vis_begin, n_vis, text_begin, text_end, causal,
                               None if text_ranges is None else list(text_ranges)[:1])


def _scaled_logits_always_causal(q, k, vis_begin, n_vis, causal=True):
    return O_scaled_logits(q, k, vis_begin, n_vis, True)


def _divergence_l2sq_without_the_cross_term(xa, xb, metric="cosine"):
    if metric == "cosine":
        return O_divergence(xa, xb, metric)
    xa, xb = np.asarray(xa, dtype=F64), np.asarray(xb, dtype=F64)
    sq = (xa * xa).sum(axis=1)[:, None] + (xb * xb).sum(axis=1)[None, :]
    return sq if metric == "l2sq" else np.sqrt(sq)


def _compress_vision_ignores_the_direction(x, pos, xi, tiles, w, keep, metric="cosine", direction="a2b"):
    return O_compress_vision(x, pos, xi, tiles, w, keep, metric, "a2b")


def _select_edges_literal_counts_tokens_not_pairs(fd, n_window, keep):
    return O_select_edges_literal(fd, n_window, 1.0 - 2.0 * (1.0 - keep)) if keep > 0.5 else O_select_edges_literal(fd, 2 * n_window, keep)


def _window_of_swapped_axes(pos, tiles, w):
    return O_window_of(pos, [(c, r) for r, c in tiles], w)


def _retention_counts_the_compression_layer_as_compressed(n_layers, layers, rho):
    return O_retention(n_layers, [l - 1 for l in layers], rho)


def _compact_kv_ignores_the_weights(kv, vis_begin, n_vis, dst, weight, survivor, mode):
    return O_compact_kv(kv, vis_begin, n_vis, dst, weight, survivor, "gather")


O_feature_divergence, O_removal_count, O_xi_from_attention = O.feature_divergence, O.removal_count, O.xi_from_attention
O_attention_rows, O_message_passing, O_window_of = O.attention_rows, O.message_passing, O.window_of
O_retention, O_compact_kv = O.retention, O.compact_kv
O_row_logsumexp, O_scaled_logits = O.row_logsumexp, O.scaled_logits
O_divergence, O_compress_vision = O.divergence, O.compress_vision
O_select_edges_literal = O.select_edges_literal

MUTATIONS = [
    ("feature_divergence", _fd_wrong_sign),
    ("feature_divergence", _fd_not_normalised_by_b),
    ("feature_divergence", _fd_norms_swapped),
    ("bipartition", _bipartition_swapped),
    ("removal_count", _removal_count_halved),
    ("removal_count", _removal_count_off_by_one),
    ("select_edges", _select_highest),
    ("select_edges", _select_farthest_partner),
    ("xi_from_attention", _xi_mean_over_heads),
    ("xi_from_attention", _xi_prompt_range_shifted),
    ("attention_rows", _attention_without_causal_mask),
    ("attention_rows", _attention_without_scale),
    ("message_passing", _message_passing_plain_mean),
    ("message_passing", _message_passing_transposed_weights),
    ("message_passing", _message_passing_without_the_zero_sum_fallback),
    ("message_passing", _message_passing_fallback_hits_every_group),
    ("row_logsumexp", _row_logsumexp_without_the_scale),
    ("xi_from_attention", _xi_first_range_only),
    ("scaled_logits", _scaled_logits_always_causal),
    ("divergence", _divergence_l2sq_without_the_cross_term),
    ("compress_vision", _compress_vision_ignores_the_direction),
    ("select_edges_literal", _select_edges_literal_counts_tokens_not_pairs),
    ("window_of", _window_of_swapped_axes),
    ("retention", _retention_counts_the_compression_layer_as_compressed),
    ("compact_kv", _compact_kv_ignores_the_weights),
]


@pytest.mark.parametrize("target,wrong", MUTATIONS, ids=[w.__name__.lstrip("_") for _, w in MUTATIONS])
def test_a_planted_mistake_fails_some_pin(monkeypatch, target, wrong):
    monkeypatch.setattr(O, target, wrong)
    failed = _first_failure()
    assert failed is not None, f"no pin noticed the mistake planted in {target}"
