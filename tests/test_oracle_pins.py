"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each pin is chosen so that a
plausible slip in the oracle (dropped term, wrong sign or index, transposed
operand, wrong set parity) makes it fail.
"""
import itertools
import math
import os

import numpy as np
import pytest
import scipy.spatial.distance
import scipy.special

import lightkv_synth as S
from oracle import gaps as G
from oracle import lightkv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([c.strip() for c in line.split(";")])
    return out


# ------------------------------------------------------------------ FD (Eq. "similarity")

def test_fd_special_vectors():
    e0, e1 = np.eye(4)[0], np.eye(4)[1]
    fd = O.feature_divergence(np.stack([e0, e0, e0]), np.stack([3.0 * e0, e1, -2.0 * e0]))
    np.testing.assert_allclose(fd[0], [0.0, 1.0, 2.0], atol=1e-15)


def test_fd_matches_library_cosine_distance_and_is_not_transposed():
    rng = np.random.default_rng(0)
    xa, xb = rng.standard_normal((5, 33)), rng.standard_normal((7, 33))
    fd = O.feature_divergence(xa, xb)
    assert fd.shape == (5, 7)
    np.testing.assert_allclose(fd, scipy.spatial.distance.cdist(xa, xb, "cosine"), atol=1e-13)
    np.testing.assert_allclose(fd, O.feature_divergence(xb, xa).T, atol=1e-15)          # symmetric
    np.testing.assert_allclose(fd, O.feature_divergence(2.5 * xa, 0.1 * xb), atol=1e-13)  # scale free
    assert (fd >= -1e-15).all() and (fd <= 2 + 1e-15).all()


def test_fd_zero_row_reads_as_one():
    fd = O.feature_divergence(np.zeros((1, 3)), np.ones((2, 3)))
    np.testing.assert_array_equal(fd, [[1.0, 1.0]])


# ------------------------------------------------------- counts (Eq. "complexity", tables)

def test_retention_printed_example():
    for n_layers, lam, rho, printed, dec in _rows("retention_examples.txt"):
        lam = [int(v) for v in lam.split(",")]
        rho = [float(v) for v in rho.split(",")]
        got = 100.0 * O.retention(int(n_layers), lam, rho)
        assert round(got, int(dec)) == float(printed)
    assert O.retention(40, [10, 20, 30], [0.5] * 3) == pytest.approx(18.75 / 40, abs=1e-15)


def test_retention_of_the_papers_schedules_is_55_percent():
    assert O.retention(40, [15, 23, 31], [0.5] * 3) == pytest.approx(0.553125)
    assert O.retention(32, [12, 18, 24], [0.5] * 3) == pytest.approx(0.546875)
    # no compression keeps everything; the three terms of the equation are all needed
    assert O.retention(10, [3, 5], [0.0, 0.0]) == 1.0
    assert O.vision_tokens_processed(100, 10, [4], [0.5]) == 100 * (4 + 6 * 0.5)
    assert O.vision_tokens_processed(8, 10, [2, 6], [0.5, 0.25]) == pytest.approx(
        8 * (2 + 4 * 0.5 + 4 * 0.5 * 0.75))


def test_first_stage_count_printed_in_the_paper():
    for rows, cols, w, rho, n_in, n_out in _rows("token_chain.txt"):
        rows, cols, w, n_in, n_out = int(rows), int(cols), int(w), int(n_in), int(n_out)
        rng = np.random.default_rng(1)
        x = rng.standard_normal((n_in, 8))
        res = O.compress_vision(x, np.arange(n_in), np.ones(n_in), [(rows, cols)], w, 1.0 - float(rho))
        assert res["n_out"] == n_out == len(res["pos_out"])


def test_fd_cost_table_ratios():
    tab = [(int(v), float(b), float(f)) for v, b, f in _rows("fd_cost_table.txt")]
    for v, bip, full in tab:
        pc = O.pair_counts(v)
        assert pc["bipartite"] == (v // 2) ** 2                      # ~ v^2 / 4
        assert pc["full"] == v * (v - 1) / 2
        # printed numbers are |A||B| * 2048 / 1e9 up to small O(v d) terms
        assert pc["bipartite"] * 2048 / 1e9 == pytest.approx(bip, rel=5e-3)
        assert full / bip == pytest.approx(4.0, rel=5e-3)            # "approximately 4x"
    for (v0, b0, _), (v1, b1, _) in zip(tab, tab[1:]):
        assert v1 == 2 * v0 and b1 / b0 == pytest.approx(4.0, rel=5e-3)
    # windowing divides the pairwise work by w^2 (paragraph "Window partitioning")
    assert O.pair_counts(576, 4)["windowed_full"] == 0.5 * 576 * (36 - 1)
    assert O.pair_counts(576, 4)["bipartite"] == 16 * 18 * 18


def test_oracle_evaluates_exactly_the_bipartite_pairs(monkeypatch):
    calls = []
    real = O.feature_divergence

    def spy(xa, xb):
        calls.append((len(xa), len(xb)))
        return real(xa, xb)

    monkeypatch.setattr(O, "feature_divergence", spy)
    rng = np.random.default_rng(2)
    O.compress_vision(rng.standard_normal((576, 4)), np.arange(576), np.ones(576), [(24, 24)], 4, 0.5)
    assert sorted(calls) == [(18, 18)] * 16
    assert sum(a * b for a, b in calls) == O.pair_counts(576, 4)["bipartite"]


def test_removal_count():
    assert O.removal_count(36, 0.5) == 18 and O.removal_count(36, 0.55) == 16
    assert O.removal_count(20, 0.55) == 9            # 0.55 * 20 = 11.000000000000002 in binary
    assert O.removal_count(16, 0.55) == 7 and O.removal_count(576, 0.55) == 259
    assert O.removal_count(7, 0.5) == 3              # floor(3.5)
    assert O.removal_count(3, 0.1) == 2              # capped at |A| = 2
    assert O.removal_count(1, 0.5) == 0 and O.removal_count(0, 0.5) == 0
    assert O.removal_count(50, 1.0) == 0
    for n in range(2, 300):
        assert O.removal_count(n, 0.5) == n // 2     # "halving"; never more than |A|


# ------------------------------------------------------------------------------- windows

def test_window_geometry():
    win = O.window_of(np.arange(576), [(24, 24)], 4)
    assert sorted(np.bincount(win)) == [36] * 16
    assert win[0] == 0 and win[5] == 0 and win[6] == 1 and win[24 * 6] == 4 and win[575] == 15
    win = O.window_of(np.arange(576), [(24, 24)], 6)
    assert sorted(np.bincount(win)) == [16] * 36
    # several tiles never share a window
    win = O.window_of(np.arange(2 * 576), [(24, 24), (24, 24)], 2)
    assert set(win[:576]) == {0, 1, 2, 3} and set(win[576:]) == {4, 5, 6, 7}
    # balanced cells when the side is not a multiple of w: 10 columns, w = 3 -> 4, 3, 3
    win = O.window_of(np.arange(30), [(3, 10)], 3)
    assert list(win[:10]) == [0, 0, 0, 0, 1, 1, 1, 2, 2, 2]
    assert list(win[10:20] - 3) == [0, 0, 0, 0, 1, 1, 1, 2, 2, 2]
    # membership depends on the ORIGINAL position only (later stages have holes)
    pos = np.array([575, 3, 300])
    np.testing.assert_array_equal(O.window_of(pos, [(24, 24)], 4),
                                  O.window_of(np.arange(576), [(24, 24)], 4)[pos])


def test_bipartition_parity():
    a, b = O.bipartition(np.array([10, 11, 12, 13, 14]))
    assert list(a) == [10, 12, 14] and list(b) == [11, 13]     # 1st, 3rd, 5th -> A


def test_euclidean_divergences_against_the_library():
    # appendix "Influence of similarity metrics": squared and plain Euclidean distance as the pair score
    import scipy.spatial.distance as D
    rng = np.random.default_rng(21)
    xa, xb = rng.standard_normal((5, 7)), rng.standard_normal((4, 7))
    np.testing.assert_allclose(O.divergence(xa, xb, "l2sq"), D.cdist(xa, xb, "sqeuclidean"), rtol=1e-13)
    np.testing.assert_allclose(O.divergence(xa, xb, "l2"), D.cdist(xa, xb, "euclidean"), rtol=1e-13)
    np.testing.assert_array_equal(O.divergence(xa, xb, "cosine"), O.feature_divergence(xa, xb))
    # on unit vectors the squared distance is twice the feature divergence
    ua, ub = xa / np.linalg.norm(xa, axis=1, keepdims=True), xb / np.linalg.norm(xb, axis=1, keepdims=True)
    np.testing.assert_allclose(O.divergence(ua, ub, "l2sq"), 2.0 * O.feature_divergence(ua, ub), rtol=1e-12, atol=1e-15)
    # unlike FD it is not scale invariant: a long vector is far from everything
    far = O.divergence(10.0 * xa[:1], xb, "l2sq")
    assert (far > O.divergence(xa[:1], xb, "l2sq")).all()
    with pytest.raises(ValueError):
        O.divergence(xa, xb, "manhattan")


# ------------------------------------------------------------------ xi (Eq. "attention-factor")

def _rand_qk(rng, n_heads, n_kv, n_seq, dh):
    return rng.standard_normal((n_heads, n_seq, dh)), rng.standard_normal((n_kv, n_seq, dh))


def test_xi_against_library_softmax_by_rows():
    rng = np.random.default_rng(3)
    n_heads, n_kv, n_text, n_vis, dh = 4, 2, 5, 9, 8
    q, k = _rand_qk(rng, n_heads, n_kv, n_text + n_vis, dh)
    xi = O.xi_from_attention(q, k, n_text, n_vis, 1, 4)
    want = np.zeros(n_vis)
    for h in range(n_heads):
        for t in range(n_vis):
            s = n_text + t
            p = scipy.special.softmax(k[h // 2][:s + 1] @ q[h, s] / math.sqrt(dh))
            want[t] += p[1:4].sum()
    np.testing.assert_allclose(xi, want, rtol=1e-12)


def test_xi_closed_form_for_zero_queries_and_bounds():
    rng = np.random.default_rng(4)
    n_heads, n_text, n_vis = 6, 7, 11
    q, k = _rand_qk(rng, n_heads, 3, n_text + n_vis, 4)
    xi = O.xi_from_attention(np.zeros_like(q), k, n_text, n_vis, 0, n_text)
    s = n_text + np.arange(n_vis)
    np.testing.assert_allclose(xi, n_heads * n_text / (s + 1.0), rtol=1e-13)
    xi = O.xi_from_attention(q, k, n_text, n_vis, 0, n_text)
    assert (xi > 0).all() and (xi < n_heads).all()
    # rows are probability rows and causal
    a = O.attention_rows(q[0], k[0], n_text, n_vis)
    np.testing.assert_allclose(a.sum(axis=1), 1.0, rtol=1e-13)
    assert a[0, n_text + 1:].sum() == 0.0 and a[0, n_text] > 0.0
    # the first vision token sees the text and itself only
    xi_all = O.xi_from_attention(q, k, n_text, 1, 0, n_text)
    self_p = sum(O.attention_rows(q[h], k[h // 2], n_text, 1)[0, n_text] for h in range(n_heads))
    assert xi_all[0] == pytest.approx(n_heads - self_p, rel=1e-13)


def test_xi_equals_exp_of_logit_minus_logsumexp():
    rng = np.random.default_rng(5)
    n_heads, n_text, n_vis, dh = 3, 4, 6, 16
    q, k = _rand_qk(rng, n_heads, n_heads, n_text + n_vis, dh)
    xi = O.xi_from_attention(q, k, n_text, n_vis, 0, n_text)
    want = np.zeros(n_vis)
    for h in range(n_heads):
        logit = q[h] @ k[h].T / math.sqrt(dh)
        for t in range(n_vis):
            s = n_text + t
            lse = scipy.special.logsumexp(logit[s, :s + 1])
            want[t] += np.exp(logit[s, :n_text] - lse).sum()
    np.testing.assert_allclose(xi, want, rtol=1e-12)


def test_xi_without_the_causal_mask_is_the_equation_as_printed():
    # causal=False: every query sees all N keys.  Library softmax row by row; zero queries give H |J| / N.
    rng = np.random.default_rng(15)
    n_heads, n_kv, n_text, n_vis, dh = 4, 2, 6, 7, 8
    n_seq = n_text + n_vis
    q, k = _rand_qk(rng, n_heads, n_kv, n_seq, dh)
    xi = O.xi_from_attention(q, k, n_text, n_vis, 1, 5, causal=False)
    want = np.zeros(n_vis)
    for h in range(n_heads):
        for t in range(n_vis):
            p = scipy.special.softmax(k[h // 2] @ q[h, n_text + t] / math.sqrt(dh))
            want[t] += p[1:5].sum()
    np.testing.assert_allclose(xi, want, rtol=1e-12)
    xi0 = O.xi_from_attention(np.zeros_like(q), k, n_text, n_vis, 0, n_text, causal=False)
    np.testing.assert_allclose(xi0, n_heads * n_text / n_seq, rtol=1e-13)
    a = O.attention_rows(q[0], k[0], n_text, n_vis, causal=False)
    np.testing.assert_allclose(a.sum(axis=1), 1.0, rtol=1e-13)
    assert (a[0, n_text + 1:] > 0).all()                   # keys behind the query are visible
    # the last query sees every key either way
    np.testing.assert_allclose(O.attention_rows(q[0], k[0], n_text, n_vis)[-1], a[-1], rtol=1e-13)


def test_xi_over_several_prompt_ranges_is_the_sum_over_the_ranges():
    rng = np.random.default_rng(16)
    n_heads, n_text, n_vis, dh = 3, 12, 5, 8
    q, k = _rand_qk(rng, n_heads, n_heads, n_text + n_vis, dh)
    parts = [O.xi_from_attention(q, k, n_text, n_vis, lo, hi) for lo, hi in ((1, 3), (5, 6), (8, 12))]
    both = O.xi_from_attention(q, k, n_text, n_vis, 0, 0, text_ranges=[(1, 3), (5, 6), (8, 12)])
    np.testing.assert_allclose(both, sum(parts), rtol=1e-13)
    whole = O.xi_from_attention(q, k, n_text, n_vis, 0, n_text)
    gaps = O.xi_from_attention(q, k, n_text, n_vis, 0, 0, text_ranges=[(0, 1), (3, 5), (6, 8)])
    np.testing.assert_allclose(both + gaps, whole, rtol=1e-13)


def test_row_logsumexp_against_the_library():
    rng = np.random.default_rng(17)
    n_text, n_vis, dh = 4, 6, 16
    q, k = rng.standard_normal((n_text + n_vis, dh)), rng.standard_normal((n_text + n_vis, dh))
    logit = q @ k.T / math.sqrt(dh)
    got = O.row_logsumexp(q, k, n_text, n_vis)
    want = [scipy.special.logsumexp(logit[n_text + t, :n_text + t + 1]) for t in range(n_vis)]
    np.testing.assert_allclose(got, want, rtol=1e-13)
    got = O.row_logsumexp(q, k, n_text, n_vis, causal=False)
    np.testing.assert_allclose(got, scipy.special.logsumexp(logit[n_text:], axis=1), rtol=1e-13)
    # shifting every logit of a row by c shifts the result by c: scale a query so that its logits are huge
    big = q.copy()
    big[n_text] *= 400.0
    assert np.isfinite(O.row_logsumexp(big, k, n_text, n_vis)).all()
    # and it is the normaliser of the attention rows
    a = O.attention_rows(q, k, n_text, n_vis)
    np.testing.assert_allclose(np.exp(logit[n_text:, :n_text] - O.row_logsumexp(q, k, n_text, n_vis)[:, None]),
                               a[:, :n_text], rtol=1e-12)


# ------------------------------------------------------------- merge (Eq. "message-passing")

def _case(seed, n=36, d=12, tiles=((6, 6),), w=1, keep=0.5):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, d))
    xi = rng.uniform(0.1, 2.0, n)
    return x, np.arange(n), xi, list(tiles), w, keep


def _groups(res, n):
    g = {}
    for i in range(n):
        g.setdefault(int(res["dst"][i]), []).append(i)
    return g


def test_merge_weights_and_convexity():
    x, pos, xi, tiles, w, keep = _case(6, keep=0.6)
    res = O.compress_vision(x, pos, xi, tiles, w, keep)
    groups = _groups(res, len(x))
    assert sorted(groups) == list(range(int(res["n_out"])))
    assert (res["weight"] >= 0).all()
    merged = 0
    for o, members in groups.items():
        wsum = res["weight"][members].sum()
        assert wsum == pytest.approx(1.0, abs=1e-14)
        np.testing.assert_allclose(res["weight"][members], xi[members] / xi[members].sum(), rtol=1e-13)
        np.testing.assert_allclose(res["x_out"][o], (res["weight"][members, None] * x[members]).sum(0),
                                   rtol=1e-12, atol=1e-14)
        assert (res["x_out"][o] <= x[members].max(0) + 1e-14).all()
        assert (res["x_out"][o] >= x[members].min(0) - 1e-14).all()
        if len(members) == 1:
            np.testing.assert_array_equal(res["x_out"][o], x[members[0]])      # bit-exact copy
            assert res["weight"][members[0]] == 1.0
        else:
            merged += len(members) - 1
    assert merged == len(x) - res["n_out"] == O.removal_count(len(x), keep)


def test_uniform_xi_is_the_group_mean_and_xi_scale_is_irrelevant():
    x, pos, xi, tiles, w, keep = _case(7)
    res = O.compress_vision(x, pos, np.ones(len(x)), tiles, w, keep)
    for o, members in _groups(res, len(x)).items():
        np.testing.assert_allclose(res["x_out"][o], x[members].mean(0), rtol=1e-13, atol=1e-15)
    r1 = O.compress_vision(x, pos, xi, tiles, w, keep)
    r2 = O.compress_vision(x, pos, 37.0 * xi, tiles, w, keep)
    np.testing.assert_allclose(r1["x_out"], r2["x_out"], rtol=1e-13)
    # a heavier token pulls the merge towards itself (xi is not inverted or ignored)
    big = np.ones(len(x))
    a0 = int(np.nonzero(r1["partner"] >= 0)[0][0])
    big[a0] = 1e6
    r3 = O.compress_vision(x, pos, big, tiles, w, keep)
    np.testing.assert_allclose(r3["x_out"][r3["dst"][a0]], x[a0], atol=1e-4)


def test_vanishing_xi_sum_falls_back_to_the_plain_group_mean():
    """A group whose xi sum is (numerically) zero cannot be normalised: it takes the plain mean of its members
    and weights 1 / size; groups with a proper sum beside it are left alone; weights still sum to one."""
    rng = np.random.default_rng(18)
    xa, xb = rng.standard_normal((3, 5)), rng.standard_normal((2, 5))
    m = np.array([[1, 0], [1, 0], [0, 1]])                 # A0, A1 -> B0;  A2 -> B1
    xi_a, xi_b = np.array([0.0, 0.0, 0.7]), np.array([0.0, 1.3])
    xb_new, w_a, w_b = O.message_passing(xa, xb, xi_a, xi_b, m)
    np.testing.assert_allclose(xb_new[0], (xb[0] + xa[0] + xa[1]) / 3.0, rtol=1e-14)
    np.testing.assert_allclose([w_b[0], w_a[0], w_a[1]], 1.0 / 3.0, rtol=1e-15)
    np.testing.assert_allclose(xb_new[1], (1.3 * xb[1] + 0.7 * xa[2]) / 2.0, rtol=1e-14)
    np.testing.assert_allclose([w_b[1], w_a[2]], [0.65, 0.35], rtol=1e-14)
    assert w_b[0] + w_a[0] + w_a[1] == pytest.approx(1.0, abs=1e-15) and w_b[1] + w_a[2] == pytest.approx(1.0, abs=1e-15)
    # an untouched B node with xi = 0 keeps its own row (a group of one)
    xb_new, w_a, w_b = O.message_passing(xa, xb, np.array([0.5, 0.5, 0.5]), np.array([0.0, 0.0]),
                                         np.array([[1, 0], [0, 0], [0, 0]]))
    np.testing.assert_allclose(xb_new[0], xa[0], rtol=1e-14)          # all of the group's mass sits on A0
    np.testing.assert_array_equal(xb_new[1], xb[1])
    assert w_b[1] == 1.0
    # through the whole step: xi = 0 everywhere gives the same result as uniform xi
    x, pos, _, tiles, w, keep = _case(19)
    r0 = O.compress_vision(x, pos, np.zeros(len(x)), tiles, w, keep)
    r1 = O.compress_vision(x, pos, np.ones(len(x)), tiles, w, keep)
    np.testing.assert_allclose(r0["x_out"], r1["x_out"], rtol=1e-14)
    np.testing.assert_allclose(r0["weight"], r1["weight"], rtol=1e-15)
    # tiny but representable sums are still normalised by xi
    tiny = np.full(len(x), 1e-20)
    tiny[0] = 3e-20
    r2 = O.compress_vision(x, pos, tiny, tiles, w, keep)
    r3 = O.compress_vision(x, pos, tiny * 1e20, tiles, w, keep)
    np.testing.assert_allclose(r2["x_out"], r3["x_out"], rtol=1e-12)


def test_direction_is_a_into_b_and_position_of_group_is_b():
    x, pos, xi, tiles, w, keep = _case(8)
    res = O.compress_vision(x, pos, xi, tiles, w, keep)
    # keep = 0.5 removes all of A: survivors are exactly the 2nd, 4th, ... tokens
    np.testing.assert_array_equal(res["pos_out"], np.arange(1, 36, 2))
    assert (res["partner"][0::2] % 2 == 1).all() and (res["partner"][1::2] == -1).all()
    assert (np.diff(res["pos_out"]) > 0).all()


def test_reverse_direction_is_the_forward_one_on_the_mirrored_window():
    """B -> A: the two sets swap roles.  Exchanging the contents of positions (0,1), (2,3), ... turns every A node
    into a B node and back, so the reverse direction on the exchanged window merges exactly the same tokens into
    exactly the same rows as the forward direction on the original."""
    x, pos, xi, tiles, w, keep = _case(23, keep=0.7)
    swap = np.arange(len(x)) ^ 1
    fwd = O.compress_vision(x, pos, xi, tiles, w, keep)
    rev = O.compress_vision(x[swap], pos, xi[swap], tiles, w, keep, direction="b2a")
    # token t of the exchanged window is token t ^ 1 of the original
    np.testing.assert_array_equal(rev["partner"][swap] >= 0, fwd["partner"] >= 0)
    merged = np.nonzero(fwd["partner"] >= 0)[0]
    np.testing.assert_array_equal(rev["partner"][merged ^ 1] ^ 1, fwd["partner"][merged])
    np.testing.assert_allclose(rev["weight"][swap], fwd["weight"], rtol=1e-14)
    by_survivor_f = {int(s): fwd["x_out"][o] for o, s in enumerate(fwd["survivor"])}
    by_survivor_r = {int(s) ^ 1: rev["x_out"][o] for o, s in enumerate(rev["survivor"])}
    assert sorted(by_survivor_f) == sorted(by_survivor_r)
    for s_ in by_survivor_f:
        np.testing.assert_allclose(by_survivor_r[s_], by_survivor_f[s_], rtol=1e-13, atol=1e-15)
    # sources are the B nodes: an odd window can lose at most floor(n / 2) tokens, and all survivors of keep = 0.5 are A
    xo, poso, xio = x[:35], pos[:35], xi[:35]
    half = O.compress_vision(xo, poso, xio, [(5, 7)], 1, 0.5, direction="b2a")
    assert int(half["n_out"]) == 18 and (half["pos_out"] % 2 == 0).all()
    assert (half["partner"][1::2] % 2 == 0).all() and (half["partner"][0::2] == -1).all()


def test_keep_one_is_identity():
    x, pos, xi, tiles, w, _ = _case(9, tiles=((6, 6),), w=2)
    res = O.compress_vision(x, pos, xi, tiles, w, 1.0)
    np.testing.assert_array_equal(res["x_out"], x)
    np.testing.assert_array_equal(res["dst"], np.arange(36))
    np.testing.assert_array_equal(res["pos_out"], pos)
    assert (res["weight"] == 1.0).all()


def test_permutation_equivariance():
    x, pos, xi, tiles, w, keep = _case(10, tiles=((6, 6),), w=2, keep=0.7)
    base = O.compress_vision(x, pos, xi, tiles, w, keep)
    perm = np.random.default_rng(0).permutation(len(x))
    res = O.compress_vision(x[perm], pos[perm], xi[perm], tiles, w, keep)
    np.testing.assert_array_equal(res["pos_out"], base["pos_out"])
    np.testing.assert_allclose(res["x_out"], base["x_out"], rtol=1e-13, atol=1e-15)
    np.testing.assert_array_equal(res["dst"], base["dst"][perm])
    np.testing.assert_allclose(res["weight"], base["weight"][perm], rtol=1e-13)


def test_duplicated_token_merges_first():
    x, pos, xi, tiles, w, _ = _case(11, n=36, d=16)
    x[13] = 1.7 * x[12]                       # local indices 12 (A) and 13 (B): FD = 0
    keep = 35.0 / 36.0                        # room for exactly one merge
    assert O.removal_count(36, keep) == 1
    res = O.compress_vision(x, pos, xi, tiles, w, keep)
    assert res["n_out"] == 35
    assert res["partner"][12] == 13 and (np.delete(res["partner"], 12) == -1).all()
    assert res["fd_best"][12] == pytest.approx(0.0, abs=1e-15)


def _brute_force(fd, r):
    """Cheapest way to attach r distinct A nodes, each to any B node."""
    n_a, n_b = fd.shape
    best_cost, best_edges = np.inf, None
    for subset in itertools.combinations(range(n_a), r):
        for assign in itertools.product(range(n_b), repeat=r):
            cost = sum(fd[a, b] for a, b in zip(subset, assign))
            if cost < best_cost - 1e-15:
                best_cost, best_edges = cost, set(zip(subset, assign))
    return best_edges


@pytest.mark.parametrize("n,keep", [(8, 0.5), (10, 0.7), (11, 0.75), (13, 0.8), (16, 0.8), (5, 0.5)])
def test_selection_agrees_with_exhaustive_matching(n, keep):
    rng = np.random.default_rng(100 + n)
    x = rng.standard_normal((n, 6))
    res = O.compress_vision(x, np.arange(n), np.ones(n), [(1, n)], 1, keep)
    ia, ib = np.arange(0, n, 2), np.arange(1, n, 2)
    fd = O.feature_divergence(x[ia], x[ib])
    r = O.removal_count(n, keep)
    want = {(int(ia[a]), int(ib[b])) for a, b in _brute_force(fd, r)} if r else set()
    got = {(i, int(p)) for i, p in enumerate(res["partner"]) if p >= 0}
    assert got == want and len(got) == r
    m = O.select_edges(fd, r)
    assert m.sum() == r and (m.sum(axis=1) <= 1).all()          # one edge per A node at most


def test_literal_edge_rule_lets_one_a_node_feed_two_b_nodes():
    """Step 2 to the letter: the floor(rho n / 2) lowest PAIRS, whatever nodes they join.  A hand case: A0 lies
    between B0 and B1 and close to both, A1 is far from everything; with two pairs allowed both go to A0."""
    xa = np.array([[1.0, 1.0, 0.0], [0.0, 0.0, 1.0]])           # A0, A1
    xb = np.array([[1.0, 0.9, 0.0], [0.9, 1.0, 0.0]])           # B0, B1
    fd = O.feature_divergence(xa, xb)
    m = O.select_edges_literal(fd, 4, 0.0)                       # rho = 1: floor(4 / 2) = 2 pairs
    np.testing.assert_array_equal(m, [[1, 1], [0, 0]])
    np.testing.assert_array_equal(O.select_edges(fd, 2), [[1, 0], [1, 0]])    # the adopted rule: one edge per A node
                                                                              # (ties go to the lower B index)
    # the count of pairs is the printed floor(rho v / 2); the number of tokens that disappear is at most that
    for n, keep in ((16, 0.5), (36, 0.5), (36, 0.7), (7, 0.5)):
        rng = np.random.default_rng(n)
        f = rng.uniform(0, 2, ((n + 1) // 2, n // 2))
        mm = O.select_edges_literal(f, n, keep)
        k = int(np.floor((1 - keep) * n / 2 + 1e-9))
        assert mm.sum() == k and (mm.sum(axis=1) > 0).sum() <= k
        assert f[mm == 1].max(initial=-1) <= f[mm == 0].min(initial=9)       # they are the lowest pairs
    # through a whole stage: halving 576 tokens this way leaves MORE than 288 (at most 144 pairs per 576 tokens),
    # which is why the library does not use this rule; A0's message reaches both B nodes with weight xi_A0
    x, pos, xi, tiles, w, keep = _case(31, n=36)
    res = O.compress_vision_literal(x, pos, xi, tiles, w, keep)
    assert int(res["n_out"]) >= 36 - 9
    ia, ib, m = res["edges"][0]
    for bi in np.nonzero(m.sum(axis=0))[0]:
        src = ia[m[:, bi] == 1]
        want = (xi[ib[bi]] * x[ib[bi]] + (xi[src, None] * x[src]).sum(0)) / (xi[ib[bi]] + xi[src].sum())
        o = int(np.nonzero(res["survivor"] == ib[bi])[0][0])
        np.testing.assert_allclose(res["x_out"][o], want, rtol=1e-13)


def test_many_a_nodes_may_share_one_b_node():
    x = np.array([[1, 0.01], [1, 0.0], [1, -0.01], [0, 1.0], [1, 0.02], [-1, 0.0]])
    res = O.compress_vision(x, np.arange(6), np.ones(6), [(1, 6)], 1, 0.5)
    assert list(res["partner"]) == [1, -1, 1, -1, 1, -1]        # all three A nodes pick B node 1
    assert res["n_out"] == 3
    np.testing.assert_allclose(res["x_out"][0], x[[0, 1, 2, 4]].mean(0))


# ------------------------------------------------------------------------- K/V operator

def test_kv_operator_is_the_same_linear_map_as_the_hidden_merge():
    x, pos, xi, tiles, w, keep = _case(12, n=36, d=24, tiles=((6, 6),), w=2, keep=0.6)
    n_text = 3
    rng = np.random.default_rng(0)
    hidden = np.concatenate([rng.standard_normal((n_text, 24)), x, rng.standard_normal((2, 24))])
    res = O.compress_sequence(hidden, n_text, 36, pos, xi, tiles, w, keep)
    kv = hidden.reshape(-1, 3, 8).transpose(1, 0, 2)                 # 3 "heads" = slices of the hidden rows
    out = O.compact_kv(kv, n_text, 36, res["dst"], res["weight"], res["survivor"], "merge")
    want = res["hidden_out"].reshape(-1, 3, 8).transpose(1, 0, 2)
    np.testing.assert_allclose(out, want, rtol=1e-12, atol=1e-14)
    np.testing.assert_array_equal(out[:, :n_text], kv[:, :n_text])   # text rows copied
    np.testing.assert_array_equal(out[:, -2:], kv[:, -2:])
    gat = O.compact_kv(kv, n_text, 36, res["dst"], res["weight"], res["survivor"], "gather")
    np.testing.assert_array_equal(gat[:, n_text:-2], kv[:, n_text + res["survivor"]])
    np.testing.assert_array_equal(pos[res["survivor"]], res["pos_out"])


# ----------------------------------------------------------- batch driver, synthetic inputs

def test_schedule_counts_on_synthetic_workload():
    wl = S.workload("tiny")
    pos = None
    counts = []
    for stage in range(wl.n_stages):
        inp = S.make_layer_inputs(wl, stage, pos)
        res = O.compress_layer(inp["hidden"], inp["q"], inp["k"], inp["pos"], inp["n_vis"], inp["vis_begin"],
                               wl.tiles, wl.windows[stage], wl.keep[stage])
        pos = [r["pos_out"] for r in res]
        counts.append([int(r["n_out"]) for r in res])
        for b, r in enumerate(res):
            assert r["hidden_out"].shape[0] == wl.n_text + r["n_out"]
            assert (r["xi"] > 0).all() and (r["xi"] < wl.n_q_heads).all()
    # 4 windows of 9 lose floor(4.5) = 4 each; then 20 -> 20 - 5; then 15 -> 15 - 7
    assert counts == [[20, 20], [15, 15], [8, 8]]


def test_generator_is_deterministic_and_bf16():
    wl = S.workload("tiny")
    a = S.make_layer_inputs(wl, 0)
    b = S.make_layer_inputs(wl, 0)
    for key in ("hidden", "q", "k", "v"):
        np.testing.assert_array_equal(a[key], b[key])
        np.testing.assert_array_equal(a[key], S.round_to_bf16(a[key]))
        np.testing.assert_array_equal(S.bf16_from_bits(S.bf16_bits(a[key])), a[key])
    one = S.make_layer_inputs(wl, 0, samples=[1])
    np.testing.assert_array_equal(one["hidden"][0], a["hidden"][1])
    # oracle's own rounding agrees with the generator's on non-tie values
    v = np.random.default_rng(0).standard_normal(1000)
    np.testing.assert_array_equal(O.to_bf16(v), S.round_to_bf16(v.astype(np.float32)).astype(np.float64))
    assert O.to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0                  # tie -> even
    assert O.to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_field_covariance_closed_form():
    gen = S._generator(7, 1)
    f = S.smooth_field(24, 24, 1024, 3.0, gen).astype(np.float64).reshape(24, 24, -1)
    assert f.var() == pytest.approx(1.0, abs=0.02)
    for lag in (1, 3):
        c = 0.5 * ((f[:, :-lag] * f[:, lag:]).mean() + (f[:-lag] * f[lag:]).mean())
        assert c == pytest.approx(math.exp(-lag * lag / 18.0), abs=0.02)


def test_gap_repair():
    wl = S.workload("cfg0")
    inp = S.make_layer_inputs(wl, 0, tensors=("hidden",))
    x = inp["hidden"][0, wl.n_text:].astype(np.float64)
    before = G.selection_gaps(x, inp["pos"][0], wl.tiles, wl.windows[0], wl.keep[0])
    fixed, rep = G.enforce_gaps(x, inp["pos"][0], wl.tiles, wl.windows[0], wl.keep[0], 1e-3, rounder=O.to_bf16)
    assert rep["ok"] and rep["partner_gap"] >= 1e-3 and rep["boundary_gap"] >= 1e-3
    assert min(before["partner_gap"], before["boundary_gap"]) < 1e-3 <= min(rep["partner_gap"], rep["boundary_gap"])
    np.testing.assert_array_equal(fixed, O.to_bf16(fixed))
