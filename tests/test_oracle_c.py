"""The two CPU oracles against each other: oracle/lightkv_oracle.py (numpy, float64) and oracle/lightkv_oracle.c
(plain C loops, double), written separately from the same passages of the paper.  Everything here runs on the
CPU and touches only oracle/ and the seeded input generator."""
import numpy as np
import pytest

import lightkv_synth as S
from oracle import c_oracle as OC
from oracle import lightkv_oracle as O


@pytest.mark.parametrize("causal", [True, False])
def test_xi_of_the_two_oracles(causal):
    rng = np.random.default_rng(61)
    n_heads, n_kv, n_text, n_vis, dh = 6, 2, 9, 23, 16
    q = rng.standard_normal((n_heads, n_text + n_vis, dh))
    k = rng.standard_normal((n_kv, n_text + n_vis, dh))
    for ranges in ([(0, n_text)], [(1, 3), (5, 9)]):
        want = O.xi_from_attention(q, k, n_text, n_vis, 0, 0, causal, text_ranges=ranges)
        got = OC.xi(q, k, n_text, n_vis, ranges, causal)
        np.testing.assert_allclose(got, want, rtol=1e-12)


@pytest.mark.parametrize("seed", range(8))
def test_a_stage_of_the_two_oracles(seed):
    rng = np.random.default_rng(700 + seed)
    tiles = [(int(rng.integers(5, 13)), int(rng.integers(5, 13))) for _ in range(int(rng.integers(1, 3)))]
    w = int(rng.integers(1, min(min(t) for t in tiles) // 2 + 1))
    keep = round(float(rng.uniform(0.5, 1.0)), 2)
    n_grid = sum(r * c for r, c in tiles)
    pos = np.sort(rng.choice(n_grid, int(rng.integers(n_grid // 2, n_grid + 1)), replace=False))
    x = rng.standard_normal((len(pos), 24))
    xi = rng.uniform(0.05, 2.0, len(pos))
    if seed == 3:
        xi[:] = 0.0                                   # the vanishing-sum branch
    a = O.compress_vision(x, pos, xi, tiles, w, keep)
    b = OC.compress(x, pos, xi, tiles, w, keep)
    assert int(a["n_out"]) == b["n_out"]
    np.testing.assert_array_equal(a["pos_out"], b["pos_out"])
    np.testing.assert_array_equal(a["dst"], b["dst"])
    np.testing.assert_allclose(a["weight"], b["weight"], rtol=1e-12)
    np.testing.assert_allclose(a["x_out"], b["x_out"], rtol=1e-11, atol=1e-13)
    kv = rng.standard_normal((3, len(pos), 8))
    want = O.compact_kv(kv, 0, len(pos), a["dst"], a["weight"], a["survivor"], "merge")
    np.testing.assert_allclose(OC.compact(kv, b["dst"], b["weight"], b["n_out"]), want, rtol=1e-11, atol=1e-13)


def test_the_two_oracles_on_a_synthetic_workload_stage():
    # the seeded generator's tensors (bf16 values), all three stages of the "small" workload chained on sample 1
    wl = S.workload("small")
    pos = None
    for st in range(wl.n_stages):
        inp = S.make_layer_inputs(wl, st, pos, samples=[1])
        nv, vb = int(inp["n_vis"][0]), inp["vis_begin"]
        xi_py = O.xi_from_attention(inp["q"][0], inp["k"][0], vb, nv, 0, vb)
        xi_c = OC.xi(inp["q"][0], inp["k"][0], vb, nv, [(0, vb)])
        np.testing.assert_allclose(xi_c, xi_py, rtol=1e-11)
        x = inp["hidden"][0, vb:vb + nv]
        a = O.compress_vision(x, inp["pos"][0, :nv], xi_py, wl.tiles, wl.windows[st], wl.keep[st])
        b = OC.compress(x, inp["pos"][0, :nv], xi_c, wl.tiles, wl.windows[st], wl.keep[st])
        np.testing.assert_array_equal(a["dst"], b["dst"])
        np.testing.assert_allclose(a["x_out"], b["x_out"], rtol=1e-10, atol=1e-12)
        pos = [a["pos_out"]]
