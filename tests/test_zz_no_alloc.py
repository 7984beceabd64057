"""lightkv_compress_layer_builtin_ws against lightkv_compress_layer, through the C ABI.

Some users of the library run where device memory cannot be allocated (inside an engine that owns
the whole memory pool, or in a phase where the runtime forbids allocation), so they cannot supply
the scratch buffer lightkv_compress_layer asks for.  The built-in-workspace entry point keeps that
scratch in a fixed array inside the library instead.  Here it is called twice in a row, the second
time on a shorter, ragged batch so that the shared array still holds the first call's contents, and
every output is compared with what the ordinary entry point returns for the same inputs.

Collected last on purpose (file name): a failure here cannot hide the other tests in a run that
stops at the first failure.  It also passes when run alone in a fresh process."""
import numpy as np
import pytest

import lightkv_synth as S
from tests import harness as H

pytestmark = pytest.mark.gpu

INDEX_OUTPUTS = ("n_vis_out", "pos_out", "dst", "grp_off", "grp_src", "status")
FLOAT_OUTPUTS = ("weight", "xi_out", "hidden_out", "k_out", "v_out")


def _same(a, b, n_vis):
    for key in INDEX_OUTPUTS:
        np.testing.assert_array_equal(a[key], b[key], err_msg=key)
    tol = H.TOL["bf16"]
    for key in FLOAT_OUTPUTS:
        x, y = a[key].astype(np.float64), b[key].astype(np.float64)
        if key in ("weight", "xi_out"):          # rows are only defined up to each sample's token count
            for s, n in enumerate(n_vis):
                np.testing.assert_allclose(x[s, :n], y[s, :n], rtol=tol["rel"], atol=0, err_msg=key)
        else:
            m = np.isfinite(y)
            assert (np.isfinite(x) == m).all(), key
            assert np.abs(x[m] - y[m]).max(initial=0.0) <= tol["max_abs"], key


def test_builtin_workspace_matches_caller_workspace_on_two_calls_in_a_row():
    import torch
    import __graft_entry__ as entry
    assert torch.cuda.is_available()
    entry.build()
    import paper_2605_00789_b200 as L

    wl = S.workload("small")
    plan = H.make_plan(wl)
    assert plan.stage_info(0).workspace_bytes <= L.BUILTIN_WS_BYTES

    full = np.arange(wl.n_vis, dtype=np.int32)
    rng = np.random.default_rng(11)
    ragged = [np.sort(rng.choice(full, 131, replace=False)).astype(np.int32), full[:60], full[:0]]
    first = H.prepare_stage(wl, 0, repair=False)
    second = H.prepare_stage(wl, 0, ragged, repair=False)

    # Free device memory is read right around the entry point itself (every buffer it is given exists by then).
    # The first call on a device loads the library's kernels and its fixed scratch array; from then on a call
    # must leave the amount of free memory where it found it.
    moved = []

    def watched(*args, **kw):
        torch.cuda.synchronize()
        before = torch.cuda.mem_get_info()[0]
        L.compress_layer_builtin_ws(*args, **kw)
        torch.cuda.synchronize()
        moved.append(before - torch.cuda.mem_get_info()[0])

    H.gpu_stage(plan, wl, 0, first, layer_fn=L.compress_layer_builtin_ws)      # loads kernels and the array
    for inp in (first, second):                   # two calls in a row on the shared array
        got = H.gpu_stage(plan, wl, 0, inp, layer_fn=watched)
        want = H.gpu_stage(plan, wl, 0, inp)
        assert int(want["status"][0]) == 0
        _same(got, want, [int(n) for n in inp["n_vis"]])
    assert moved == [0, 0], f"free device memory moved across the calls: {moved}"
    plan.close()
