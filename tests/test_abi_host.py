"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and rejects bad
arguments on the host before anything is launched (no GPU needed)."""
import ctypes as C
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    entry.build()
    import paper_2605_00789_b200 as pkg
    return pkg


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "lightkv.h")).read()
    declared = set(re.findall(r"\b(lightkv_[a-z_]+)\s*\(", header))
    assert declared == set(L.lightkv.EXPORTS)
    lib = L.library()
    for name in declared:
        assert getattr(lib, name) is not None
    assert L.version() == 200
    assert L.status_string(0) == "ok" and "workspace" in L.status_string(-3)


def test_struct_layouts_match_the_header(L, tmp_path):
    """Ask the C compiler for the size of every struct and the offset of its last field."""
    import subprocess
    src = tmp_path / "layout.c"
    src.write_text('''#include <stdio.h>
#include <stddef.h>
#include "lightkv.h"
int main(void) {
  printf("%zu %zu\\n", sizeof(lightkv_config_t), offsetof(lightkv_config_t, direction));
  printf("%zu %zu\\n", sizeof(lightkv_stage_info_t), offsetof(lightkv_stage_info_t, reserved));
  printf("%zu %zu\\n", sizeof(lightkv_layer_args_t), offsetof(lightkv_layer_args_t, seq_start_out));
  printf("%zu %zu\\n", sizeof(lightkv_kv_args_t), offsetof(lightkv_kv_args_t, dst_seq_start));
  return 0;
}
''')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c99", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    rows = [tuple(int(v) for v in line.split()) for line in subprocess.check_output([str(exe)]).decode().splitlines()]
    k = L.lightkv
    got = [(C.sizeof(k._Config), k._Config.direction.offset),
           (C.sizeof(k._StageInfo), k._StageInfo.reserved.offset),
           (C.sizeof(k._LayerArgs), k._LayerArgs.seq_start_out.offset),
           (C.sizeof(k._KvArgs), k._KvArgs.dst_seq_start.offset)]
    assert got == rows


def _plan(L, **kw):
    args = dict(batch=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, n_layers=8, tiles=[(6, 6)],
                layers=[2, 4], windows=[2, 1], keep=[0.5, 0.5], max_text=16)
    args.update(kw)
    return L.Plan(**args)


def test_plan_counts_and_retention(L):
    p = _plan(L, tiles=[(24, 24)], layers=[12, 18, 24], windows=[4, 2, 1], keep=[0.5] * 3, n_layers=32,
              hidden=4096, n_q_heads=32, n_kv_heads=32, head_dim=128, batch=1, max_text=64)
    caps = [(p.stage_info(s).cap_in, p.stage_info(s).cap_out, p.stage_info(s).n_windows,
             p.stage_info(s).counts_exact) for s in range(3)]
    assert caps == [(576, 288, 16, 1), (288, 144, 4, 1), (144, 72, 1, 1)]
    assert p.retention() == pytest.approx(0.546875)
    p = _plan(L, tiles=[(24, 24)], layers=[15, 23, 31], windows=[4, 2, 1], keep=[0.5] * 3, n_layers=40)
    assert p.retention() == pytest.approx(0.553125)
    p = _plan(L, tiles=[(24, 24)], layers=[10, 20, 30], windows=[4, 2, 1], keep=[0.5] * 3, n_layers=40)
    assert p.retention() == pytest.approx(0.46875)
    # data-dependent counts: capacities are upper bounds
    p = _plan(L, tiles=[(24, 24)], layers=[12], windows=[4], keep=[0.55], n_layers=32)
    info = p.stage_info(0)
    assert info.counts_exact == 0 and 320 <= info.cap_out <= 576 and info.workspace_bytes > 0
    # odd windows (9 tokens) under keep 0.5 leave one data-dependent A node per window
    p = _plan(L)
    assert p.stage_info(0).counts_exact == 0 and p.stage_info(0).cap_out >= 20


@pytest.mark.parametrize("kw", [
    dict(batch=0), dict(hidden=65), dict(head_dim=12), dict(n_q_heads=3), dict(keep=[0.4, 0.5]),
    dict(keep=[0.5, 1.5]), dict(windows=[7, 1]), dict(windows=[0, 1]), dict(layers=[4, 2]),
    dict(layers=[2, 9]), dict(tiles=[(0, 6)]), dict(dtype=7), dict(xi_mode=9), dict(engine=5),
    dict(ragged_input=2), dict(divergence=3), dict(direction=2),
])
def test_plan_rejects_bad_configs(L, kw):
    with pytest.raises(L.LightKVError, match="invalid argument"):
        _plan(L, **kw)


def test_plan_unsupported(L):
    with pytest.raises(L.LightKVError, match="unsupported"):
        _plan(L, tiles=[(6, 6)] * 33)
    with pytest.raises(L.LightKVError, match="unsupported"):
        _plan(L, tiles=[(64, 64)], windows=[64, 1])
    # a window may hold at most 65535 tokens (16-bit counters of the window build): 256 x 256 is one too many
    _plan(L, tiles=[(255, 257)], windows=[1, 1])
    with pytest.raises(L.LightKVError, match="unsupported"):
        _plan(L, tiles=[(256, 256)], windows=[1, 1])
    _plan(L, tiles=[(510, 514)], windows=[2], layers=[2], keep=[0.5])        # cells of 255 x 257
    with pytest.raises(L.LightKVError, match="unsupported"):
        _plan(L, tiles=[(510, 514)], windows=[2, 1])                           # one window at the second stage


def test_ragged_input_plans_hold_for_any_subset_of_the_grid(L):
    """With ragged_input the capacities are bounds over every subset of positions: (cap_in + n_windows) / 2 A
    nodes and ceil(keep cap_in) + n_windows survivors; a full-grid plan keeps the exact counts."""
    kw = dict(tiles=[(24, 24)], layers=[12, 18, 24], windows=[6, 4, 2], keep=[0.5] * 3, n_layers=32, hidden=4096,
              n_q_heads=32, n_kv_heads=32, head_dim=128, batch=1, max_text=64)
    exact = [L.Plan(**kw).stage_info(s) for s in range(3)]
    assert [(i.cap_in, i.cap_out, i.counts_exact) for i in exact[:2]] == [(576, 288, 1), (288, 144, 1)]
    ragged = [L.Plan(ragged_input=True, **kw).stage_info(s) for s in range(3)]
    assert [(i.cap_in, i.cap_out, i.counts_exact) for i in ragged] == \
        [(576, 288 + 36, 0), (324, 162 + 16, 0), (178, 89 + 4, 0)]
    assert all(r.workspace_bytes >= e.workspace_bytes for r, e in zip(ragged, exact))


@pytest.mark.parametrize("seed", range(6))
def test_ragged_capacities_bound_what_the_oracle_produces_on_random_subsets(L, seed):
    """The capacities of a ragged_input plan must hold whatever subset of the grid a sample enters with: run the
    oracle stage by stage on random subsets (both message directions) and compare its counts with the plan's."""
    import numpy as np
    from oracle import lightkv_oracle as O
    rng = np.random.default_rng(400 + seed)
    tiles = [(int(rng.integers(6, 15)), int(rng.integers(6, 15))) for _ in range(int(rng.integers(1, 3)))]
    smallest = min(min(t) for t in tiles)
    windows = sorted((int(rng.integers(1, min(6, smallest) + 1)) for _ in range(3)), reverse=True)
    keep = [float(k) for k in rng.uniform(0.5, 0.95, size=3).round(2)]
    direction = ["a2b", "b2a"][seed % 2]
    plan = L.Plan(batch=1, hidden=64, n_q_heads=2, n_kv_heads=2, head_dim=16, n_layers=8, tiles=tiles,
                  layers=[2, 4, 6], windows=windows, keep=keep, max_text=8, ragged_input=True,
                  direction=L.DIR_A2B if direction == "a2b" else L.DIR_B2A)
    n_grid = sum(r * c for r, c in tiles)
    for trial in range(4):
        n0 = int(rng.integers(max(2, n_grid // 3), n_grid + 1))
        pos = np.sort(rng.choice(n_grid, n0, replace=False))
        for st in range(3):
            info = plan.stage_info(st)
            assert len(pos) <= info.cap_in
            win = O.window_of(pos, tiles, windows[st])
            counts = np.bincount(win, minlength=info.n_windows)
            src = (counts + 1) // 2 if direction == "a2b" else counts // 2
            assert src.sum() <= info.cap_a and (counts - src).sum() <= info.cap_b, (st, src.sum(), info.cap_a, info.cap_b)
            x = rng.standard_normal((len(pos), 8))
            res = O.compress_vision(x, pos, np.ones(len(pos)), tiles, windows[st], keep[st], direction=direction)
            assert int(res["n_out"]) <= info.cap_out, (st, int(res["n_out"]), info.cap_out)
            pos = res["pos_out"]


@pytest.mark.parametrize("seed", range(6))
def test_exact_plans_agree_with_the_oracle_on_full_grids(L, seed):
    """Where the plan calls its counts exact (the host simulation of the schedule), the oracle on a full grid must
    produce exactly those counts, stage after stage; elsewhere the capacities must still bound them."""
    import numpy as np
    from oracle import lightkv_oracle as O
    rng = np.random.default_rng(500 + seed)
    side = int(rng.choice([8, 12, 16, 24]))
    tiles = [(side, side)] * int(rng.integers(1, 3))
    windows = [[4, 2, 1], [2, 2, 1], [4, 4, 2], [3, 2, 1]][seed % 4]
    keep = [0.5, 0.5, 0.5] if seed % 2 == 0 else [0.5, 0.75, 0.5]
    plan = L.Plan(batch=1, hidden=64, n_q_heads=2, n_kv_heads=2, head_dim=16, n_layers=8, tiles=tiles,
                  layers=[2, 4, 6], windows=windows, keep=keep, max_text=8)
    pos = np.arange(sum(r * c for r, c in tiles))
    for st in range(3):
        info = plan.stage_info(st)
        x = rng.standard_normal((len(pos), 8))
        res = O.compress_vision(x, pos, np.ones(len(pos)), tiles, windows[st], keep[st])
        assert len(pos) <= info.cap_in and int(res["n_out"]) <= info.cap_out
        if info.counts_exact:
            assert len(pos) == info.cap_in and int(res["n_out"]) == info.cap_out
        pos = res["pos_out"]


def test_prompt_ranges_and_stream_events_are_checked_on_the_host(L):
    p = _plan(L)
    lib = L.library()
    a = L.lightkv._LayerArgs()
    a.struct_size = C.sizeof(a)
    a.vis_begin = 12
    for f in ("hidden", "n_vis_out", "pos_out", "dst", "weight", "grp_off", "grp_src", "workspace", "q", "k"):
        setattr(a, f, 0x1000)
    a.hidden_out = 0x2000
    a.hidden_row_stride = a.hidden_out_row_stride = 64
    a.hidden_batch_stride = a.hidden_out_batch_stride = 64 * 64
    a.q_row_stride = a.k_row_stride = 16
    a.workspace_bytes = 1 << 30

    def ranges(*pairs):
        flat = [v for pr in pairs for v in pr]
        a._keep = (C.c_int32 * len(flat))(*flat)
        a.text_ranges, a.n_text_ranges = a._keep, len(pairs)
        return lib.lightkv_compress_layer(p.handle, C.byref(a))

    a.n_text_ranges = 9
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # more ranges than the library takes
    a.n_text_ranges = 2
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # ranges announced, none given
    assert ranges((4, 8), (6, 10)) == -1                                     # overlapping
    assert ranges((6, 10), (0, 4)) == -1                                     # not ascending
    assert ranges((0, 4), (8, 13)) == -1                                     # reaches into the vision block
    assert ranges((5, 3)) == -1                                              # end before begin
    a.n_text_ranges = 0
    a.bidirectional = 2
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1
    a.bidirectional = 0
    a.aux_stream = 0x10
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # second stream without fork / join events
    a.fork_event = 0x20
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # ... with only one of them
    a.aux_stream, a.fork_event = None, None
    given = _plan(L, xi_mode=L.XI_GIVEN)
    a.xi, a.lse_out = 0x1000, 0x3000
    assert lib.lightkv_compress_layer(given.handle, C.byref(a)) == -1        # lse_out needs ATTN_FULL


def test_calls_reject_bad_arguments_before_any_launch(L):
    p = _plan(L)
    lib = L.library()
    a = L.lightkv._LayerArgs()
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # struct_size
    a.struct_size = C.sizeof(a)
    a.stage = 5
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # stage
    a.stage = 0
    a.vis_begin, a.text_end = 4, 9
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # J outside the text rows
    a.text_end = 4
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # NULL buffers
    for f in ("hidden", "n_vis_out", "pos_out", "dst", "weight", "grp_off", "grp_src", "workspace"):
        setattr(a, f, 0x1000)
    a.hidden_out = 0x2000
    a.hidden_row_stride = a.hidden_out_row_stride = 64
    a.hidden_batch_stride = a.hidden_out_batch_stride = 64 * 64
    a.workspace_bytes = 16
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -3            # workspace too small
    a.workspace_bytes = 1 << 30
    a.hidden = 0x1008
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # misaligned rows
    a.hidden = 0x1000
    a.hidden_row_stride = 60
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # row stride below hidden
    a.hidden_row_stride = 64
    assert lib.lightkv_compress_layer(p.handle, C.byref(a)) == -1            # ATTN_FULL without q / k
    assert lib.lightkv_compress_layer(None, C.byref(a)) == -1

    kv = L.lightkv._KvArgs()
    assert lib.lightkv_compact_kv(p.handle, C.byref(kv)) == -1
    kv.struct_size = C.sizeof(kv)
    kv.mode = 3
    assert lib.lightkv_compact_kv(p.handle, C.byref(kv)) == -1
    kv.mode = 0
    for f in ("n_vis_out", "grp_off", "grp_src", "weight", "k_src", "v_src"):
        setattr(kv, f, 0x1000)
    kv.k_dst, kv.v_dst = 0x1000, 0x3000
    kv.src_row_stride = kv.dst_row_stride = 16
    assert lib.lightkv_compact_kv(p.handle, C.byref(kv)) == -1               # K in place, V not
    kv.k_dst = kv.v_dst = 0x1000
    kv.dst_head_stride = 16 * 64
    assert lib.lightkv_compact_kv(p.handle, C.byref(kv)) == -1               # in place with two addressings
    kv.dst_head_stride = 0
    kv.k_dst = kv.v_dst = 0x3000
    kv.page_size = 16
    assert lib.lightkv_compact_kv(p.handle, C.byref(kv)) == -1               # paged without block tables
    assert lib.lightkv_plan_stage_info(p.handle, 9, C.byref(L.lightkv._StageInfo())) == -1
    assert lib.lightkv_plan_retention(None) < 0


def test_builtin_workspace_entry_rejects_oversized_stages_on_the_host(L):
    lib = L.library()
    a = L.lightkv._LayerArgs()
    p = _plan(L)
    assert lib.lightkv_compress_layer_builtin_ws(p.handle, C.byref(a)) == -1     # struct_size
    assert lib.lightkv_compress_layer_builtin_ws(None, C.byref(a)) == -1
    a.struct_size = C.sizeof(a)
    a.stage = 7
    assert lib.lightkv_compress_layer_builtin_ws(p.handle, C.byref(a)) == -1     # stage
    # 64 samples x 32 heads x 2880 tokens of per-head xi alone exceed the built-in array
    big = _plan(L, batch=64, hidden=4096, n_q_heads=32, n_kv_heads=32, head_dim=128, n_layers=32,
                tiles=[(24, 24)] * 5, layers=[12], windows=[6], keep=[0.5], max_text=128)
    assert big.stage_info(0).workspace_bytes > L.BUILTIN_WS_BYTES
    a.stage = 0
    assert lib.lightkv_compress_layer_builtin_ws(big.handle, C.byref(a)) == -3   # before any CUDA call
    header = open(os.path.join(ROOT, "include", "lightkv.h")).read()
    assert re.search(r"#define LIGHTKV_BUILTIN_WS_BYTES \(8u << 20\)", header) and L.BUILTIN_WS_BYTES == 8 << 20


def test_missing_library_fails_loudly(L, monkeypatch):
    from paper_2605_00789_b200 import lightkv
    monkeypatch.setattr(lightkv, "_LIB", None)
    monkeypatch.setattr(lightkv, "_HERE", "/nonexistent")
    with pytest.raises(L.LightKVError, match="missing"):
        lightkv.library()
