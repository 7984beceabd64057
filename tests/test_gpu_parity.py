"""Parity of the CUDA path (through the C ABI) with the CPU oracle on seeded synthetic inputs.

Index sets (survivors, dst, positions, counts, group lists) must be bit-exact on inputs whose
selection margins are >= 1e-3; merged hidden states and K/V within max-abs 2e-2 and relative 1e-2
(bf16 storage, fp32 accumulation) or 1e-5 relative (fp32 mode)."""
import dataclasses

import numpy as np
import pytest

import lightkv_synth as S
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    import torch
    import __graft_entry__ as entry
    assert torch.cuda.is_available()
    entry.build()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("engine", ["simt", "auto"])
@pytest.mark.parametrize("xi_mode", ["attn", "lse", "given", "uniform"])
def test_tiny_schedule(dtype, engine, xi_mode):
    stats = H.run_schedule(S.workload("tiny"), dtype=dtype, xi_mode=xi_mode, engine=engine)
    assert [s["n_out"] for s in stats] == [[20, 20], [15, 15], [8, 8]]


@pytest.mark.parametrize("dtype,engine", [("bf16", "simt"), ("bf16", "auto"), ("fp32", "simt")])
def test_small_ragged_multitile_gqa(dtype, engine):
    # two tiles of different shape, windows that do not divide the grid, GQA, keep 0.55 / 0.6 / 0.5
    H.run_schedule(S.workload("small"), dtype=dtype, engine=engine)


@pytest.mark.parametrize("kv_mode,paged", [("gather", 0), ("merge", 16), ("gather", 16), ("merge", 5)])
def test_small_kv_modes_and_paged_cache(kv_mode, paged):
    H.run_schedule(S.workload("small"), kv_mode=kv_mode, paged=paged, stages=[0])


def test_small_lse_mode_on_tensor_cores():
    # row log-sum-exp supplied by the caller: only the prompt key tiles are visited (tcgen05 path, GQA)
    H.run_schedule(S.workload("small"), xi_mode="lse")
    wl = dataclasses.replace(S.workload("cfg0"), n_text=200)      # prompt keys spanning two key tiles
    H.run_schedule(wl, xi_mode="lse")


@pytest.mark.parametrize("kv_mode", ["merge", "gather"])
def test_small_token_major_kv_cache(kv_mode):
    # K/V stored [B, N, H_kv, dh]: the same call with other strides
    H.run_schedule(S.workload("small"), kv_mode=kv_mode, kv_layout="bnhd", stages=[0, 1])


@pytest.mark.parametrize("w", [4, 6, 1])
@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_cfg0_single_step(w, engine):
    wl = dataclasses.replace(S.workload("cfg0"), windows=(w,))
    stats = H.run_schedule(wl, engine=engine)
    assert stats[0]["n_out"] == [{4: 320, 6: 324, 1: 317}[w]]


@pytest.mark.parametrize("name", ["cfg1", "cfg1r"])
def test_cfg1_full_schedule(name):
    stats = H.run_schedule(S.workload(name))
    if name == "cfg1":
        assert [s["n_out"] for s in stats] == [[288], [144], [72]]


@pytest.mark.parametrize("name", ["small", "cfg1"])
def test_second_stream_inside_compress_layer(name):
    # window build + FD on aux_stream beside xi: same results as the oracle, run after run
    import torch
    aux = torch.cuda.Stream()
    for _ in range(2):
        H.run_schedule(S.workload(name), aux_stream=aux)


@pytest.mark.parametrize("name", ["small", "cfg1"])
def test_kv_compaction_behind_the_map_event(name):
    # lightkv_compact_kv on a second stream behind map_event (recorded once the merge map is complete, before
    # the hidden-state merge), together with the second stream inside the call
    import torch
    aux, kv_stream = torch.cuda.Stream(), torch.cuda.Stream()
    for _ in range(2):
        H.run_schedule(S.workload(name), aux_stream=aux, kv_stream=kv_stream)


def test_cfg0_fp32_mode():
    H.run_schedule(dataclasses.replace(S.workload("cfg0"), hidden=1024, n_q_heads=8, n_kv_heads=8), dtype="fp32")


def test_text_after_and_prompt_subrange():
    wl = S.workload("small")
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0)
    # move the last 4 text rows behind the vision block: [15 text | vision | 4 text], J = [2, 12)
    vb, after = wl.n_text - 4, 4
    for key in ("hidden", "q", "k", "v"):
        a = inp[key]
        axis = 1 if key == "hidden" else 2
        a = np.concatenate([np.take(a, range(0, vb), axis), np.take(a, range(wl.n_text, a.shape[axis]), axis),
                            np.take(a, range(vb, wl.n_text), axis)], axis)
        inp[key] = np.ascontiguousarray(a)
    inp["vis_begin"] = vb
    assert len(set(inp["n_vis"])) == 1        # full grids: every sample has the same length here
    gpu = H.gpu_stage(plan, wl, 0, inp, n_text_after=after, text_range=(2, 12))
    ref = H.oracle_stage(wl, 0, inp, n_text_after=after, text_range=(2, 12))
    H.compare_stage(wl, 0, inp, ref, gpu, n_text_after=after)
    for b, r in enumerate(ref):
        n_out = int(r["n_out"])
        np.testing.assert_array_equal(gpu["hidden_out"][b, vb + n_out:vb + n_out + after],
                                      inp["hidden"][b, vb + int(inp["n_vis"][b]):][:after])


def test_ragged_batch_and_empty_sample():
    wl = S.workload("small")
    plan = H.make_plan(wl)
    full = np.arange(wl.n_vis, dtype=np.int32)
    rng = np.random.default_rng(5)
    pos = [full, np.sort(rng.choice(full, 97, replace=False)).astype(np.int32), full[:0]]
    inp = H.prepare_stage(wl, 0, pos)
    gpu = H.gpu_stage(plan, wl, 0, inp)
    ref = H.oracle_stage(wl, 0, inp)
    H.compare_stage(wl, 0, inp, ref, gpu)
    assert int(gpu["n_vis_out"][2]) == 0


def test_keep_one_is_identity_on_device():
    wl = dataclasses.replace(S.workload("small"), keep=(1.0, 1.0, 1.0))
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0, repair=False)
    gpu = H.gpu_stage(plan, wl, 0, inp)
    n = wl.n_vis
    assert (gpu["n_vis_out"] == n).all()
    np.testing.assert_array_equal(gpu["hidden_out"][:, :wl.n_text + n], inp["hidden"])
    np.testing.assert_array_equal(gpu["k_out"][:, :, :wl.n_text + n], inp["k"])
    np.testing.assert_array_equal(gpu["dst"][:, :n], np.tile(np.arange(n), (wl.batch, 1)))
    assert (gpu["weight"][:, :n] == 1.0).all()


def test_device_status_word_flags_unsorted_positions():
    wl = S.workload("tiny")
    plan = H.make_plan(wl, xi_mode="uniform")
    inp = H.prepare_stage(wl, 0, repair=False)
    inp["pos"][1, [3, 4]] = inp["pos"][1, [4, 3]]
    gpu = H.gpu_stage(plan, wl, 0, inp, xi_mode="uniform")
    assert int(gpu["status"][0]) & 1


def test_vanishing_xi_gives_the_group_mean_and_the_status_bit():
    # xi = 0 for every token of sample 0: the sum over a group vanishes, the merge falls back to the plain
    # group mean (as the oracle does) and the ZERO_WEIGHT bit is raised; the other samples are unaffected
    wl = S.workload("small")
    plan = H.make_plan(wl, xi_mode="given")
    inp = H.prepare_stage(wl, 0)
    inp["xi"] = np.random.default_rng(5).uniform(0.05, 3.0, size=inp["pos"].shape).astype(np.float32)
    inp["xi"][0] = 0.0
    gpu = H.gpu_stage(plan, wl, 0, inp, xi_mode="given")
    ref = H.oracle_stage(wl, 0, inp, "given")
    H.compare_stage(wl, 0, inp, ref, gpu, expect_status=2)
    plan.close()


def test_run_to_run_bit_repeatability():
    wl = S.workload("small")
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0, repair=False)
    a = H.gpu_stage(plan, wl, 0, inp)
    b = H.gpu_stage(plan, wl, 0, inp)
    for key in ("hidden_out", "k_out", "v_out", "weight", "xi_out", "dst", "grp_src", "grp_off", "pos_out"):
        np.testing.assert_array_equal(a[key], b[key])


# ---- prompt ranges, rows without the causal mask, the row log-sum-exp as an output ---------------------------

@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_prompt_ranges_bidirectional_rows_and_lse_out(engine):
    wl = S.workload("small")                                   # 19 text rows, head_dim 128 (tcgen05 with "auto")
    H.run_schedule(wl, engine=engine, stages=[0], text_ranges=[(1, 4), (7, 8), (10, 19)], want_lse=True)
    H.run_schedule(wl, engine=engine, stages=[0, 1], bidirectional=True, want_lse=True)
    H.run_schedule(wl, engine=engine, stages=[0], bidirectional=True, xi_mode="lse", text_ranges=[(0, 3), (9, 19)])


def test_prompt_ranges_over_several_key_tiles():
    # 200 prompt rows = four 64-key tiles; J = three ranges with holes, cut by tile borders
    wl = dataclasses.replace(S.workload("cfg0"), n_text=200, hidden=256)
    ranges = [(3, 50), (60, 70), (100, 190)]
    H.run_schedule(wl, text_ranges=ranges, want_lse=True)
    H.run_schedule(wl, text_ranges=ranges, xi_mode="lse")
    H.run_schedule(wl, text_ranges=ranges, bidirectional=True, want_lse=True)


def test_bidirectional_rows_with_text_behind_the_vision_block():
    # [15 text | vision | 4 text], no causal mask: the rows behind the vision block are keys too (not in J)
    wl = S.workload("small")
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0)
    vb, after = wl.n_text - 4, 4
    for key in ("hidden", "q", "k", "v"):
        a = inp[key]
        axis = 1 if key == "hidden" else 2
        a = np.concatenate([np.take(a, range(0, vb), axis), np.take(a, range(wl.n_text, a.shape[axis]), axis),
                            np.take(a, range(vb, wl.n_text), axis)], axis)
        inp[key] = np.ascontiguousarray(a)
    inp["vis_begin"] = vb
    gpu = H.gpu_stage(plan, wl, 0, inp, n_text_after=after, text_range=(2, 12), bidirectional=True, want_lse=True)
    ref = H.oracle_stage(wl, 0, inp, n_text_after=after, text_range=(2, 12), causal=False)
    H.compare_stage(wl, 0, inp, ref, gpu, n_text_after=after)
    H.check_lse_out(inp, gpu, wl.n_q_heads, wl.n_kv_heads, range(wl.batch), causal=False, n_text_after=after)


@pytest.mark.parametrize("name", ["small", "cfg1"])
def test_the_librarys_own_row_lse_feeds_the_lse_mode(name):
    """ATTN_FULL hands out the row log-sum-exp it saw (lse_out); given back as the input of ATTN_LSE, only the
    prompt keys are visited and xi, the merge map and the merged rows agree with ATTN_FULL and the oracle."""
    wl = S.workload(name)
    full, lse_plan = H.make_plan(wl), H.make_plan(wl, xi_mode="lse")
    inp = H.prepare_stage(wl, 0)
    a = H.gpu_stage(full, wl, 0, inp, want_lse=True)
    b = H.gpu_stage(lse_plan, wl, 0, inp, xi_mode="lse", lse=a["lse_out_dev"])
    ref = H.oracle_stage(wl, 0, inp)
    H.compare_stage(wl, 0, inp, ref, a)
    H.compare_stage(wl, 0, inp, ref, b)
    H.check_lse_out(inp, a, wl.n_q_heads, wl.n_kv_heads, range(wl.batch))
    for key in ("dst", "grp_src", "grp_off", "pos_out"):
        np.testing.assert_array_equal(a[key], b[key])
    nv = int(inp["n_vis"][0])
    np.testing.assert_allclose(a["xi_out"][:, :nv], b["xi_out"][:, :nv], rtol=2e-3)


@pytest.mark.parametrize("name", ["small", "cfg1"])
def test_logits_far_above_the_first_tiles_maximum_take_the_safe_pass(name):
    """The tensor-core xi kernel subtracts the maximum of a row's FIRST key tile and checks its sums at the end.
    Here one late key of one KV head is scaled by 128, so that many rows meet a logit far more than 88 above
    that reference: their sums leave the fp32 range, the CTA repeats the item with a running maximum, and the
    result still matches the oracle (the other heads keep xi away from zero)."""
    wl = S.workload(name)
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0)
    late = inp["vis_begin"] + int(inp["n_vis"].min()) * 2 // 3
    inp["k"][:, 0, late] *= 128.0                              # a power of two: still bf16 values
    logit = inp["q"][0, 0, late + 1:] @ inp["k"][0, 0, late] / np.sqrt(wl.head_dim)
    first = (inp["q"][0, 0, late + 1:] @ inp["k"][0, 0, :64].T / np.sqrt(wl.head_dim)).max(axis=1)
    assert (logit - first > 100).any()                         # the case really leaves the fp32 range
    gpu = H.gpu_stage(plan, wl, 0, inp, want_lse=True)
    del gpu["k_out"], gpu["v_out"]      # the scaled key row is outside the value range the bf16 K/V tolerance is meant for
    H.compare_stage(wl, 0, inp, H.oracle_stage(wl, 0, inp), gpu)
    H.check_lse_out(inp, gpu, wl.n_q_heads, wl.n_kv_heads, range(inp["hidden"].shape[0]), atol=2e-2)
    plan.close()


# ---- K/V compaction inside the cache's own rows / pages ---------------------------------------------------------

@pytest.mark.parametrize("kv_mode,paged,layout", [("merge", 0, "bhnd"), ("gather", 0, "bhnd"), ("merge", 16, "bhnd"),
                                                  ("merge", 5, "bhnd"), ("gather", 16, "bhnd"), ("merge", 0, "bnhd")])
def test_in_place_kv_compaction(kv_mode, paged, layout):
    # destination = source: groups are merged over their surviving token's row, then rows move forward plane by
    # plane; compared with the oracle like the out-of-place form (ragged windows, two tiles, GQA, three stages)
    H.run_schedule(S.workload("small"), kv_mode=kv_mode, paged=paged, kv_layout=layout, kv_in_place=True)


def test_in_place_kv_compaction_long_rows_and_text_behind():
    # 2304 tokens per sample: a plane is swept in many chunks (sources of a chunk lie inside the next chunks'
    # destinations); text rows behind the vision block move forward with it
    wl = S.Workload(name="inpl", config_id=140, batch=2, tiles=((48, 48),), n_text=37, hidden=64, n_q_heads=4,
                    n_kv_heads=2, head_dim=64, n_layers=16, layers=(3, 7), windows=(6, 3), keep=(0.55, 0.5))
    H.run_schedule(wl, xi_mode="given", kv_in_place=True)
    plan = H.make_plan(wl, xi_mode="uniform")
    inp = H.prepare_stage(wl, 0)
    vb, after = wl.n_text - 9, 9
    for key in ("hidden", "q", "k", "v"):
        a = inp[key]
        axis = 1 if key == "hidden" else 2
        a = np.concatenate([np.take(a, range(0, vb), axis), np.take(a, range(wl.n_text, a.shape[axis]), axis),
                            np.take(a, range(vb, wl.n_text), axis)], axis)
        inp[key] = np.ascontiguousarray(a)
    inp["vis_begin"] = vb
    gpu = H.gpu_stage(plan, wl, 0, inp, xi_mode="uniform", n_text_after=after, kv_in_place=True)
    ref = H.oracle_stage(wl, 0, inp, "uniform", n_text_after=after)
    H.compare_stage(wl, 0, inp, ref, gpu, n_text_after=after)
    plan.close()


def test_in_place_equals_out_of_place_bit_for_bit():
    wl = S.workload("cfg1")
    plan = H.make_plan(wl)
    inp = H.prepare_stage(wl, 0, repair=False)
    a = H.gpu_stage(plan, wl, 0, inp)
    b = H.gpu_stage(plan, wl, 0, inp, kv_in_place=True)
    np.testing.assert_array_equal(a["k_out"], b["k_out"])
    np.testing.assert_array_equal(a["v_out"], b["v_out"])
    plan.close()


# ---- packed (ragged) batches: samples back to back on one row axis ----------------------------------------------

@pytest.mark.parametrize("engine,xi_mode,in_place", [("auto", "attn", False), ("simt", "attn", False),
                                                     ("auto", "lse", False), ("auto", "attn", True)])
def test_packed_batch_with_row_offsets(engine, xi_mode, in_place):
    """Three samples of different lengths (one of them empty) stored without padding: every tensor has one row
    axis and seq_start / seq_start_out say where a sample begins.  Same results as the padded form."""
    import torch
    import paper_2605_00789_b200 as L
    wl = S.workload("small")
    plan = H.make_plan(wl, xi_mode=xi_mode, engine=engine)
    full = np.arange(wl.n_vis, dtype=np.int32)
    rng = np.random.default_rng(6)
    pos = [full, np.sort(rng.choice(full, 101, replace=False)).astype(np.int32), full[:0]]
    inp = H.prepare_stage(wl, 0, pos)
    info = plan.stage_info(0)
    vb, bsz = inp["vis_begin"], 3
    lens = [vb + int(n) for n in inp["n_vis"]]
    start = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    start_out = (np.arange(bsz + 1) * (vb + info.cap_out)).astype(np.int32)
    dev = "cuda"

    def pack(a, axis):          # [B, (H,) N, w] -> [1, (H,) total, w]
        return np.concatenate([np.take(a[b], range(lens[b]), axis - 1) for b in range(bsz)], axis - 1)[None]

    hid = H.to_device(pack(inp["hidden"], 1), "bf16", dev)
    q, k, v = (H.to_device(pack(inp[n], 2), "bf16", dev) for n in ("q", "k", "v"))
    out = L.StageBuffers(plan, 0, vb + info.cap_out, dev)
    hidden_out = torch.full((1, int(start_out[-1]), wl.hidden), float("nan"), dtype=torch.bfloat16, device=dev)
    pos_pad = np.pad(inp["pos"], ((0, 0), (0, info.cap_in - inp["pos"].shape[1])), constant_values=-1)
    kw = dict(vis_begin=vb, q=q, k=k, n_vis=torch.from_numpy(inp["n_vis"]).to(dev), pos=torch.from_numpy(pos_pad).to(dev),
              seq_start=torch.from_numpy(start[:-1].copy()).to(dev), seq_start_out=torch.from_numpy(start_out[:-1].copy()).to(dev),
              hidden_out=hidden_out)
    if xi_mode == "lse":
        lse = H.oracle_lse(inp, wl.n_q_heads, wl.n_kv_heads)                      # [B, H, N] padded
        kw["lse"] = torch.from_numpy(pack(lse[:, :, :, None], 2)[..., 0].astype(np.float32)).to(dev)   # [1, H, total]
    L.compress_layer(plan, 0, hid, out, **kw)
    if in_place:
        k_dst, v_dst, dst_start = k, v, kw["seq_start"]
    else:
        k_dst = torch.full((1, wl.n_kv_heads, int(start_out[-1]), wl.head_dim), float("nan"), dtype=torch.bfloat16, device=dev)
        v_dst, dst_start = k_dst.clone(), kw["seq_start_out"]
    L.compact_kv(plan, 0, out, k, v, k_dst, v_dst, vis_begin=vb, n_vis=kw["n_vis"], src_seq_start=kw["seq_start"],
                 dst_seq_start=dst_start)
    torch.cuda.synchronize()
    gpu = {name: getattr(out, name).cpu().numpy() for name in
           ("n_vis_out", "pos_out", "dst", "weight", "grp_off", "grp_src", "xi_out", "status")}
    n_out = gpu["n_vis_out"]
    ho = hidden_out.float().cpu().numpy()[0]
    kd, vd = k_dst.float().cpu().numpy()[0], v_dst.float().cpu().numpy()[0]
    so = start if in_place else start_out
    gpu["hidden_out"] = np.stack([ho[start_out[b]:start_out[b] + vb + info.cap_out] for b in range(bsz)])
    rows = vb + info.cap_out
    gpu["k_out"] = np.stack([np.pad(kd[:, so[b]:so[b] + vb + n_out[b]], ((0, 0), (0, rows - vb - n_out[b]), (0, 0))) for b in range(bsz)])
    gpu["v_out"] = np.stack([np.pad(vd[:, so[b]:so[b] + vb + n_out[b]], ((0, 0), (0, rows - vb - n_out[b]), (0, 0))) for b in range(bsz)])
    ref = H.oracle_stage(wl, 0, inp, xi_mode)
    H.compare_stage(wl, 0, inp, ref, gpu)
    plan.close()


# ---- the variants the paper ablates: Euclidean pair scores, reverse message direction ---------------------------

@pytest.mark.parametrize("metric", ["l2sq", "l2"])
@pytest.mark.parametrize("dtype,engine", [("bf16", "auto"), ("bf16", "simt"), ("fp32", "simt")])
def test_euclidean_pair_scores(metric, dtype, engine):
    H.run_schedule(S.workload("small"), dtype=dtype, engine=engine, metric=metric)
    if dtype == "bf16" and metric == "l2sq":
        H.run_schedule(S.workload("cfg1"), engine=engine, metric=metric)      # windows of 36 / 72 / 144 tokens


@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_reverse_direction_b_into_a(engine):
    # odd windows: the destinations (A) outnumber the sources (B); keep 0.5 on even windows removes all of B
    H.run_schedule(S.workload("small"), engine=engine, direction="b2a")
    H.run_schedule(S.workload("tiny"), engine=engine, direction="b2a", xi_mode="given")
    stats = H.run_schedule(S.workload("cfg1"), engine=engine, direction="b2a")
    assert [s["n_out"] for s in stats] == [[288], [144], [72]]
    H.run_schedule(S.workload("cfg1r"), engine=engine, direction="b2a", metric="l2sq", stages=[0, 1])


# ---- persistent CTAs that take more than one work item ---------------------------------------------------------

def _sm_count():
    import torch
    return torch.cuda.get_device_properties(0).multi_processor_count


@pytest.mark.parametrize("head_dim", [64, 128])
def test_lse_mode_persistent_ctas_walk_several_items(head_dim):
    # 4 samples x 8 heads x 16 query tiles = 512 work items for at most 3 CTAs per SM: every CTA of the xi kernel
    # takes a second item (its barriers and rings run on across items); 130 prompt rows span three key tiles
    wl = S.Workload(name="lsewalk", config_id=130, batch=4, tiles=((64, 32),), n_text=130, hidden=64, n_q_heads=8,
                    n_kv_heads=4, head_dim=head_dim, n_layers=16, layers=(3,), windows=(4,), keep=(0.5,))
    assert 16 * wl.n_q_heads * wl.batch > 3 * _sm_count()
    H.run_schedule(wl, xi_mode="lse")
    H.run_schedule(wl, xi_mode="lse", text_ranges=[(2, 60), (70, 129)])


def test_cfg2_lse_mode_full_size_sampled():
    # the benchmark shape in ATTN_LSE mode (5888 work items walked by 3 CTAs per SM), bench.py's streams; the
    # log-sum-exp input comes from plain torch ops, the oracle derives xi from Q and K alone
    stats = H.run_schedule(S.workload("cfg2"), xi_mode="lse", lse_source="torch", oracle_samples=[0, 5],
                           **_bench_streams())
    assert [s["n_out"] for s in stats] == [[1440] * 8, [720] * 8, [360] * 8]


@pytest.mark.parametrize("hidden,ragged", [(64, False), (72, True)])
def test_fd_persistent_ctas_take_several_tiles(hidden, ragged):
    # 160 samples x 36 windows of 16 tokens: three tiles of sixteen windows per sample (a tile holds at most 128 A
    # nodes), 480 tiles for the 2 x SMs persistent CTAs of the tensor-core FD kernel, so most CTAs take a second
    # tile (ring phases and the accumulator barrier run on); the ragged variant gives every sample its own subset
    # of the grid under a plan built for subsets
    wl = S.Workload(name="fdmulti", config_id=131, batch=160, tiles=((24, 24),), n_text=4, hidden=hidden,
                    n_q_heads=2, n_kv_heads=1, head_dim=64, n_layers=16, layers=(3,), windows=(6,), keep=(0.5,))
    first = None
    if ragged:
        rng = np.random.default_rng(77)
        full = np.arange(wl.n_vis, dtype=np.int32)
        first = [np.sort(rng.choice(full, int(rng.integers(500, 577)), replace=False)).astype(np.int32)
                 for _ in range(wl.batch)]
    stats = H.run_schedule(wl, xi_mode="uniform", oracle_samples=[0, 17, 159], ragged=ragged, first_pos=first)
    info = stats[0]["info"]
    assert info.uses_tensor_cores == 1 and info.fd_tiles * wl.batch > 2 * _sm_count()


# ---- subsets of the grid: capacities ---------------------------------------------------------------------------

def _near_full_subset():
    """576-token grid, windows 6 / 4 / 2 (not nested): a sample that misses 8 positions reaches the second stage
    with 146 A nodes, two more than the full grid's 144 (found with the oracle, seed fixed)."""
    wl = dataclasses.replace(S.workload("cfg1r"), batch=2, hidden=64, n_q_heads=2, n_kv_heads=2, head_dim=64, n_text=8)
    rng = np.random.default_rng(9000)
    full = np.arange(576, dtype=np.int32)
    n_missing = int(rng.integers(1, 12))
    subset = np.sort(rng.choice(full, 576 - n_missing, replace=False)).astype(np.int32)
    return wl, [subset, full]


def test_near_full_subset_through_two_stages_under_a_ragged_plan():
    wl, first = _near_full_subset()
    stats = H.run_schedule(wl, stages=[0, 1], ragged=True, first_pos=first)
    assert stats[1]["info"].cap_a >= 146 and stats[1]["info"].counts_exact == 0


def test_subset_given_to_a_full_grid_plan_raises_the_count_bit():
    """The same subset under a plan built for full grids: at the second stage it has more A nodes than the plan
    holds.  The sample then passes through unmerged (cut at cap_out), the COUNT bit is raised, nothing is written
    out of a row, and the full-grid sample beside it still matches the oracle."""
    wl, first = _near_full_subset()
    plan = H.make_plan(wl, batch=2)
    inp0 = H.prepare_stage(wl, 0, first)
    g0 = H.gpu_stage(plan, wl, 0, inp0)
    H.compare_stage(wl, 0, inp0, H.oracle_stage(wl, 0, inp0), g0)           # stage 0 holds any subset
    pos1 = [g0["pos_out"][b, :int(g0["n_vis_out"][b])] for b in range(2)]
    info = plan.stage_info(1)
    assert info.cap_a == 144 and info.cap_out == 144
    inp1 = H.prepare_stage(wl, 1, pos1)
    g1 = H.gpu_stage(plan, wl, 1, inp1)
    assert int(g1["status"][0]) == 8
    sub = {k: (v[[1]] if isinstance(v, np.ndarray) and v.shape[:1] == (2,) else v) for k, v in inp1.items()}
    H.compare_stage(wl, 1, inp1, H.oracle_stage(wl, 1, sub), g1, samples=[1], expect_status=8)
    vb = inp1["vis_begin"]
    assert int(g1["n_vis_out"][0]) == info.cap_out
    np.testing.assert_array_equal(g1["pos_out"][0, :144], pos1[0][:144])
    np.testing.assert_array_equal(g1["hidden_out"][0, vb:vb + 144], inp1["hidden"][0, vb:vb + 144])
    plan.close()


# ---- seeded random geometries ---------------------------------------------------------------------

def _random_workload(seed):
    """Tiles, windows, keep ratios, head layout and sizes drawn from a seeded generator: ragged windows, several
    tiles per sample, 600 to 4500 tokens (one to eight CTAs per sample in the selection kernel), hidden sizes
    that are and are not multiples of 64, head sizes with and without a tensor-core path."""
    rng = np.random.default_rng(7000 + seed)
    n_tiles = int(rng.integers(1, 4))
    big = seed % 3 == 0
    tiles = tuple((int(rng.integers(18, 50 if big else 30)), int(rng.integers(18, 46 if big else 26)))
                  for _ in range(n_tiles))
    smallest = min(min(t) for t in tiles)
    windows = tuple(sorted((int(rng.integers(1, min(7, smallest // 2))) for _ in range(3)), reverse=True))
    n_kv = int(rng.choice([1, 2, 4]))
    return S.Workload(name=f"rand{seed}", config_id=100 + seed, batch=int(rng.integers(1, 4)), tiles=tiles,
                      n_text=int(rng.integers(1, 180)), hidden=int(rng.choice([64, 72, 192, 320, 520])),
                      n_q_heads=n_kv * int(rng.choice([1, 2])), n_kv_heads=n_kv,
                      head_dim=int(rng.choice([64, 128, 128, 32])), n_layers=16, layers=(3, 7, 11),
                      windows=windows, keep=tuple(float(k) for k in rng.uniform(0.5, 0.9, size=3).round(2)))


@pytest.mark.parametrize("seed", range(16))
def test_random_geometry(seed):
    wl = _random_workload(seed)
    # K/V side: merge or gather, contiguous or paged caches (pages of 16 or 5 tokens), both cache layouts
    H.run_schedule(wl, xi_mode=["attn", "given", "lse"][seed % 3], dtype="fp32" if seed == 4 else "bf16",
                   engine="simt" if seed == 4 else "auto", kv_mode=["merge", "gather"][(seed // 2) % 2],
                   paged=[0, 16, 0, 5][seed % 4], kv_layout="bnhd" if seed % 4 == 2 else "bhnd")


def test_selection_over_eight_ctas_ragged_windows():
    # 4480 tokens per sample (a cluster of eight CTAs in the selection kernel), windows that do not divide
    # the grid, a single large window at the last stage (1344 tokens: the per-window rank loops at length)
    wl = S.Workload(name="sel8", config_id=120, batch=2, tiles=((70, 64),), n_text=9, hidden=64, n_q_heads=2,
                    n_kv_heads=1, head_dim=64, n_layers=16, layers=(3, 7, 11), windows=(6, 3, 1),
                    keep=(0.6, 0.5, 0.7))
    stats = H.run_schedule(wl, xi_mode="given")
    assert stats[0]["n_out"][0] < 4480 * 0.6 + 40


@pytest.mark.parametrize("engine", ["simt", "auto"])
def test_windows_of_one_and_two_tokens(engine):
    # a 6 x 8 grid cut 6 x 6: windows of one token (no B node: nothing to merge) and of two (one A, one B);
    # then 3 x 3 and a single window over what is left
    wl = S.Workload(name="w12", config_id=122, batch=2, tiles=((6, 8),), n_text=3, hidden=64, n_q_heads=2,
                    n_kv_heads=1, head_dim=64, n_layers=16, layers=(3, 7, 11), windows=(6, 3, 1),
                    keep=(0.5, 0.6, 0.5))
    stats = H.run_schedule(wl, engine=engine)
    assert stats[0]["n_out"] == [36, 36]          # twelve two-token windows lose one token each


def test_selection_with_several_tokens_per_thread():
    # 9600 tokens per sample: more than the 8 x 1024 threads of the largest cluster, so every phase of the
    # selection kernel loops and its prefix sums take the two-pass path
    wl = S.Workload(name="sel9600", config_id=121, batch=1, tiles=((100, 96),), n_text=7, hidden=64, n_q_heads=2,
                    n_kv_heads=2, head_dim=64, n_layers=16, layers=(3, 7, 11), windows=(6, 3, 2),
                    keep=(0.6, 0.5, 0.7))
    H.run_schedule(wl, xi_mode="given", stages=[0, 1])


# ---- full benchmark shapes, compared on the samples the oracle can finish in seconds -----------------

def _bench_streams():
    # the schedule bench.py times: second stream inside the call (window build and FD beside xi), K/V
    # compaction on a third stream behind the map event
    import torch
    return dict(aux_stream=torch.cuda.Stream(), kv_stream=torch.cuda.Stream())


def test_cfg2_full_size_sampled():
    stats = H.run_schedule(S.workload("cfg2"), oracle_samples=[0, 5], **_bench_streams())
    assert [s["n_out"] for s in stats] == [[1440] * 8, [720] * 8, [360] * 8]


def test_cfg2_full_size_one_stream():
    H.run_schedule(S.workload("cfg2"), oracle_samples=[3], stages=[0])


def test_cfg3_full_schedule_sampled():
    stats = H.run_schedule(S.workload("cfg3"), oracle_samples=[0, 31], **_bench_streams())
    assert [s["n_out"] for s in stats] == [[288] * 32, [144] * 32, [72] * 32]


def test_cfg4_gqa_video_full_schedule_sampled():
    # all three stages: later stages have few large tiles (128 x 128 entries), which the FD kernel splits
    # over clusters of CTAs, and 8192 -> 2048 tokens per sample for the clustered selection kernel
    stats = H.run_schedule(S.workload("cfg4"), oracle_samples=[1], **_bench_streams())
    assert [s["n_out"] for s in stats] == [[4096] * 2, [2048] * 2, [1024] * 2]


def test_cfg4g_large_windows_uniform_xi():
    # windows of 512, 1024 and 2048 tokens: FD tiles of 128 x 128 entries combined across B blocks (atomic
    # minimum on the keys), the rank loops of the selection kernel over up to 1024 A entries
    H.run_schedule(S.workload("cfg4g"), xi_mode="uniform", oracle_samples=[0])
