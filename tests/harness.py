"""Shared test plumbing: feed one seeded synthetic stage to the CPU oracle and to the CUDA library
(through the C ABI binding) and compare them element by element.

Inputs come from lightkv_synth, conditioned by oracle.gaps so that every selection decision has a
margin of at least 1e-3 (index-set parity is only claimed on such inputs).  Nothing here computes any
part of the method."""
from __future__ import annotations

import numpy as np

import lightkv_synth as S
from oracle import gaps as G
from oracle import lightkv_oracle as O

GAP = 1e-3
# bf16 storage, fp32 accumulation: max-abs 2e-2 and relative 1e-2; fp32 mode: 1e-5 relative
TOL = {"bf16": dict(max_abs=2e-2, rel=1e-2), "fp32": dict(max_abs=None, rel=1e-5)}


def prepare_stage(wl, stage, pos=None, dtype="bf16", samples=None, repair=True, tensors=("hidden", "q", "k", "v"),
                  metric="cosine", direction="a2b"):
    """Synthetic inputs of one stage with the selection margins enforced on the hidden states."""
    inp = S.make_layer_inputs(wl, stage, pos, dtype=dtype, samples=samples, tensors=tensors)
    rounder = O.to_bf16 if dtype == "bf16" else (lambda a: np.asarray(a, dtype=np.float32).astype(np.float64))
    reports = []
    if repair:
        vb = inp["vis_begin"]
        for b in range(inp["hidden"].shape[0]):
            nv = int(inp["n_vis"][b])
            fixed, rep = G.enforce_gaps(inp["hidden"][b, vb:vb + nv], inp["pos"][b, :nv], wl.tiles,
                                        wl.windows[stage], wl.keep[stage], GAP, rounder=rounder, metric=metric,
                                        direction=direction)
            assert rep["ok"], rep
            inp["hidden"][b, vb:vb + nv] = fixed.astype(np.float32)
            reports.append(rep)
    inp["gap_reports"] = reports
    return inp


def oracle_stage(wl, stage, inp, xi_mode="attn", n_text_after=0, text_range=None, text_ranges=None, causal=True,
                 metric="cosine", direction="a2b"):
    tb, te = (0, inp["vis_begin"]) if text_range is None else text_range
    q = inp.get("q") if xi_mode in ("attn", "lse") else None
    k = inp.get("k") if xi_mode in ("attn", "lse") else None
    xi = inp.get("xi") if xi_mode == "given" else None
    return O.compress_layer(inp["hidden"], q, k, inp["pos"], inp["n_vis"], inp["vis_begin"], wl.tiles,
                            wl.windows[stage], wl.keep[stage], text_begin=tb, text_end=te, xi=xi,
                            n_text_after=n_text_after, causal=causal, text_ranges=text_ranges, metric=metric,
                            direction=direction)


def oracle_lse(inp, n_heads, n_kv, causal=True, n_text_after=0, samples=None):
    """Row log-sum-exp of the scaled logits of the vision rows, [B, H, N] (what a fused attention would hand
    over; rows outside the vision block stay 0).  Sample b's keys are its own vis_begin + n_vis[b] + n_text_after rows."""
    q, k = inp["q"], inp["k"]
    b, h, n, dh = q.shape
    vb = inp["vis_begin"]
    out = np.zeros((b, h, n))
    for bi in (range(b) if samples is None else samples):
        nv = int(inp["n_vis"][bi])
        n_seq = vb + nv + n_text_after
        for hi in range(h):
            out[bi, hi, vb:vb + nv] = O.row_logsumexp(q[bi, hi, :n_seq], k[bi, hi // (n_heads // n_kv), :n_seq],
                                                     vb, nv, causal)
    return out


def torch_lse(q, k, group):
    """The same row log-sum-exp (causal) computed with plain torch ops on the device in fp32, for every row: an
    INPUT of the lse mode at sizes where the float64 oracle would take minutes (the oracle side of the
    comparison never uses it: it derives xi from Q and K alone)."""
    import torch
    b, h, n, dh = q.shape
    out = torch.empty((b, h, n), dtype=torch.float32, device=q.device)
    mask = torch.ones((n, n), dtype=torch.bool, device=q.device).tril_()
    for i in range(b):
        kk = k[i].float().repeat_interleave(group, dim=0)
        for h0 in range(0, h, 8):
            logits = torch.matmul(q[i, h0:h0 + 8].float(), kk[h0:h0 + 8].transpose(1, 2)) / dh ** 0.5
            out[i, h0:h0 + 8] = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1)
    return out


def to_device(arr, dtype, device="cuda"):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(arr))
    if arr.dtype == np.float32 and dtype == "bf16":
        return t.to(device).to(torch.bfloat16)          # values are bf16-representable: exact
    return t.to(device)


def make_plan(wl, dtype="bf16", xi_mode="attn", engine="auto", batch=None, max_text=None, ragged=False,
              metric="cosine", direction="a2b"):
    import paper_2605_00789_b200 as L
    xm = {"attn": L.XI_ATTN_FULL, "lse": L.XI_ATTN_LSE, "given": L.XI_GIVEN, "uniform": L.XI_UNIFORM}[xi_mode]
    return L.Plan(batch or wl.batch, wl.hidden, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_layers,
                  wl.tiles, wl.layers, wl.windows, wl.keep, max_text if max_text is not None else wl.n_text + 64,
                  dtype=L.BF16 if dtype == "bf16" else L.FP32, xi_mode=xm,
                  engine=L.ENGINE_AUTO if engine == "auto" else L.ENGINE_SIMT, ragged_input=ragged,
                  divergence={"cosine": L.FD_COSINE, "l2sq": L.FD_L2SQ, "l2": L.FD_L2}[metric],
                  direction=L.DIR_A2B if direction == "a2b" else L.DIR_B2A)


def gpu_stage(plan, wl, stage, inp, dtype="bf16", xi_mode="attn", n_text_after=0, text_range=None,
              lse=None, kv_mode="merge", paged=0, device="cuda", layer_fn=None, aux_stream=None,
              kv_layout="bhnd", kv_stream=None, text_ranges=None, bidirectional=False, want_lse=False,
              kv_in_place=False):
    """Run lightkv_compress_layer (or `layer_fn`, a binding function with the same signature) +
    lightkv_compact_kv on the device; returns numpy outputs."""
    import torch
    import paper_2605_00789_b200 as L
    info = plan.stage_info(stage)
    vb = inp["vis_begin"]
    bsz = inp["hidden"].shape[0]
    hidden = to_device(inp["hidden"], dtype, device)
    n_seq = hidden.shape[1]
    assert n_seq <= vb + info.cap_in + n_text_after
    kw = {}
    if aux_stream is not None:
        kw["aux_stream"] = aux_stream
    kv_kw = {}
    if kv_stream is not None:
        # K/V compaction on a second stream behind the call's map event (recorded before the hidden-state merge)
        kw["map_event"] = torch.cuda.Event()
        kw["map_event"].record()
        kv_kw["stream"] = kv_stream
    if xi_mode in ("attn", "lse"):
        kw["q"], kw["k"] = to_device(inp["q"], dtype, device), to_device(inp["k"], dtype, device)
    if xi_mode == "lse":
        if isinstance(lse, str):          # "torch": computed on the device with plain torch ops
            kw["lse"] = torch_lse(kw["q"], kw["k"], inp["q"].shape[1] // inp["k"].shape[1])
        elif isinstance(lse, torch.Tensor):   # already on the device (e.g. the lse_out of an earlier call)
            kw["lse"] = lse
        else:
            kw["lse"] = torch.from_numpy(lse.astype(np.float32)).to(device)
    if text_ranges is not None:
        kw["text_ranges"] = text_ranges
    if bidirectional:
        kw["bidirectional"] = True
    lse_out = None
    if want_lse:
        lse_out = torch.full((bsz, inp["q"].shape[1], n_seq), float("nan"), dtype=torch.float32, device=device)
        kw["lse_out"] = lse_out
    cap_pad = info.cap_in - inp["pos"].shape[1]
    assert cap_pad >= 0
    pos = np.pad(inp["pos"], ((0, 0), (0, cap_pad)), constant_values=-1)
    if xi_mode == "given":
        kw["xi"] = torch.from_numpy(np.pad(inp["xi"], ((0, 0), (0, cap_pad))).astype(np.float32)).to(device)
    tb, te = (0, vb) if text_range is None else text_range
    n_seq_out = vb + info.cap_out + n_text_after
    out = L.StageBuffers(plan, stage, n_seq_out, device)
    out.hidden_out.fill_(float("nan"))
    (layer_fn or L.compress_layer)(plan, stage, hidden, out, vis_begin=vb, n_text_after=n_text_after,
                                   text_begin=tb, text_end=te, n_vis=torch.from_numpy(inp["n_vis"]).to(device),
                                   pos=torch.from_numpy(pos).to(device), **kw)
    res = {"out": out}
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    if "k" in inp and "v" in inp:
        k_src, v_src = to_device(inp["k"], dtype, device), to_device(inp["v"], dtype, device)
        hkv, dh = k_src.shape[1], k_src.shape[3]
        mode = L.KV_MERGE if kv_mode == "merge" else L.KV_GATHER
        if kv_stream is not None:
            kv_stream.wait_stream(torch.cuda.current_stream())     # the K/V source tensors were just written
            kv_stream.wait_event(kw["map_event"])
        if paged:
            # scatter the contiguous K/V into shuffled pages, compact page pool -> page pool, gather back
            nblk_s = (n_seq + paged - 1) // paged
            nblk_d = (n_seq_out + paged - 1) // paged
            # the block tables must cover the stage's capacity (the host cannot know the device-side counts)
            mb = max(nblk_s, nblk_d, (vb + info.cap_in + n_text_after + paged - 1) // paged)
            g = torch.Generator().manual_seed(1234 + stage)
            perm_s = torch.randperm(bsz * mb, generator=g).reshape(bsz, mb).to(torch.int32)
            perm_d = torch.randperm(bsz * mb, generator=g).reshape(bsz, mb).to(torch.int32)
            pool = lambda: torch.full((bsz * mb, hkv, paged, dh), float("nan"), dtype=tdt, device=device)
            ks, vs, kd, vd = pool(), pool(), pool(), pool()
            for b in range(bsz):
                for blk in range(nblk_s):
                    lo, hi = blk * paged, min(n_seq, (blk + 1) * paged)
                    ks[perm_s[b, blk], :, :hi - lo] = k_src[b, :, lo:hi]
                    vs[perm_s[b, blk], :, :hi - lo] = v_src[b, :, lo:hi]
            if kv_in_place:     # the page pool shrinks inside its own pages: one pool, one block table
                kd, vd, perm_d = ks, vs, perm_s
            table_s = perm_s.to(device)
            table_d = table_s if kv_in_place else perm_d.to(device)
            L.compact_kv(plan, stage, out, ks, vs, kd, vd, vis_begin=vb, n_text_after=n_text_after, mode=mode,
                         n_vis=torch.from_numpy(inp["n_vis"]).to(device), page_size=paged,
                         src_block_table=table_s, dst_block_table=table_d)
            torch.cuda.synchronize()
            k_dst = torch.full((bsz, hkv, n_seq_out, dh), float("nan"), dtype=tdt, device=device)
            v_dst = k_dst.clone()
            for b in range(bsz):
                for blk in range(nblk_d):
                    lo, hi = blk * paged, min(n_seq_out, (blk + 1) * paged)
                    k_dst[b, :, lo:hi] = kd[perm_d[b, blk], :, :hi - lo]
                    v_dst[b, :, lo:hi] = vd[perm_d[b, blk], :, :hi - lo]
        else:
            k_dst = torch.full((bsz, hkv, n_seq_out, dh), float("nan"), dtype=tdt, device=device)
            v_dst = k_dst.clone()
            if kv_layout == "bnhd":      # token-major storage [B, N, H_kv, dh] handed over as strided views
                as_bnhd = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
                k_src, v_src, k_dst, v_dst = as_bnhd(k_src), as_bnhd(v_src), as_bnhd(k_dst), as_bnhd(v_dst)
                assert k_src.stride(1) == dh and k_src.stride(2) == hkv * dh
            if kv_in_place:     # destination = source (the shorter sequences end up at the front of their rows)
                k_dst, v_dst = k_src, v_src
            L.compact_kv(plan, stage, out, k_src, v_src, k_dst, v_dst, vis_begin=vb, n_text_after=n_text_after,
                         mode=mode, n_vis=torch.from_numpy(inp["n_vis"]).to(device), **kv_kw)
            if kv_in_place:
                k_dst, v_dst = k_dst[:, :, :n_seq_out], v_dst[:, :, :n_seq_out]
        torch.cuda.synchronize()
        res["k_out"], res["v_out"] = k_dst.float().cpu().numpy(), v_dst.float().cpu().numpy()
    torch.cuda.synchronize()
    for name in ("n_vis_out", "pos_out", "dst", "weight", "grp_off", "grp_src", "xi_out", "status"):
        res[name] = getattr(out, name).cpu().numpy()
    res["hidden_out"] = out.hidden_out.float().cpu().numpy()
    if lse_out is not None:
        res["lse_out"] = lse_out.cpu().numpy()
        res["lse_out_dev"] = lse_out
    return res


def _check_close(got, want, dtype, what):
    tol = TOL[dtype]
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    diff = np.abs(got - want)
    rel = np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300)
    assert rel <= tol["rel"], f"{what}: relative error {rel:.3e} > {tol['rel']}"
    if tol["max_abs"] is not None:
        assert diff.max() <= tol["max_abs"], f"{what}: max abs error {diff.max():.3e}"
    else:   # fp32 mode: element-wise relative to the row scale
        scale = np.abs(want).max(axis=-1, keepdims=True) + 1e-30
        assert (diff / scale).max() <= 10 * tol["rel"], f"{what}: element error {(diff / scale).max():.3e}"
    return float(diff.max()), float(rel)


def compare_stage(wl, stage, inp, ref, gpu, dtype="bf16", kv_mode="merge", n_text_after=0, samples=None,
                  xi_rel=None, expect_status=0):
    """Index sets bit-exact; weights, xi, merged hidden states and K/V within tolerance.
    `ref` is the oracle's per-sample result list for the samples in `samples` (default: all)."""
    vb = inp["vis_begin"]
    samples = list(range(len(ref))) if samples is None else samples
    stats = {"hidden_max_abs": 0.0, "hidden_rel": 0.0, "kv_max_abs": 0.0}
    assert int(gpu["status"][0]) == expect_status, f"device status word {int(gpu['status'][0])}"
    for r, b in zip(ref, samples):
        nv, n_out = int(inp["n_vis"][b]), int(r["n_out"])
        assert int(gpu["n_vis_out"][b]) == n_out, (b, int(gpu["n_vis_out"][b]), n_out)
        np.testing.assert_array_equal(gpu["pos_out"][b, :n_out], r["pos_out"])
        np.testing.assert_array_equal(gpu["dst"][b, :nv], r["dst"])
        # CSR form of the same map: slot o gathers exactly the tokens with dst == o, survivor first
        off, src = gpu["grp_off"][b], gpu["grp_src"][b]
        assert off[0] == 0 and off[n_out] == nv
        for o in range(n_out):
            members = src[off[o]:off[o + 1]]
            assert members[0] == r["survivor"][o]
            assert sorted(members) == sorted(np.nonzero(r["dst"] == o)[0])
        xr = xi_rel if xi_rel is not None else (2e-3 if dtype == "bf16" else 2e-5)
        np.testing.assert_allclose(gpu["xi_out"][b, :nv], r["xi"], rtol=xr, atol=0)
        np.testing.assert_allclose(gpu["weight"][b, :nv], r["weight"], rtol=2 * xr, atol=0)
        n_seq_out = vb + n_out + n_text_after
        want = r["hidden_out"]
        ma, rel = _check_close(gpu["hidden_out"][b, :n_seq_out], want, dtype, f"hidden_out[{b}]")
        stats["hidden_max_abs"] = max(stats["hidden_max_abs"], ma)
        stats["hidden_rel"] = max(stats["hidden_rel"], rel)
        # tokens that were not merged are copied bit-exactly
        single = np.array([off[o + 1] - off[o] == 1 for o in range(n_out)], dtype=bool)
        np.testing.assert_array_equal(gpu["hidden_out"][b, vb:vb + n_out][single],
                                      inp["hidden"][b, vb + r["survivor"]][single])
        np.testing.assert_array_equal(gpu["hidden_out"][b, :vb], inp["hidden"][b, :vb])
        if "k_out" in gpu:
            for name in ("k", "v"):
                n_seq = vb + nv + n_text_after
                want = O.compact_kv(inp[name][b][:, :n_seq], vb, nv, r["dst"], r["weight"], r["survivor"], kv_mode)
                ma, _ = _check_close(gpu[name + "_out"][b][:, :n_seq_out], want, dtype, f"{name}_out[{b}]")
                stats["kv_max_abs"] = max(stats["kv_max_abs"], ma)
    return stats


def check_lse_out(inp, gpu, n_heads, n_kv, samples, causal=True, n_text_after=0, atol=2e-3):
    """lse_out of the vision rows against the oracle's row log-sum-exp (natural log); rows outside the vision
    block must not have been written (they still hold the NaN fill)."""
    vb = inp["vis_begin"]
    want = oracle_lse(inp, n_heads, n_kv, causal, n_text_after, samples=samples)
    for b in samples:
        nv = int(inp["n_vis"][b])
        got = gpu["lse_out"][b]
        np.testing.assert_allclose(got[:, vb:vb + nv], want[b][:, vb:vb + nv], rtol=0, atol=atol)
        assert np.isnan(got[:, :vb]).all() and np.isnan(got[:, vb + nv:]).all()


def run_schedule(wl, dtype="bf16", xi_mode="attn", engine="auto", kv_mode="merge", paged=0, samples=None,
                 stages=None, oracle_samples=None, aux_stream=None, kv_layout="bhnd", kv_stream=None,
                 lse_source="oracle", ragged=False, first_pos=None, text_ranges=None, bidirectional=False,
                 want_lse=False, expect_status=0, metric="cosine", direction="a2b", kv_in_place=False):
    """All stages of a workload, chained through the surviving positions; returns per-stage stats.
    first_pos: per-sample positions entering stage 0 (a subset of the grid); ragged: plan built for subsets."""
    bsz = wl.batch if samples is None else len(samples)
    plan = make_plan(wl, dtype, xi_mode, engine, batch=bsz, ragged=ragged, metric=metric, direction=direction)
    pos = first_pos
    all_stats = []
    for stage in (range(wl.n_stages) if stages is None else stages):
        inp = prepare_stage(wl, stage, pos, dtype, samples=samples, metric=metric, direction=direction)
        if xi_mode == "given":
            rng = np.random.default_rng(stage)
            inp["xi"] = rng.uniform(0.05, 3.0, size=inp["pos"].shape).astype(np.float32)
        lse = None
        if xi_mode == "lse":
            lse = "torch" if lse_source == "torch" else oracle_lse(inp, wl.n_q_heads, wl.n_kv_heads,
                                                                   causal=not bidirectional)
        gpu = gpu_stage(plan, wl, stage, inp, dtype, xi_mode, lse=lse, kv_mode=kv_mode, paged=paged,
                        aux_stream=aux_stream, kv_layout=kv_layout, kv_stream=kv_stream, text_ranges=text_ranges,
                        bidirectional=bidirectional, want_lse=want_lse, kv_in_place=kv_in_place)
        osamp = list(range(bsz)) if oracle_samples is None else oracle_samples
        sub = {key: (val[osamp] if isinstance(val, np.ndarray) and val.shape[:1] == (bsz,) else val)
               for key, val in inp.items()}
        ref = oracle_stage(wl, stage, sub, xi_mode, text_ranges=text_ranges, causal=not bidirectional,
                           metric=metric, direction=direction)
        stats = compare_stage(wl, stage, inp, ref, gpu, dtype, kv_mode, samples=osamp, expect_status=expect_status)
        if want_lse:
            check_lse_out(inp, gpu, wl.n_q_heads, wl.n_kv_heads, osamp, causal=not bidirectional)
        stats["n_out"] = [int(v) for v in gpu["n_vis_out"]]
        stats["info"] = plan.stage_info(stage)
        all_stats.append(stats)
        # chain on the device result (equal to the oracle's on the compared samples)
        pos = [gpu["pos_out"][b, :int(gpu["n_vis_out"][b])] for b in range(bsz)]
    plan.close()
    return all_stats


def smoke_check():
    """One small stage on cuda:0 against the oracle."""
    import torch
    assert torch.cuda.is_available(), "smoke needs a CUDA device"
    wl = S.workload("small")
    stats = run_schedule(wl, dtype="bf16", xi_mode="attn", stages=[0])
    print("smoke ok", stats)
