#!/usr/bin/env python
"""Benchmark of the LightKV compression hot path on B200 (one JSON line on stdout).

A step = one pass of the whole hot path over one batch: for every stage of the workload's schedule,
lightkv_compress_layer (window build, xi, FD + best partner, selection + merge map, hidden merge) and
lightkv_compact_kv on that layer's K/V, chained through the surviving positions on the device.
Inputs are seeded synthetic tensors (lightkv_synth), regenerated per compression layer and resident
in HBM before the timed region.  `value` is vision tokens entering compression stages per second.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

N > 1 (under torchrun): every rank compresses its own batch (no data-path collective, weak scaling);
the time is the max over ranks.  --impl reference times the CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import lightkv_synth as S  # noqa: E402

KERNELS = ("window_build", "xi", "fd_best_partner", "select_map", "merge_hidden", "kv_compact")

# dram__bytes_read.sum + dram__bytes_write.sum per launch from the committed ncu captures (profiles/),
# of the stage-0 launch, keyed by (workload, kernel); null where no capture exists.
NCU_TRAFFIC_BYTES = {
    ("cfg2", "xi"): 401.05e6,                # profiles/xi_tc_kernel_cfg2_stage0.txt
    ("cfg2", "fd_best_partner"): 192.91e6,   # profiles/fd_tc_kernel_cfg2_stage0.txt
    ("cfg2", "merge_hidden"): 264.93e6,      # profiles/merge_rows_kernel_cfg2_stage0.txt
    ("cfg2", "kv_compact"): 563.41e6,        # profiles/kv_compact_kernel_cfg2_stage0.txt
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.file = index, None, None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ------------------------------------------------------------------------------------- multi-rank
# Samples are independent and the path has no exchange step: rank r compresses its own batch (samples
# r*batch .. r*batch + batch - 1 of the seeded generator).  The only communication is the timing protocol.

def rank_samples(rank: int, batch: int):
    return [rank * batch + b for b in range(batch)]


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Slowest rank's value (all-reduce MAX over the default process group); identity for one rank."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(tokens_per_rank_step: int, world: int, ms_step_max: float) -> float:
    """Units all ranks processed per second, timed by the slowest rank."""
    return world * tokens_per_rank_step / (ms_step_max / 1e3)


# ------------------------------------------------------------------------------------------ workload

def causal_lse(torch, q, k, group):
    """Row log-sum-exp of the scaled causal logits, [B, H, N] fp32 (what a fused attention kernel hands over);
    plain torch, one sample at a time: an input of the lse mode, computed outside every timed region."""
    b, h, n, dh = q.shape
    out = torch.empty((b, h, n), dtype=torch.float32, device=q.device)
    mask = torch.ones((n, n), dtype=torch.bool, device=q.device).tril_()
    for i in range(b):
        kk = k[i].float().repeat_interleave(group, dim=0)
        for h0 in range(0, h, 8):
            logits = torch.matmul(q[i, h0:h0 + 8].float(), kk[h0:h0 + 8].transpose(1, 2)) / dh ** 0.5
            out[i, h0:h0 + 8] = torch.logsumexp(logits.masked_fill(~mask, float("-inf")), dim=-1)
    return out


def build_inputs(wl, plan, L, torch, device, sample_offset, kv_layout="bhnd", xi_mode="full"):
    """Generate every stage's inputs on the host (pinned) and upload them.  Stage i+1 is sampled at the
    positions that survive stage i (taken from one untimed run of the library itself)."""
    samples = rank_samples(sample_offset // wl.batch, wl.batch)
    stages, pos = [], None
    for st in range(wl.n_stages):
        info = plan.stage_info(st)
        inp = S.make_layer_inputs(wl, st, pos, samples=samples)
        host, dev = {}, {}
        for name in ("hidden", "q", "k", "v"):
            t = torch.from_numpy(S.bf16_bits(inp[name]).view(np.int16)).view(torch.bfloat16).pin_memory()
            host[name] = t
            if name in ("k", "v") and kv_layout == "bnhd":      # token-major cache, handed over as a strided view
                store = torch.empty((t.shape[0], t.shape[2], t.shape[1], t.shape[3]), dtype=t.dtype, device=device)
                dev[name] = store.permute(0, 2, 1, 3)
                dev[name].copy_(t, non_blocking=True)
            else:
                dev[name] = t.to(device, non_blocking=True)
        n_seq = host["hidden"].shape[1]
        pos_pad = np.full((wl.batch, info.cap_in), -1, dtype=np.int32)
        pos_pad[:, :inp["pos"].shape[1]] = inp["pos"]
        if xi_mode == "lse":
            dev["lse"] = causal_lse(torch, dev["q"], dev["k"], wl.n_q_heads // wl.n_kv_heads)
        dev["pos"] = torch.from_numpy(pos_pad).to(device)
        dev["n_vis"] = torch.from_numpy(inp["n_vis"]).to(device)
        n_seq_out = wl.n_text + info.cap_out
        out = L.StageBuffers(plan, st, n_seq_out, device)
        if kv_layout == "bnhd":
            k_dst = torch.empty((wl.batch, n_seq_out, wl.n_kv_heads, wl.head_dim), dtype=torch.bfloat16,
                                device=device).permute(0, 2, 1, 3)
            v_dst = torch.empty((wl.batch, n_seq_out, wl.n_kv_heads, wl.head_dim), dtype=torch.bfloat16,
                                device=device).permute(0, 2, 1, 3)
        else:
            k_dst = torch.empty((wl.batch, wl.n_kv_heads, n_seq_out, wl.head_dim), dtype=torch.bfloat16, device=device)
            v_dst = torch.empty_like(k_dst)
        host_out = {"hidden": torch.empty(out.hidden_out.shape, dtype=torch.bfloat16).pin_memory(),
                    "k": torch.empty(k_dst.shape, dtype=torch.bfloat16).pin_memory(),
                    "v": torch.empty(k_dst.shape, dtype=torch.bfloat16).pin_memory(),
                    "n_vis_out": torch.empty((wl.batch,), dtype=torch.int32).pin_memory(),
                    "pos_out": torch.empty(out.pos_out.shape, dtype=torch.int32).pin_memory()}
        stg = dict(info=info, host=host, dev=dev, out=out, k_dst=k_dst, v_dst=v_dst, host_out=host_out,
                   n_vis=inp["n_vis"].copy(), n_seq=n_seq, n_seq_out=n_seq_out)
        stages.append(stg)
        run_stage(L, plan, wl, st, stg, stg["dev"]["pos"], stg["dev"]["n_vis"])
        torch.cuda.synchronize()
        n_out = out.n_vis_out.cpu().numpy()
        pos_out = out.pos_out.cpu().numpy()
        stg["n_out"] = n_out.copy()
        pos = [pos_out[b, :n_out[b]] for b in range(wl.batch)]
        if int(out.status.item()) != 0:
            raise RuntimeError(f"device status word {int(out.status.item())} at stage {st}")
    return stages


def run_stage(L, plan, wl, st, stg, pos, n_vis, trace=None, side=None, aux=None):
    k_dst, v_dst = (stg["dev"]["k"], stg["dev"]["v"]) if stg.get("kv_in_place") else (stg["k_dst"], stg["v_dst"])
    return _run_stage(L, plan, wl, st, stg, pos, n_vis, trace, side, aux, k_dst, v_dst)


def _run_stage(L, plan, wl, st, stg, pos, n_vis, trace, side, aux, k_dst, v_dst):
    """lightkv_compress_layer on the current stream, then lightkv_compact_kv either on the same stream or,
    when `side` is given, on that stream behind the call's map event (the compaction only needs the stage's
    merge map, which is complete before the hidden-state merge starts)."""
    import torch
    d = stg["dev"]
    map_event = stg.get("map_event") if side is not None else None
    L.compress_layer(plan, st, d["hidden"], stg["out"], vis_begin=wl.n_text, q=d["q"], k=d["k"], n_vis=n_vis,
                     pos=pos, trace_events=trace, aux_stream=aux, lse=d.get("lse"), map_event=map_event)
    if side is None:
        L.compact_kv(plan, st, stg["out"], d["k"], d["v"], k_dst, v_dst, vis_begin=wl.n_text, n_vis=n_vis)
    else:
        if map_event is not None:
            side.wait_event(map_event)
        else:
            side.wait_stream(torch.cuda.current_stream())
        L.compact_kv(plan, st, stg["out"], d["k"], d["v"], k_dst, v_dst, vis_begin=wl.n_text, n_vis=n_vis,
                     stream=side)


def run_step(L, plan, wl, stages, traces=None, kv_events=None, side=None, aux=None):
    """The whole hot path once; stage i+1 reads positions and counts stage i left on the device.
    With `side`, the K/V compaction of stage i (HBM bound) runs on that second stream while stage i+1's
    compression (bound by the xi contraction) proceeds on the current one; the step ends with a join.
    With `aux`, the library itself runs window build + FD beside the xi contraction (aux_stream)."""
    import torch
    pos, n_vis = stages[0]["dev"]["pos"], stages[0]["dev"]["n_vis"]
    for st, stg in enumerate(stages):
        run_stage(L, plan, wl, st, stg, pos, n_vis, trace=None if traces is None else traces[st], side=side, aux=aux)
        if kv_events is not None:
            kv_events[st].record()
        pos, n_vis = stg["out"].pos_out, stg["out"].n_vis_out
    if side is not None:
        torch.cuda.current_stream().wait_stream(side)


def algorithmic_work(wl, stages, xi_mode="full"):
    """Per stage and per kernel: algorithmic bytes (HBM streams) or flops (xi) of one launch."""
    e = 2  # bf16
    per_stage = []
    nt = wl.n_text
    for stg in stages:
        work = {}
        n_in = stg["n_vis"].astype(np.float64)
        n_out = stg["n_out"].astype(np.float64)
        # xi, ATTN_FULL: 2*dh flops per (head, query, visible key); query t sees n_text + t + 1 keys
        work["xi"] = float((2.0 * wl.n_q_heads * wl.head_dim * (n_in * (nt + 1) + n_in * (n_in - 1) / 2)).sum())
        if xi_mode == "lse":
            # only the prompt keys are visited: HBM bound on one read of Q_v and K_text (+ 4 B of log-sum-exp in and
            # 4 B of per-head xi out per (head, query))
            work["xi"] = float((wl.n_q_heads * n_in * (wl.head_dim * e + 8) + wl.n_kv_heads * nt * wl.head_dim * e).sum())
        # FD: one read of the vision rows (+ 8 bytes of keys per A node)
        work["fd_best_partner"] = float((n_in * wl.hidden * e + 4 * n_in).sum())
        # hidden merge: every input row read once, every output row written once
        work["merge_hidden"] = float(((nt + n_in) * wl.hidden * e + (nt + n_out) * wl.hidden * e).sum())
        # K/V: same for K and V, all KV heads
        work["kv_compact"] = float((2 * wl.n_kv_heads * wl.head_dim * e * ((nt + n_in) + (nt + n_out))).sum())
        work["window_build"] = float((n_in * 4 * 5).sum())
        work["select_map"] = float((n_in * 4 * 10).sum())
        per_stage.append(work)
    return per_stage


def oracle_sample_inputs(wl):
    """Inputs of sample 0 for every stage of the schedule (generated once, untimed); the positions are
    chained through the oracle's own results."""
    from oracle import lightkv_oracle as O
    per_stage, pos = [], None
    for st in range(wl.n_stages):
        inp = S.make_layer_inputs(wl, st, pos, samples=[0])
        per_stage.append(inp)
        if st + 1 < wl.n_stages:      # advance the positions cheaply with uniform xi
            res = O.compress_layer(inp["hidden"], None, None, inp["pos"], inp["n_vis"], inp["vis_begin"], wl.tiles,
                                   wl.windows[st], wl.keep[st])
            pos = [res[0]["pos_out"]]
    return per_stage


def oracle_sample_run(wl, per_stage, stage_list):
    """The CPU oracle (compression + K/V compaction) on the prepared inputs of the given stages.
    Returns (seconds, vision tokens entering the stages it ran)."""
    from oracle import lightkv_oracle as O
    t_total, tokens = 0.0, 0
    for st in stage_list:
        inp = per_stage[st]
        t0 = time.perf_counter()
        res = O.compress_layer(inp["hidden"], inp["q"], inp["k"], inp["pos"], inp["n_vis"], inp["vis_begin"],
                               wl.tiles, wl.windows[st], wl.keep[st])
        r = res[0]
        nv = int(inp["n_vis"][0])
        for name in ("k", "v"):
            O.compact_kv(inp[name][0][:, :inp["vis_begin"] + nv], inp["vis_begin"], nv, r["dst"], r["weight"],
                         r["survivor"], "merge")
        t_total += time.perf_counter() - t0
        tokens += nv
    return t_total, tokens


def c_oracle_sample(wl, unit, per_stage):
    """The plain C oracle (oracle/lightkv_oracle.c: simple loops, double precision, one thread) on the last stage of
    sample 0: xi, the compression stage and the K/V compaction.  Returns a cpu_baseline-style dict."""
    from oracle import c_oracle as OC
    st = wl.n_stages - 1
    inp = per_stage[st]
    nv, vb = int(inp["n_vis"][0]), inp["vis_begin"]
    t0 = time.perf_counter()
    xi = OC.xi(inp["q"][0][:, :vb + nv], inp["k"][0][:, :vb + nv], vb, nv, [(0, vb)])
    r = OC.compress(inp["hidden"][0, vb:vb + nv], inp["pos"][0, :nv], xi, wl.tiles, wl.windows[st], wl.keep[st])
    for name in ("k", "v"):
        OC.compact(inp[name][0][:, vb:vb + nv], r["dst"], r["weight"], r["n_out"])
    t = time.perf_counter() - t0
    return {"value": nv / t, "unit": unit, "cores": 1, "kind": "oracle (plain C)",
            "sample": f"sample 0 of {wl.batch}, last stage only ({nv} vision tokens, {t:.1f} s)"}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------------ main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="cfg2", choices=sorted(S.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--engine", default="auto", choices=["auto", "simt"])
    ap.add_argument("--xi-mode", default="full", choices=["full", "lse"],
                    help="full: xi from Q and K alone (the benchmark); lse: the row log-sum-exp of the layer's attention "
                         "is an input (computed once with torch before the timed region), only prompt keys are visited")
    ap.add_argument("--kv-layout", default="bhnd", choices=["bhnd", "bnhd"],
                    help="K/V cache layout: [B,H_kv,N,dh] (head-major) or [B,N,H_kv,dh] (token-major)")
    ap.add_argument("--kv-in-place", action="store_true",
                    help="compact K/V inside the cache's own rows (destination = source) instead of into a second buffer")
    ap.add_argument("--graph", type=int, default=1, choices=[0, 1],
                    help="1: replay the step from a CUDA graph captured once (timed region only)")
    ap.add_argument("--streams", type=int, default=2, choices=[1, 2],
                    help="2: HBM-bound kernels (window build + FD, K/V compaction) on second streams beside the xi contraction")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    wl = S.workload(args.workload)
    metric, unit = "vision_tokens_compressed_per_s", "tokens/s"
    config = {"workload": f"{wl.name}: {wl.n_stages}-stage schedule layers={list(wl.layers)} windows={list(wl.windows)} "
                          f"keep={list(wl.keep)}, batch {wl.batch}, {wl.n_vis} vision + {wl.n_text} text tokens, "
                          f"hidden {wl.hidden}, {wl.n_q_heads}q/{wl.n_kv_heads}kv heads x {wl.head_dim}, "
                          f"xi from {'full causal attention' if args.xi_mode == 'full' else 'the prompt keys + a given row log-sum-exp'}, "
                          f"K/V merge{' in place' if args.kv_in_place else ''}, K/V layout {args.kv_layout}",
              "batch_per_gpu": wl.batch}
    # L2 policy of the device-timed arm, a function of the workload alone so that both arms print the same config:
    # a step streams every stage's inputs once; where the first stage's inputs are less than twice the L2, the L2
    # is flushed between timed steps by writing a 256 MB buffer outside the timed intervals
    stage0_bytes = 2 * wl.batch * (wl.n_text + wl.n_vis) * (wl.hidden + (wl.n_q_heads + 2 * wl.n_kv_heads) * wl.head_dim)
    flush_l2 = stage0_bytes < 2 * 126e6
    config["l2"] = ("L2 flushed between timed steps (256 MB write, untimed)" if flush_l2 else
                    f"inputs larger than L2 ({stage0_bytes / 1e6:.0f} MB read by the first stage alone, L2 is 126 MB)")

    if args.impl == "reference":
        if rank != 0:
            return
        # A step is the oracle on sample 0: all stages if the K + W steps then fit in about two and a half
        # minutes of CPU work, else the last stage only.  Inputs are generated once, outside the timed steps.
        budget = 150.0
        per_stage = oracle_sample_inputs(wl)
        n_iter = args.steps + args.warmup
        t_last, _ = oracle_sample_run(wl, per_stage, [wl.n_stages - 1])
        full = t_last * 12 * n_iter < budget                         # the full schedule costs ~10x its last stage
        stage_list = list(range(wl.n_stages)) if full else [wl.n_stages - 1]
        times, tokens = [], 0
        for i in range(n_iter):
            t, tokens = oracle_sample_run(wl, per_stage, stage_list)
            if i >= args.warmup:
                times.append(t)
        ms = 1e3 * sum(times) / len(times)
        value = tokens / (ms / 1e3)
        sample = f"sample 0 of {wl.batch}, " + ("all stages" if full else "last stage only") + f" ({tokens} vision tokens per step)"
        line = {"impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
                "cpu_baseline": {"value": value, "unit": unit, "cores": blas_threads(), "kind": "oracle", "sample": sample},
                "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
                "gpu_launches": 0}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    if local_rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    import paper_2605_00789_b200 as L

    plan = L.Plan(wl.batch, wl.hidden, wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.n_layers, wl.tiles, wl.layers,
                  wl.windows, wl.keep, wl.n_text, dtype=L.BF16,
                  xi_mode=L.XI_ATTN_FULL if args.xi_mode == "full" else L.XI_ATTN_LSE,
                  engine=L.ENGINE_AUTO if args.engine == "auto" else L.ENGINE_SIMT)
    stages = build_inputs(wl, plan, L, torch, device, sample_offset=rank * wl.batch, kv_layout=args.kv_layout,
                          xi_mode=args.xi_mode)
    for s in stages:
        s["kv_in_place"] = args.kv_in_place
    tokens_per_step = int(sum(int(s["n_vis"].sum()) for s in stages))
    n_stages = len(stages)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    side = torch.cuda.Stream(device=device) if args.streams == 2 else None
    aux = torch.cuda.Stream(device=device) if args.streams == 2 else None
    if side is not None:
        for s in stages:              # recorded by the library after the merge map of the stage is complete
            s["map_event"] = torch.cuda.Event()
            s["map_event"].record()   # torch creates the CUDA event lazily; the C ABI needs a live handle
    for _ in range(args.warmup):
        run_step(L, plan, wl, stages, side=side, aux=aux)

    # The step's launches (18 kernels on three streams) are captured once into a CUDA graph and replayed:
    # the library's calls are plain stream work, so the caller may do that.  Plumbing only; if the capture is
    # refused the step is launched call by call and the JSON says so.
    step_graph = None
    if args.graph:
        try:
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                run_step(L, plan, wl, stages, side=side, aux=aux)
            step_graph = g
        except Exception as exc:      # noqa: BLE001
            print(f"bench: graph capture refused ({exc}); launching call by call", file=sys.stderr)
            torch.cuda.synchronize()

    def one_step():
        if step_graph is not None:
            step_graph.replay()
        else:
            run_step(L, plan, wl, stages, side=side, aux=aux)
    for _ in range(2):
        one_step()

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record()                    # torch creates the CUDA event lazily; the C ABI needs a live handle
        return e
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device) if flush_l2 else None

    # timed region: K whole steps in the benchmark's schedule (--streams 2: K/V compaction of a stage on a
    # second stream, overlapping the next stage's compression).  The clock sampler runs from here to the
    # end of the per-kernel pass.
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    if flush_buf is None:
        t_begin, t_end = ev(), ev()
        t_begin.record()
        for i in range(args.steps):
            one_step()
        t_end.record()
        barrier()
        ms_local = t_begin.elapsed_time(t_end)
    else:
        pairs = [(ev(), ev()) for _ in range(args.steps)]
        for a_ev, b_ev in pairs:
            flush_buf.fill_(1)
            a_ev.record()
            one_step()
            b_ev.record()
        barrier()
        ms_local = sum(a_ev.elapsed_time(b_ev) for a_ev, b_ev in pairs)
    ms_total = max_over_ranks(ms_local, world, device)
    ms_step = ms_total / args.steps
    value = whole_job_throughput(tokens_per_step, world, ms_step)
    for st, s in enumerate(stages):     # the timed steps left the same counts as the untimed first run, no status bit
        if int(s["out"].status.item()) != 0 or not np.array_equal(s["out"].n_vis_out.cpu().numpy(), s["n_out"]):
            raise RuntimeError(f"timed steps disagree with the first run at stage {st}")

    # per-kernel pass: the same steps on ONE stream, with the library's trace events between its launches
    # (TRACE_EVENTS per (step, stage) + one after compact_kv), so that every kernel is timed alone
    ksteps = max(3, min(args.steps, 10))
    traces = [[[ev() for _ in range(L.TRACE_EVENTS)] for _ in range(n_stages)] for _ in range(ksteps)]
    kv_ev = [[ev() for _ in range(n_stages)] for _ in range(ksteps)]
    k_begin, k_end = ev(), ev()
    barrier()
    k_begin.record()
    for i in range(ksteps):
        run_step(L, plan, wl, stages, traces[i], kv_ev[i])
    k_end.record()
    barrier()
    clocks = sampler.stop()
    ms_step_one_stream = max_over_ranks(k_begin.elapsed_time(k_end), world, device) / ksteps
    # the same one-stream schedule without events between the launches, replayed from a graph: the difference
    # to the pass above is what recording an event after every kernel costs (launch latencies are exposed)
    ms_one_stream_graph = None
    if args.graph:
        try:
            torch.cuda.synchronize()
            g1 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g1):
                run_step(L, plan, wl, stages)
            g1.replay()
            barrier()
            c_begin, c_end = ev(), ev()
            c_begin.record()
            for _ in range(ksteps):
                g1.replay()
            c_end.record()
            barrier()
            ms_one_stream_graph = max_over_ranks(c_begin.elapsed_time(c_end), world, device) / ksteps
        except Exception as exc:      # noqa: BLE001
            print(f"bench: one-stream graph capture refused ({exc})", file=sys.stderr)
            torch.cuda.synchronize()

    ktime = {k: 0.0 for k in KERNELS}       # ms per step, summed over stages
    kstage = [{k: 0.0 for k in KERNELS} for _ in range(n_stages)]
    for i in range(ksteps):
        for st in range(n_stages):
            e = traces[i][st]
            for j, name in enumerate(L.TRACE_NAMES):
                kstage[st][name] += e[j].elapsed_time(e[j + 1]) / ksteps
            kstage[st]["kv_compact"] += e[-1].elapsed_time(kv_ev[i][st]) / ksteps
    for st in range(n_stages):
        for k in KERNELS:
            ktime[k] += kstage[st][k]
    work_stage = algorithmic_work(wl, stages, args.xi_mode)
    work = {k: sum(w[k] for w in work_stage) for k in KERNELS}
    peaks = measured_peaks()

    def rate(k, amount, ms):
        # xi from full attention rows is a contraction: every launch is timed alone between two events (a pass of
        # a few milliseconds at full clocks), so the peak that applies is the burst one; with the caller's row
        # log-sum-exp it only streams Q_v and the prompt keys and is judged against the copy bandwidth
        sec = ms / 1e3
        if k == "xi" and args.xi_mode == "full":
            return amount / sec / 1e12, peaks["bf16_tflops"], "TFLOP/s", "tensor"
        return amount / sec / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"

    kernels = {}
    for k in KERNELS:
        ach, peak, u, bound = rate(k, work[k], ktime[k])
        kernels[k] = {"ms_per_step": round(ktime[k], 4), "share": round(ktime[k] / sum(ktime.values()), 4),
                      "bound": bound, "achieved": round(ach, 2), "peak": peak, "unit": u, "frac": round(ach / peak, 4)}
    # roofline object: the kernel with the largest share, at its largest launch (stage 0), so that `achieved`
    # and `traffic` are both per launch
    top = max(KERNELS, key=lambda k: ktime[k])
    ach, peak, u, bound = rate(top, work_stage[0][top], kstage[0][top])
    roofline = {"kernel": top, "launch": "stage 0", "bound": bound, "achieved": round(ach, 2), "peak": peak, "unit": u,
                "frac": round(ach / peak, 4), "traffic": NCU_TRAFFIC_BYTES.get((wl.name, top)),
                "algorithmic": work_stage[0][top], "us": round(1e3 * kstage[0][top], 1),
                "peak_source": f"of {peaks['source']}"}
    if bound == "tensor":
        roofline["peak_kind"] = "bf16_tflops (burst: the launch is timed alone between two events)"
        roofline["frac_of_sustained"] = round(ach / peaks["bf16_tflops_sustained"], 4)
    if top == "xi" and args.xi_mode == "full":
        # one exponential per logit on the special-function unit (16 per clock per SM) is the narrower bound
        logits = work_stage[0]["xi"] / (2.0 * wl.head_dim)
        sfu_peak = 16.0 * 148 * 1.965e9
        roofline["sfu"] = {"achieved_exp_per_s": logits / (kstage[0]["xi"] / 1e3), "peak_exp_per_s": sfu_peak,
                           "frac": round(logits / (kstage[0]["xi"] / 1e3) / sfu_peak, 4),
                           "note": "16 ex2/clk/SM x 148 SMs x 1.965 GHz"}

    # end to end through the public API with host buffers: H2D of every stage's inputs from pinned
    # memory, the step, D2H of every stage's results
    e2e = None
    if not args.no_e2e:
        h2d = sum(t.numel() * t.element_size() for s in stages for t in s["host"].values())
        d2h = sum(t.numel() * t.element_size() for s in stages for t in s["host_out"].values())

        cin, cout = torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
        kv_side = side if side is not None else torch.cuda.current_stream()

        def e2e_step():
            """One step from pinned host inputs to pinned host outputs: every stage's inputs go up on a copy
            stream while earlier stages compute, results come down on another as soon as they exist."""
            main = torch.cuda.current_stream()
            cin.wait_stream(main)                       # the previous step no longer reads the device inputs
            ready = []
            with torch.cuda.stream(cin):
                for s in stages:
                    for name, t in s["host"].items():
                        s["dev"][name].copy_(t, non_blocking=True)
                    e = torch.cuda.Event()
                    e.record(cin)
                    ready.append(e)
            pos, n_vis = stages[0]["dev"]["pos"], stages[0]["dev"]["n_vis"]
            for st, s in enumerate(stages):
                main.wait_event(ready[st])
                run_stage(L, plan, wl, st, s, pos, n_vis, side=side, aux=aux)
                cout.wait_stream(main)
                cout.wait_stream(kv_side)
                with torch.cuda.stream(cout):
                    s["host_out"]["hidden"].copy_(s["out"].hidden_out, non_blocking=True)
                    s["host_out"]["k"].copy_(s["k_dst"], non_blocking=True)
                    s["host_out"]["v"].copy_(s["v_dst"], non_blocking=True)
                    s["host_out"]["n_vis_out"].copy_(s["out"].n_vis_out, non_blocking=True)
                    s["host_out"]["pos_out"].copy_(s["out"].pos_out, non_blocking=True)
                pos, n_vis = s["out"].pos_out, s["out"].n_vis_out
            if side is not None:
                main.wait_stream(side)
            main.wait_stream(cout)
        e2e_steps = max(3, min(args.steps, 10))
        for _ in range(2):
            e2e_step()
        barrier()
        a, b = ev(), ev()
        a.record()
        for _ in range(e2e_steps):
            e2e_step()
        b.record()
        barrier()
        ms_e2e = max_over_ranks(a.elapsed_time(b) / e2e_steps, world, device)
        e2e = {"value": whole_job_throughput(tokens_per_step, world, ms_e2e), "unit": unit, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        per_stage = oracle_sample_inputs(wl)                 # generated once, outside every timed interval
        t, tok = oracle_sample_run(wl, per_stage, range(n_stages))
        cpu = {"value": tok / t, "unit": unit, "cores": blas_threads(), "kind": "oracle",
               "sample": f"sample 0 of {wl.batch}, all {n_stages} stages ({tok} vision tokens, {t:.1f} s)"}
        # the same oracle held to one thread, on the last stage of sample 0 (the smallest; bounded CPU time)
        try:
            from threadpoolctl import threadpool_limits
            with threadpool_limits(limits=1):
                t1, tok1 = oracle_sample_run(wl, per_stage, [n_stages - 1])
            cpu["one_thread"] = {"value": tok1 / t1, "unit": unit, "cores": 1,
                                 "sample": f"sample 0 of {wl.batch}, last stage only ({tok1} vision tokens, {t1:.1f} s)"}
        except Exception as exc:      # noqa: BLE001
            cpu["one_thread"] = {"unavailable": str(exc)}
        # the plain C oracle (one thread by construction) on the same last stage of sample 0
        try:
            cpu["c_oracle_one_thread"] = c_oracle_sample(wl, unit, per_stage)
        except Exception as exc:      # noqa: BLE001
            cpu["c_oracle_one_thread"] = {"unavailable": str(exc)}

    if rank == 0:
        # per stage: window build, xi (+ its second launch for rows that left the fp32 range; none with a given
        # log-sum-exp), FD, selection, hidden merge, K/V compaction (+ the move kernel when in place)
        launches_per_step = n_stages * (6 + (1 if args.xi_mode == "full" else 0) + (1 if args.kv_in_place else 0))
        line = {"metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": config,
                "us_per_compression_layer": 1e3 * ms_step / n_stages,
                "schedule": ("streams: window build + FD beside xi inside lightkv_compress_layer (aux_stream); "
                             "lightkv_compact_kv of stage i behind the stage's map event, beside its hidden-state merge and lightkv_compress_layer of stage i+1"
                             if side is not None else "one stream"),
                "cuda_graph": step_graph is not None,
                "ms_per_step_one_stream": ms_step_one_stream,
                "ms_per_step_one_stream_graph": ms_one_stream_graph,
                "per_kernel_note": ("kernels / us_by_stage / roofline come from the one-stream pass with an event after "
                                    "every launch (ms_per_step_one_stream); ms_per_step_one_stream_graph is the same "
                                    "schedule without those events"),
                "roofline": roofline, "kernels": kernels,
                "us_by_stage": [{k: round(1e3 * v, 1) for k, v in ks.items()} for ks in kstage], "cpu_baseline": cpu, "e2e": e2e, "clocks": clocks,
                "gpu_launches": launches_per_step * args.steps,
                "engine": {st: int(plan.stage_info(st).uses_tensor_cores) for st in range(n_stages)}}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
