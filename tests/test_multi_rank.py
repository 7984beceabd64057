"""The N > 1 path of the benchmark on CPU: two gloo ranks.

The compression step has no exchange between samples, so several GPUs only ever mean "every rank takes
its own batch".  What is multi-rank is the protocol around it: which samples a rank draws, the
max-over-ranks timing and the whole-job throughput.  Those run here as two processes over gloo."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    import lightkv_synth as S
    wl = S.workload("tiny")
    samples = bench.rank_samples(rank, wl.batch)
    inp = S.make_layer_inputs(wl, 0, samples=samples, tensors=("hidden",))
    digest = float(np.abs(inp["hidden"]).sum())
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)            # rank 1 is the slow one
    gathered = [None] * world
    dist.all_gather_object(gathered, (samples, digest))
    dist.barrier()
    if rank == 0:
        torch.save({"ms": ms, "gathered": gathered,
                    "value": bench.whole_job_throughput(1000, world, ms)}, out)
    dist.destroy_process_group()


def test_two_ranks_take_disjoint_batches_and_time_by_the_slowest(tmp_path):
    out = str(tmp_path / "r0.pt")
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    res = torch.load(out, weights_only=False)
    assert res["ms"] == 15.0                                        # max over ranks, not rank 0's own 10 ms
    assert res["value"] == 2 * 1000 / 15e-3                         # both ranks' tokens over the slowest time
    (s0, d0), (s1, d1) = res["gathered"]
    assert s0 == [0, 1] and s1 == [2, 3]                            # disjoint, consecutive sample ids
    assert d0 != d1                                                 # different samples -> different tensors


def test_single_rank_is_the_identity():
    import bench
    assert bench.max_over_ranks(3.25, 1) == 3.25
    assert bench.rank_samples(0, 4) == [0, 1, 2, 3]
