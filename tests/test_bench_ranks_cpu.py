"""The N>1 logic of bench.py on CPU: two gloo ranks, distinct per-rank batches, MAX-over-ranks timing,
whole-job aggregation.  (The data path itself has no collective: heads are independent.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2608_01563_b200 import inputs as synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.WORKLOADS["tiny"]
    wr = bench.rank_workload(w, rank)
    q = synth.make_inputs(wr)[0]
    # each rank reports a different time; everyone must end up with the maximum
    mx = bench.max_over_ranks([10.0 + rank, 5.0 - rank], dist, "cpu")
    out[rank] = (wr.seed, float(q.sum()), mx, bench.whole_job_tflops(w, world, 4, mx[0]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_batches_and_take_max_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29000 + os.getpid() % 2000
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    (s0, q0, m0, v0), (s1, q1, m1, v1) = out[0], out[1]
    assert s0 != s1 and q0 != q1                  # different batches per rank
    assert m0 == m1 == [11.0, 5.0]                # MAX over ranks, on every rank
    import bench
    from paper_2608_01563_b200 import inputs as synth
    w = synth.WORKLOADS["tiny"]
    assert v0 == v1
    assert abs(v0 - 2 * bench.flops(w, "sum") * 4 / 11e-3 / 1e12) < 1e-12 * v0 + 1e-30


def test_flop_convention():
    import bench
    from paper_2608_01563_b200 import inputs as synth
    w = synth.WORKLOADS["gpt2_small"]
    assert abs(bench.flops(w, "fwd") / 1e9 - 12.885) < 0.01       # 4 * 96 * 1024^2/2 * 64
    assert abs(bench.flops(w, "bwd") / bench.flops(w, "fwd") - 2.5) < 1e-12
    w = synth.WORKLOADS["long_context"]
    assert abs(bench.flops(w, "sum") / 1e9 - 481.0) < 0.1
