"""The N > 1 path of the benchmark is "replicas only": no data-path collective, one reduction of the
timings at the end.  Checked with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2504_12329_b200 import workloads as W
    w = bench.rank_workload(W.CONFIGS["tiny_pair"], rank)
    prompt, force = W.workload_inputs(w)
    # rank r "ran" for (1 + r) seconds and wrote 100 * (r + 1) tokens
    dev_s, e2e_s, n = bench.aggregate_over_ranks(1.0 + rank, 2.0 + rank, 100.0 * (rank + 1), dist, "cpu")
    out.put((rank, w.input_seed, prompt[:4].tolist(), int((force >= 0).sum()), dev_s, e2e_s, n))
    dist.destroy_process_group()


def test_two_gloo_ranks_replicas_only():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, seed0, p0, f0, d0, e0, n0), (r1, seed1, p1, f1, d1, e1, n1) = res
    assert seed0 != seed1 and p0 != p1                 # independent replicas
    assert f0 > 0 and f1 > 0
    assert (d0, e0, n0) == (d1, e1, n1) == (2.0, 3.0, 300.0)   # max of the times, sum of the tokens


def test_single_process_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(1.5, 2.5, 10.0) == (1.5, 2.5, 10.0)
