"""Host logic of the multi-GPU bench path on CPU: two gloo ranks take disjoint scenario ranges and agree on the
maximum step time (no collective touches the data path)."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import bench


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    S = 8
    w = bench.make_workload("c4", S, rank * S, 28)
    first = w.first_scenario
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    x = w.host_inputs([0])
    out.put((rank, first, ms, int(x.view(np.uint32).sum()), bench.whole_job_value(world, S, ms)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_disjoint_scenarios_and_max_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, f0, ms0, h0, v0), (r1, f1, ms1, h1, v1) = res
    assert (f0, f1) == (0, 8) and h0 != h1                  # disjoint scenario ranges, different inputs
    assert ms0 == ms1 == 15.0                               # the slower rank's time on both
    assert v0 == v1 == 2 * 8 / 15e-3                        # whole-job scenarios per second
