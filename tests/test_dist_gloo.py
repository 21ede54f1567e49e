"""world_size-2 gloo run of the multi-GPU plumbing on CPU: worker sharding, the barrier and the
max-over-ranks clock that bench.py uses; each rank runs the oracle on its own workers and the union must
equal the single-process result (the data path has no collective)."""
import os
import sys

import numpy as np
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, size, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(size), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from oracle import kimad_oracle as ko
    from paper_2312_08053_b200 import dist as kd
    from paper_2312_08053_b200 import workloads

    kd.init_distributed("gloo")
    wl = workloads.workload(2, 256, n_workers=5)
    mine = kd.shard_workers(wl.n_workers, rank, size)
    grads = workloads.gradients(wl, 0, workers=mine).numpy()
    bw = workloads.bandwidth_trace(wl, 4)[2][mine]
    kd.barrier()
    r = ko.step(wl.layer_sizes, len(mine), wl.ratio_grid, wl.D, 0, grads, np.zeros_like(grads), bw, wl.t_target)
    kd.barrier()
    slowest = kd.max_over_ranks(10.0 + rank)
    q.put((rank, mine, r.k.tolist(), slowest))
    import torch.distributed as dist

    dist.destroy_process_group()


def test_two_rank_gloo_sharding_and_clock():
    from oracle import kimad_oracle as ko
    from paper_2312_08053_b200 import dist as kd
    from paper_2312_08053_b200 import workloads

    assert kd.shard_workers(5, 0, 2) == [0, 1, 2] and kd.shard_workers(5, 1, 2) == [3, 4]
    assert sum((kd.shard_workers(7, r, 3) for r in range(3)), []) == list(range(7))
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=240) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = workloads.workload(2, 256, n_workers=5)
    grads = workloads.gradients(wl, 0).numpy()
    ref = ko.step(wl.layer_sizes, 5, wl.ratio_grid, wl.D, 0, grads, np.zeros_like(grads),
                  workloads.bandwidth_trace(wl, 4)[2], wl.t_target)
    merged = got[0][2] + got[1][2]
    assert merged == ref.k.tolist()
    assert got[0][3] == got[1][3] == 11.0  # every rank sees the slowest rank's time
