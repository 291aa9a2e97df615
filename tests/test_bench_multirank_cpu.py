"""The N > 1 plumbing of the benchmark (replicas only: barrier, max-over-ranks time, summed
units, distinct seeds per rank) on CPU with gloo, world size 2."""
import os

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2112_04291_b200 import multirank, workloads


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, w, lr = multirank.env_rank()
    assert (r, w, lr) == (rank, world, rank)
    multirank.init("gloo")
    multirank.barrier(w, cuda=False)
    # each rank draws its own replica's gradients
    wl = workloads.make("c1", n=4096, workers=2, seed=multirank.rank_seed(r))
    digest = float(np.abs(wl.grads[0]).sum())
    ms_local = 10.0 * (rank + 1)            # rank 1 is the slow one
    units_local = 4.0 * wl.n * wl.workers
    rate, ms = multirank.job_throughput(units_local, ms_local, w)
    mx = multirank.max_over_ranks(digest, w)
    sm = multirank.sum_over_ranks(digest, w)
    out.put((rank, rate, ms, digest, mx, sm))
    multirank.barrier(w, cuda=False)
    torch.distributed.destroy_process_group()


def test_two_ranks_gloo():
    world, port = 2, 29533
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, rate0, ms0, d0, mx0, sm0), (r1, rate1, ms1, d1, mx1, sm1) = res
    assert ms0 == ms1 == 20.0                                  # the slowest rank's time
    assert rate0 == rate1 == (2 * 4.0 * 4096 * 2) / 20e-3      # units of both ranks over that time
    assert d0 != d1                                            # distinct seeds per rank
    assert mx0 == mx1 == max(d0, d1) and abs(sm0 - (d0 + d1)) < 1e-9


def test_single_process_defaults():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert multirank.env_rank() == (0, 1, 0)
    assert multirank.job_throughput(100.0, 5.0, 1) == (100.0 / 5e-3, 5.0)
    assert multirank.rank_seed(3) == 3000
