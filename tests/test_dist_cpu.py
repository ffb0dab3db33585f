"""Multi-rank plumbing on CPU (gloo, world_size 2): max-over-ranks timing and batch sharding."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2012_00596_b200 import dist as npd


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, lr, w = npd.init("gloo")
    npd.barrier()
    ms = 10.0 if rank == 0 else 25.0                 # rank 1 is the slow replica
    value, ms_step = npd.whole_job_throughput(units_per_rank_step=3.0, steps=5, ms_local=ms)
    q.put((rank, r, w, npd.max_over_ranks(ms), value, ms_step))
    torch.distributed.destroy_process_group()


def test_two_rank_aggregation():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, r, w, mx, value, ms_step in res:
        assert r == rank and w == 2 and mx == 25.0
        assert abs(value - (3.0 + 3.0) * 5 / 0.025) < 1e-6 and abs(ms_step - 5.0) < 1e-9


def test_shard_batch_covers_everything_once():
    for n, world in [(32, 2), (64, 8), (7, 4), (3, 8)]:
        spans = [npd.shard_batch(n, r, world) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == n
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        assert max(hi - lo for lo, hi in spans) - min(hi - lo for lo, hi in spans) <= 1


def test_single_rank_is_identity():
    assert npd.max_over_ranks(3.5) == 3.5 and npd.sum_over_ranks(2.0) == 2.0
