"""World-size-2 checks (gloo, CPU) of the only multi-rank logic: sharding independent sequences over ranks and
reducing timings/totals.  There is no data-path collective."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_09649_b200 import dist_util, workloads


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, batch, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, _, w = dist_util.init("gloo")
    lo, hi = workloads.shard_sequences(batch, r, w)
    dist_util.barrier()
    ms = dist_util.max_over_ranks(10.0 + r)          # slowest rank defines the step time
    total = dist_util.sum_over_ranks(hi - lo)        # units processed by the whole job
    q.put((r, lo, hi, ms, total))
    dist.destroy_process_group()


def test_sequences_shard_without_overlap_world2():
    for batch in (8, 5):
        ctx = mp.get_context("spawn")
        q = ctx.Queue()
        port = _free_port()
        procs = [ctx.Process(target=_worker, args=(r, 2, port, batch, q)) for r in range(2)]
        for p in procs:
            p.start()
        res = sorted(q.get(timeout=120) for _ in procs)
        for p in procs:
            p.join(60)
            assert p.exitcode == 0
        (r0, lo0, hi0, ms0, t0), (r1, lo1, hi1, ms1, t1) = res
        assert lo0 == 0 and hi0 == lo1 and hi1 == batch and abs((hi0 - lo0) - (hi1 - lo1)) <= 1
        assert ms0 == ms1 == 11.0 and t0 == t1 == batch


def test_shard_covers_all_sequences_any_world():
    for batch in (1, 4, 7, 32):
        for world in (1, 2, 3, 4, 8):
            spans = [workloads.shard_sequences(batch, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == batch
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
