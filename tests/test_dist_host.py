"""Host-side multi-process logic on CPU (gloo, world_size 2): every rank runs its own units, the step time
is the max over ranks and the job's throughput the units of all ranks over that time.  No GPU and no
data-path collective is involved."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_09307_b200.dist import aggregate_throughput, max_over_ranks


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        units = 16 + rank                                 # the ranks' own batches
        step_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
        tmax = max_over_ranks(step_ms)
        thr = aggregate_throughput(units, tmax * 1e-3)
        out.put((rank, units, tmax, thr))
    finally:
        dist.destroy_process_group()


def test_two_ranks_agree_on_max_time_and_total_throughput():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [16, 17]
    assert all(abs(r[2] - 15.0) < 1e-9 for r in res)       # max over ranks
    assert all(abs(r[3] - 33 / 15e-3) < 1e-6 for r in res) # all units / slowest time
