"""The N > 1 benchmark path ("replicas only") on CPU: two gloo ranks aggregate their timings."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2505_13544_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    units, ms = replicas.aggregate(100.0 * (rank + 1), 5.0 + 3.0 * rank)
    per_s, ms2 = replicas.throughput(100.0 * (rank + 1), 5.0 + 3.0 * rank)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, units, ms, per_s, ms2))


def test_two_rank_aggregation():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, units, ms, per_s, ms2 in results:
        assert units == 300.0            # sum of the ranks' tokens
        assert ms == ms2 == 8.0          # slowest rank's time
        assert per_s == 300.0 / 8e-3


def test_single_process_is_identity():
    assert replicas.aggregate(7.0, 2.0) == (7.0, 2.0)
    assert replicas.throughput(10.0, 500.0) == (20.0, 500.0)
