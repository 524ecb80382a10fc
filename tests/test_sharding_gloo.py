"""Replica sharding over processes, on CPU with the gloo backend (world size 2).

Each rank runs the oracle on its slice of the replicas with `replica_offset` set; results
and summed counters must equal one process running all replicas.
"""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import Oracle
from paper_2603_20661_b200 import synth
from paper_2603_20661_b200.sharding import max_over_ranks, replica_shard, sum_counters
from tests.helpers import run_workload


def test_replica_shard_partitions():
    for n, w in ((16, 8), (5, 2), (3, 4), (256, 3)):
        got = [replica_shard(n, w, r) for r in range(w)]
        assert got[0][0] == 0 and sum(c for _, c in got) == n
        for (o1, c1), (o2, _) in zip(got, got[1:]):
            assert o1 + c1 == o2
        assert max(c for _, c in got) - min(c for _, c in got) <= 1


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = synth.make_workload("zipf1k", n_replicas=5, n_requests=1500, n_peers=96)
    off, cnt = replica_shard(5, world, rank)
    part = synth.slice_replicas(wl, off, off + cnt)
    o = Oracle(part.settings, part.peers); o.bind_requests(part.requests)
    run_workload(o, part)
    tot = sum_counters(o.stats()[-1])
    t = max_over_ranks(float(rank + 1))
    q.put((rank, off, cnt, o.results()["exec_a"], o.table("credit"), tot, t))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_one_process():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]; s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=120) for _ in procs], key=lambda g: g[0])
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    wl = synth.make_workload("zipf1k", n_replicas=5, n_requests=1500, n_peers=96)
    o = Oracle(wl.settings, wl.peers); o.bind_requests(wl.requests)
    run_workload(o, wl)
    full = o.results()["exec_a"]; credit = o.table("credit")
    for rank, off, cnt, ex, cr, tot, t in got:
        assert np.array_equal(ex, full[off:off + cnt]) and np.array_equal(cr, credit[off:off + cnt])
        assert np.array_equal(tot, o.stats()[-1])
        assert t == 2.0
