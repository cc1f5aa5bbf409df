"""Row-block sharding over 2 gloo ranks on CPU: the union of the per-rank joins, shifted by
each rank's row offset, is the whole join (Theorem 1's block decomposition).  The per-rank
join here is the CPU oracle -- this test covers the host-side sharding logic only."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2006_12608_b200 import sharding
from paper_2006_12608_b200 import workloads as W


def test_row_blocks_partition_the_rows():
    for n in (0, 1, 7, 128, 1000):
        for world in (1, 2, 3, 8):
            blocks = [sharding.row_block(n, world, r) for r in range(world)]
            assert blocks[0][0] == 0 and sum(b[1] for b in blocks) == n
            for (s0, c0), (s1, _c1) in zip(blocks, blocks[1:]):
                assert s0 + c0 == s1
            assert max(b[1] for b in blocks) - min(b[1] for b in blocks) <= 1
    with pytest.raises(ValueError):
        sharding.row_block(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    from oracle import simjoin_oracle as O
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.make_workload(4, n=1001, m=700, planted=60)          # every rank draws the same inputs
        start, rows = sharding.row_block(w.n, world, rank)
        local, cnt = O.join(w.P[start:start + rows], w.Q, w.kind, w.threshold, w.dtype, threads=1)
        local = local + np.array([start, 0], dtype=np.int32)         # what simjoin_set_offsets does on the GPU
        counts = sharding.exchange_counts(cnt)
        allp = sharding.gather_pairs(torch.from_numpy(local), counts).numpy()
        whole, wcnt = O.join(w.P, w.Q, w.kind, w.threshold, w.dtype, threads=1)
        ok = sum(counts) == wcnt and np.array_equal(allp, whole) and counts[rank] == cnt
        q.put((rank, bool(ok), counts))
    finally:
        dist.destroy_process_group()


def test_two_rank_sharded_join_equals_whole_join():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(ok for (_r, ok, _c) in results), results
    assert results[0][2] == results[1][2] and min(results[0][2]) > 0
