"""World-size-2 CPU (gloo) test of the multi-GPU host logic: head slicing, gather in head
order, max-over-ranks timing reduction.  The per-head work stands in for the GPU plan by the
oracle's Stage 2 (any per-head function works: the path has no data-path collective)."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2609_34814_b200 import dist as wd


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, total_heads, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from oracle import waveal_oracle as wo
    wd.init(backend="gloo")
    mine = wd.head_slice(rank, world, total_heads)
    rng_rows = 24
    local = []
    for h in mine:
        nnz = np.random.default_rng(h).integers(1, 9, size=rng_rows)
        local.append(wo.stage2_order(np.arange(rng_rows), nnz, 8))
    local = torch.from_numpy(np.stack(local)) if local else torch.zeros((0, rng_rows), dtype=torch.int64)
    full = wd.gather_heads(local, total_heads)
    t = wd.max_over_ranks(1.0 + rank)
    s = wd.sum_over_ranks(float(len(mine)))
    wd.barrier()
    q.put((rank, full.numpy(), t, s, list(mine)))
    wd.shutdown()


def test_head_slice_partitions():
    for total in (1, 5, 40, 41):
        for world in (1, 2, 3, 8):
            got = [h for r in range(world) for h in wd.head_slice(r, world, total)]
            assert got == list(range(total))
            sizes = [len(wd.head_slice(r, world, total)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_gloo():
    from oracle import waveal_oracle as wo
    world, total = 2, 5
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, total, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    expect = np.stack([wo.stage2_order(np.arange(24), np.random.default_rng(h).integers(1, 9, size=24), 8)
                       for h in range(total)])
    for rank, full, t, s, mine in res:
        assert np.array_equal(full, expect)
        assert t == 2.0 and s == float(total)
    assert sorted(h for r in res for h in r[4]) == list(range(total))
