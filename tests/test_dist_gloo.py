"""CPU (gloo) tests of the multi-GPU host logic with 2 and 3 ranks: head slicing, gather in head
order, max- and sum-over-ranks reductions.  Each rank runs, for its slice of the heads, the
oracle's whole per-head plan (guard, Algorithm 1, Eq. 4, Algorithm 2) in place of the GPU plan
- the path has no data-path collective, so the gathered result must equal what one process
computes for all heads, also when the heads do not divide evenly."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from paper_2609_34814_b200 import dist as wd


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


ROWS = 64


def _plan_of_head(h):
    """Planned row order of head h of the small 64-block config (every step of the plan)."""
    from oracle import waveal_oracle as wo
    from paper_2609_34814_b200 import inputs as I
    cfg = I.CONFIGS["tiny"]
    mask = I.make_mask(cfg, h)
    assert mask.shape[0] == ROWS
    return wo.plan_head(mask, 16, 5, cfg.plan_seed, h, mode=wo.MODE_FORCE_REORDER)["row_order"]


def _worker(rank, world, port, total_heads, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from oracle import waveal_oracle as wo
    wd.init(backend="gloo")
    mine = wd.head_slice(rank, world, total_heads)
    local = [_plan_of_head(h) for h in mine]
    local = torch.from_numpy(np.stack(local)) if local else torch.zeros((0, ROWS), dtype=torch.int64)
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


@pytest.mark.parametrize("world,total", [(2, 5), (3, 40)])
def test_head_split_over_gloo_ranks(world, total):
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
    expect = np.stack([_plan_of_head(h) for h in range(total)])       # what a single process computes
    assert len({tuple(r) for r in expect.tolist()}) > 1               # heads differ, so the order is checked
    for rank, full, t, s, mine in res:
        assert np.array_equal(full, expect)
        assert t == float(world) and s == float(total)
    assert sorted(h for r in res for h in r[4]) == list(range(total))
