"""World-size-2 gloo test of the host-side multi-GPU logic (sharding and timing reduction)."""
import os
import socket

import torch.multiprocessing as mp

from paper_2104_08378_b200 import distributed as D


def test_shard_range_covers_everything_once():
    for total, world, mult in [(8192, 2, 16), (8192, 8, 16), (100, 3, 16), (48, 8, 16), (0, 2, 16)]:
        seen = []
        for r in range(world):
            b, e = D.shard_range(total, r, world, mult)
            assert b % mult == 0 and b <= e <= total
            seen.append((b, e))
        assert seen[0][0] == 0 and seen[-1][1] == total
        assert all(seen[i][1] == seen[i + 1][0] for i in range(world - 1))


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, _, w = D.init("gloo")
    D.barrier()
    mx = D.max_over_ranks(1.0 + rank)          # slowest rank decides the step time
    sm = D.sum_over_ranks(10.0 * (rank + 1))   # units processed by all ranks
    b, e = D.shard_range(8192, r, w, 16)
    out.put((rank, mx, sm, b, e))
    D.barrier()


def test_gloo_world_size_2():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 2.0, 30.0, 0, 4096), (1, 2.0, 30.0, 4096, 8192)]
