"""The benchmark's cross-rank plumbing on CPU: two gloo ranks, barrier + maximum of a timing over the ranks.
The path does not shard (replicas only), so this is all that ever crosses ranks."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench
    r = bench.Ranks("gloo")
    assert (r.rank, r.world) == (rank, world)
    r.barrier()
    got = [r.reduce_max(10.0 * (rank + 1) + k) for k in range(3)]     # the slowest rank's time is the reported one
    r.barrier()
    r.close()
    out.put((rank, got))


def test_two_gloo_ranks_report_the_maximum_over_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(rk, 2, port, out)) for rk in range(2)]
    for p in procs:
        p.start()
    res = dict(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [20.0, 21.0, 22.0]


def test_a_single_rank_needs_no_process_group():
    for k in ("RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    sys.path.insert(0, ROOT)
    import bench
    r = bench.Ranks("gloo")
    assert r.world == 1 and r.reduce_max(3.5) == 3.5
    r.barrier()
    r.close()
