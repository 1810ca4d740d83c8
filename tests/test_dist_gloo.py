"""world_size-2 gloo test (CPU) of the multi-GPU plumbing: disjoint session shards, barrier, max over ranks."""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2609_17652_b200 import dist as fdist
    r, w, _ = fdist.init_from_env(world, backend="gloo")
    mine = fdist.sessions_of_rank(r, w, 16)
    fdist.barrier()
    slowest = fdist.max_over_ranks(10.0 + r)          # rank 1 is "slower"
    total = fdist.sum_over_ranks(float(len(mine)))
    fdist.barrier()
    fdist.shutdown()
    q.put((r, mine, slowest, total))


def test_two_ranks_shard_sessions_and_reduce_times():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    (r0, s0, m0, t0), (r1, s1, m1, t1) = res
    assert sorted(s0 + s1) == list(range(16)) and not set(s0) & set(s1)
    assert m0 == m1 == 11.0 and t0 == t1 == 16.0


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    from paper_2609_17652_b200 import dist as fdist
    assert fdist.max_over_ranks(3.5) == 3.5
    assert fdist.sessions_of_rank(0, 1, 4) == [0, 1, 2, 3]
    fdist.barrier()
