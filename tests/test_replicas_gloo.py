"""World-size-2 check (gloo, CPU) of the benchmark's multi-rank plumbing: rendezvous, distinct replica inputs,
barrier and max-over-ranks of the per-rank time."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2602_02159_b200 import replicas, workloads as wl
    r, w, _ = replicas.init("gloo")
    assert (r, w) == (rank, world)
    s = wl.Shape(256, 192, 2, 2, 64, 64, "bf16")
    t = wl.gen_qkv(s, replicas.replica_seed(5, rank), threads=1)
    replicas.barrier()
    slowest = replicas.max_over_ranks(10.0 + 3.0 * rank)          # rank 1 is the slow one
    out.put((rank, slowest, int(t["K"].astype(np.int64).sum())))
    replicas.barrier()
    replicas.shutdown()


def test_two_replicas_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    assert all(abs(r[1] - 13.0) < 1e-12 for r in res)             # every rank reports the slowest rank's time
    assert res[0][2] != res[1][2]                                 # replicas hold different inputs


def test_single_process_is_a_no_op():
    from paper_2602_02159_b200 import replicas
    assert replicas.max_over_ranks(4.5) == 4.5
    assert replicas.replica_seed(7, 0) == 7 and replicas.replica_seed(7, 3) == 3007
    replicas.barrier()
