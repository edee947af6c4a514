"""World-size-2 check (gloo, CPU) of the one exchange step of a head-sharded layer: the mean over ranks of the
per-rank attention-sink scores (Eq. 6 is a mean over all heads), and the dealing out of heads to ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import focus_oracle as fo
from paper_2602_02159_b200 import head_shards, workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs():
    s = wl.Shape(640, 512, 8, 4, 64, 64, "f32")
    t = wl.gen_qkv(s, 77, threads=1)
    active = np.array([3, 4, 5, 40, 41, 90], dtype=np.int64) + s.M
    return s, t, active


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    s, t, active = _inputs()
    qh, kvh = head_shards.local_heads(s.H, s.Hkv, rank, world)
    # this rank's S over its own heads (here by the oracle: the test is about the exchange, not about the kernels)
    Q = wl.storage_to_f64(t["Q"], s.dtype)[active - s.M][:, qh]
    K = wl.storage_to_f64(t["K"], s.dtype)[kvh]
    S_local = torch.from_numpy(fo.sink_scores(Q, K, 1.0 / np.sqrt(s.d)).astype(np.float32))
    S = head_shards.mean_over_ranks(S_local.clone())
    out.put((rank, S.numpy()))
    dist.barrier()
    dist.destroy_process_group()


def test_mean_of_the_ranks_scores_is_the_score_over_all_heads():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert np.array_equal(res[0], res[1]), "every rank must hold the same averaged scores"
    s, t, active = _inputs()
    S_all = fo.sink_scores(wl.storage_to_f64(t["Q"], s.dtype)[active - s.M], wl.storage_to_f64(t["K"], s.dtype),
                           1.0 / np.sqrt(s.d))
    assert np.abs(res[0] - S_all).max() <= 1e-6 * S_all.max()
    # and so is the sink set (no candidate of this case sits within rounding of the threshold)
    n_sink = 6
    assert fo.find_sinks(res[0].astype(np.float64), n_sink, 0, s.M).tolist() == fo.find_sinks(S_all, n_sink, 0, s.M).tolist()


def test_heads_are_dealt_out_in_whole_kv_groups():
    assert head_shards.local_heads(32, 8, 0, 4) == (slice(0, 8), slice(0, 2))
    assert head_shards.local_heads(32, 8, 3, 4) == (slice(24, 32), slice(6, 8))
    assert head_shards.local_heads(28, 4, 1, 2) == (slice(14, 28), slice(2, 4))
    assert head_shards.local_heads(8, 8, 0, 1) == (slice(0, 8), slice(0, 8))
    with pytest.raises(ValueError):
        head_shards.local_heads(28, 4, 0, 3)


def test_without_a_process_group_the_scores_stay_as_they_are():
    x = torch.arange(5, dtype=torch.float32)
    assert head_shards.mean_over_ranks(x.clone()).equal(x)
