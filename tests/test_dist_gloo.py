"""Multi-process host logic of the benchmark (replicas, max-over-ranks) on CPU with gloo."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2609_35140_b200 import dist as tdist
from paper_2609_35140_b200 import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, lr, w = tdist.init("gloo")
    assert (r, w) == (rank, world)
    tdist.barrier()
    agg = tdist.max_over_ranks({"train": 1.0 + rank, "decode0": 5.0 - rank, "total": 10.0})
    tot = tdist.sum_over_ranks(100.0 * (rank + 1))
    wl = synth.get_workload(0)
    q0, _, _, _ = synth.make_qkv(wl, "cpu", tdist.replica_seed_offset(rank))
    out.put((rank, agg, tot, float(q0.float().sum())))
    tdist.barrier()
    tdist.finalize()


def test_two_ranks_reduce_and_draw_distinct_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, agg, tot, _ in res:
        assert agg == {"decode0": 5.0, "total": 10.0, "train": 2.0}
        assert tot == 300.0
    assert res[0][3] != res[1][3]          # replicas hold different data of the same shape


def test_shard_sequences_is_a_partition():
    for n in (1, 7, 16, 64, 256):
        for world in (1, 2, 3, 8):
            parts = [tdist.shard_sequences(n, r, world) for r in range(world)]
            flat = [i for p in parts for i in p]
            assert flat == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1


def test_single_process_is_identity():
    assert tdist.max_over_ranks({"a": 3.0}) == {"a": 3.0}
    assert tdist.sum_over_ranks(2.5) == 2.5
    assert tdist.env_world()[2] >= 1
