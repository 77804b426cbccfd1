"""Host logic of multi-GPU runs (independent replicas), on CPU with the gloo backend, world size 2."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2402_11131_b200 import replicas, workloads as W
    # every rank runs the same seeded workload (a replica): identical inputs, no exchange on the path
    st = W.make_step(W.CONFIGS["tiny"])
    digest = int(st.layer(0).k_cache.astype("int64").sum())
    seconds = [0.002, 0.005][rank]                       # rank 1 is the slow replica
    slowest = replicas.max_over_ranks(seconds)
    total = replicas.aggregate_throughput(1000.0, seconds)
    out.put((rank, replicas.world_size(), slowest, total, digest))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_agree_on_the_slowest_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    rows = [out.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    rows.sort()
    assert [r[1] for r in rows] == [2, 2]
    assert all(abs(r[2] - 0.005) < 1e-12 for r in rows)              # max over ranks, on both ranks
    assert all(abs(r[3] - 2 * 1000.0 / 0.005) < 1e-6 for r in rows)  # all ranks' units / slowest time
    assert rows[0][4] == rows[1][4]                                  # replicas: the same seeded inputs


def test_single_process_is_the_identity():
    from paper_2402_11131_b200 import replicas
    assert replicas.world_size() == 1
    assert replicas.max_over_ranks(0.25) == 0.25
    assert replicas.aggregate_throughput(10.0, 0.5) == 20.0
