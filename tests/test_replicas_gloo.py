"""The N > 1 layout (independent replicas; only a MAX over per-rank times) on CPU with gloo, world_size 2."""
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
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2609_36062_b200 import replicas
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        seconds = 0.5 if rank == 0 else 2.0                 # rank 1 is the slow one
        tmax = replicas.max_over_ranks([seconds, 10.0 - rank])
        value = replicas.aggregate_throughput(units_per_rank=1000.0, seconds_this_rank=seconds)
        heads = list(replicas.head_slice(7, rank, world))
        out.put((rank, tmax, value, heads))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_disjoint_heads():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, tmax0, v0, h0), (r1, tmax1, v1, h1) = results
    assert tmax0 == tmax1 == [2.0, 10.0]                    # element-wise max over ranks, same on every rank
    assert v0 == v1 == 2 * 1000.0 / 2.0                     # all units / slowest time
    assert sorted(h0 + h1) == list(range(7)) and not set(h0) & set(h1)


def test_single_process_is_the_identity():
    from paper_2609_36062_b200 import replicas
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.aggregate_throughput(10.0, 2.0) == 5.0
    assert list(replicas.head_slice(5, 0, 1)) == [0, 1, 2, 3, 4]
