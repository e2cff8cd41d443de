"""The multi-GPU plan on CPU: two gloo ranks own disjoint contexts that together cover all, generate different
synthetic contexts, agree on the reduced (maximum) time, and would report the same aggregate."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2403_11805_b200 import sharding, synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = sharding.contexts_of_rank(64, rank, world)
    sh = synth.KVShape("t", 1, 1, 1, 16, 32, 16, 16, seed=1)
    sig = float(synth.kv_tensor(sh, context=mine[0]).float().sum())            # this rank's first context
    ms = sharding.max_over_ranks([1.0 + rank, 5.0 - rank], dist)
    gathered = [None] * world
    dist.all_gather_object(gathered, (mine, sig, ms))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_contexts_and_reduce_times():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (m0, s0, t0), (m1, s1, t1) = gathered
    assert sorted(m0 + m1) == list(range(64)) and not set(m0) & set(m1)
    assert m0[:3] == [0, 2, 4] and m1[:3] == [1, 3, 5]
    assert s0 != s1                       # different contexts, different data
    assert t0 == t1 == [2.0, 5.0]         # both ranks hold the maximum


def test_single_rank_is_the_identity():
    assert sharding.contexts_of_rank(5, 0, 1) == [0, 1, 2, 3, 4]
    assert sharding.max_over_ranks([3.5]) == [3.5]
