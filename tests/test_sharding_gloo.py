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


def _head_worker(rank, world, port, out):
    import numpy as np
    import oracle
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sh = synth.KVShape("tp", 2, 4, 8, 32, 96, 16, 32, seed=3)     # 2 layers, 4 KV heads read by 8 query heads
    W = 8
    kv, q = synth.kv_tensor(sh), synth.q_window(sh, W)
    (k0, k1), (q0, q1) = sharding.heads_of_rank(sh.n_kv_heads, sh.n_q_heads, rank, world)
    kv_mine = kv[:, :, k0:k1].contiguous().view(torch.int16).numpy().view(np.uint16)
    q_mine = q[:, q0:q1].contiguous().view(torch.int16).numpy().view(np.uint16)
    od = oracle.make_desc(sh.n_layers, k1 - k0, q1 - q0, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size)
    local = torch.from_numpy(oracle.chunk_tolerance(od, kv_mine, q_mine, W).astype(np.float32))
    combined = sharding.combine_head_sharded_scores(local, dist)
    bits, order = oracle.assign_bits(combined.numpy(), (1 / 3, 1 / 3, 1 / 3))
    gathered = [None] * world
    dist.all_gather_object(gathered, (combined.numpy().tobytes(), bits.tobytes(), order.tobytes()))
    if rank == 0:
        out.put(gathered)
    dist.barrier()
    dist.destroy_process_group()


def test_head_sharded_scores_combine_to_the_whole_model_score():
    import numpy as np
    import oracle
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_head_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert gathered[0] == gathered[1]                      # same score bits, same levels, same order on both ranks
    combined = np.frombuffer(gathered[0][0], dtype=np.float32)
    sh = synth.KVShape("tp", 2, 4, 8, 32, 96, 16, 32, seed=3)
    kv = synth.kv_tensor(sh).view(torch.int16).numpy().view(np.uint16)
    q = synth.q_window(sh, 8).view(torch.int16).numpy().view(np.uint16)
    od = oracle.make_desc(sh.n_layers, sh.n_kv_heads, sh.n_q_heads, sh.head_dim, sh.n_tokens, sh.chunk_len, sh.group_size)
    whole = oracle.chunk_tolerance(od, kv, q, 8)
    assert np.allclose(combined, whole, rtol=1e-6, atol=0)


def test_heads_of_rank_blocks():
    assert sharding.heads_of_rank(8, 32, 1, 4) == ((2, 4), (8, 16))
    assert sharding.heads_of_rank(1, 8, 0, 1) == ((0, 1), (0, 8))
    import pytest
    with pytest.raises(ValueError):
        sharding.heads_of_rank(1, 8, 0, 2)                 # one KV head cannot be split
    t = torch.tensor([0.25, 0.5])
    assert torch.equal(sharding.combine_head_sharded_scores(t), t)


def test_launcher_starts_one_process_per_rank():
    """sharding.launch_ranks (what `bench.py --gpus N` becomes when it is started as one plain process): two ranks
    come up with the rendezvous on 127.0.0.1, rank 0 prints one JSON line, a failing rank fails the launch."""
    import json
    import subprocess
    import sys
    here = os.path.dirname(os.path.abspath(__file__))
    code = ("import sys; from paper_2403_11805_b200 import sharding; "
            "sys.exit(sharding.launch_ranks(sys.argv[1], sys.argv[2:], 2))")
    env = dict(os.environ, PYTHONPATH=os.path.dirname(here))
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    run = subprocess.run([sys.executable, "-c", code, os.path.join(here, "rank_stub.py"), "--steps", "3"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert run.returncode == 0, run.stderr[-2000:]
    lines = [json.loads(l) for l in run.stdout.splitlines() if l.startswith("{")]
    assert lines == [{"n_gpus": 2, "ms_per_step": 11.0, "argv": ["--steps", "3"]}]
    bad = subprocess.run([sys.executable, "-c", code, os.path.join(here, "rank_stub.py"), "--fail"],
                         env=env, capture_output=True, text=True, timeout=300)
    assert bad.returncode != 0


def test_bench_refuses_a_rank_count_it_was_not_started_with():
    """Under a launcher, bench.py's --gpus must equal WORLD_SIZE (checked before any CUDA call)."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0")
    run = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "4"], env=env, capture_output=True,
                         text=True, timeout=300)
    assert run.returncode != 0 and "WORLD_SIZE=2" in run.stderr
