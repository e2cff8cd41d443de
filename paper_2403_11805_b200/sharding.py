"""How the path spreads over several GPUs.  Contexts are independent (Sec. 3.1), so by default each rank owns whole
contexts and nothing of the data path crosses ranks; only the timing is reduced (maximum over ranks).  Where a
context's KV heads are split over the ranks instead (tensor-parallel serving), the codec still works per rank on its
own heads and only the per-chunk scores of Eq. 1 are exchanged."""
import os
import socket
import subprocess
import sys

import torch


def contexts_of_rank(n_contexts: int, rank: int, world: int):
    """Round-robin ownership: context c belongs to rank c % world."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    return list(range(rank, n_contexts, world))


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def heads_of_rank(n_kv_heads: int, n_q_heads: int, rank: int, world: int):
    """Tensor-parallel serving: a rank holds a contiguous block of KV heads and the query heads that read them.
    Returns ((kv_first, kv_end), (q_first, q_end)).  Every rank holds the same number of heads."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    if n_kv_heads % world or n_q_heads % n_kv_heads:
        raise ValueError("heads must split evenly over the ranks")
    per = n_kv_heads // world
    rep = n_q_heads // n_kv_heads
    return (rank * per, (rank + 1) * per), (rank * per * rep, (rank + 1) * per * rep)


def combine_head_sharded_scores(local_scores: torch.Tensor, dist=None):
    """Eq. 1 is a mean over layers, heads and a chunk's tokens.  When every rank scored the chunks from its own,
    equally many heads, the information density of the whole model is the mean of the ranks' results: one sum
    all-reduce of n_chunks fp32 values (the only exchange on the path), then a division by the number of ranks.
    Every rank receives the same bits, so the rank -> bits rule and the eviction order come out the same everywhere."""
    t = local_scores.to(torch.float32).clone()
    if dist is not None and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        t /= dist.get_world_size()
    return t


def launch_ranks(script: str, argv, n_ranks: int, env=None) -> int:
    """Start `script argv...` as n_ranks processes of one node (one per GPU) under torch.distributed.run, with the
    rendezvous on 127.0.0.1 and a free port, and wait for them.  Each process finds RANK, LOCAL_RANK and WORLD_SIZE
    in its environment.  Output passes through; the return value is the launcher's exit code (non-zero if any rank
    failed).  Unless the caller's environment says otherwise, NCCL's initialisation log is switched on and sent to
    stderr, so that the communicator's rank count can be read from a run's log without touching stdout."""
    if n_ranks < 1:
        raise ValueError("need at least one rank")
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    child_env = dict(os.environ if env is None else env)
    if "NCCL_DEBUG" not in child_env:
        child_env.update(NCCL_DEBUG="INFO", NCCL_DEBUG_SUBSYS="INIT", NCCL_DEBUG_FILE="/dev/stderr")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_ranks}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), script] + list(argv)
    return subprocess.run(cmd, env=child_env).returncode
