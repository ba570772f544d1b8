"""Host-side helpers for running the routing decision on several GPUs.

The path shards by rows: sequences are independent, so every rank decides its own sequences against
a replicated LM head and there is no data-path collective.  What crosses ranks is only bookkeeping:
which sequences a rank owns, the slowest rank's time, and the totals.

A head too large for one GPU shards by vocabulary rows instead (tensor-parallel head): every rank runs the
head kernels on its rows of W_head and leaves five words of softmax statistics per row; one all-gather
of those (20 bytes per row and rank) is the path's only collective, after which each rank merges and
decides (binding.shard_stats / binding.shard_route).

Nothing here computes any part of the decision; it works on CPU tensors with the gloo backend and on
CUDA tensors with NCCL.
"""
from __future__ import annotations

import os
import socket
import subprocess
from typing import List, Optional, Tuple


def rank_rows(n_rows: int, rank: int, world: int) -> Tuple[int, int]:
    """[begin, end) of the sequences rank `rank` decides when n_rows are dealt to `world` ranks
    in contiguous, balanced blocks (sizes differ by at most one, earlier ranks take the extra)."""
    if world < 1 or not (0 <= rank < world) or n_rows < 0:
        raise ValueError("bad sharding arguments")
    base, extra = divmod(n_rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def global_index(local_idx, begin: int):
    """Sequence ids of a rank's compacted list in the numbering of the whole batch."""
    return local_idx + begin


def reduce_step_stats(ms: float, units: float, launches: int, dist=None, device="cpu"):
    """(slowest rank's ms, units summed over ranks, launches summed over ranks).

    `dist` is torch.distributed (initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms), float(units), int(launches)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    s = torch.tensor([units, float(launches)], dtype=torch.float64, device=device)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    return float(t[0].item()), float(s[0].item()), int(round(float(s[1].item())))


def gather_counts(count: int, dist=None, device="cpu"):
    """Every rank's llm_count, in rank order: the offsets that turn per-rank index lists into one
    global list are their exclusive prefix sums."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return [int(count)]
    import torch
    mine = torch.tensor([int(count)], dtype=torch.int64, device=device)
    out = [torch.zeros_like(mine) for _ in range(dist.get_world_size())]
    dist.all_gather(out, mine)
    return [int(o.item()) for o in out]


def vocab_shard(V: int, rank: int, world: int, align: int = 16) -> Tuple[int, int]:
    """[begin, end) of the W_head rows rank `rank` holds when a vocabulary of V entries is split into
    `world` contiguous shards.  Boundaries are multiples of `align` rows (whole tensor-core tile units),
    sizes differ by at most `align`, and the last shard takes the ragged end."""
    if world < 1 or not (0 <= rank < world) or V < 0 or align < 1:
        raise ValueError("bad sharding arguments")
    b, e = rank_rows(-(-V // align), rank, world)
    return min(b * align, V), min(e * align, V)


def empty_shard_stats(R: int, device="cpu"):
    """Statistics of a shard that holds no vocabulary entry (the empty set of the merge): what a rank
    contributes when the split leaves it no rows.  The head kernels need at least two rows per shard."""
    import torch
    import struct
    ninf = struct.unpack("<i", struct.pack("<f", float("-inf")))[0]
    row = torch.tensor([ninf, 0, 0, ninf, 2**31 - 1], dtype=torch.int32, device=device)
    return row.repeat(R, 1)


def gather_shard_stats(stats, dist=None, out=None):
    """All-gather of the per-row shard statistics ([R, 5] int32, every rank the same R) into
    [world, R, 5] in rank order = ascending vocabulary order, the order the merge wants."""
    import torch
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        g = stats.unsqueeze(0)
        if out is not None:
            out.copy_(g)
            return out
        return g
    world = dist.get_world_size()
    if out is None:
        out = torch.empty((world,) + tuple(stats.shape), dtype=stats.dtype, device=stats.device)
    # the ranks' blocks concatenated along the first axis: the form every backend accepts
    dist.all_gather_into_tensor(out.view((world * stats.shape[0],) + tuple(stats.shape[1:])), stats.contiguous())
    return out


def spawn_ranks(n_ranks: int, argv: List[str], port: Optional[int] = None, extra_env: Optional[dict] = None,
                timeout: Optional[float] = None) -> int:
    """Run the command line `argv` as n_ranks processes of one node, one per GPU, with the environment
    torch.distributed reads (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT): what a
    launcher would do, for callers that were started without one.  The ranks inherit stdout and stderr.
    Returns 0 if every rank exited 0, else the first non-zero exit code; once a rank has failed the others
    are terminated (by process id) instead of being left waiting at a rendezvous."""
    if n_ranks < 1:
        raise ValueError("n_ranks must be at least 1")
    if port is None:
        with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as sk:
            sk.bind(("127.0.0.1", 0))
            port = int(sk.getsockname()[1])
    procs = []
    for r in range(n_ranks):
        env = dict(os.environ)
        env.update({"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n_ranks), "LOCAL_WORLD_SIZE": str(n_ranks),
                    "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        if extra_env:
            env.update(extra_env)
        procs.append(subprocess.Popen(list(argv), env=env))
    import time
    deadline = None if timeout is None else time.monotonic() + timeout
    rc = 0
    pending = list(procs)
    while pending:
        for p in list(pending):
            code = p.poll()
            if code is not None:
                pending.remove(p)
                if code != 0 and rc == 0:
                    rc = code
        if rc != 0 or (deadline is not None and time.monotonic() > deadline):
            for p in pending:
                p.terminate()
            for p in pending:
                try:
                    p.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    p.kill()
            if rc == 0:
                rc = 124
            break
        time.sleep(0.05)
    return rc
