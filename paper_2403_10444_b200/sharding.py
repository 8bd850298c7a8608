"""Host logic of the multi-GPU path: the batch of sequences is split across ranks.

Verifying one sequence (Algorithm 1 or 2 on its gamma drafted tokens) needs nothing from any
other sequence, so the data path has no exchange step: every rank verifies its own contiguous
slice of the batch with the single-GPU entry points.  What crosses ranks is control data only:
the emitted tokens and lengths when a caller wants them in one place, and the timing maximum.
The functions work on any initialised ``torch.distributed`` backend (NCCL on GPUs, gloo on
CPU); with no process group they behave as a single rank.
"""
from __future__ import annotations

from typing import Callable, Dict, Optional, Tuple

import torch


def world(group=None) -> Tuple[int, int]:
    """(rank, world_size) of the process group, (0, 1) without one."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(group), dist.get_world_size(group)
    return 0, 1


def shard_bounds(B: int, rank: int, world_size: int) -> Tuple[int, int]:
    """Contiguous balanced split of B sequences: the first B % world_size ranks get one more."""
    if B < 0 or world_size < 1 or not 0 <= rank < world_size:
        raise ValueError("bad shard request B=%d rank=%d world=%d" % (B, rank, world_size))
    q, r = divmod(B, world_size)
    lo = rank * q + min(rank, r)
    return lo, lo + q + (1 if rank < r else 0)


def shard_inputs(inputs: Dict[str, object], rank: int, world_size: int) -> Dict[str, object]:
    """This rank's slice (views, no copies) of a batch given as the dict of make_inputs."""
    B = inputs["draft_tokens"].shape[0]
    lo, hi = shard_bounds(B, rank, world_size)
    return {k: (v[lo:hi] if torch.is_tensor(v) else v) for k, v in inputs.items()}


def verify_sharded(fn: Callable, inputs: Dict[str, object], gather: bool = True, group=None):
    """Verify this rank's slice of ``inputs`` with ``fn`` (one of the single-GPU entry points,
    called as fn(target, draft, tokens, uniforms, temperature) -> (out_tokens, out_len)) and,
    when ``gather``, return the whole batch's (out_tokens, out_len) on every rank.

    An empty slice (more ranks than sequences) is not passed to ``fn``.
    """
    import torch.distributed as dist
    rank, ws = world(group)
    B, g = inputs["draft_tokens"].shape
    mine = shard_inputs(inputs, rank, ws)
    lo, hi = shard_bounds(B, rank, ws)
    dev = inputs["draft_tokens"].device
    if hi > lo:
        ot, ol = fn(mine["target_logits"], mine["draft_logits"], mine["draft_tokens"], mine["uniforms"],
                    mine["temperature"])[:2]
        ot, ol = torch.as_tensor(ot).to(dev, torch.int32), torch.as_tensor(ol).to(dev, torch.int32)
    else:
        ot = torch.empty((0, g + 1), dtype=torch.int32, device=dev)
        ol = torch.empty((0,), dtype=torch.int32, device=dev)
    if not gather or ws == 1:
        return ot, ol
    # equal-sized pieces for all_gather: pad to the largest slice, cut after the exchange
    width = -(-B // ws)
    piece = torch.full((width, g + 2), -1, dtype=torch.int32, device=dev)
    piece[: hi - lo, : g + 1] = ot
    piece[: hi - lo, g + 1] = ol
    pieces = [torch.empty_like(piece) for _ in range(ws)]
    dist.all_gather(pieces, piece, group=group)
    rows = []
    for r in range(ws):
        a, b = shard_bounds(B, r, ws)
        rows.append(pieces[r][: b - a])
    full = torch.cat(rows, dim=0)
    return full[:, : g + 1].contiguous(), full[:, g + 1].contiguous()


def max_over_ranks(value: float, device: Optional[torch.device] = None, group=None) -> float:
    """The largest ``value`` any rank holds (device-timed milliseconds of a step)."""
    import torch.distributed as dist
    _, ws = world(group)
    if ws == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def whole_job_rate(units_per_rank: int, ms_per_step: float, group=None) -> float:
    """Units all ranks processed per second given the (already maximal) step time."""
    _, ws = world(group)
    return ws * units_per_rank / (ms_per_step * 1e-3)


def rank_command(script: str, argv, n_ranks: int, port: Optional[int] = None):
    """The command that starts ``n_ranks`` processes of ``script argv`` on this node, one per GPU,
    through ``torch.distributed.run`` with the rendezvous on 127.0.0.1."""
    import socket
    import sys
    if n_ranks < 1:
        raise ValueError("n_ranks must be at least 1")
    if port is None:
        with socket.socket() as s:          # a port that is free now
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n_ranks),
            "--master-addr", "127.0.0.1", "--master-port", str(port), script, *argv]


def launch_ranks(script: str, argv, n_ranks: int, port: Optional[int] = None, env=None) -> int:
    """Run :func:`rank_command` to its end and return its exit status (non-zero if any rank failed)."""
    import subprocess
    return subprocess.call(rank_command(script, argv, n_ranks, port), env=env)
