"""Data-parallel plumbing of the layer: one process per GPU, token shards, three collectives.

The layer shards along the tokens (the batch axis the paper's variance lemma averages over):
every rank holds ``tokens`` rows of A and dY and a replica of W.  Nothing of the method's
arithmetic lives here; this module only
  - starts the ranks (``spawn_ranks``) when no launcher has done so,
  - reads the launcher's environment (``init_from_env``),
  - says where a rank's rows sit in the whole batch (``TokenShard``: the ``index_offset`` that
    makes a shard draw the thresholds its rows have in the unsharded tensor),
  - and wraps the collectives of a step: one max-reduction of the per-tensor maxima of A and dY
    (so that every rank quantizes with the step sizes of the whole batch) and one sum-reduction
    of the weight gradient.
It works with any ``torch.distributed`` backend (``nccl`` on GPUs, ``gloo`` in the CPU tests).
"""
from __future__ import annotations

import os
import signal
import socket
import subprocess
import sys
import time
from dataclasses import dataclass
from typing import Optional, Sequence

import torch
import torch.distributed as dist

LAUNCH_VARS = ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")


def launched_by_env() -> bool:
    """True when a launcher (torch.distributed.run, or spawn_ranks) has set the rank variables."""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv: Sequence[str], env: Optional[dict] = None, timeout: Optional[float] = None) -> int:
    """Starts ``n`` copies of ``python argv...`` on this node, one per rank, with RANK, LOCAL_RANK,
    WORLD_SIZE, LOCAL_WORLD_SIZE, MASTER_ADDR (127.0.0.1) and MASTER_PORT (a free port) set, and
    waits for them.  The children inherit stdout / stderr, so whatever rank 0 prints is this
    process's output.  If a rank fails, the others (exactly the processes started here) are
    terminated.  Returns 0 if every rank exited with 0, else the first non-zero exit code."""
    if n < 1:
        raise ValueError("need at least one rank")
    base = dict(os.environ if env is None else env)
    base.update({"WORLD_SIZE": str(n), "LOCAL_WORLD_SIZE": str(n), "MASTER_ADDR": "127.0.0.1",
                 "MASTER_PORT": str(free_port())})
    procs = []
    for r in range(n):
        e = dict(base)
        e.update({"RANK": str(r), "LOCAL_RANK": str(r)})
        procs.append(subprocess.Popen([sys.executable, *argv], env=e))
    deadline = None if timeout is None else time.monotonic() + timeout
    rc = 0
    pending = set(range(n))
    while pending:
        for r in sorted(pending):
            code = procs[r].poll()
            if code is None:
                continue
            pending.discard(r)
            if code != 0 and rc == 0:
                rc = code
        timed_out = deadline is not None and time.monotonic() > deadline
        if (rc != 0 or timed_out) and pending:
            for r in pending:                       # the other ranks would wait for the failed one forever
                procs[r].send_signal(signal.SIGTERM)
            for r in pending:
                try:
                    procs[r].wait(10)
                except subprocess.TimeoutExpired:
                    procs[r].kill()
                    procs[r].wait()
            pending.clear()
            if rc == 0:
                rc = 124
        if pending:
            time.sleep(0.05)
    return rc


@dataclass(frozen=True)
class TokenShard:
    """Rows [rank * tokens, (rank + 1) * tokens) of a batch of world * tokens tokens."""
    rank: int
    world: int
    tokens: int

    @property
    def first_row(self) -> int:
        return self.rank * self.tokens

    def index_offset(self, cols: int) -> int:
        """Flat index of the shard's first element in the whole [world * tokens, cols] tensor:
        the ``index_offset`` of the shard's quantization points."""
        return self.first_row * cols


def init_from_env(backend: str, device=None):
    """(rank, local_rank, world) from the launcher's variables; joins the process group when
    world > 1 (rendezvous through MASTER_ADDR / MASTER_PORT)."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", str(rank)))
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (device is not None and backend == "nccl") else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, local, world


def reduce_absmax(absmax: torch.Tensor, world: int) -> None:
    """In place: element-wise maximum over the ranks of a small vector of maxima (one collective
    for all operands of a step)."""
    if world > 1:
        dist.all_reduce(absmax, op=dist.ReduceOp.MAX)


def reduce_sum(t: torch.Tensor, world: int) -> None:
    """In place: sum over the ranks (the weight gradient, as int32 sums or as fp32 values)."""
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM)


def int32_sums_fit(world: int, tokens: int, bits_a: int, bits_b: int) -> bool:
    """Whether the int32 sums of a contraction over all world * tokens tokens cannot overflow for
    codes of the given widths (the bound the library applies to one product)."""
    qa, qb = (1 << (bits_a - 1)) - 1, (1 << (bits_b - 1)) - 1
    return world * tokens * qa * qb < (1 << 31)


def finish() -> None:
    if dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()
