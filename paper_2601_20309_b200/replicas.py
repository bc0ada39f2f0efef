"""Start N independent replicas of a command on one node, one process per GPU.

The rotation path has no exchange step (the paper's tensor-parallel run adds no inter-GPU traffic,
section 5.3.5): every GPU has its own pool, its own host link and its own lists.  A multi-GPU run is
therefore N copies of the single-GPU program that only meet to agree on a start time and to add up
their figures.  ``spawn`` is what ``bench.py --gpus N`` uses when it was not started by a launcher
(no ``WORLD_SIZE`` in the environment): it sets the rendezvous variables a ``torch.distributed``
process group reads, starts the ranks, passes rank 0's output through and returns the exit codes.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Sequence, Tuple


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rank_env(rank: int, world: int, port: int, base: Optional[dict] = None) -> dict:
    """Environment of one replica: the variables ``torch.distributed`` rendezvous reads."""
    env = dict(os.environ if base is None else base)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                "LOCAL_WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    return env


def spawn(world: int, argv: Sequence[str], timeout_s: Optional[float] = None,
          capture: bool = False) -> Tuple[List[int], str]:
    """Run ``argv`` as ``world`` processes with ranks 0..world-1.  Rank 0's standard output is passed
    through (or returned when ``capture``); the other ranks' output is dropped, their errors are not.
    Returns (exit codes by rank, rank 0's output if captured).  A rank that outlives ``timeout_s`` is
    killed (only the processes started here) and reported with exit code -9."""
    if world < 1:
        raise ValueError("world must be at least 1")
    port = free_port()
    procs = []
    for rank in range(world):
        out = (subprocess.PIPE if capture else None) if rank == 0 else subprocess.DEVNULL
        procs.append(subprocess.Popen(list(argv), env=rank_env(rank, world, port), stdout=out, text=True))
    codes, text = [], ""
    for rank, p in enumerate(procs):
        try:
            o, _ = p.communicate(timeout=timeout_s)
            if rank == 0 and capture:
                text = o or ""
            codes.append(p.returncode)
        except subprocess.TimeoutExpired:
            p.kill()
            p.communicate()
            codes.append(-9)
    return codes, text


def main_spawn(world: int) -> int:
    """Re-run the current program (``sys.argv``) as ``world`` replicas; returns the worst exit code."""
    codes, _ = spawn(world, [sys.executable] + sys.argv)
    bad = [c for c in codes if c != 0]
    return bad[0] if bad else 0
