"""One process per GPU on one node.

``spawn_ranks`` re-runs a script under ``python -m torch.distributed.run`` with N local ranks; every
rank finds its place through ``rank_env``.  Ranks share nothing but the rendezvous: streams are
independent units, so the benchmark's data path needs no collective and the launcher starts no
communication of its own.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from typing import List, Optional, Tuple


def rank_env() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) from the environment a torch launcher sets; (0, 0, 1) without one."""
    e = os.environ
    return int(e.get("RANK", 0)), int(e.get("LOCAL_RANK", 0)), int(e.get("WORLD_SIZE", 1))


def under_launcher() -> bool:
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_command(n: int, script: str, argv: List[str], port: Optional[int] = None) -> List[str]:
    """The command line that starts `script argv` as n ranks of one node (rendezvous on 127.0.0.1)."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port if port else free_port()),
            script, *argv]


def spawn_ranks(n: int, script: str, argv: List[str], port: Optional[int] = None, capture: bool = False,
                env: Optional[dict] = None, timeout: Optional[float] = None):
    """Runs `script argv` as n ranks and waits.  Returns the exit code, or (exit code, stdout, stderr)
    with capture=True.  The ranks inherit stdout, so whatever rank 0 prints is this process's output."""
    if n < 1:
        raise ValueError("need at least one rank")
    cmd = launch_command(n, script, argv, port)
    child_env = dict(os.environ if env is None else env)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "LOCAL_WORLD_SIZE", "GROUP_RANK"):
        child_env.pop(k, None)
    if capture:
        p = subprocess.run(cmd, env=child_env, capture_output=True, text=True, timeout=timeout)
        return p.returncode, p.stdout, p.stderr
    return subprocess.run(cmd, env=child_env, timeout=timeout).returncode
