"""Start one process per GPU on this node with the environment torch.distributed expects.

`spawn_ranks` is what ``bench.py --gpus N`` uses when it was not started under a launcher: it
re-runs a command N times with RANK / LOCAL_RANK / WORLD_SIZE / MASTER_ADDR / MASTER_PORT set, lets
every rank inherit stdout and stderr (rank 0 prints the result line), and returns the worst exit
code.  If one rank fails the others are terminated by their own process ids.
"""
from __future__ import annotations

import os
import socket
import subprocess
import time


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rank_environment(rank: int, nranks: int, port: int, base=None) -> dict:
    env = dict(os.environ if base is None else base)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(nranks),
                "LOCAL_WORLD_SIZE": str(nranks), "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    return env


def spawn_ranks(cmd: list, nranks: int, port: int | None = None, env=None, timeout: float | None = None) -> int:
    """Run `cmd` as ranks 0..nranks-1 on this node; returns 0 if every rank exited 0."""
    if nranks < 1:
        raise ValueError("nranks must be positive")
    port = free_port() if port is None else port
    procs = [subprocess.Popen(cmd, env=rank_environment(r, nranks, port, env)) for r in range(nranks)]
    deadline = None if timeout is None else time.monotonic() + timeout
    worst = 0
    pending = set(range(nranks))
    while pending:
        for r in sorted(pending):
            rc = procs[r].poll()
            if rc is not None:
                pending.discard(r)
                if rc != 0 and worst == 0:
                    worst = rc
        failed = worst != 0 or (deadline is not None and time.monotonic() > deadline)
        if failed and pending:
            for r in pending:
                procs[r].terminate()
            for r in pending:
                try:
                    procs[r].wait(timeout=10)
                except subprocess.TimeoutExpired:
                    procs[r].kill()
            if worst == 0:
                worst = 124
            break
        if pending:
            time.sleep(0.05)
    return worst
