"""Start one process per GPU on a single node.

`spawn_ranks(n, argv)` runs `argv` n times with the environment a `torch.distributed` program expects
(RANK, LOCAL_RANK, WORLD_SIZE, LOCAL_WORLD_SIZE, MASTER_ADDR=127.0.0.1, MASTER_PORT) and waits for all of them.
It is what `bench.py --gpus N` uses when it is started as a plain `python bench.py` instead of through
`python -m torch.distributed.run`: the ranks then rendezvous over the loopback address, which also works where
the container's hostname does not resolve.
"""
from __future__ import annotations

import os
import socket
import subprocess
import time
from typing import Mapping, Optional, Sequence


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def rank_environment(rank: int, world: int, port: int, base: Optional[Mapping[str, str]] = None) -> dict:
    env = dict(os.environ if base is None else base)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), LOCAL_WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    return env


def spawn_ranks(n: int, argv: Sequence[str], *, port: Optional[int] = None, env: Optional[Mapping[str, str]] = None,
                stdout=None, timeout_s: Optional[float] = None) -> int:
    """Run `argv` as ranks 0..n-1 and wait.  Rank 0 writes to `stdout` (None = inherit), the other ranks inherit.
    Returns 0 if every rank exited 0; otherwise the first non-zero exit code, after the ranks still running have been
    terminated (by their own process ids).  `timeout_s` bounds the whole run."""
    if n < 1:
        raise ValueError("need at least one rank")
    port = free_port() if port is None else int(port)
    procs = []
    try:
        for r in range(n):
            procs.append(subprocess.Popen(list(argv), env=rank_environment(r, n, port, env), stdout=stdout if r == 0 else None))
        deadline = None if timeout_s is None else time.monotonic() + timeout_s
        rc = 0
        pending = set(range(n))
        while pending and rc == 0:
            for r in sorted(pending):
                code = procs[r].poll()
                if code is not None:
                    pending.discard(r)
                    if code != 0:
                        rc = code
                        break
            if deadline is not None and time.monotonic() > deadline:
                rc = 124
            if pending and rc == 0:
                time.sleep(0.02)
        return rc
    finally:
        for p in procs:
            if p.poll() is None:
                p.terminate()
        for p in procs:
            try:
                p.wait(timeout=10)
            except subprocess.TimeoutExpired:
                p.kill()
                p.wait()
