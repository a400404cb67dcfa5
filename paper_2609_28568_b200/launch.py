"""Start one process per GPU on this node (the paper's arrangement: one process per rank).

`bench.py --gpus N` is normally started N times by `torch.distributed.run`; when it is started
once, directly, it calls `spawn_ranks` to start the N ranks itself. Only process plumbing lives
here: environment variables of the rendezvous and waiting for the children.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys
import time


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return int(s.getsockname()[1])


def spawn_ranks(n: int, argv: list[str], python: str | None = None, env_extra: dict | None = None,
                timeout: float | None = None) -> int:
    """Run `python argv...` as ranks 0..n-1 of one node and wait for all of them.

    Every child gets RANK, LOCAL_RANK, WORLD_SIZE, LOCAL_WORLD_SIZE, MASTER_ADDR (127.0.0.1) and a
    free MASTER_PORT. Rank 0 inherits this process's stdout (it prints the result line); the other
    ranks' stdout goes to stderr so that stdout carries one result only. NCCL's communicator set-up
    lines are switched on (unless the caller chose a debug level) so that a log shows how many ranks
    joined. Returns the largest exit code; a rank that fails ends the others.
    """
    if n < 1:
        raise ValueError("need at least one rank")
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ)
        env.update({"RANK": str(r), "LOCAL_RANK": str(r), "WORLD_SIZE": str(n), "LOCAL_WORLD_SIZE": str(n),
                    "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        if env_extra:
            env.update({k: str(v) for k, v in env_extra.items()})
        procs.append(subprocess.Popen([python or sys.executable, *argv], env=env,
                                      stdout=None if r == 0 else sys.stderr))
    rc = 0
    deadline = None if timeout is None else time.monotonic() + timeout
    try:
        pending = list(procs)
        while pending:
            for p in list(pending):
                try:
                    code = p.wait(timeout=0.2)
                except subprocess.TimeoutExpired:
                    continue
                pending.remove(p)
                if code != 0:
                    rc = max(rc, code if code > 0 else 1)
                    for q in pending:   # one rank failed: the others would wait at a barrier for ever
                        q.terminate()
            if deadline is not None and pending and time.monotonic() > deadline:
                for q in pending:
                    q.terminate()
                rc = max(rc, 124)
                deadline = None
    finally:
        for p in procs:
            if p.poll() is None:
                p.kill()
    return rc
