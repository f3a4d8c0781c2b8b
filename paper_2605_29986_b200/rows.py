"""Row sharding for several GPUs: rows are independent, so ranks take contiguous row blocks and the
data path has no collective. Pure host logic (no CUDA, no arithmetic of the path): how the rows are
split, how N ranks are started on one node, and how their timings are combined."""
from __future__ import annotations

import os
import socket
import sys
from typing import List, Optional, Sequence, Tuple


def shard_rows(B: int, rank: int, world: int) -> Tuple[int, int]:
    """Half-open row range [lo, hi) of `rank` when B rows are split as evenly as possible over `world` ranks."""
    base, extra = divmod(B, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def max_over_ranks(seconds: float, dist, device=None) -> float:
    """Slowest rank's time: the figure a multi-GPU throughput is computed from."""
    import torch
    t = torch.tensor([seconds], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0])


def dist_env(env=None) -> Tuple[int, int, int]:
    """(rank, local rank, world size) as a launcher left them in the environment; (0, 0, 1) without one."""
    env = os.environ if env is None else env
    return int(env.get("RANK", "0")), int(env.get("LOCAL_RANK", "0")), int(env.get("WORLD_SIZE", "1"))


def launched_by_torchrun(env=None) -> bool:
    env = os.environ if env is None else env
    return "WORLD_SIZE" in env and "RANK" in env


def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def torchrun_command(script: str, n: int, argv: Sequence[str], port: Optional[int] = None) -> List[str]:
    """The command that starts `n` ranks of `script` on this node, one per GPU, rendezvous on 127.0.0.1."""
    if n < 1:
        raise ValueError("need at least one rank")
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr",
            "127.0.0.1", "--master-port", str(port or free_port()), script] + list(argv)


def need_spawn(gpus: int, env=None) -> bool:
    """True when several GPUs were asked for and no launcher has started the ranks yet."""
    return gpus > 1 and not launched_by_torchrun(env)


def spawn_ranks(script: str, n: int, argv: Sequence[str]) -> int:
    """Run `script` as `n` ranks and wait; returns the launcher's exit code."""
    import subprocess
    return subprocess.call(torchrun_command(script, n, argv))


def init_ranks(backend: str = "nccl", device=None):
    """Join the process group the launcher prepared. Returns (rank, local rank, world, dist or None)."""
    rank, local_rank, world = dist_env()
    if world <= 1:
        return rank, local_rank, world, None
    import torch.distributed as dist
    kwargs = {}
    if device is not None:
        kwargs["device_id"] = device
    dist.init_process_group(backend, **kwargs)
    return rank, local_rank, world, dist
