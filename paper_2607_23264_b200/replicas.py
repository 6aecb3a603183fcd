"""Host-side logic of a multi-GPU run: independent replicas of the layer, one process per GPU.

Nothing on the data path is sharded and no collective moves activations (EP=1): every rank runs the whole
layer on its own batch of tokens with replicated expert weights.  torch.distributed is used only to line the
ranks up (barrier) and to reduce the timing to the slowest rank.  The same functions run on CPU with the
gloo backend, which is how they are tested.
"""
from __future__ import annotations

import numpy as np


def rank_batch(x_bits: np.ndarray, rank: int) -> np.ndarray:
    """The batch of one rank: the seeded batch with its rows rotated by 17*rank, so ranks differ."""
    return x_bits if rank == 0 else np.roll(x_bits, rank * 17, axis=0)


def init_process_group(world: int, backend: str, device=None, force: bool = False):
    """Join the job's process group (rendezvous from the MASTER_* / RANK / WORLD_SIZE environment).

    A single process needs no group; `force` joins one all the same (a launcher started this process as the only
    rank), so that a one-rank run takes the same path as an N-rank run."""
    import torch.distributed as dist
    if world <= 1 and not force:
        return False
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)
    return True


def _in_group() -> bool:
    import torch.distributed as dist
    return dist.is_available() and dist.is_initialized()


def barrier(world: int):
    import torch.distributed as dist
    if world > 1 or _in_group():
        dist.barrier()


def max_over_ranks(value: float, world: int, device="cpu") -> float:
    """Slowest rank's figure (e.g. the device time of the timed region)."""
    import torch
    import torch.distributed as dist
    if world <= 1 and not _in_group():
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tokens_per_second(tokens_per_rank: int, world: int, steps: int, slowest_ms: float) -> float:
    """Whole-job throughput: all ranks' tokens over the slowest rank's time."""
    return tokens_per_rank * world * steps / (slowest_ms * 1e-3)


def launcher_command(n_gpus: int, script: str, argv, port: int, python: str = "python"):
    """Command and extra environment that start `script argv` as n_gpus ranks on this node, one per GPU.

    The ranks meet over 127.0.0.1 (a container's host name may not resolve).  NCCL's own log stays on at INFO level
    unless the caller's environment already sets it, so that a run's output shows how many ranks joined."""
    if n_gpus < 2:
        raise ValueError("a launcher is needed for two or more ranks only")
    cmd = [python, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), script, *argv]
    env = {"NCCL_DEBUG": "INFO"}
    return cmd, env
