"""Multi-GPU plumbing for the benchmark: one process per GPU, no data-path collective.

The hot path shards without any exchange step: a KV head together with the query heads that share it
(and, above that, a batch element) is an independent unit, so ranks either run replicas of the
workload (weak scaling) or each take a contiguous range of KV heads of one workload (strong
scaling).  torch.distributed is used only for the start barrier and for the maximum over ranks of
the measured time.  Works with the ``nccl`` backend on GPUs and with ``gloo`` on CPUs."""
from __future__ import annotations

import os

import torch


def env_world():
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without a launcher."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0")))


def head_shard(rank: int, world: int, Hq: int, Hkv: int):
    """Contiguous range of KV heads of this rank and the query heads that go with them.

    Returns (kv_lo, kv_hi, q_lo, q_hi).  KV heads are dealt as evenly as possible (the first
    ``Hkv % world`` ranks get one more); a rank beyond the number of KV heads gets an empty range."""
    if Hq % Hkv:
        raise ValueError("Hq must be a multiple of Hkv")
    G = Hq // Hkv
    base, extra = divmod(Hkv, world)
    lo = rank * base + min(rank, extra)
    hi = lo + base + (1 if rank < extra else 0)
    return lo, hi, lo * G, hi * G


def init(backend: str, device=None):
    """Join the process group when launched with WORLD_SIZE > 1; returns torch.distributed or None."""
    rank, world, _ = env_world()
    if world <= 1:
        return None
    import torch.distributed as dist
    if not dist.is_initialized():
        kwargs = dict(device_id=device) if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, **kwargs)
    return dist


def barrier(dist):
    if dist is not None:
        dist.barrier()
    if torch.cuda.is_available():
        torch.cuda.synchronize()


def max_over_ranks(value: float, dist, device="cpu") -> float:
    """Largest ``value`` over all ranks (every rank gets it)."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, dist, device="cpu") -> float:
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())
