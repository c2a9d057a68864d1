"""Multi-GPU plumbing.  The decode path shards by request: every GPU owns a pool and a disjoint set
of requests, and no step of the path exchanges data between them.  What is left for
`torch.distributed` is the rendezvous, the barrier around the timed region and the max-over-ranks
of the device time.  Works with NCCL (one process per GPU) and with gloo (CPU tests).

The path also shards by KV head (Eq. 11: the query-state tensor is laid out by "query heads per GPU"): every rank
of a tensor-parallel group holds a pool over the same requests with its slice of the heads; scoring, working
sets, selection and compaction are per (layer, KV head), and the one exchange is the mean of Eq. 8: two integers
per boundary request (sum of K^S, sum of K^L), added up over the ranks between gp_decode_step_local and
gp_decode_step_finish."""
from __future__ import annotations

import os
from typing import List, Tuple


def env_world() -> Tuple[int, int, int]:
    """(rank, local rank, world size) from the torchrun environment; (0, 0, 1) when absent."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend: str) -> Tuple[int, int, int]:
    import torch.distributed as dist
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def finish() -> None:
    """Leaves the process group (a no-op for a single process)."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()
        dist.destroy_process_group()


def shard_seed(base_seed: int, rank: int) -> int:
    """Weak scaling: rank r decodes its own set of requests, drawn with this seed.  Rank 0 keeps the
    configuration's own seed."""
    return base_seed + 1000 * rank


def shard_requests(n_requests: int, rank: int, world: int) -> List[int]:
    """Strong-scaling split of a fixed request list: contiguous, sizes differ by at most one."""
    base, extra = divmod(n_requests, world)
    lo = rank * base + min(rank, extra)
    return list(range(lo, lo + base + (1 if rank < extra else 0)))


def barrier(device=None) -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        if device is not None and dist.get_backend() == "nccl":
            dist.barrier(device_ids=[device])
        else:
            dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = f"cuda:{device}" if (device is not None and dist.get_backend() == "nccl") else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    dev = f"cuda:{device}" if (device is not None and dist.get_backend() == "nccl") else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def job_throughput(units_this_rank: float, ms_this_rank: float, device=None) -> Tuple[float, float]:
    """Whole-job throughput: units of all ranks over the slowest rank's time.  Returns (units/s, ms)."""
    ms = max_over_ranks(ms_this_rank, device)
    units = sum_over_ranks(units_this_rank, device)
    return units / (ms * 1e-3), ms


def kv_head_slice(n_q_heads: int, n_kv_heads: int, rank: int, world: int) -> Tuple[slice, slice]:
    """The query heads and KV heads rank `rank` of `world` holds: whole GQA groups, contiguous, equally many each."""
    if n_kv_heads % world or n_q_heads % n_kv_heads:
        raise ValueError("the KV heads must divide evenly over the ranks, the query heads over the KV heads")
    per = n_kv_heads // world
    g = n_q_heads // n_kv_heads
    return slice(rank * per * g, (rank + 1) * per * g), slice(rank * per, (rank + 1) * per)


def complete_boundary_sums(sums, group=None) -> None:
    """Adds the per-request sums of K^S and K^L up over the ranks, in place (`sums`: an int32 tensor, on the device
    for NCCL, on the host for gloo).  One all-reduce; a no-op for a single process."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)


def shard_sums_tensor(pool):
    """The pool's array of sums (gp_shard_sums) as a tensor that shares its memory: a view into the pool's blob."""
    import torch
    from . import binding as B
    ptr, n = B.gp_shard_sums(pool.handle)
    off = ptr - pool.blob.data_ptr()
    return pool.blob[off:off + 4 * n].view(torch.int32)


def sharded_decode_step(pool, req_ids, q, k, v, out, actions, group=None) -> None:
    """One decode step of a pool that holds this rank's KV heads: the local half, the all-reduce of the sums, the
    decisions and compaction.  q, k, v, out are this rank's head slices; every rank passes the same req_ids."""
    from . import binding as B
    n = int(req_ids.numel())
    B.gp_decode_step_local(pool.handle, req_ids.data_ptr(), n, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                           actions.data_ptr(), pool.stream())
    complete_boundary_sums(shard_sums_tensor(pool), group)
    B.gp_decode_step_finish(pool.handle, req_ids.data_ptr(), n, actions.data_ptr(), pool.stream())
