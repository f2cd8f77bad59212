"""Host-side sharding of the hot path across ranks (one process per GPU).

(head, query block) work items never exchange data, so the path shards without any data-path
collective.  Two ways are provided:
  * independent problems: rank r processes its own layer (bench.py --gpus N, weak scaling);
  * one layer split by KV-head group: rank r owns a contiguous range of KV heads and the
    query heads that read them; outputs stay head-sharded (the layout tensor-parallel attention
    already has).
The only communication is the reduction of the timing (max over ranks) and of the work counters
(sum over ranks) for reporting.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def kv_head_shard(hq: int, hkv: int, world: int, rank: int):
    """Contiguous, balanced KV-head range of `rank` and the query-head range reading it.

    Returns (kv_lo, kv_hi, q_lo, q_hi); ranks beyond the number of KV heads get empty ranges."""
    if hq % hkv != 0 or not 0 <= rank < world:
        raise ValueError("bad head counts or rank")
    group = hq // hkv
    base, extra = divmod(hkv, world)
    kv_lo = rank * base + min(rank, extra)
    kv_hi = kv_lo + base + (1 if rank < extra else 0)
    return kv_lo, kv_hi, kv_lo * group, kv_hi * group


def shard_tensors(q, k, v, world: int, rank: int):
    """Slices [B,H,N,d] tensors (torch or numpy) to the heads of `rank`."""
    kv_lo, kv_hi, q_lo, q_hi = kv_head_shard(q.shape[1], k.shape[1], world, rank)
    return q[:, q_lo:q_hi], k[:, kv_lo:kv_hi], v[:, kv_lo:kv_hi]


def reduce_job(ms_local: float, units_local: float, device=None):
    """(max over ranks of the time, sum over ranks of the work).  Works with any backend; without an
    initialised process group it returns its arguments."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(units_local)
    if device is None:
        device = torch.device("cuda", torch.cuda.current_device()) if dist.get_backend() == "nccl" else torch.device("cpu")
    t_max = torch.tensor([ms_local], dtype=torch.float64, device=device)
    t_sum = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t_max, op=dist.ReduceOp.MAX)
    dist.all_reduce(t_sum, op=dist.ReduceOp.SUM)
    return float(t_max.item()), float(t_sum.item())
