"""Request sharding across GPUs.  The path is independent per request (own history, own logits
rows, own state), so ranks never exchange data: a rank takes a contiguous range of requests and
runs the same three kernels on it.  Only timings and counters are reduced for the report.

The one exchange the path can need is under a vocabulary-parallel output layer, where every rank
holds a slice of each logits row: hvd_verify_keys gives one 8-byte key per row and rank,
reduce_keys_over_ranks takes their element-wise maximum (8 bytes per row cross the links, not the
logits), hvd_commit_keys finishes the step on every rank."""
from __future__ import annotations

import numpy as np


def request_cost(hist_len, K, V, elt) -> np.ndarray:
    """Bytes a step streams for each request: its history plus its K+1 logits rows."""
    return 4 * np.asarray(hist_len, np.int64) + (np.asarray(K, np.int64) + 1) * int(V) * int(elt)


def partition_requests(cost, world: int) -> np.ndarray:
    """Boundaries [world+1] of contiguous request ranges with near-equal summed cost: range r is
    [bounds[r], bounds[r+1]).  Every request lands in exactly one range; ranges may be empty when
    there are fewer requests than ranks."""
    cost = np.asarray(cost, np.float64)
    B = len(cost)
    csum = np.concatenate([[0.0], np.cumsum(cost)])
    total = csum[-1]
    bounds = np.zeros(world + 1, np.int64)
    for r in range(1, world):
        target = total * r / world
        j = int(np.searchsorted(csum, target, side="left"))
        # pick the neighbour whose prefix cost is closest to the target
        if j > 0 and abs(csum[j - 1] - target) <= abs(csum[min(j, B)] - target):
            j -= 1
        bounds[r] = min(max(j, bounds[r - 1]), B)
    bounds[world] = B
    return bounds


def max_over_ranks(value: float, device=None) -> float:
    """Maximum of a host scalar over all ranks (identity without an initialised process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(value: float, device=None) -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def vocab_shards(V: int, world: int) -> np.ndarray:
    """Boundaries [world+1] of near-equal contiguous vocabulary slices: rank r holds [b[r], b[r+1])."""
    return (np.arange(world + 1, dtype=np.int64) * int(V)) // int(world)


def reduce_keys_over_ranks(keys, group=None):
    """Element-wise MAX of the int64 row keys of hvd_verify_keys over all ranks, in place (identity
    without an initialised process group).  The keys are in signed order, so the plain MAX picks the
    larger logit and, among equal logits, the lower global index."""
    import torch
    import torch.distributed as dist
    assert keys.dtype == torch.int64
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(keys, op=dist.ReduceOp.MAX, group=group)
    return keys
