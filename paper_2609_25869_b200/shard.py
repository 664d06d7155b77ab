"""Head-sharded driver: one request's heads split over the ranks of a ``torch.distributed`` job.

Heads are independent problems (Section 2.1 defines masked attention per head), so the split needs no exchange on the
data path: rank r prepares a plan for its own contiguous range of heads from its slice of the mask and runs the forward
on its slices of Q, K, V.  Only a caller that wants the whole output on every rank pays a collective afterwards
(``all_gather_heads``: NCCL on GPUs, gloo in the CPU tests); the attention itself launches none.

    lo, hi = head_range(H, rank, world)
    out = forward_local(mask[lo:hi], q[lo:hi], k[lo:hi], v[lo:hi], B_Q, B_KV, N, d)
"""
from __future__ import annotations

from typing import List, Tuple


def head_range(H: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous, balanced split of ``H`` heads: the first ``H % world`` ranks get one head more; a rank beyond the
    number of heads gets an empty range."""
    if H < 0 or world < 1 or not 0 <= rank < world:
        raise ValueError("head_range: need H >= 0 and 0 <= rank < world")
    base, extra = divmod(H, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def head_ranges(H: int, world: int) -> List[Tuple[int, int]]:
    return [head_range(H, r, world) for r in range(world)]


def forward_local(mask, q, k, v, B_Q: int, B_KV: int, N: int, d: int, plan_id: int = -1, N_kv: int = 0,
                  dtype: str = "bf16", cache=None, stream=None):
    """Plan + forward for this rank's heads (CUDA tensors already sliced to them).  Returns ``(O, LSE, plan info)``;
    with no local head the result is empty and nothing is launched.  ``cache``: a ``bsa.PlanCache`` to reuse plans."""
    import torch
    from . import bsa
    h = q.shape[0]
    if h == 0:
        return torch.empty_like(q), torch.empty((0, N), dtype=torch.float32, device=q.device), None
    if cache is not None:
        plan, _ = cache.get(mask, B_Q, B_KV, N, h, d, plan_id=plan_id, stream=stream, N_kv=N_kv, dtype=dtype)
    else:
        plan = bsa.plan_create(mask, B_Q, B_KV, N, h, d, plan_id=plan_id, stream=stream, N_kv=N_kv, dtype=dtype)
    try:
        O, LSE = plan.forward(q, k, v, stream=stream)
        info = plan.info()  # synchronises: the plan may be destroyed afterwards
    finally:
        plan.destroy()
    return O, LSE, info


def all_gather_heads(local, H: int, dist, group=None):
    """Concatenate every rank's ``[h_r, ...]`` tensor along the head axis on every rank.  Ranges may differ by one
    head, so each rank pads to the largest range before the (equal-size) all-gather and the padding is cut off."""
    import torch
    world = dist.get_world_size(group)
    ranges = head_ranges(H, world)
    hmax = max(hi - lo for lo, hi in ranges)
    pad = torch.zeros((hmax,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[: local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    return torch.cat([p[: hi - lo] for p, (lo, hi) in zip(parts, ranges)], dim=0)
