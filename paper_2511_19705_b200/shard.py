"""Layer-parallel sharding of a weight set over ranks (one process per GPU).

Every matrix (pair) of every decoder layer is an independent optimisation problem, so the data path needs no
collective: rank r takes layers r, r + world, r + 2 world, ...  The only exchanges are a barrier and a
max-reduction of the measured time (and a gather of per-layer results on the host), which this module wraps so
that they can be tested on CPU with the gloo backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def layers_of_rank(n_layers: int, world: int, rank: int) -> list[int]:
    """Round-robin assignment; every layer belongs to exactly one rank."""
    if world < 1 or not (0 <= rank < world):
        raise ValueError("bad world / rank")
    return list(range(rank, n_layers, world))


def max_over_ranks(value: float, device="cpu") -> float:
    """The largest `value` over all ranks (the job's time is its slowest rank's); identity without a process group."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_results(local: dict) -> dict:
    """Union of the per-layer result dictionaries of all ranks (keys = layer indices), on every rank."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return dict(local)
    parts = [None] * dist.get_world_size()
    dist.all_gather_object(parts, local)
    out = {}
    for p in parts:
        for k, v in p.items():
            if k in out:
                raise RuntimeError(f"layer {k} was processed by two ranks")
            out[k] = v
    return out
