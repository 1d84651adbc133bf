"""Aggregation with the coordinates sharded over several GPUs, one process per GPU.

Every rank holds the same n gradients restricted to its own contiguous range of columns.
Squared distances add over disjoint column sets, so the distance step runs locally on the
slice; the n x n partial matrices (at most 32 KB each) are all-gathered into every rank's own
memory (`torch.distributed`, NCCL over NVLink on GPUs) and added there in rank order, which
gives every rank the bit-identical matrix; the selection is then replicated and the
coordinate phase runs on the local slice.  The output stays sharded the same way.  This is
the only exchange of the whole rule: n*n fp64 values per rank, whatever d is.

The stages are the C entry points of include/gar.h (`gar_pairwise_distances`,
`gar_reduce_partials`, `gar_select`, `gar_coordinate_phase`); `Stages` only names them so
that a host-logic test can run the same orchestration with stand-ins on CPU ranks.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable

import torch
import torch.distributed as dist

from . import binding as B

_NO_DISTANCES = ("average", "median")
_PREAGG = ("average", "multi_krum", "multi_bulyan")


@dataclass
class Stages:
    distances: Callable = B.gar_pairwise_distances            # slice [n, d_local] -> [n, n] float64
    reduce: Callable = B.gar_reduce_partials                  # [world, n, n] -> [n, n], summed in rank order
    select: Callable = B.gar_select                           # (rule, D, n, f) -> selection
    coordinate: Callable = B.gar_coordinate_phase             # (slice, selection, theta, preagg) -> [d_local]
    theta: Callable = B.gar_theta


def gather_partials(part: torch.Tensor, group=None) -> torch.Tensor:
    """All ranks' partial matrices, stacked in rank order: [world, n, n].  Remote data lands in
    this rank's own buffer; the sum is done locally afterwards."""
    world = dist.get_world_size(group)
    parts = [torch.empty_like(part) for _ in range(world)]
    dist.all_gather(parts, part.contiguous(), group=group)
    return torch.stack(parts, dim=0).contiguous()


def sharded_aggregate(rule: str, grads_slice: torch.Tensor, f: int, group=None, stages: Stages | None = None):
    """GAR(f, [G_1..G_n]) of `rule` when this rank holds the columns `grads_slice` ([n, d_local],
    d_local may be 0 on a rank that got no columns).  Returns (out_slice, selection, D): the
    aggregated vector restricted to this rank's columns, the selection every rank made, and
    the full distance matrix (None for the rules that need none)."""
    st = stages or Stages()
    n, d_local = grads_slice.shape
    D = None
    if rule not in _NO_DISTANCES:
        if d_local > 0:
            part = st.distances(grads_slice)
        else:
            part = torch.zeros(n, n, dtype=torch.float64, device=grads_slice.device)
        D = st.reduce(gather_partials(part, group))
    sel = st.select(rule, D, n, f) if D is not None else st.select(rule, None, n, f, device=grads_slice.device)
    theta = st.theta(rule, n, f)
    if d_local > 0:
        out = st.coordinate(grads_slice, sel, theta, int(rule in _PREAGG))
    else:
        out = torch.empty(0, dtype=torch.float32, device=grads_slice.device)
    return out, sel, D
