"""Host-side plumbing for running on several GPUs: which rank owns which matrices, and how per-rank
timings are combined.  No optimizer arithmetic lives here.

Every matrix's update is independent of every other matrix (Algorithm 1 is written per parameter), so the
step shards by whole matrices with no data-path collective.  Two uses:

  * weak scaling (the benchmark): every rank owns a full parameter set of the same shape;
  * a ZeRO-1-style deployment (the distributed Muon scheme the paper's related-work section cites): one
    parameter set is split across ranks with `partition()`, each rank steps the matrices it owns
    (`local_views()` gives the slices of the full tensors, which is what a handle is built over), and
    `exchange()` then brings every rank's copy of the parameters up to date - one broadcast per owned slice,
    in place, no staging copy.  That exchange is the only collective; it follows the step, it is not fused
    with it (there is no computation left to overlap it with).
"""
from __future__ import annotations

import os
from dataclasses import dataclass
from typing import List, Sequence, Tuple


@dataclass(frozen=True)
class Share:
    """Matrices [start, start + count) of stacked descriptor `spec` (count >= 1)."""
    spec: int
    start: int
    count: int


def step_cost(rows: int, cols: int, ns_steps: int = 5) -> float:
    """Relative cost of one matrix per step: Newton-Schulz flops (4 s^2 l + 2 s^3 per iteration) plus the
    elementwise passes expressed in the same unit (40 bytes per element at ~200 flop per byte)."""
    s, l = min(rows, cols), max(rows, cols)
    return ns_steps * (4.0 * s * s * l + 2.0 * s ** 3) + 8000.0 * rows * cols


def partition(shapes: Sequence[Tuple[int, int, int]], world: int, ns_steps: int = 5) -> List[List[Share]]:
    """Splits descriptors `shapes[i] = (batch, rows, cols)` over `world` ranks by whole matrices.

    Stacked descriptors are cut into contiguous slices (an even share per rank first); what is left over is
    placed largest-first on the least loaded rank.  Every matrix lands on exactly one rank; the load of two
    ranks differs by at most the cost of the most expensive single matrix."""
    if world < 1:
        raise ValueError("world must be >= 1")
    load = [0.0] * world
    out: List[List[Share]] = [[] for _ in range(world)]
    leftovers = []   # (cost, spec, index)
    for i, (batch, rows, cols) in enumerate(shapes):
        c = step_cost(rows, cols, ns_steps)
        even = batch // world
        if even:
            for r in range(world):
                out[r].append(Share(i, r * even, even))
                load[r] += even * c
        for b in range(even * world, batch):
            leftovers.append((c, i, b))
    leftovers.sort(key=lambda t: (-t[0], t[1], t[2]))
    for c, i, b in leftovers:
        r = min(range(world), key=lambda k: (load[k], k))
        last = out[r][-1] if out[r] else None
        if last is not None and last.spec == i and last.start + last.count == b:
            out[r][-1] = Share(i, last.start, last.count + 1)
        else:
            out[r].append(Share(i, b, 1))
        load[r] += c
    return out


def loads(shapes: Sequence[Tuple[int, int, int]], shares: List[List[Share]], ns_steps: int = 5) -> List[float]:
    return [sum(sh.count * step_cost(shapes[sh.spec][1], shapes[sh.spec][2], ns_steps) for sh in rank) for rank in shares]


def local_views(tensors, shares: Sequence[Share]):
    """The slices of the full per-descriptor tensors (batch, rows, cols) that `shares` names, as views:
    stepping them steps the owner's part of the full parameter set in place."""
    return [tensors[sh.spec][sh.start: sh.start + sh.count] for sh in shares]


def share_shapes(shapes: Sequence[Tuple[int, int, int]], shares: Sequence[Share]) -> List[Tuple[int, int, int]]:
    """(count, rows, cols) of every share: the descriptor list of the owner's handle."""
    return [(sh.count, shapes[sh.spec][1], shapes[sh.spec][2]) for sh in shares]


def exchange(params, all_shares: List[List[Share]], dist=None) -> int:
    """After every rank has stepped the matrices it owns: make all ranks' full parameter tensors equal by
    broadcasting each owned slice from its owner, in place.  `params` are this rank's full tensors
    (batch, rows, cols).  Returns the bytes this rank received.  With dist=None (one process) there is nothing
    to do.  Slices are contiguous (stacked descriptors are cut along the batch axis), so no packing is needed;
    the broadcasts are issued asynchronously and waited for together."""
    if dist is None or len(all_shares) == 1:
        return 0
    me = dist.get_rank()
    works, received = [], 0
    for owner, lst in enumerate(all_shares):
        for sh in lst:
            view = params[sh.spec][sh.start: sh.start + sh.count]
            works.append(dist.broadcast(view, src=owner, async_op=True))
            if owner != me:
                received += view.numel() * view.element_size()
    for w in works:
        w.wait()
    return received


def env_rank() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) for a plain launch."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")))


def max_over_ranks(value: float, dist=None, device=None) -> float:
    """The slowest rank's figure: what a whole-job time is.  `dist` is torch.distributed (already
    initialised) or None for a single process."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, slowest_seconds: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return units_per_rank * world / slowest_seconds
