"""Host-side sharding of the candidate space over ranks (one process per GPU).

Candidates are independent, so a rank evaluates a contiguous range of candidate indices and
the only exchange is one (cost, index) pair per rank followed by a lexicographic minimum.
Ranges are balanced by the recurrence work of their candidates, which depends on the number of
pipeline stages of the owning configuration.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import numpy as np


def recurrence_cells(N: int, PP: int) -> float:
    """Cell updates of the plain recurrence for one candidate (no window)."""
    if PP == 1:
        return 1.0
    w = N - PP + 1
    return 2.0 * w + (PP - 2) * w * (w + 1) / 2.0


def shard_ranges(pconfs: np.ndarray, n_rc: int, N: int, world: int, overhead: float = 256.0) -> List[Tuple[int, int]]:
    """Splits [0, n_cand) into `world` contiguous (first, count) ranges of about equal work.

    `pconfs` is the configuration table (fields PP, nmap, offset); a candidate's work is the
    recurrence cell count of its configuration plus a constant per-candidate overhead."""
    nmap = pconfs["nmap"].astype(np.float64) * n_rc
    per = np.array([recurrence_cells(N, int(pp)) + overhead for pp in pconfs["PP"]])
    cum = np.concatenate([[0.0], np.cumsum(nmap * per)])
    total = cum[-1]
    n_cand = int(pconfs["offset"][-1]) + int(pconfs["nmap"][-1]) * n_rc
    cuts = [0]
    for r in range(1, world):
        target = total * r / world
        p = int(np.searchsorted(cum, target, side="right") - 1)
        p = min(max(p, 0), len(per) - 1)
        inside = int((target - cum[p]) / per[p])
        cut = int(pconfs["offset"][p]) + min(inside, int(nmap[p]))
        cuts.append(max(cut, cuts[-1]))
    cuts.append(n_cand)
    return [(cuts[r], cuts[r + 1] - cuts[r]) for r in range(world)]


def combine_minima(pairs: Sequence[Tuple[int, int]]) -> Tuple[int, int]:
    """Lexicographic minimum of (cost, index) pairs: lowest cost, lowest index on ties."""
    return min(pairs)


def exchange_minimum(cost: int, index: int, device=None) -> Tuple[int, int]:
    """All-gathers one (cost, index) pair per rank over torch.distributed and reduces it locally.

    Works with NCCL (CUDA tensors) and gloo (CPU tensors); with one process it is the identity."""
    import torch
    import torch.distributed as dist
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return cost, index
    mine = torch.tensor([cost, index], dtype=torch.int64, device=device)
    gathered = [torch.empty_like(mine) for _ in range(dist.get_world_size())]
    dist.all_gather(gathered, mine)
    return combine_minima([(int(g[0]), int(g[1])) for g in gathered])


NO_CANDIDATE = (1 << 62, (1 << 63) - 1)      # what a rank with an empty range contributes


def exchange_minimum_tensor(pair, first: int):
    """The same exchange without a host round trip: `pair` is the rank's (cost, index within its range) as a
    2-element int64 tensor on the device the process group communicates on (what hap_argmin returns; NO_CANDIDATE for
    an empty range); `first` is the start of the rank's range.  Returns the global (cost, index) as a tensor on that
    device; nothing is read back here, so the caller decides when to synchronise."""
    import torch
    import torch.distributed as dist
    mine = pair.clone()
    mine[1] = torch.where(mine[0] < NO_CANDIDATE[0], mine[1] + first, mine[1])      # "no candidate" keeps its index
    if not dist.is_available() or not dist.is_initialized() or dist.get_world_size() == 1:
        return mine
    world = dist.get_world_size()
    gathered = torch.empty((world, 2), dtype=torch.int64, device=mine.device)
    dist.all_gather_into_tensor(gathered, mine.reshape(1, 2))
    cost = gathered[:, 0]
    best = cost.min()
    index = torch.where(cost == best, gathered[:, 1], torch.full_like(cost, NO_CANDIDATE[1])).min()
    return torch.stack([best, index])
