"""CPU oracle of the shard selection under a cache budget (Section 3.2, last paragraph).

TEST INFRASTRUCTURE ONLY (see ``ciera_oracle.py``); plain Python loops, no tuning.

What Section 3.2 defines: every shard has a gain g_i (seconds saved per iteration if it is
compressed) and costs M_i = (W - 1) * S_e^i bytes of exponent cache on each GPU.  Candidates are the
shards whose gain is positive; they are taken in order of gain per cached byte, best first, as long
as the budget allows.

Readings taken here (the paper gives no pseudo-code for this step):
  * ties in g_i / M_i keep the shards' original order;
  * "until the budget is exhausted" = walk down the ranking and stop at the first shard that no
    longer fits (a plain greedy prefix; later, smaller shards are not tried);
  * a shard without values (M_i = 0) is never selected.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple


def cache_footprint(n_values: int, world_size: int, with_sender_cache: bool = False) -> int:
    """M_i = (W - 1) * S_e^i, S_e^i = one exponent byte per value.  ``with_sender_cache`` adds the
    S_e^i of a sender-side exponent cache (exact comparison in place of the block hash)."""
    return (world_size - 1 + (1 if with_sender_cache else 0)) * n_values


def select_shards(gains: Sequence[float], footprints: Sequence[int], budget: int) -> Tuple[List[int], List[bool], int]:
    """Returns (ranking, selected flags, cache bytes used)."""
    n = len(gains)
    assert len(footprints) == n
    candidates = [i for i in range(n) if gains[i] > 0.0 and footprints[i] > 0]
    rest = [i for i in range(n) if not (gains[i] > 0.0 and footprints[i] > 0)]
    # descending g_i / M_i; Python's sort is stable, so ties keep the original order
    ranking = sorted(candidates, key=lambda i: -(gains[i] / footprints[i])) + rest
    selected = [False] * n
    used = 0
    for i in ranking[: len(candidates)]:
        if used + footprints[i] > budget:
            break
        selected[i] = True
        used += footprints[i]
    return ranking, selected, used
