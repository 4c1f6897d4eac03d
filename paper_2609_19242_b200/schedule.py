"""Host-side CSBP partition (appendix B): which corrupted blocks and which clean positions a rank owns.

Dual-end block parallelism pairs block b with block B-1-b (0-indexed), because the attention work of a
block grows linearly with its index and the two of a pair add up to the same amount for every pair
(Eq. aligned-pair-work).  Complete pairs are dealt out as evenly as possible; an unpaired middle block
goes to the rank with the least work so far.  The clean sequence is cut into 2P chunks and rank r owns
chunks r and 2P-1-r (zigzag), the same early-late pairing.  This module only builds index lists and the
per-rank tables the packed attention calls take; it does no attention arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple


def block_work(b: int, M: int) -> int:
    """Visible (query, key) pairs of the M corrupted queries of 0-indexed block b: (b+1) M^2
    (Eq. block-work-by-position with the paper's 1-indexed b)."""
    return (b + 1) * M * M


def dual_end_blocks(n_blocks: int, P: int, block_size: int = 1) -> List[List[int]]:
    """B_r for r = 0..P-1: sorted block indices owned by each rank."""
    if n_blocks <= 0 or P <= 0:
        raise ValueError("n_blocks and P must be positive")
    owned: List[List[int]] = [[] for _ in range(P)]
    load = [0] * P
    n_pairs = n_blocks // 2
    for p in range(n_pairs):
        r = p % P                                   # every pair carries the same work: round robin is even
        for b in (p, n_blocks - 1 - p):
            owned[r].append(b)
            load[r] += block_work(b, block_size)
    if n_blocks % 2 == 1:
        mid = n_blocks // 2
        r = min(range(P), key=lambda x: (load[x], x))
        owned[r].append(mid)
        load[r] += block_work(mid, block_size)
    return [sorted(x) for x in owned]


def zigzag_chunks(L: int, P: int) -> List[List[Tuple[int, int]]]:
    """C_r for r = 0..P-1 as position ranges [(begin, end), (begin, end)]: chunks r and 2P-1-r of 2P."""
    if L % (2 * P) != 0:
        raise ValueError("L must be divisible by 2P for zigzag sharding")
    c = L // (2 * P)
    return [[(r * c, (r + 1) * c), ((2 * P - 1 - r) * c, (2 * P - r) * c)] for r in range(P)]


@dataclass(frozen=True)
class RankPlan:
    rank: int
    blocks: List[int]                       # owned corrupted blocks, ascending
    block_prefix: List[int]                 # clean keys visible to each owned block: block index * M
    clean_ranges: List[Tuple[int, int]]     # owned clean query positions


def csbp_plan(L: int, block_size: int, P: int) -> List[RankPlan]:
    """The per-rank launch description of Algorithm 1: packed blocks with their prefix table, and the
    clean position ranges, for every rank."""
    if L % block_size != 0:
        raise ValueError("L must be a multiple of block_size")
    B = L // block_size
    blocks = dual_end_blocks(B, P, block_size)
    chunks = zigzag_chunks(L, P)
    return [RankPlan(r, blocks[r], [b * block_size for b in blocks[r]], chunks[r]) for r in range(P)]
