"""Reference two-stage planner (Section 5 of arXiv 2207.05022) -- TEST INFRASTRUCTURE ONLY.

Plain Python following the paper's order: compute planning (Section 5.3), then IO planning with
accumulated IO budgets in two passes (Section 5.4), then the preload rule (Section 1: the first shards
in layer order that fit the buffer).  Only tests, the smoke check and the benchmark's CPU leg may
import it; it shares no code with the C++ planner.

Notation: T target latency, N x M stored model, (n, m) submodel, T_comp(m) delay of one layer with m
shards, T_io(k) delay of loading one k-bit shard, S preload buffer, AIB(k) accumulated IO budget.

Readings where the paper is silent (listed with the others in the design notes):
 * which n layers: the first n; which m shards of a layer: the m most important, lower index on ties;
 * pass 1 tries every stored version 2,3,4,5,6,32; if not even 2 bits is valid the plan keeps 2 bits
   and is flagged invalid (the pipeline will stall);
 * pass 2 visits each shard once, most important first, and gives it the highest version that keeps
   every budget from its layer onward non-negative;
 * when the buffer's contents are not given, |S| is first credited as bonus time at the 6-bit version's
   bytes-per-microsecond, the preload prefix is read off that plan, and the plan is redone with it.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

VERSIONS = (2, 3, 4, 5, 6, 32)
EPS = 1e-9


@dataclass
class PlannerResult:
    n: int
    m: int
    pass1_bits: int
    valid: bool
    keep: List[List[int]]       # [N][M]
    bits: List[List[int]]
    preload: List[List[int]]
    aib: List[float]            # [n]


def compute_planning(T: float, N: int, M: int, t_comp: Sequence[float]) -> Optional[Tuple[int, int]]:
    """Section 5.3: all (n, m) with n * T_comp(m) <= T; most shards wins, deeper wins a tie."""
    best = None
    for n in range(1, N + 1):
        for m in range(1, M + 1):
            if n * t_comp[m] <= T + EPS:
                if best is None or n * m > best[0] * best[1] or (n * m == best[0] * best[1] and n > best[0]):
                    best = (n, m)
    return best


def initial_aib(n: int, t_comp_m: float, aib0: float) -> List[float]:
    """Section 5.4: AIB(0) = delay of filling S; AIB(k) = AIB(k-1) + T_comp."""
    aib = [aib0]
    for _ in range(1, n):
        aib.append(aib[-1] + t_comp_m)
    return aib


def charge(aib: List[float], layer: int, delay: float) -> None:
    """A shard of layer k delays layer k and every later layer (Section 5.4, budget update)."""
    for k in range(layer, len(aib)):
        aib[k] -= delay


def is_valid(aib: Sequence[float]) -> bool:
    return all(b >= -EPS for b in aib)


def io_planning(n: int, t_comp_m: float, t_io: Dict[int, float], shards: List[Tuple[int, int]],
                importance: Dict[Tuple[int, int], float], preloaded: Dict[Tuple[int, int], int],
                bonus: float = 0.0):
    """Section 5.4 with S given (`bonus` adds to AIB(0); used only while S is still to be chosen).
    Returns (bits per shard, remaining AIB, pass-1 bitwidth, valid)."""
    aib = initial_aib(n, t_comp_m, bonus + sum(t_io[b] for b in preloaded.values()))
    bits: Dict[Tuple[int, int], int] = {}
    for s, b in preloaded.items():           # fill S' with S first
        bits[s] = b
        charge(aib, s[0], t_io[b])
    todo = [s for s in shards if s not in preloaded]
    uniform = None
    for k in VERSIONS:                        # first pass: lowest version upward
        trial = list(aib)
        for s in todo:
            charge(trial, s[0], t_io[k])
        if not is_valid(trial):
            break
        uniform = k
    valid = uniform is not None
    k1 = uniform if valid else VERSIONS[0]
    for s in todo:
        bits[s] = k1
        charge(aib, s[0], t_io[k1])
    if valid:                                 # second pass: spend what is left by importance
        for s in sorted(todo, key=lambda q: -importance[q]):   # stable: equal scores keep layer order
            higher = [k for k in VERSIONS if VERSIONS.index(k) > VERSIONS.index(bits[s])]
            for k in reversed(higher):
                trial = list(aib)
                charge(trial, s[0], t_io[k] - t_io[bits[s]])
                if is_valid(trial):
                    aib = trial
                    bits[s] = k
                    break
    return bits, aib, k1, valid


def plan(T: float, N: int, M: int, t_comp: Sequence[float], t_io_list: Sequence[float],
         shard_bytes_list: Sequence[int], importance_grid: Sequence[Sequence[float]],
         preload_bytes: int, preloaded_bits: Optional[Sequence[Sequence[int]]] = None) -> PlannerResult:
    t_io = dict(zip(VERSIONS, t_io_list))
    nbytes = dict(zip(VERSIONS, shard_bytes_list))
    nm = compute_planning(T, N, M, t_comp)
    fits = nm is not None
    n, m = nm if fits else (1, 1)
    shards: List[Tuple[int, int]] = []
    for l in range(n):
        ranked = sorted(range(M), key=lambda i: -importance_grid[l][i])
        shards += [(l, i) for i in sorted(ranked[:m])]
    importance = {s: importance_grid[s[0]][s[1]] for s in shards}

    if preloaded_bits is not None:
        S = {s: int(preloaded_bits[s[0]][s[1]]) for s in shards if preloaded_bits[s[0]][s[1]] in VERSIONS}
        bits, aib, k1, valid = io_planning(n, t_comp[m], t_io, shards, importance, S)
    else:
        rate = t_io[6] / nbytes[6] if nbytes[6] else 0.0
        # bonus-budget plan: no shard is marked preloaded yet, AIB(0) = time worth of |S|
        bits0, _, _, _ = io_planning(n, t_comp[m], t_io, shards, importance, {}, bonus=rate * preload_bytes)
        S, used = {}, 0
        for s in shards:                       # first shards in layer order that fit
            if used + nbytes[bits0[s]] > preload_bytes:
                break
            used += nbytes[bits0[s]]
            S[s] = bits0[s]
        bits, aib, k1, valid = io_planning(n, t_comp[m], t_io, shards, importance, S)

    keep = [[0] * M for _ in range(N)]
    bgrid = [[0] * M for _ in range(N)]
    pgrid = [[0] * M for _ in range(N)]
    for s in shards:
        keep[s[0]][s[1]] = 1
        bgrid[s[0]][s[1]] = bits[s]
        pgrid[s[0]][s[1]] = 1 if s in S else 0
    return PlannerResult(n, m, k1, bool(valid and fits), keep, bgrid, pgrid, list(aib))


def retain_after_run(keep: Sequence[Sequence[int]], bits: Sequence[Sequence[int]], shard_bytes_list: Sequence[int],
                     buffer_bytes: int) -> Tuple[List[List[int]], int]:
    """Section 3.2 (caching between back-to-back executions) with Section 5.5's eviction order: loaded
    shards are dropped from the top layer down until what remains fits the buffer.  Returns the grid of
    retained versions (0 = not cached) and the bytes used."""
    nbytes = dict(zip(VERSIONS, shard_bytes_list))
    N, M = len(keep), len(keep[0])
    loaded = [(l, i) for l in range(N) for i in range(M) if keep[l][i]]
    total = sum(nbytes[bits[l][i]] for l, i in loaded)
    while loaded and total > buffer_bytes:          # evict the topmost remaining shard
        l, i = loaded.pop()
        total -= nbytes[bits[l][i]]
    # the walk from the bottom stops at the first shard that does not fit: a shard above an evicted one
    # is evicted too, which the pop-from-the-top loop guarantees
    grid = [[0] * M for _ in range(N)]
    for l, i in loaded:
        grid[l][i] = bits[l][i]
    return grid, total
