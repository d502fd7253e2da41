"""Two-stage planner oracle (Section 5.3, 5.4) against the paper's worked example, an event-by-event
pipeline simulation and brute force.  No GPU needed."""
import itertools

import numpy as np
import pytest

from oracle import sti_planner_oracle as po

VERS = po.VERSIONS


# ---------------------------------------------------------------------------------------------
# an independent check of validity: play the IO/compute pipeline of Section 5.5 event by event
# ---------------------------------------------------------------------------------------------
def simulate_pipeline(n, t_comp_m, t_io, bits, preload):
    """IO loads the non-preloaded shards one after another in layer order from time 0; layer k computes
    once layer k-1 is done and all its shards have arrived.  Returns (finish time, total stall)."""
    io_clock, done, stall = 0.0, 0.0, 0.0
    for l in range(n):
        for i, b in enumerate(bits[l]):
            if b and not preload[l][i]:
                io_clock += t_io[b]
        start = max(done, io_clock)
        stall += start - done
        done = start + t_comp_m
    return done, stall


def random_instance(rng, N=None, M=None):
    N = N or int(rng.integers(1, 7))
    M = M or int(rng.integers(1, 6))
    base = rng.uniform(0.5, 2.0)
    t_comp = [0.0] + list(np.cumsum(rng.uniform(0.2, 1.0, M)) + base)       # increasing in m
    per_bit = rng.uniform(0.05, 0.4)
    t_io = [per_bit * b + rng.uniform(0, 0.05) for b in VERS]
    t_io = list(np.maximum.accumulate(t_io))
    nbytes = [int(1000 * b) + 64 for b in VERS]
    imp = rng.uniform(0, 1, (N, M)).round(3)
    T = float(rng.uniform(0.5, 1.5) * N * t_comp[M] * rng.uniform(0.2, 1.2))
    S = int(rng.integers(0, 3 * M) * 3000)
    return dict(T=T, N=N, M=M, t_comp=t_comp, t_io=t_io, nbytes=nbytes, imp=imp, S=S)


def run_oracle(inst, preloaded=None):
    return po.plan(inst["T"], inst["N"], inst["M"], inst["t_comp"], inst["t_io"], inst["nbytes"],
                   inst["imp"].tolist(), inst["S"], preloaded)


# ------------------------------------------------------------------ pins from the paper's text
def test_aib_worked_example():
    """Section 5.4's mini example: 2x3 submodel, T = 2 s, T_comp = 1 s, three 2-bit shards of layer 0
    preloaded (0.6 s, so 0.2 s each): budgets start at 0.6 / 1.6 s, are 0 / 1.0 s once S is placed,
    and a candidate that costs layer 1 1.1 s ends at -0.1 s and is rejected."""
    aib = po.initial_aib(2, 1.0, 0.6)
    assert aib == pytest.approx([0.6, 1.6])
    for _ in range(3):
        po.charge(aib, 0, 0.2)
    assert aib == pytest.approx([0.0, 1.0])
    ok = list(aib)
    po.charge(ok, 1, 1.0)
    assert po.is_valid(ok) and ok[1] == pytest.approx(0.0)
    bad = list(aib)
    po.charge(bad, 1, 1.1)
    assert bad[1] == pytest.approx(-0.1) and not po.is_valid(bad)
    # no spare budget in layer 0: any further layer-0 shard is rejected
    l0 = list(aib)
    po.charge(l0, 0, 0.2)
    assert not po.is_valid(l0)


def test_two_passes_on_the_example_geometry():
    """Same geometry, passes of Section 5.4: 3-bit (0.3 s) x 3 = 0.9 s fits in 1.0 s, 4-bit (0.4 s) x 3
    does not, so pass 1 picks 3; the 0.1 s left upgrades the single most important shard to 4 bits."""
    t_io = {2: 0.2, 3: 0.3, 4: 0.4, 5: 0.5, 6: 0.6, 32: 3.2}
    shards = [(l, i) for l in range(2) for i in range(3)]
    imp = {s: 0.1 for s in shards}
    imp[(1, 2)] = 0.9
    S = {(0, 0): 2, (0, 1): 2, (0, 2): 2}
    bits, aib, k1, valid = po.io_planning(2, 1.0, t_io, shards, imp, S)
    assert valid and k1 == 3
    assert [bits[(1, i)] for i in range(3)] == [3, 3, 4]
    assert [bits[(0, i)] for i in range(3)] == [2, 2, 2]
    assert aib == pytest.approx([0.0, 0.0])


def test_too_small_budget_keeps_two_bits_and_stops():
    """Section 5.4: if not even 2-bit shards fit they are still chosen and allocation stops."""
    t_io = {2: 0.6, 3: 0.7, 4: 0.8, 5: 0.9, 6: 1.0, 32: 4.0}
    shards = [(l, i) for l in range(2) for i in range(3)]
    bits, aib, k1, valid = po.io_planning(2, 1.0, t_io, shards, {s: 1.0 for s in shards}, {})
    assert not valid and k1 == 2 and set(bits.values()) == {2}
    assert min(aib) < 0


def test_compute_planning_prefers_more_shards_then_depth():
    """Section 5.3: most shards first, the deeper submodel on a tie."""
    t_comp = [0.0] + [float(m) for m in range(1, 7)]                       # T_comp(m) = m
    assert po.compute_planning(12.0, 6, 6, t_comp) == (6, 2)               # (2,6),(3,4),(4,3),(6,2) tie -> deepest
    assert po.compute_planning(12.0, 3, 6, t_comp) == (3, 4)
    assert po.compute_planning(11.9, 3, 6, t_comp) == (2, 5)               # 10 shards beat (3,3) = 9
    assert po.compute_planning(0.5, 3, 6, t_comp) is None
    flat = [0.0] + [1.0] * 6                                               # width is free: always all M
    assert po.compute_planning(2.5, 6, 6, flat) == (2, 6)


# ------------------------------------------------------------------ properties and brute force
@pytest.mark.parametrize("seed", range(40))
def test_valid_plans_never_stall_and_are_maximal(seed):
    rng = np.random.default_rng(seed)
    inst = random_instance(rng)
    r = run_oracle(inst)
    t_io = dict(zip(VERS, inst["t_io"]))
    tc = inst["t_comp"][r.m]
    # the submodel: first n layers, the m most important shards of each
    for l in range(inst["N"]):
        assert sum(r.keep[l]) == (r.m if l < r.n else 0)
        if l < r.n:
            kept = [i for i in range(inst["M"]) if r.keep[l][i]]
            dropped = [i for i in range(inst["M"]) if not r.keep[l][i]]
            assert all(inst["imp"][l][a] >= inst["imp"][l][b] for a in kept for b in dropped)
    # preload = a prefix of the kept shards in layer order, within |S|
    order = [(l, i) for l in range(r.n) for i in range(inst["M"]) if r.keep[l][i]]
    flags = [r.preload[l][i] for l, i in order]
    assert flags == sorted(flags, reverse=True)
    used = sum(inst["nbytes"][VERS.index(r.bits[l][i])] for (l, i), f in zip(order, flags) if f)
    assert used <= inst["S"]
    finish, stall = simulate_pipeline(r.n, tc, t_io, r.bits, r.preload)
    if r.valid:
        assert stall == pytest.approx(0.0, abs=1e-7)
        assert finish <= inst["T"] + 1e-7
        assert min(r.aib) >= -1e-9
        # budgets consumed: no streamed shard can move up one version without a stall
        for l, i in order:
            if r.preload[l][i] or r.bits[l][i] == 32:
                continue
            up = [row[:] for row in r.bits]
            up[l][i] = VERS[VERS.index(r.bits[l][i]) + 1]
            if t_io[up[l][i]] > t_io[r.bits[l][i]] + 1e-9:
                assert simulate_pipeline(r.n, tc, t_io, up, r.preload)[1] > 1e-9
        # pass 1 is the highest uniform version the pipeline sustains for the streamed shards
        best = None
        for k in VERS:
            uni = [[(r.bits[l][i] if r.preload[l][i] else k) if r.keep[l][i] else 0
                    for i in range(inst["M"])] for l in range(inst["N"])]
            if simulate_pipeline(r.n, tc, t_io, uni, r.preload)[1] <= 1e-9:
                best = k
            else:
                break
        if any(not f for f in flags):
            assert r.pass1_bits == best
            assert all(VERS.index(r.bits[l][i]) >= VERS.index(best) for (l, i), f in zip(order, flags) if not f)


def test_brute_force_compute_planning():
    rng = np.random.default_rng(7)
    for _ in range(50):
        inst = random_instance(rng)
        cands = [(n, m) for n in range(1, inst["N"] + 1) for m in range(1, inst["M"] + 1)
                 if n * inst["t_comp"][m] <= inst["T"]]
        got = po.compute_planning(inst["T"], inst["N"], inst["M"], inst["t_comp"])
        if not cands:
            assert got is None
            continue
        top = max(n * m for n, m in cands)
        assert got == max((c for c in cands if c[0] * c[1] == top), key=lambda c: c[0])


def test_importance_pass_matches_exhaustive_greedy_on_tiny_case():
    """Tiny case, every assignment enumerated: the plan is the lexicographically best (in importance
    order) among the valid assignments at or above the uniform level."""
    t_io = {2: 0.2, 3: 0.3, 4: 0.45, 5: 0.5, 6: 0.7, 32: 2.0}
    shards = [(0, 0), (1, 0), (1, 1), (2, 0)]
    imp = {(0, 0): 0.2, (1, 0): 0.9, (1, 1): 0.4, (2, 0): 0.7}
    bits, aib, k1, valid = po.io_planning(3, 1.0, t_io, shards, imp, {}, bonus=0.25)
    assert valid
    ranked = sorted(shards, key=lambda s: -imp[s])
    best = None
    for combo in itertools.product(VERS, repeat=len(shards)):
        if any(VERS.index(b) < VERS.index(k1) for b in combo):
            continue
        a = po.initial_aib(3, 1.0, 0.25)
        for s, b in zip(shards, combo):
            po.charge(a, s[0], t_io[b])
        if not po.is_valid(a):
            continue
        key = tuple(VERS.index(dict(zip(shards, combo))[s]) for s in ranked)
        if best is None or key > best:
            best = key
    assert tuple(VERS.index(bits[s]) for s in ranked) == best


def test_more_time_never_shrinks_the_submodel():
    rng = np.random.default_rng(3)
    inst = random_instance(rng, N=6, M=5)
    sizes = []
    for T in np.linspace(0.2, 1.5, 14) * inst["N"] * inst["t_comp"][inst["M"]]:
        inst["T"] = float(T)
        r = run_oracle(inst)
        sizes.append(r.n * r.m)
    assert sizes == sorted(sizes)


# ------------------------------------------------------------------ caching between back-to-back runs
def test_retained_shards_are_the_longest_bottom_up_prefix_that_fits():
    """Section 5.5: eviction goes from the top layer down until the buffer is filled, so what stays is a
    prefix of the loaded shards in layer order; checked against brute force over all prefixes."""
    rng = np.random.default_rng(21)
    for _ in range(60):
        inst = random_instance(rng)
        r = run_oracle(inst)
        order = [(l, i) for l in range(inst["N"]) for i in range(inst["M"]) if r.keep[l][i]]
        sizes = [inst["nbytes"][VERS.index(r.bits[l][i])] for l, i in order]
        budget = int(rng.integers(0, sum(sizes) + 2000))
        grid, used = po.retain_after_run(r.keep, r.bits, inst["nbytes"], budget)
        best = max(k for k in range(len(order) + 1) if sum(sizes[:k]) <= budget)
        kept = [(l, i) for l, i in order if grid[l][i]]
        assert kept == order[:best] and used == sum(sizes[:best])
        assert all(grid[l][i] == r.bits[l][i] for l, i in kept)
    assert po.retain_after_run([[1, 1]], [[2, 3]], [10, 20, 30, 40, 50, 60], 0) == ([[0, 0]], 0)
    assert po.retain_after_run([[1, 1]], [[2, 3]], [10, 20, 30, 40, 50, 60], 29) == ([[2, 0]], 10)
    assert po.retain_after_run([[1, 1]], [[2, 3]], [10, 20, 30, 40, 50, 60], 30) == ([[2, 3]], 30)


def test_replanning_with_cached_shards_spends_the_freed_io_time():
    """Section 3.2: with more shards cached the next plan stays stall-free (pipeline simulation) and no
    streamed shard gets a lower uniform version than before."""
    rng = np.random.default_rng(22)
    for _ in range(40):
        inst = random_instance(rng, N=int(rng.integers(2, 7)), M=int(rng.integers(2, 6)))
        first = run_oracle(inst)
        if not first.valid:
            continue
        t_io = dict(zip(VERS, inst["t_io"]))
        grown = inst["S"] + int(rng.integers(1, 6)) * 4000
        cached, _ = po.retain_after_run(first.keep, first.bits, inst["nbytes"], grown)
        second = run_oracle(inst, cached)
        assert (second.n, second.m) == (first.n, first.m) and second.valid
        assert second.preload == [[1 if c else 0 for c in row] for row in cached]
        assert all(second.bits[l][i] == cached[l][i] for l in range(inst["N"]) for i in range(inst["M"]) if cached[l][i])
        assert simulate_pipeline(second.n, inst["t_comp"][second.m], t_io, second.bits, second.preload)[1] <= 1e-7
        if any(k and not c for kr, cr in zip(second.keep, cached) for k, c in zip(kr, cr)):
            assert VERS.index(second.pass1_bits) >= VERS.index(first.pass1_bits)
