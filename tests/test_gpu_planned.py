"""A plan produced by sti_plan_auto, executed by the layer pipeline, equals the oracle's forward of the
same plan: a submodel that is narrower than the store, mixed versions including raw 32-bit shards, and a
preload prefix that ends in the middle of a layer."""
import numpy as np
import pytest

import workloads as W
from oracle import sti_oracle as O

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


def test_planned_submodel_matches_oracle():
    from paper_2207_05022_b200 import build
    from gpu_util import run_model, rel_err, REL_TOL
    build.build_library()
    N, M = 24, 16
    # synthetic device tables: 3 layers of 12 shards fit the target; budgets leave room for upgrades
    t_comp = [0.0] + [40.0 + 2.0 * m for m in range(1, M + 1)]
    t_io = [1.0, 1.5, 2.0, 2.5, 3.0, 16.0]
    nbytes = [197828, 296164, 394500, 492836, 591172, 3145728]
    imp = np.random.default_rng(5).uniform(0, 1, (N, M)).astype(np.float32)
    plan = sti.sti_plan_auto(3 * 64.0 + 1.0, N, M, t_comp, t_io, nbytes, imp, 9_000_000)
    assert (plan["n"], plan["m"]) == (3, 12) and plan["valid"]
    kept = plan["bits"][plan["keep"] > 0]
    assert len(np.unique(kept)) >= 2                                   # pass 2 raised some shards
    assert 0 < plan["preload"][1].sum() < 12                           # prefix ends inside layer 1
    work = W.make_planned(plan["keep"], plan["bits"], plan["preload"], batch=2, seq=48, workers=3)
    ref = O.run_workload(work)
    with sti.Session(work) as s:
        y = run_model(s, work)
        y2 = run_model(s, work)
        mem = sti.sti_plan_memory(s.plan)
    assert np.array_equal(y, y2)
    assert mem["preload_bytes"] > 0 and mem["pinned_bytes"] > 0
    e = rel_err(y, ref)
    print("planned 3x12 submodel rel err: %.3e" % e)
    assert e <= REL_TOL
