"""The library's two-stage planner (sti_plan_auto) equals the oracle planner exactly.  No GPU needed."""
import numpy as np
import pytest

from oracle import sti_planner_oracle as po
from test_planner_oracle import random_instance, run_oracle

VERS = po.VERSIONS


@pytest.fixture(scope="module")
def sti():
    from paper_2207_05022_b200 import build
    build.build_library()
    import paper_2207_05022_b200 as pkg
    return pkg


@pytest.mark.parametrize("given_buffer", [False, True])
def test_library_planner_equals_oracle(sti, given_buffer):
    rng = np.random.default_rng(11 + given_buffer)
    for _ in range(150):
        inst = random_instance(rng)
        pre = None
        if given_buffer:
            pre = np.zeros((inst["N"], inst["M"]), np.uint8)
            k = int(rng.integers(0, inst["N"] * inst["M"] + 1))
            flat = pre.reshape(-1)
            flat[:k] = rng.choice(VERS, size=k)
        want = run_oracle(inst, None if pre is None else pre.tolist())
        got = sti.sti_plan_auto(inst["T"], inst["N"], inst["M"], inst["t_comp"], inst["t_io"], inst["nbytes"],
                                inst["imp"], inst["S"], pre)
        assert (got["n"], got["m"], got["pass1_bits"], got["valid"]) == (want.n, want.m, want.pass1_bits, want.valid)
        assert got["keep"].tolist() == want.keep
        assert got["bits"].tolist() == want.bits
        assert got["preload"].tolist() == want.preload
        np.testing.assert_allclose(got["aib_us"][:want.n], want.aib, rtol=0, atol=1e-9)


def test_library_planner_rejects_bad_arguments(sti):
    import ctypes as C
    lib = sti.load_library()
    assert lib.sti_plan_auto(None, None, None) == 1
    with pytest.raises(sti.StiError):
        sti.sti_plan_auto(-1.0, 2, 2, [0, 1, 2], [1, 2, 3, 4, 5, 6], [1] * 6, np.ones((2, 2)), 0)
    with pytest.raises(sti.StiError):                                      # IO delays must not decrease with bits
        sti.sti_plan_auto(5.0, 2, 2, [0, 1, 2], [6, 5, 4, 3, 2, 1], [1] * 6, np.ones((2, 2)), 0)
    with pytest.raises(ValueError):
        sti.sti_plan_auto(5.0, 2, 2, [0, 1], [1, 2, 3, 4, 5, 6], [1] * 6, np.ones((2, 2)), 0)
    del C


def test_library_retention_equals_oracle(sti):
    rng = np.random.default_rng(31)
    for _ in range(100):
        inst = random_instance(rng)
        r = run_oracle(inst)
        total = sum(inst["nbytes"][VERS.index(b)] for row in r.bits for b in row if b)
        budget = int(rng.integers(0, total + 3000))
        want, want_used = po.retain_after_run(r.keep, r.bits, inst["nbytes"], budget)
        got, used = sti.sti_preload_after_run(np.array(r.keep), np.array(r.bits), inst["nbytes"], budget)
        assert got.tolist() == want and used == want_used
    with pytest.raises(sti.StiError):                                      # a kept shard with an unknown version
        sti.sti_preload_after_run(np.ones((1, 2)), np.array([[2, 7]]), [1] * 6, 10)
