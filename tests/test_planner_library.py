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
