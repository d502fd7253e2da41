"""Execution modes must not change results: CUDA-graph replay vs plain stream launches, programmatic
dependent launch on/off, repeated forwards, and the plain-ALU debug GEMM vs the tensor-core GEMM."""
import os

import numpy as np
import pytest

import workloads as W
from workloads.shards import ATTN, FFN
from oracle import sti_oracle as O

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _workload():
    shape = W.ModelShape(n_layers=4, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    bits = [2, 3, 4, 5, 6]
    attn = [[W.UnitPlan((l + i) % 3 != 0, bits[(l + i) % 5], l < 2) for i in range(4)] for l in range(4)]
    ffn = [[W.UnitPlan((l + i) % 4 != 1, bits[(l + 2 * i) % 5], l < 2) for i in range(4)] for l in range(4)]
    return W.build_workload("modes", shape, 2, 150, "f32", attn, ffn, seed=31, ring_slots=2)


def _run(work, env):
    from gpu_util import run_model
    old = {k: os.environ.get(k) for k in env}
    os.environ.update(env)
    try:
        with sti.Session(work) as s:           # the switches are read when the context / plan is set up
            first = run_model(s, work)
            second = run_model(s, work)        # with graphs on, this one replays the captured graph
            launches = sti.sti_ctx_launch_count(s.ctx)
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    assert np.array_equal(first, second)
    return first, launches


def test_graph_and_dependent_launch_modes_are_bit_identical():
    from gpu_util import rel_err, REL_TOL
    work = _workload()
    ref = O.run_workload(work)
    base, n_base = _run(work, {})
    assert rel_err(base, ref) <= REL_TOL
    for env in ({"STI_NO_GRAPH": "1"}, {"STI_NO_PDL": "1"}, {"STI_NO_GRAPH": "1", "STI_NO_PDL": "1"}):
        y, n = _run(work, env)
        assert np.array_equal(y, base), env
        assert n == n_base, env                  # the launch accounting does not depend on the mode
    y_simt, _ = _run(work, {"STI_DEBUG_SIMT": "1", "STI_NO_GRAPH": "1"})
    assert rel_err(y_simt, ref) <= REL_TOL
    assert rel_err(y_simt, base) <= 2e-3         # same bf16 operands, only the summation order differs


def test_tile_shapes_do_not_change_results_beyond_rounding():
    from gpu_util import rel_err, REL_TOL
    work = _workload()
    ref = O.run_workload(work)
    for tune in ("qkv_n=32,f1_n=32,o_group=1,f2_group=1", "qkv_n=64,f1_n=128,o_group=16,f2_group=4,f2_n=128,o_n=128",
                 "ln1_ctas=1,ln2_ctas=40",        # LayerNorm rows packed 16 per CTA / two float4 per thread
                 "ln1_ctas=0,ln2_ctas=0"):        # one row per CTA
        y, _ = _run(work, {"STI_TUNE": tune})
        assert rel_err(y, ref) <= REL_TOL, tune


def test_load_then_execute_order_gives_the_same_result():
    """The Load&Exec order (every streamed layer copied before layer 0 starts) against the layerwise pipeline."""
    from gpu_util import run_model
    work = _workload()                                   # layers 2 and 3 streamed
    with sti.Session(work) as s:                         # two ring slots = two streamed layers
        piped = run_model(s, work)
        sti.sti_plan_set_overlap(s.plan, False)
        loaded_first = run_model(s, work)
        again = run_model(s, work)
        sti.sti_plan_set_overlap(s.plan, True)
        back = run_model(s, work)
    assert np.array_equal(piped, loaded_first) and np.array_equal(piped, again) and np.array_equal(piped, back)
    # one slot per streamed layer is required: three streamed layers do not fit two slots
    import dataclasses
    attn = [[dataclasses.replace(u, resident=l < 1) for u in row] for l, row in enumerate(work.attn_plan)]
    ffn = [[dataclasses.replace(u, resident=l < 1) for u in row] for l, row in enumerate(work.ffn_plan)]
    with sti.Session(dataclasses.replace(work, attn_plan=attn, ffn_plan=ffn)) as s:
        with pytest.raises(sti.StiError) as err:
            sti.sti_plan_set_overlap(s.plan, False)
        assert "state" in str(err.value)
