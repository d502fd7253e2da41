"""Host-made faults (no GPU fault, trap or hang anywhere): a shard copy that reaches the copy engine late, a pinned
allocation that fails, and a bad argument that must not change how later forwards run."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import ATTN, FFN

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _work(n_layers=4, resident_layers=1, seq=64):
    shape = W.ModelShape(n_layers=n_layers, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    attn = [[W.UnitPlan(True, 3 + (l + i) % 3, l < resident_layers) for i in range(4)] for l in range(n_layers)]
    ffn = [[W.UnitPlan(True, 2 + (l + i) % 4, l < resident_layers) for i in range(4)] for l in range(n_layers)]
    return W.build_workload("faults", shape, 1, seq, "f32", attn, ffn, seed=31, ring_slots=2)


def _forward(sess, work, x):
    y = torch.empty_like(x)
    sti.sti_model_forward(sess.plan, x.data_ptr(), y.data_ptr(), work.batch, work.seq)
    sti.sti_sync(sess.ctx)
    return y


def test_slow_shard_copy_shows_up_as_that_layers_stall_and_nowhere_else():
    work = _work()
    x = torch.from_numpy(work.x_dev).cuda()
    delay_us, layer = 4000, 2
    with sti.Session(work) as s:
        y_graph = _forward(s, work, x)                       # ordinary (graph-replayed) forward
        sti.sti_plan_set_profiling(s.plan, 1)
        for _ in range(2):
            y_plain = _forward(s, work, x)
        base = sti.sti_get_stats(s.plan)
        sti.sti_plan_inject(s.plan, sti.STI_INJECT_SLOW_COPY, layer, delay_us)
        y_slow = _forward(s, work, x)
        slow = sti.sti_get_stats(s.plan)
        sti.sti_plan_inject(s.plan, sti.STI_INJECT_NONE)
        y_after = _forward(s, work, x)
        after = sti.sti_get_stats(s.plan)
    assert torch.equal(y_slow, y_plain) and torch.equal(y_graph, y_plain) and torch.equal(y_after, y_plain)
    assert slow.stall_us[layer] > 0.5 * delay_us, list(slow.stall_us[:4])
    for l in range(4):
        if l != layer:
            assert slow.stall_us[l] < 0.1 * delay_us, (l, list(slow.stall_us[:4]))
        assert base.stall_us[l] < 0.1 * delay_us and after.stall_us[l] < 0.1 * delay_us
    assert slow.total_us > base.total_us + 0.5 * delay_us   # the pipeline waited, it did not skip the layer


def test_pinned_allocation_failure_is_reported_and_the_plan_can_be_destroyed():
    work = _work(n_layers=2, resident_layers=0)
    with sti.Session(work, finalize=False) as s:
        sti.sti_plan_inject(s.plan, sti.STI_INJECT_PINNED_ALLOC_FAILURE, 0, 1)
        with pytest.raises(sti.StiError) as e:
            sti.sti_plan_finalize(s.plan)
        assert e.value.status == 7                           # STI_ERR_OOM
        with pytest.raises(sti.StiError) as e:
            sti.sti_plan_finalize(s.plan)
        assert e.value.status == 5                           # the half-built plan stays unusable
        with pytest.raises(sti.StiError) as e:
            sti.sti_plan_inject(s.plan, sti.STI_INJECT_PINNED_ALLOC_FAILURE, 0, 0)
        assert e.value.status == 5
    with sti.Session(work) as s:                             # the context's device is fine: a fresh plan works
        x = torch.from_numpy(work.x_dev).cuda()
        assert torch.isfinite(_forward(s, work, x)).all()


def test_bad_argument_does_not_change_later_forwards():
    work = _work(n_layers=2, resident_layers=2)
    x = torch.from_numpy(work.x_dev).cuda()
    with sti.Session(work) as s:
        y0 = _forward(s, work, x)
        launches = sti.sti_ctx_launch_count(s.ctx)
        y = torch.empty_like(x)
        with pytest.raises(sti.StiError) as e:               # activations must be 16-byte aligned
            sti.sti_model_forward(s.plan, x.data_ptr() + 4, y.data_ptr(), work.batch, work.seq)
        assert e.value.status == 1
        with pytest.raises(sti.StiError) as e:
            sti.sti_plan_inject(s.plan, 99, 0, 0)
        assert e.value.status == 1
        assert sti.sti_ctx_launch_count(s.ctx) == launches   # nothing was launched for the refused call
        assert torch.equal(_forward(s, work, x), y0)


def test_randomised_copy_delays_change_neither_results_nor_guard_words():
    # stream-order check of the pipeline: whenever a layer's copy reaches the copy engine, the layer computes on
    # its own bytes (two ring slots for seven streamed layers, so every slot is reused three times per forward),
    # and nothing writes past a slot or past the preload buffer
    work = _work(n_layers=8, resident_layers=1)
    x = torch.from_numpy(work.x_dev).cuda()
    rng = np.random.default_rng(8)
    with sti.Session(work) as s:
        assert sti.sti_plan_check_guards(s.plan) == 0          # right after the upload
        y_ref = _forward(s, work, x)
        assert sti.sti_plan_check_guards(s.plan) == 0
        sti.sti_plan_set_profiling(s.plan, 1)                  # forwards launched kernel by kernel: delays apply
        for _ in range(12):
            layer = int(rng.integers(1, 8))
            sti.sti_plan_inject(s.plan, sti.STI_INJECT_SLOW_COPY, layer, int(rng.integers(50, 1500)))
            y = _forward(s, work, x)
            assert torch.equal(y, y_ref), layer
            st = sti.sti_get_stats(s.plan)
            assert all(st.streamed_bytes[l] > 0 for l in range(1, 8)) and st.streamed_bytes[0] == 0
        sti.sti_plan_inject(s.plan, sti.STI_INJECT_NONE)
        sti.sti_plan_set_profiling(s.plan, 0)
        assert torch.equal(_forward(s, work, x), y_ref)
        assert sti.sti_plan_check_guards(s.plan) == 0
        mem = sti.sti_plan_memory(s.plan)
        assert mem["ring_bytes"] > 0 and mem["preload_bytes"] > 0


def test_guard_words_of_a_fully_resident_plan():
    work = _work(n_layers=2, resident_layers=2)
    x = torch.from_numpy(work.x_dev).cuda()
    with sti.Session(work) as s:
        _forward(s, work, x)
        assert sti.sti_plan_check_guards(s.plan) == 0
        assert sti.sti_plan_memory(s.plan)["ring_bytes"] == 0
