"""Back-to-back executions on the device (Section 3.2, Section 5.5): three executions with a growing preload buffer.
What the eviction rule keeps after a run stays in DEVICE memory: the next plan adopts those shards (device-to-device)
and uploads only the others.  Every execution's output is checked against the oracle forward of its own plan, the
bytes uploaded / adopted / streamed against what the plans say."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import ATTN, FFN
from oracle import sti_oracle as O
from oracle import sti_planner_oracle as P

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")

N, M = 4, 4            # layers x shards per layer (shard i = head i + FFN slice i)
VERSIONS = (2, 3, 4, 5, 6, 32)


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _workload(keep, bits, preload, seed=41):
    shape = W.ModelShape(n_layers=N, hidden=256, n_heads=M, head_dim=64, ffn=1024, n_ffn_slices=M)
    grid = lambda: [[W.UnitPlan(bool(keep[l][i]), int(bits[l][i]) if keep[l][i] else 2, bool(preload[l][i]))
                     for i in range(M)] for l in range(N)]
    return W.build_workload("b2b", shape, 1, 64, "f32", grid(), grid(), seed=seed, ring_slots=2)


def _shard_bytes():
    """Bytes of one shard (head + FFN slice) per stored version, from the generator's own blobs."""
    ones = np.ones((N, M), np.uint8)
    out = []
    for k in VERSIONS:
        w = _workload(ones, ones * k, ones * 0)
        out.append(w.packed_bytes() // (N * M))
    return out


def _unit_bytes(work, key):
    b = work.blobs[key]
    return b.packed_bytes if isinstance(b.packed_bytes, int) else b.packed_bytes()


def test_three_executions_with_a_growing_buffer_keep_their_shards_on_the_device():
    shard_bytes = _shard_bytes()
    t_comp = [0.0] + [40.0] * M                                     # flat compute delay, as on this device
    t_io = [b / 50e3 for b in shard_bytes]                          # 50 GB/s in us
    importance = np.random.default_rng(5).uniform(0, 1, (N, M)).astype(np.float32)
    target_us = 400.0
    buffers = [shard_bytes[0] * 5, shard_bytes[2] * 8, shard_bytes[4] * 14]      # the first holds layer 0 and a bit
    prev = None                                                     # (session, plan grids, workload)
    sessions = []
    try:
        for step, buf in enumerate(buffers):
            cached = None
            if prev is not None:
                cached, _ = sti.sti_preload_after_run(prev["plan"]["keep"], prev["plan"]["bits"], shard_bytes, buf)
                want_cached = P.retain_after_run(prev["plan"]["keep"], prev["plan"]["bits"], shard_bytes, buf)[0]
                assert np.array_equal(cached, want_cached)          # the library's eviction rule = the oracle's
            plan = sti.sti_plan_auto(target_us, N, M, t_comp, t_io, shard_bytes, importance, buf, cached)
            assert plan["valid"]
            work = _workload(plan["keep"], plan["bits"], plan["preload"])
            # build the session by hand: adopt what the previous plan holds on the device, upload the rest
            sess = sti.Session.__new__(sti.Session)
            sh = work.shape
            sess.work, sess.plan = work, 0
            sess.desc = sti.StiModelDesc(n_layers=sh.n_layers, hidden=sh.hidden, n_heads=sh.n_heads, head_dim=64,
                                         ffn=sh.ffn, n_ffn_slices=sh.n_ffn_slices, max_batch=1, max_seq=64,
                                         act_dtype=0, ln_eps=work.ln_eps)
            sess.ctx = prev["sess"].ctx if prev else sti.sti_ctx_create(sess.desc, 0)
            if not prev:
                for l, p in enumerate(work.dense):
                    sti.sti_ctx_set_layer_params(sess.ctx, l, p["bq"], p["bk"], p["bv"], p["bo"], p["b1"], p["b2"],
                                                 p["ln1_g"], p["ln1_b"], p["ln2_g"], p["ln2_b"])
            attn = [(u.keep, u.bits, u.resident) for layer in work.attn_plan for u in layer]
            ffn = [(u.keep, u.bits, u.resident) for layer in work.ffn_plan for u in layer]
            sess.plan = sti.sti_plan_create(sess.ctx, attn, ffn, work.ring_slots)
            sessions.append(sess)
            adopted = uploaded_resident = 0
            for (l, kind, idx), b in work.blobs.items():
                is_cached = cached is not None and cached[l][idx] != 0
                if is_cached:
                    assert plan["preload"][l][idx] and plan["bits"][l][idx] == cached[l][idx]
                    sti.sti_shard_adopt(sess.plan, prev["sess"].plan, l, kind, idx)
                    adopted += 1
                else:
                    sti.sti_shard_upload(sess.plan, l, kind, idx, b.bits, b.codes, b.centroids, b.outlier_off, b.outlier_val)
                    uploaded_resident += int(plan["preload"][l][idx])
            sti.sti_plan_finalize(sess.plan)
            fill = sti.sti_plan_fill_stats(sess.plan)
            if cached is not None:
                assert adopted == 2 * int(((cached != 0) & (plan["keep"] != 0)).sum()) and adopted > 0
                assert fill["adopted_bytes"] > 0
            if uploaded_resident == 0:
                assert fill["uploaded_bytes"] == 0                  # nothing it already holds goes up again
            # what must stay for the NEXT execution is decided now, before the run that loads it
            if step + 1 < len(buffers):
                keep_next, _ = sti.sti_preload_after_run(plan["keep"], plan["bits"], shard_bytes, buffers[step + 1])
                mask = (keep_next != 0).astype(np.uint8)
                retained = sti.sti_plan_retain(sess.plan, mask, mask)
                streamed_kept = ((keep_next != 0) & (plan["preload"] == 0)).sum()
                assert (retained > 0) == (streamed_kept > 0)
            # run and check against the oracle forward of THIS plan
            x = torch.from_numpy(work.x_dev).cuda()
            y = torch.empty_like(x)
            sti.sti_plan_set_profiling(sess.plan, 0)
            sti.sti_model_forward(sess.plan, x.data_ptr(), y.data_ptr(), 1, 64)     # also moves the shards to keep
            sti.sti_sync(sess.ctx)
            ref = O.run_workload(work)
            err = float(np.abs(y.cpu().numpy().astype(np.float64) - ref).max() / np.abs(ref).max())
            assert err <= 2e-2, (step, err)
            y2 = torch.empty_like(x)
            sti.sti_model_forward(sess.plan, x.data_ptr(), y2.data_ptr(), 1, 64)    # graph-replayed from here on
            sti.sti_sync(sess.ctx)
            assert torch.equal(y, y2)
            # streamed bytes of the run = the plan's non-preloaded shards
            sti.sti_plan_set_profiling(sess.plan, 1)
            sti.sti_model_forward(sess.plan, x.data_ptr(), y2.data_ptr(), 1, 64)
            st = sti.sti_get_stats(sess.plan)
            sti.sti_plan_set_profiling(sess.plan, 0)
            streamed = sum(st.streamed_bytes[:st.n_layers])
            want_keys = [k for k in work.blobs if not plan["preload"][k[0]][k[2]]]
            assert abs(streamed - sum(_unit_bytes(work, k) for k in want_keys)) <= 64 * len(want_keys) + 64
            prev = {"sess": sess, "plan": plan, "work": work, "streamed": streamed}
            if step:
                assert int((cached != 0).sum()) >= prev_cached      # the cache only grows with the buffer
            prev_cached = 0 if cached is None else int((cached != 0).sum())
        assert prev_cached > 0
    finally:
        ctx = sessions[0].ctx if sessions else 0
        for s in sessions:
            if s.plan:
                sti.sti_plan_destroy(s.plan)
        if ctx:
            sti.sti_ctx_destroy(ctx)


def test_adopt_and_retain_argument_checks():
    ones = np.ones((N, M), np.uint8)
    work = _workload(ones, ones * 3, ones * 0)                      # everything streamed
    with sti.Session(work) as s:
        attn = [(True, 3, True)] * (N * M)
        other = sti.sti_plan_create(s.ctx, attn, attn, 2)
        try:
            with pytest.raises(sti.StiError) as e:                  # streamed and not retained: not on the device
                sti.sti_shard_adopt(other, s.plan, 0, ATTN, 0)
            assert e.value.status == 5
            mask = np.zeros((N, M), np.uint8)
            mask[0, 0] = 1
            assert sti.sti_plan_retain(s.plan, mask, mask * 0) > 0
            with pytest.raises(sti.StiError) as e:                  # marked, but the retaining forward has not run
                sti.sti_shard_adopt(other, s.plan, 0, ATTN, 0)
            assert e.value.status == 5
            with pytest.raises(sti.StiError) as e:                  # one retained set per plan
                sti.sti_plan_retain(s.plan, mask, mask)
            assert e.value.status == 5
            x = torch.from_numpy(work.x_dev).cuda()
            y = torch.empty_like(x)
            sti.sti_model_forward(s.plan, x.data_ptr(), y.data_ptr(), 1, 64)
            sti.sti_sync(s.ctx)
            sti.sti_shard_adopt(other, s.plan, 0, ATTN, 0)          # now it is
            wrong_bits = sti.sti_plan_create(s.ctx, [(True, 4, True)] * (N * M), attn, 2)
            with pytest.raises(sti.StiError) as e:
                sti.sti_shard_adopt(wrong_bits, s.plan, 0, ATTN, 0)
            assert e.value.status == 2
            sti.sti_plan_destroy(wrong_bits)
        finally:
            sti.sti_plan_destroy(other)
