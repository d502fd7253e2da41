"""GPU parity: the CUDA path through the C ABI against the CPU oracle on the same seeded inputs.
Bit-exact for unpacked indexes and dequantized weights (fp32 and bf16); <= 2e-2 relative max-abs
for layer and model outputs."""
import numpy as np
import pytest
import torch

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


def _small_shape(n_layers=1):
    return W.ModelShape(n_layers=n_layers, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)


def _plan(shape, bits_fn, keep_fn=lambda l, kind, i: True, res_fn=lambda l: True):
    attn = [[W.UnitPlan(keep_fn(l, ATTN, i), bits_fn(l, ATTN, i), res_fn(l)) for i in range(shape.n_heads)]
            for l in range(shape.n_layers)]
    ffn = [[W.UnitPlan(keep_fn(l, FFN, i), bits_fn(l, FFN, i), res_fn(l)) for i in range(shape.n_ffn_slices)]
           for l in range(shape.n_layers)]
    return attn, ffn


def _check_decode(work, sess, units):
    from gpu_util import O as _O  # noqa: F401
    sh = work.shape
    for (l, kind, idx) in units:
        blob = work.blobs[(l, kind, idx)]
        ref, ref_codes = O.decode_unit(blob.bits, blob.codes, blob.centroids, blob.outlier_off, blob.outlier_val,
                                       sh.hidden, sh.head_dim, sh.slice_width, kind, return_codes=True)
        for m, (name, (r, c)) in enumerate(W.unit_matrix_shapes(sh, kind)):
            w = torch.zeros(r * c, dtype=torch.float32, device="cuda")
            codes = torch.zeros(r * c, dtype=torch.uint8, device="cuda")
            wb = torch.zeros(r * c, dtype=torch.int16, device="cuda")
            torch.cuda.synchronize()
            sti.sti_shard_decode(sess.plan, l, kind, idx, m, w.data_ptr(), codes.data_ptr(), wb.data_ptr())
            sti.sti_sync(sess.ctx)
            got = w.cpu().numpy().reshape(r, c)
            assert np.array_equal(got.view(np.uint32), ref[name].view(np.uint32)), (l, kind, idx, name, "fp32")
            if blob.bits != 32:
                assert np.array_equal(codes.cpu().numpy().reshape(r, c), ref_codes[name]), (l, kind, idx, name, "codes")
            want_bf16 = (O.bf16_rne(ref[name]).view(np.uint32) >> 16).astype(np.uint16)
            assert np.array_equal(wb.cpu().numpy().view(np.uint16).reshape(r, c), want_bf16), (l, kind, idx, name, "bf16")


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6, 32])
def test_decode_bit_exact_small(bits):
    shape = _small_shape()
    attn, ffn = _plan(shape, lambda l, k, i: bits)
    work = W.build_workload("dec", shape, 1, 8, "f32", attn, ffn, seed=bits, outlier_stress=0.0015)
    with sti.Session(work) as s:
        _check_decode(work, s, [(0, ATTN, 0), (0, ATTN, 3), (0, FFN, 1)])


def test_decode_bit_exact_bert_base_and_large_shapes():
    for shape, seed in ((W.BERT_BASE.with_layers(1), 1), (W.BERT_LARGE.with_layers(1), 2)):
        bits = [2, 3, 4, 5, 6]
        attn, ffn = _plan(shape, lambda l, k, i: bits[(i + k) % 5], keep_fn=lambda l, k, i: i < 5,
                          res_fn=lambda l: False)          # streamed: decode copies the layer first
        work = W.build_workload("dec", shape, 1, 8, "f32", attn, ffn, seed=seed)
        with sti.Session(work) as s:
            _check_decode(work, s, [(0, ATTN, i) for i in range(5)] + [(0, FFN, i) for i in range(5)])


def _layer_case(work, lens=None, layer=0):
    from gpu_util import run_layer, rel_err, REL_TOL
    a, f = O.decode_layer(work, layer)
    ref = O.layer_forward(work.x, work.dense[layer], a, f, eps=work.ln_eps, seq_lens=lens)
    with sti.Session(work) as s:
        y = run_layer(s, work, layer, lens=lens)
    assert np.isfinite(y).all()
    e = rel_err(y, ref)
    assert e <= REL_TOL, e
    return e


@pytest.mark.parametrize("batch,seq,act", [(1, 8, "f32"), (2, 5, "bf16"), (1, 128, "f32"), (1, 200, "bf16"),
                                           (3, 130, "f32"), (2, 512, "bf16")])
def test_layer_small_model_shapes(batch, seq, act):
    shape = _small_shape()
    bits = [2, 3, 4, 5, 6]
    attn, ffn = _plan(shape, lambda l, k, i: bits[(i * 2 + k) % 5])
    work = W.build_workload("layer", shape, batch, seq, act, attn, ffn, seed=batch * 100 + seq,
                            outlier_stress=0.0015)
    _layer_case(work)


def test_layer_dropped_units_raw_bits_and_padding_mask():
    shape = _small_shape()
    attn, ffn = _plan(shape, lambda l, k, i: 32 if i == 1 else 3 + i % 3, keep_fn=lambda l, k, i: i != 2)
    work = W.build_workload("layer", shape, 2, 70, "f32", attn, ffn, seed=5)
    _layer_case(work, lens=[70, 33])
    # nothing kept at all: biases and the two LayerNorms only
    attn, ffn = _plan(shape, lambda l, k, i: 4, keep_fn=lambda l, k, i: False)
    work = W.build_workload("layer", shape, 1, 16, "f32", attn, ffn, seed=6)
    _layer_case(work)


def test_config1_and_config2_layers():
    e1 = _layer_case(W.make_config(1))
    e2 = _layer_case(W.make_config(2))
    print("rel err cfg1 %.3e cfg2 %.3e" % (e1, e2))


def test_bert_large_layer_seq256():
    _layer_case(W.make_config(4, n_layers=1))


def test_model_small_resident_vs_streamed_bit_identical():
    from gpu_util import run_model, rel_err, REL_TOL
    shape = _small_shape(n_layers=5)
    bits = [2, 3, 4, 5, 6]
    keep = lambda l, k, i: (l + i + k) % 4 != 0
    outs = {}
    for name, res_fn in (("resident", lambda l: True), ("streamed", lambda l: l < 1), ("cold", lambda l: False)):
        attn, ffn = _plan(shape, lambda l, k, i: bits[(l + i + k) % 5], keep_fn=keep, res_fn=res_fn)
        work = W.build_workload("model", shape, 2, 96, "f32", attn, ffn, seed=21, ring_slots=2)
        with sti.Session(work) as s:
            outs[name] = run_model(s, work)
            outs[name + "_again"] = run_model(s, work)
            if name == "streamed":
                outs["host"] = run_model(s, work, host=True)
                mem = sti.sti_plan_memory(s.plan)
                assert mem["preload_bytes"] > 0 and mem["pinned_bytes"] > 0 and mem["ring_bytes"] > 0
    ref = O.run_workload(work)
    assert rel_err(outs["resident"], ref) <= REL_TOL
    for k in outs:
        assert np.array_equal(outs[k], outs["resident"]), k      # residency never changes results


def test_config3_model_reduced_depth():
    from gpu_util import run_model, rel_err, REL_TOL
    work = W.make_config(3, n_layers=5)           # layers 0-2 preloaded, 3-4 streamed
    ref = O.run_workload(work)
    with sti.Session(work) as s:
        sti.sti_plan_set_profiling(s.plan, True)
        y = run_model(s, work)
        st = sti.sti_get_stats(s.plan)
    assert rel_err(y, ref) <= REL_TOL
    assert st.n_layers == 5 and st.total_us > 0
    assert st.copy_us[0] == 0 and st.copy_us[4] > 0 and st.streamed_bytes[3] > 0 and st.resident_bytes[0] > 0


def test_error_paths_on_device():
    shape = _small_shape()
    attn, ffn = _plan(shape, lambda l, k, i: 4)
    work = W.build_workload("err", shape, 1, 8, "f32", attn, ffn, seed=1)
    missing = dict(work.blobs)
    del missing[(0, FFN, 2)]
    work_missing = W.Workload(**{**work.__dict__, "blobs": missing})
    with pytest.raises(sti.StiError) as e:
        sti.Session(work_missing)
    assert e.value.status == 6                              # STI_ERR_SHARD_MISSING before any launch
    with sti.Session(work, finalize=False) as s:
        b = work.blobs[(0, ATTN, 0)]
        with pytest.raises(sti.StiError) as e:
            sti.sti_shard_upload(s.plan, 0, ATTN, 0, 3, b.codes, b.centroids)
        assert e.value.status == 2                          # bits differ from the plan's
        with pytest.raises(sti.StiError) as e:
            sti.sti_shard_upload(s.plan, 0, ATTN, 0, 4, b.codes[:-4], b.centroids)
        assert e.value.status == 4                          # wrong size
        x = torch.zeros(1, 8, 256, device="cuda")
        with pytest.raises(sti.StiError) as e:
            sti.sti_layer_forward(s.plan, 0, x.data_ptr(), x.data_ptr(), 4, 8)
        assert e.value.status == 3                          # batch*seq beyond the context's maximum
