"""GPU parity of the device quantizer (Section 6) against the CPU oracle on the same seeded weights: index
streams, outlier offsets, values and counts bit-exact; centroids equal up to one fp32 unit in the last place
(both sides round an fp64 mean once, the summation orders differ).  Every case runs through both methods of the
library (rank selection, the default, and the stable sort it falls back to)."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import ATTN, FFN, make_unit_weights
from oracle import sti_quantizer_oracle as Q

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _run(units, bits, max_out=4096, method=None, want_sorted=False):
    """units: [n_units][n] fp32 on the host -> (words, centroids, offsets, values, counts) from the device."""
    n_units, n = units.shape
    w = torch.from_numpy(units).cuda()
    K = 1 << bits
    codes = torch.zeros((n_units, n * bits // 32), dtype=torch.int32, device="cuda")
    cents = torch.zeros((n_units, K), dtype=torch.float32, device="cuda")
    off = torch.zeros((n_units, max_out), dtype=torch.int32, device="cuda")
    val = torch.zeros((n_units, max_out), dtype=torch.float32, device="cuda")
    cnt = torch.zeros(n_units, dtype=torch.int32, device="cuda")
    ws_bytes = sti.sti_quantize_workspace_bytes(n_units, n)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    by_sort = torch.full((n_units,), 7, dtype=torch.uint8, device="cuda")
    if method is None:
        sti.sti_quantize_units(w.data_ptr(), n_units, n, bits, codes.data_ptr(), cents.data_ptr(), off.data_ptr(),
                               val.data_ptr(), max_out, cnt.data_ptr(), ws.data_ptr(), ws_bytes)
    else:
        sti.sti_quantize_units_by(w.data_ptr(), n_units, n, bits, codes.data_ptr(), cents.data_ptr(), off.data_ptr(),
                                  val.data_ptr(), max_out, cnt.data_ptr(), ws.data_ptr(), ws_bytes, method,
                                  by_sort.data_ptr())
    torch.cuda.synchronize()
    res = (codes.cpu().numpy().view(np.uint32), cents.cpu().numpy(), off.cpu().numpy().view(np.uint32),
           val.cpu().numpy(), cnt.cpu().numpy())
    return res + (by_sort.cpu().numpy(),) if want_sorted else res


def _ulp_diff(a, b):
    ia, ib = a.view(np.int32).astype(np.int64), b.view(np.int32).astype(np.int64)
    ia = np.where(ia < 0, -(ia & 0x7FFFFFFF), ia)
    ib = np.where(ib < 0, -(ib & 0x7FFFFFFF), ib)
    return np.abs(ia - ib)


def _check(units, bits, max_out=4096):
    """Both methods against the oracle; returns which units the default method handed to the sort."""
    refs = [Q.quantize_unit(units[u], bits) for u in range(units.shape[0])]
    _check_one(units, bits, max_out, refs, sti.STI_QUANTIZE_SORT)
    return _check_one(units, bits, max_out, refs, sti.STI_QUANTIZE_SELECT)


def _check_one(units, bits, max_out, refs, method):
    words, cents, off, val, cnt, by_sort = _run(units, bits, max_out, method, want_sorted=True)
    assert set(np.unique(by_sort)) <= {0, 1}
    if method == sti.STI_QUANTIZE_SORT:
        assert by_sort.all()
    _compare(units, bits, max_out, refs, words, cents, off, val, cnt)
    return by_sort


def _compare(units, bits, max_out, refs, words, cents, off, val, cnt):
    for u in range(units.shape[0]):
        rw, rc, ro, rv = refs[u]
        assert cnt[u] == ro.size, (u, bits)
        m = min(ro.size, max_out)
        assert np.array_equal(off[u, :m], ro[:m]) and np.array_equal(val[u, :m].view(np.uint32), rv[:m].view(np.uint32))
        assert _ulp_diff(cents[u], rc).max() <= 1, (u, bits)
        if np.array_equal(cents[u].view(np.uint32), rc.view(np.uint32)):
            assert np.array_equal(words[u], rw), (u, bits)
        else:       # a centroid one unit off can only move an outlier's nearest-centroid index; everything else is exact
            codes = np.asarray(__import__("oracle.sti_oracle", fromlist=["x"]).unpack_codes(words[u], units.shape[1], bits))
            ref = np.asarray(__import__("oracle.sti_oracle", fromlist=["x"]).unpack_codes(rw, units.shape[1], bits))
            inl = np.ones(units.shape[1], bool)
            inl[ro] = False
            assert np.array_equal(codes[inl], ref[inl]), (u, bits)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
def test_bert_base_units_every_bitwidth(bits):
    shape = W.BERT_BASE
    units = np.stack([np.concatenate([m.reshape(-1) for m in make_unit_weights(shape, 11, l, ATTN, i)])
                      for l, i in ((0, 0), (1, 5), (2, 11))])
    assert not _check(units, bits).any()                  # Gaussian-like weights never need the sort


def test_bert_large_ffn_unit_with_heavy_tails():
    shape = W.BERT_LARGE
    mats = make_unit_weights(shape, 12, 3, FFN, 7, outlier_stress=0.0015)       # 524,288 weights, ~0.15 % outliers
    units = np.concatenate([m.reshape(-1) for m in mats])[None, :]
    assert not _check(units, 3).any()
    assert not _check(units, 6).any()


def test_ties_constant_and_tiny_units():
    rng = np.random.default_rng(5)
    few_values = rng.choice(np.linspace(-0.05, 0.05, 9).astype(np.float32), size=8192)      # massive ties
    signed_zero = few_values.copy()
    signed_zero[::7] = np.float32(-0.0)
    signed_zero[3::7] = np.float32(0.0)
    const = np.full(8192, 0.0125, np.float32)
    ramp = np.arange(8192, dtype=np.float32) * np.float32(1e-5) - np.float32(0.04)
    units = np.stack([few_values, signed_zero, const, ramp])
    for bits in (2, 4, 6):
        by_sort = _check(units, bits)
        assert by_sort[2] == 1                             # zero variance: no value bins to select in
    _check(rng.standard_normal((2, 32)).astype(np.float32) * np.float32(0.02), 5)            # fewer weights than 2 clusters' worth
    _check(rng.standard_normal((1, 1056)).astype(np.float32) * np.float32(0.02), 3)          # ragged last chunk


def test_units_the_selection_hands_to_the_sort():
    """Many equal values: one value bin holds more members than the counting selection accepts.  Mixed in one launch
    with units that the selection does itself."""
    rng = np.random.default_rng(6)
    n = 65536
    ties = rng.choice(np.linspace(-0.05, 0.05, 9).astype(np.float32), size=n)
    normal = (rng.standard_normal(n) * 0.03).astype(np.float32)
    half = normal.copy()
    half[: n // 2] = np.float32(0.01)                     # half the unit is one value
    units = np.stack([normal, ties, half, normal[::-1].copy()])
    for bits in (2, 5):
        by_sort = _check(units, bits)
        assert list(by_sort) == [0, 1, 1, 0]


def test_selection_is_deterministic():
    shape = W.BERT_LARGE
    units = np.stack([np.concatenate([m.reshape(-1) for m in make_unit_weights(shape, 14, 0, ATTN, i)]) for i in range(3)])
    a = _run(units, 6)
    b = _run(units, 6)
    for x, y in zip(a, b):
        assert np.array_equal(x.view(np.uint32) if x.dtype == np.float32 else x, y.view(np.uint32) if y.dtype == np.float32 else y)


def test_outlier_lists_shorter_than_the_outliers_found():
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    mats = make_unit_weights(shape, 13, 0, FFN, 1, outlier_stress=0.01)
    units = np.concatenate([m.reshape(-1) for m in mats])[None, :]
    _check(units, 4, max_out=16)          # count reported in full, lists truncated, index stream complete


def test_argument_checks():
    w = torch.zeros(64, device="cuda")
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    p = buf.data_ptr()
    with pytest.raises(sti.StiError) as e:
        sti.sti_quantize_units(w.data_ptr(), 1, 64, 7, p, p, p, p, 4, p, p, 4096)
    assert e.value.status == 2
    with pytest.raises(sti.StiError) as e:
        sti.sti_quantize_units(w.data_ptr(), 1, 48, 4, p, p, p, p, 4, p, p, 4096)
    assert e.value.status == 3
    with pytest.raises(sti.StiError) as e:
        sti.sti_quantize_units(w.data_ptr(), 1, 64, 4, p, p, p, p, 4, p, p, 100)
    assert e.value.status == 4
    big = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    q = big.data_ptr()
    with pytest.raises(sti.StiError) as e:                               # no such method
        sti.sti_quantize_units_by(w.data_ptr(), 1, 64, 4, q, q, q, q, 4, q, q, 1 << 16, 2)
    assert e.value.status == 1
    with pytest.raises(sti.StiError) as e:                               # weights not 16-byte aligned
        sti.sti_quantize_units(w.data_ptr() + 4, 1, 32, 4, q, q, q, q, 4, q, q, 1 << 16)
    assert e.value.status == 1


def test_device_quantized_units_run_through_the_layer():
    """fp32 weights -> sti_quantize_units -> sti_shard_upload -> sti_layer_forward, against the oracle's forward
    on the oracle's own quantization of the same weights."""
    from gpu_util import run_layer, rel_err, REL_TOL
    from oracle import sti_oracle as O
    from workloads.shards import ShardBlob
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    bits_of = {ATTN: [2, 3, 5, 6], FFN: [4, 6, 3, 2]}
    attn = [[W.UnitPlan(True, bits_of[ATTN][i], True) for i in range(4)]]
    ffn = [[W.UnitPlan(True, bits_of[FFN][i], True) for i in range(4)]]
    work = W.build_workload("quantized_on_device", shape, 1, 96, "f32", attn, ffn, seed=19, ring_slots=2)
    blobs = {}
    for (l, kind, idx), ref_blob in work.blobs.items():
        flat = np.concatenate([m.reshape(-1) for m in make_unit_weights(shape, 19, l, kind, idx)])[None, :]
        words, cents, off, val, cnt = _run(flat, ref_blob.bits)
        n_out = int(cnt[0])
        blobs[(l, kind, idx)] = ShardBlob(bits=ref_blob.bits, codes=words[0].copy(), centroids=cents[0].copy(),
                                          outlier_off=off[0, :n_out].copy(), outlier_val=val[0, :n_out].copy())
        assert np.array_equal(words[0], ref_blob.codes)          # the generator's blob is the same quantization
    import dataclasses
    work_dev = dataclasses.replace(work, blobs=blobs)
    ref = O.run_workload(work)
    with sti.Session(work_dev) as s:
        y = run_layer(s, work_dev, 0)
    assert rel_err(y, ref) <= REL_TOL
