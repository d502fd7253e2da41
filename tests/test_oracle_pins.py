"""Pins for the CPU oracle: each function is checked against something other than itself
(brute force, closed forms, a third-party CPU library, invariants the paper states)."""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import workloads as W
from workloads.shards import ATTN, FFN
from oracle import sti_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- unpack (Section 4.2)
def _pack_bit_by_bit(codes, k):
    """Independent packer: one big Python integer, index i at bits [i*k, i*k+k)."""
    big = 0
    for i, c in enumerate(codes):
        big |= int(c) << (i * k)
    nbytes = (len(codes) * k + 31) // 32 * 4
    return np.frombuffer(big.to_bytes(nbytes, "little"), dtype="<u4").copy()


@pytest.mark.parametrize("k", [1, 2, 3, 4, 5, 6, 7, 8])
def test_unpack_round_trip_bit_by_bit(k):
    rng = np.random.default_rng(k)
    for n in (32, 64, 96, 128, 160, 1024):
        codes = rng.integers(0, 1 << k, size=n)
        words = _pack_bit_by_bit(codes, k)
        got = O.unpack_codes(words, n, k)
        assert got.dtype == np.uint8
        assert np.array_equal(got, codes)
    # every code value at every position modulo 32 (covers all word-straddling offsets)
    n = 32 * (1 << k)
    codes = np.array([(i + i // 32) % (1 << k) for i in range(n)])
    assert np.array_equal(O.unpack_codes(_pack_bit_by_bit(codes, k), n, k), codes)


@pytest.mark.parametrize("k", [2, 3, 4, 5, 6])
def test_unpack_single_set_code_lands_in_one_position(k):
    n = 128
    for i in (0, 1, 10, 31, 32, 63, 127):
        codes = np.zeros(n, dtype=int)
        codes[i] = (1 << k) - 1
        words = _pack_bit_by_bit(codes, k)
        # the set bits are exactly stream bits [i*k, i*k+k)
        bits = np.unpackbits(words.view(np.uint8), bitorder="little")
        assert bits.sum() == k and bits[i * k:i * k + k].all()
        assert np.array_equal(O.unpack_codes(words, n, k), codes)


@pytest.mark.parametrize("k", [2, 3, 4, 5, 6])
def test_generator_packer_agrees_with_bit_by_bit(k):
    rng = np.random.default_rng(100 + k)
    codes = rng.integers(0, 1 << k, size=4096).astype(np.uint8)
    assert np.array_equal(W.pack_codes(codes, k), _pack_bit_by_bit(codes, k))


def test_stream_size_closed_forms_and_paper_storage_figure():
    golden = {}
    with open(os.path.join(GOLDEN, "paper_sizes.txt")) as fh:
        for line in fh:
            if line.strip() and not line.startswith("#"):
                name, value, _unit = line.split()
                golden[name] = float(value)
    shape = W.BERT_BASE
    n_layer = shape.n_heads * W.unit_weight_count(shape, ATTN) + shape.n_ffn_slices * W.unit_weight_count(shape, FFN)
    assert n_layer == 4 * 768 * 768 + 2 * 768 * 3072 == 7_077_888
    n_model = 12 * n_layer
    total = 0
    for k in (2, 3, 4, 5, 6):
        words = O.stream_words(n_model, k)
        assert words * 4 == n_model * k // 8
        # Section 4.2: size shrinks by 32/k against fp32
        assert (n_model * 4) / (words * 4) == pytest.approx(golden["compression_ratio_numerator"] / k)
        total += words * 4
    # Section 7.2: the five versions k=2..6 take 215 MB; code streams alone are 212.3 MB, the
    # dictionaries and outliers make up the rest => no per-index padding in the format
    assert total == 212_336_640
    assert abs(total / 1e6 - golden["stored_versions_k2_to_k6"]) / golden["stored_versions_k2_to_k6"] < 0.02


# ---------------------------------------------------------------- dequantize (Section 4.2, 6)
def test_dequantize_brute_force_tiny_shard():
    rng = np.random.default_rng(7)
    for k in (2, 3, 4, 5, 6):
        n = 64 * 32
        codes = rng.integers(0, 1 << k, size=n)
        table = {c: np.float32(rng.standard_normal()) for c in range(1 << k)}
        cent = np.array([table[c] for c in range(1 << k)], dtype=np.float32)
        off = np.sort(rng.choice(n, size=5, replace=False)).astype(np.uint32)
        val = rng.standard_normal(5).astype(np.float32)
        want = [table[int(c)] for c in codes]
        for o, v in zip(off, val):
            want[int(o)] = v
        got = O.dequantize(codes, cent, off, val)
        assert got.dtype == np.float32
        assert np.array_equal(got, np.array(want, dtype=np.float32))
        # outlier positions return the preserved value exactly; all-equal table -> constant matrix
        assert np.array_equal(got[off], val)
        const = O.dequantize(codes, np.full(1 << k, 0.25, np.float32), off[:0], val[:0])
        assert np.all(const == np.float32(0.25))


def test_bf16_rounding_matches_third_party_and_ties_to_even():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(10000).astype(np.float32) * 0.02,
                        np.array([1.0, -1.0, 0.0, 1.00390625, 1.01171875, 3.0e-39, 65504.0], np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_rne(x), want)
    # 1 + 2^-8 is exactly halfway between 1 and 1 + 2^-7: ties go to the even mantissa (1.0)
    assert O.bf16_rne(np.array([1.00390625], np.float32))[0] == np.float32(1.0)
    assert O.bf16_rne(np.array([1.01171875], np.float32))[0] == np.float32(1.015625)


def test_decode_unit_shapes_follow_table_1_and_alignment():
    shape = W.ModelShape(1, 128, 2, 64, 256, 2)
    for kind in (ATTN, FFN):
        for bits in (2, 3, 5, 32):
            mats = W.make_unit_weights(shape, 5, 0, kind, 1)
            blob = W.quantize_unit(mats, bits)
            dec, codes = O.decode_unit(blob.bits, blob.codes, blob.centroids, blob.outlier_off, blob.outlier_val,
                                       shape.hidden, shape.head_dim, shape.slice_width, kind, return_codes=True)
            names = [n for n, _ in W.unit_matrix_shapes(shape, kind)]
            assert list(dec) == names
            for (name, shp), m in zip(W.unit_matrix_shapes(shape, kind), mats):
                assert dec[name].shape == shp
                if bits == 32:
                    assert np.array_equal(dec[name], m)          # raw version is the original weights
                else:
                    cent = blob.centroids
                    # every decoded value is a centroid or a preserved outlier
                    ok = np.isin(dec[name], cent) | np.isin(dec[name], blob.outlier_val)
                    assert ok.all()
                    assert codes[name].max() < (1 << bits)


# ---------------------------------------------------------------- quantizer invariants (Section 6)
def test_quantizer_invariants():
    shape = W.BERT_BASE
    mats = W.make_unit_weights(shape, 0, 0, ATTN, 0)
    flat = np.concatenate([m.reshape(-1) for m in mats])
    prev_mse = None
    for k in (2, 3, 4, 5, 6):
        blob = W.quantize_unit(mats, k)
        dec, codes = O.decode_unit(k, blob.codes, blob.centroids, blob.outlier_off, blob.outlier_val,
                                   shape.hidden, shape.head_dim, shape.slice_width, ATTN, return_codes=True)
        w = np.concatenate([dec[n].reshape(-1) for n in ("Q", "K", "V", "O")])
        c = np.concatenate([codes[n].reshape(-1) for n in ("Q", "K", "V", "O")])
        inl = np.ones(flat.size, bool)
        inl[blob.outlier_off] = False
        hist = np.bincount(c[inl], minlength=1 << k)
        assert hist.max() - hist.min() <= 1                              # equal population
        assert np.all(np.diff(blob.centroids) > 0)                       # sorted clusters
        # centroid = arithmetic mean of its cluster  =>  sums agree
        assert w[inl].astype(np.float64).sum() == pytest.approx(flat[inl].astype(np.float64).sum(), rel=1e-4, abs=1e-3)
        assert np.array_equal(w[~inl], flat[~inl])                       # outliers kept as-is
        mse = float(((w - flat) ** 2).mean())
        assert prev_mse is None or mse < prev_mse
        prev_mse = mse
    # log-likelihood < -4 under N(0, 0.02^2)  <=>  |z| > 3.7397;  two-sided tail = erfc(z / sqrt 2)
    z = math.sqrt(2.0 * (4.0 - 0.5 * math.log(2.0 * math.pi * 0.02 ** 2)))
    expect = math.erfc(z / math.sqrt(2.0))
    frac = blob.outlier_off.size / flat.size
    assert 0.5 * expect < frac < 1.6 * expect
    assert np.all(np.diff(blob.outlier_off.astype(np.int64)) > 0)


# ---------------------------------------------------------------- layer forward
def _tiny_workload(seed=0, keep_originals=True, bits=4, batch=2, seq=5, act="f32"):
    shape = W.ModelShape(n_layers=1, hidden=128, n_heads=2, head_dim=64, ffn=512, n_ffn_slices=2)
    attn = [[W.UnitPlan(True, bits, True) for _ in range(2)]]
    ffn = [[W.UnitPlan(True, bits, True) for _ in range(2)]]
    return W.build_workload("tiny", shape, batch, seq, act, attn, ffn, seed=seed, keep_originals=keep_originals)


def _dense_bert_layer_torch(x, dense, wq, wk, wv, wo, f1, f2, n_heads, eps, seq_lens=None):
    """Independently written ordinary BERT layer on full matrices, third-party CPU ops, fp64."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    x = t(x)
    B, L, d = x.shape
    hd = wq.shape[0] // n_heads
    q = F.linear(x, t(wq), t(dense["bq"].reshape(-1))).view(B, L, n_heads, hd).transpose(1, 2)
    k = F.linear(x, t(wk), t(dense["bk"].reshape(-1))).view(B, L, n_heads, hd).transpose(1, 2)
    v = F.linear(x, t(wv), t(dense["bv"].reshape(-1))).view(B, L, n_heads, hd).transpose(1, 2)
    mask = None
    if seq_lens is not None:
        mask = torch.zeros(B, 1, 1, L, dtype=torch.bool)
        for b, n in enumerate(seq_lens):
            mask[b, :, :, :n] = True
    a = F.scaled_dot_product_attention(q, k, v, attn_mask=mask)
    a = a.transpose(1, 2).reshape(B, L, n_heads * hd)
    h1 = F.layer_norm(x + F.linear(a, t(wo), t(dense["bo"])), (d,), t(dense["ln1_g"]), t(dense["ln1_b"]), eps)
    u = F.gelu(F.linear(h1, t(f1), t(dense["b1"].reshape(-1))))
    y = F.layer_norm(h1 + F.linear(u, t(f2), t(dense["b2"])), (d,), t(dense["ln2_g"]), t(dense["ln2_b"]), eps)
    return y.numpy()


def _assemble(attn_units, ffn_units):
    hs, js = sorted(attn_units), sorted(ffn_units)
    wq = np.concatenate([attn_units[h]["Q"] for h in hs], axis=0)
    wk = np.concatenate([attn_units[h]["K"] for h in hs], axis=0)
    wv = np.concatenate([attn_units[h]["V"] for h in hs], axis=0)
    wo = np.concatenate([attn_units[h]["O"] for h in hs], axis=1)
    f1 = np.concatenate([ffn_units[j]["F1"] for j in js], axis=0)
    f2 = np.concatenate([ffn_units[j]["F2"] for j in js], axis=1)
    return wq, wk, wv, wo, f1, f2


@pytest.mark.parametrize("seq_lens", [None, [5, 3]])
def test_all_units_kept_equals_dense_layer(seq_lens):
    w = _tiny_workload()
    a, f = O.decode_layer(w, 0)
    y = O.layer_forward(w.x, w.dense[0], a, f, eps=1e-12, seq_lens=seq_lens)
    y_dense = _dense_bert_layer_torch(w.x, w.dense[0], *_assemble(a, f), n_heads=2, eps=1e-12, seq_lens=seq_lens)
    if seq_lens is not None:      # padded query rows are defined but the dense mask treats them the same
        pass
    assert np.abs(y - y_dense).max() < 1e-9


def test_full_precision_plan_equals_dense_layer_on_original_weights():
    w = _tiny_workload(bits=32)
    a, f = O.decode_layer(w, 0)
    orig_a = {h: dict(zip(("Q", "K", "V", "O"), w.originals[(0, ATTN, h)])) for h in range(2)}
    orig_f = {j: dict(zip(("F1", "F2"), w.originals[(0, FFN, j)])) for j in range(2)}
    for h in range(2):
        for n in ("Q", "K", "V", "O"):
            assert np.array_equal(a[h][n], orig_a[h][n])
    y = O.layer_forward(w.x, w.dense[0], a, f)
    y_dense = _dense_bert_layer_torch(w.x, w.dense[0], *_assemble(orig_a, orig_f), n_heads=2, eps=1e-12)
    assert np.abs(y - y_dense).max() < 1e-9


def test_bert_base_layer_against_dense_torch():
    w = W.make_config(1)
    a, f = O.decode_layer(w, 0)
    y = O.layer_forward(w.x, w.dense[0], a, f)
    y_dense = _dense_bert_layer_torch(w.x, w.dense[0], *_assemble(a, f), n_heads=12, eps=1e-12)
    assert np.abs(y - y_dense).max() < 1e-9


def test_dropped_unit_contributes_zero():
    w = _tiny_workload()
    a, f = O.decode_layer(w, 0)
    # dropping head 1 == keeping it with an all-zero output slice; same for FFN slice 0
    a_zero = {0: a[0], 1: dict(a[1], O=np.zeros_like(a[1]["O"]))}
    f_zero = {0: dict(f[0], F2=np.zeros_like(f[0]["F2"])), 1: f[1]}
    y_drop = O.layer_forward(w.x, w.dense[0], {0: a[0]}, {1: f[1]})
    y_zero = O.layer_forward(w.x, w.dense[0], a_zero, f_zero)
    assert np.array_equal(y_drop, y_zero)
    # dense layer with only the kept head / slice (biases sliced with their unit)
    d = dict(w.dense[0])
    d_kept = dict(d, bq=d["bq"][:1], bk=d["bk"][:1], bv=d["bv"][:1], b1=d["b1"][1:])
    y_dense = _dense_bert_layer_torch(w.x, d_kept, *_assemble({0: a[0]}, {1: f[1]}), n_heads=1, eps=1e-12)
    assert np.abs(y_drop - y_dense).max() < 1e-9
    # nothing kept at all: only b_o, b_2 and the two LayerNorms act
    y_none = O.layer_forward(w.x, w.dense[0], {}, {})
    p = {k: v.astype(np.float64) for k, v in w.dense[0].items()}
    h1 = O.layer_norm(w.x.astype(np.float64) + p["bo"], p["ln1_g"], p["ln1_b"], 1e-12)
    assert np.abs(y_none - O.layer_norm(h1 + p["b2"], p["ln2_g"], p["ln2_b"], 1e-12)).max() < 1e-12


def test_kept_unit_order_does_not_matter():
    w = _tiny_workload(seed=4)
    a, f = O.decode_layer(w, 0)
    y = O.layer_forward(w.x, w.dense[0], a, f)
    # relabel: swap units 0 and 1 together with their sliced biases
    d = w.dense[0]
    d_sw = dict(d, bq=d["bq"][::-1], bk=d["bk"][::-1], bv=d["bv"][::-1], b1=d["b1"][::-1])
    y_sw = O.layer_forward(w.x, d_sw, {0: a[1], 1: a[0]}, {0: f[1], 1: f[0]})
    assert np.abs(y - y_sw).max() < 1e-9


def test_closed_forms_single_token_identical_tokens_zero_input():
    w = _tiny_workload(seed=2, batch=1, seq=1)
    a, f = O.decode_layer(w, 0)
    p = {k: v.astype(np.float64) for k, v in w.dense[0].items()}
    x = w.x.astype(np.float64)
    # seq = 1: softmax over one key is 1, so each head's output is its value vector
    attn = p["bo"].copy()
    for h in a:
        v = x[0] @ a[h]["V"].astype(np.float64).T + p["bv"][h]
        attn = attn + v @ a[h]["O"].astype(np.float64).T
    y, inter = O.layer_forward(x, w.dense[0], a, f, return_intermediates=True)
    assert np.abs(inter["h1"][0] - O.layer_norm(x[0] + attn, p["ln1_g"], p["ln1_b"], 1e-12)).max() < 1e-10
    # identical tokens: uniform attention, every row of the output equal
    xx = np.repeat(x, 6, axis=1)
    yy = O.layer_forward(xx, w.dense[0], a, f)
    assert np.abs(yy - yy[:, :1]).max() < 1e-10
    assert np.abs(yy[:, 0] - y[:, 0]).max() < 1e-10
    # zero input: the query/key/value are the biases, still identical rows
    y0 = O.layer_forward(np.zeros((1, 4, 128)), w.dense[0], a, f)
    assert np.abs(y0 - y0[:, :1]).max() < 1e-12


def test_softmax_layernorm_gelu_closed_forms():
    s = np.array([[0.0, math.log(3.0)], [5.0, 5.0]])
    assert np.allclose(O.softmax_rows(s), [[0.25, 0.75], [0.5, 0.5]], atol=1e-15)
    big = np.array([[1000.0, 1000.0 + math.log(3.0)]])
    assert np.allclose(O.softmax_rows(big), [[0.25, 0.75]], atol=1e-12)      # max-subtracted
    v = np.array([[1.0, 2.0, 3.0, 4.0]])
    ln = O.layer_norm(v, np.ones(4), np.zeros(4), 0.0)
    assert np.allclose(ln, (v - 2.5) / math.sqrt(1.25))
    ln2 = O.layer_norm(v, np.full(4, 2.0), np.full(4, 0.5), 0.0)
    assert np.allclose(ln2, 2.0 * ln + 0.5)
    xs = np.linspace(-4, 4, 41)
    want = np.array([0.5 * t * (1.0 + math.erf(t / math.sqrt(2.0))) for t in xs])
    assert np.allclose(O.gelu_erf(xs), want, atol=1e-15)
    assert np.allclose(O.gelu_erf(xs), F.gelu(torch.from_numpy(xs)).numpy(), atol=1e-12)


def test_model_forward_is_layer_composition():
    shape = W.ModelShape(n_layers=3, hidden=128, n_heads=2, head_dim=64, ffn=512, n_ffn_slices=2)
    attn = [[W.UnitPlan(True, 3 + (l + i) % 3, l == 0) for i in range(2)] for l in range(3)]
    ffn = [[W.UnitPlan(i != l % 2, 2 + l, l == 0) for i in range(2)] for l in range(3)]
    w = W.build_workload("tiny3", shape, 1, 7, "f32", attn, ffn, seed=11)
    outs = O.run_workload(w, return_all=True)
    h = w.x
    for l in range(3):
        a, f = O.decode_layer(w, l)
        assert sorted(f) == w.kept(l, FFN)
        h = O.layer_forward(h, w.dense[l], a, f)
        assert np.array_equal(h, outs[l])
    # residency flags are not an input of the arithmetic at all
    assert np.array_equal(O.run_workload(w), outs[-1])
