"""Pins of the quantizer oracle (Section 6) against things other than itself: a brute-force restatement in
plain Python on tiny inputs, the invariants the paper's construction fixes (equal population, centroid = mean,
ascending centroids, error falling with the bitwidth), the closed-form outlier rate of exactly Gaussian weights,
degenerate inputs, and bit streams read back by the separately pinned unpacker."""
import math
from fractions import Fraction

import numpy as np
import pytest

from oracle import sti_oracle as O
from oracle import sti_quantizer_oracle as Q


def _brute_force(w32, bits):
    """Every step with Python numbers: exact rational sums, sorted() on (value, index)."""
    w = [float(v) for v in w32]
    n, K = len(w), 1 << bits
    mu = float(sum(Fraction(v) for v in w) / n)
    var = float(sum((Fraction(v) - Fraction(mu)) ** 2 for v in w) / n)
    out = []
    for i, v in enumerate(w):
        if var > 0.0:
            ll = -0.5 * math.log(2.0 * math.pi * var) - (v - mu) ** 2 / (2.0 * var)
            if ll < -4.0:
                out.append(i)
    inl = sorted((i for i in range(n) if i not in set(out)), key=lambda i: (w[i], i))
    codes, cents = [0] * n, [0.0] * K
    for c in range(K):
        lo, hi = (c * len(inl)) // K, ((c + 1) * len(inl)) // K
        if hi > lo:
            cents[c] = float(np.float32(float(sum(Fraction(w[i]) for i in inl[lo:hi]) / (hi - lo))))
            for i in inl[lo:hi]:
                codes[i] = c
    for i in out:
        best = min(range(K), key=lambda c: (abs(w[i] - cents[c]), c))
        codes[i] = best
    return codes, cents, out


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("n", [64, 97, 200])
def test_brute_force_on_tiny_arrays_with_ties_and_an_outlier(bits, n):
    rng = np.random.default_rng(100 * bits + n)
    w = (rng.standard_normal(n) * 0.02).astype(np.float32)
    w[5] = w[11] = w[40]                      # ties: original index order decides
    w[17] = np.float32(0.31)                  # far out: log-likelihood below -4
    codes, cents, off, val = Q.quantize(w, bits)
    bc, bcent, bout = _brute_force(w, bits)
    assert list(off) == bout and 17 in bout
    assert np.array_equal(val, w[off])
    assert list(codes) == bc
    assert np.array_equal(cents, np.asarray(bcent, np.float32))


def test_outlier_slot_takes_nearest_centroid_lower_index_on_a_tie():
    # 8 inliers in 4 clusters of 2 with centroids -3e-3, -1e-3, 1e-3, 3e-3 (x 1) and one huge value
    base = np.array([-3.5, -2.5, -1.5, -0.5, 0.5, 1.5, 2.5, 3.5], np.float32) * np.float32(1e-3)
    w = np.concatenate([np.tile(base, 40), np.array([0.9], np.float32)])
    codes, cents, off, _ = Q.quantize(w, 2)
    assert list(off) == [w.size - 1] and codes[-1] == 3
    assert np.all(np.diff(cents) > 0)


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
def test_equal_population_mean_and_order_invariants(bits):
    rng = np.random.default_rng(7)
    w = (rng.standard_normal(196608) * 0.02).astype(np.float32)
    codes, cents, off, val = Q.quantize(w, bits)
    K = 1 << bits
    inl = np.ones(w.size, bool)
    inl[off] = False
    hist = np.bincount(codes[inl], minlength=K)
    assert hist.max() - hist.min() <= 1                                   # equal population
    assert np.all(np.diff(cents.astype(np.float64)) > 0)                  # sorted clusters
    total = float((cents.astype(np.float64) * hist).sum())
    assert abs(total - float(w[inl].astype(np.float64).sum())) <= 1e-6 * float(np.abs(w[inl]).sum())   # centroid = mean
    assert np.all(np.diff(off.astype(np.int64)) > 0) and np.array_equal(val, w[off])
    # every inlier sits in the cluster whose value range contains it
    lo = np.array([w[inl][codes[inl] == c].min() for c in range(K)])
    hi = np.array([w[inl][codes[inl] == c].max() for c in range(K)])
    assert np.all(hi[:-1] <= lo[1:])


def test_error_falls_with_bitwidth_and_outlier_rate_matches_closed_form():
    rng = np.random.default_rng(8)
    sigma = 0.02
    w = (rng.standard_normal(524288) * sigma).astype(np.float32)
    mse = []
    for bits in (2, 3, 4, 5, 6):
        codes, cents, off, val = Q.quantize(w, bits)
        deq = cents[codes].astype(np.float64)
        deq[off] = val
        mse.append(float(((deq - w) ** 2).mean()))
    assert all(a > b for a, b in zip(mse, mse[1:]))
    p = Q.outlier_fraction_closed_form(sigma)
    assert abs(p - 2.0 * (1.0 - 0.5 * (1.0 + math.erf(3.74 / math.sqrt(2.0))))) < 2e-5     # |z| > 3.74 for sigma 0.02
    n_out = Q.quantize(w, 4)[2].size
    assert abs(n_out - p * w.size) <= 5.0 * math.sqrt(p * w.size)


def test_constant_array_has_no_outliers_and_fewer_weights_than_clusters():
    w = np.full(256, 0.0125, np.float32)
    codes, cents, off, _ = Q.quantize(w, 3)
    assert off.size == 0 and np.all(cents == np.float32(0.0125))
    assert np.array_equal(codes, np.repeat(np.arange(8, dtype=np.uint8), 32))          # rank decides, in index order
    codes, cents, off, _ = Q.quantize(np.array([0.3, -0.1, 0.2], np.float32), 2)
    assert off.size == 0
    assert sorted(codes.tolist()) == sorted(set(codes.tolist())) and set(codes.tolist()) <= {0, 1, 2, 3}
    assert np.count_nonzero(cents) == 3


@pytest.mark.parametrize("bits", [2, 3, 4, 5, 6])
def test_bit_stream_reads_back(bits):
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 1 << bits, size=4096, dtype=np.uint8)
    words = Q.pack_stream(codes, bits)
    assert words.size == 4096 * bits // 32
    assert np.array_equal(O.unpack_codes(words, codes.size, bits), codes)
    big = 0
    for i, c in enumerate(codes[:64].tolist()):
        big |= c << (i * bits)
    assert [int(x) for x in words[: 64 * bits // 32]] == [(big >> (32 * j)) & 0xFFFFFFFF for j in range(64 * bits // 32)]


def test_agrees_with_the_input_generator_written_separately():
    import workloads as W
    from workloads.shards import ATTN, quantize_unit, make_unit_weights
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    mats = make_unit_weights(shape, 3, 0, ATTN, 1, outlier_stress=0.0015)
    for bits in (2, 5):
        blob = quantize_unit(mats, bits)
        words, cents, off, val = Q.quantize_unit(np.concatenate([m.reshape(-1) for m in mats]), bits)
        assert np.array_equal(words, blob.codes) and np.array_equal(off, blob.outlier_off)
        assert np.array_equal(val, blob.outlier_val) and np.array_equal(cents, blob.centroids)


@pytest.mark.parametrize("bits", [2, 4, 6])
def test_index_is_the_count_of_boundary_elements_not_above(bits):
    """The property the device's selecting method rests on: in the stable sorted order (= the order of (value,
    offset) pairs) cluster c starts at rank floor(c n'/2^k), so an inlier's index is the number of those boundary
    elements, c = 1 .. 2^k - 1, whose pair is not above its own.  Checked on arrays with many ties, where the
    offset decides, and with fewer inliers than clusters, where boundaries coincide."""
    rng = np.random.default_rng(40 + bits)
    cases = [(rng.standard_normal(4096) * 0.03).astype(np.float32),
             rng.choice(np.linspace(-0.05, 0.05, 7).astype(np.float32), size=2048),
             (rng.standard_normal(24) * 0.02).astype(np.float32)]
    for w in cases:
        codes, _, out_off, _ = Q.quantize(w, bits)
        inl = np.setdiff1d(np.arange(w.size), out_off)
        # -0 and +0 compare equal; the pair order is (value, offset)
        order = sorted(inl, key=lambda i: (float(w[i]), int(i)))
        n_in, K = len(order), 1 << bits
        bounds = [order[(c * n_in) // K] for c in range(1, K)] if n_in else []
        for i in inl:
            count = sum(1 for b in bounds if (float(w[b]), int(b)) <= (float(w[i]), int(i)))
            assert codes[i] == count
