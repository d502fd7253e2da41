"""CPU oracle of the shard quantizer (test infrastructure: only tests, the smoke check and the benchmark's
CPU baseline may import it; it shares no code with the CUDA path).

Section 6 of the paper (its outlier-aware quantization with one Gaussian, after GOBO), step by step, in fp64:
  1. fit one Gaussian component to the flat weight array (maximum likelihood: mean and 1/n variance);
  2. a weight whose log-likelihood under that Gaussian is below -4 is an outlier, kept verbatim with its offset;
  3. the other weights are sorted (ties in original order) and cut into 2^k clusters of equal population,
     cluster c = sorted[floor(c n'/2^k) : floor((c+1) n'/2^k));
  4. the arithmetic mean of a cluster is its centroid (fp32); every member gets the cluster's k-bit index;
  5. an outlier's slot also holds a k-bit index (Section 6: outliers, too, are represented as k-bit integers in the matrix):
     the nearest centroid, the lower index on a tie (reading: the paper does not say which);
  6. the indexes are written as a bit stream, index i at bits [i k, i k + k), least-significant bit first,
     in little-endian 32-bit words (Section 4.2 gives sizes only; this is the library's upload format).
"""
from __future__ import annotations

import math
from typing import Tuple

import numpy as np

LOGLIK_THRESHOLD = -4.0


def fit_gaussian(w: np.ndarray) -> Tuple[float, float]:
    """Step 1: maximum-likelihood mean and variance of a single component."""
    x = np.asarray(w, dtype=np.float64).reshape(-1)
    mu = float(x.sum() / x.size)
    var = float(((x - mu) ** 2).sum() / x.size)
    return mu, var


def log_likelihood(w: np.ndarray, mu: float, var: float) -> np.ndarray:
    """log N(w; mu, var), element by element."""
    x = np.asarray(w, dtype=np.float64).reshape(-1)
    with np.errstate(divide="ignore", invalid="ignore"):
        return -0.5 * np.log(2.0 * np.pi * var) - (x - mu) ** 2 / (2.0 * var)


def quantize(w: np.ndarray, bits: int):
    """Steps 1-5 on one flat fp32 array.  Returns (codes uint8[n], centroids float32[2^bits],
    outlier offsets uint32 ascending, outlier values float32)."""
    flat = np.ascontiguousarray(w, dtype=np.float32).reshape(-1)
    n = flat.size
    K = 1 << bits
    mu, var = fit_gaussian(flat)
    ll = log_likelihood(flat, mu, var)
    is_out = ll < LOGLIK_THRESHOLD                       # NaN (zero variance) compares false: no outliers
    out_off = np.flatnonzero(is_out).astype(np.uint32)
    inliers = np.flatnonzero(~is_out)
    order = inliers[np.argsort(flat[inliers], kind="stable")]
    n_in = order.size
    codes = np.zeros(n, dtype=np.uint8)
    centroids = np.zeros(K, dtype=np.float32)
    for c in range(K):
        lo, hi = (c * n_in) // K, ((c + 1) * n_in) // K
        members = order[lo:hi]
        if members.size:
            centroids[c] = np.float32(flat[members].astype(np.float64).sum() / members.size)
            codes[members] = c
    cent64 = centroids.astype(np.float64)
    for o in out_off:
        d = np.abs(np.float64(flat[o]) - cent64)
        codes[o] = int(np.argmin(d))                     # first minimum = lower index on a tie
    return codes, centroids, out_off, flat[out_off].copy()


def pack_stream(codes: np.ndarray, bits: int) -> np.ndarray:
    """Step 6: one index after the other into 32-bit words (plain loop over the indexes)."""
    codes = np.asarray(codes, dtype=np.uint64).reshape(-1)
    if (codes.size * bits) % 32:
        raise ValueError("the stream must fill whole 32-bit words")
    words = np.zeros(codes.size * bits // 32, dtype=np.uint64)
    pos = np.arange(codes.size, dtype=np.uint64) * np.uint64(bits)
    wi, sh = (pos >> np.uint64(5)).astype(np.int64), pos & np.uint64(31)
    np.add.at(words, wi, (codes << sh) & np.uint64(0xFFFFFFFF))            # disjoint bit fields: add = or
    spill = (sh + np.uint64(bits)) > np.uint64(32)
    np.add.at(words, wi[spill] + 1, codes[spill] >> (np.uint64(32) - sh[spill]))
    return words.astype(np.uint32)


def quantize_unit(w: np.ndarray, bits: int):
    """One shard unit -> (words, centroids, outlier offsets, outlier values)."""
    codes, centroids, off, val = quantize(w, bits)
    return pack_stream(codes, bits), centroids, off, val


def outlier_fraction_closed_form(sigma: float) -> float:
    """For exactly Gaussian weights of standard deviation sigma: P(log N(w) < -4) = 2 (1 - Phi(z*)),
    z*^2 = 2 (4 - 0.5 ln(2 pi sigma^2))."""
    z2 = 2.0 * (-LOGLIK_THRESHOLD - 0.5 * math.log(2.0 * math.pi * sigma * sigma))
    if z2 <= 0.0:
        return 1.0
    return math.erfc(math.sqrt(z2) / math.sqrt(2.0))
