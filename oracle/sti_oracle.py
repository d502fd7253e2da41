"""CPU oracle for shard decode and the elastic transformer-layer forward.

TEST INFRASTRUCTURE ONLY.  This module is the plain, slow, obviously-correct
statement of what the execution path computes, written from the paper
(arXiv 2207.05022).  Only the test-suite, the smoke check and the benchmark's
CPU-baseline leg may import it; the library never does, and nothing here
imports the library.  Floating point is fp64 throughout unless a function says
otherwise; there is no blocking, fusion or reordering beyond what each cited
passage states.

What each function follows:

* `unpack_codes`   - Section 4.2 (a shard's weight matrix holds k-bit indexes
  into its centroid dictionary).  The paper does not fix the bit order;
  the stream format is the upload format of the library: index i of a matrix
  occupies stream bits [i*k, i*k+k), least-significant bit first, in
  little-endian 32-bit words.
* `dequantize`     - Section 4.2 (decompression replaces each index by its
  centroid, then outliers overwrite their positions) and Section 6 (outliers keep
  their original weights and offsets in the shard).
* `decode_unit`    - Table 1 (matrix shapes of a vertical slice) and
  Section 4.2 (one stored copy of a shard per fidelity version).
* `layer_forward`  - Section 2.1 (MHA over heads backed by Q, K, V, output
  layer O, two FFN layers), Section 4.2 (any subset of shards executes; a
  shard is one head plus 1/M of the FFN neurons), Section 6 (biases and
  layernorm stay in full fidelity).  The constants the paper takes from BERT
  (post-LN order, erf-GELU, 1/sqrt(head_dim) scaling, LayerNorm epsilon) are
  BERT's.
* `model_forward`  - Section 5.5 (layers 0..n-1 in order).

Readings of points the paper leaves open (also listed in the design notes):
Q/K/V slices take a head's output rows and O takes the head's input columns;
biases bq/bk/bv/b1 are sliced with their unit while b_o and b_2 are always
added once; a dropped unit contributes exactly zero with no rescaling; padded
keys get probability exactly zero when sequence lengths are given.

Pins (see tests/test_oracle_pins.py): bit-by-bit packer round trip, closed-form
sizes (32/k ratio, 215 MB), brute-force dictionary lookup, dense-layer equality
with all units kept, third-party (torch CPU) layer, dropped-unit-is-zero,
permutation invariance, softmax/LayerNorm closed forms.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
from scipy.special import erf as _scipy_erf

ATTN = 0
FFN = 1
RAW_BITS = 32


# ----------------------------------------------------------------------------
# Section 4.2: k-bit indexes
# ----------------------------------------------------------------------------
def unpack_codes(words: np.ndarray, n: int, bits: int) -> np.ndarray:
    """Indexes 0..n-1 of one matrix from its bit stream (uint32 words)."""
    if not 1 <= bits <= 8:
        raise ValueError("bits out of range")
    words = np.ascontiguousarray(words, dtype=np.uint32)
    if n * bits > words.size * 32:
        raise ValueError("stream too short")
    ext = np.concatenate([words, np.zeros(1, np.uint32)]).astype(np.uint64)
    start = np.arange(n, dtype=np.uint64) * np.uint64(bits)       # first stream bit of index i
    word = (start >> np.uint64(5)).astype(np.int64)
    shift = start & np.uint64(31)
    two_words = ext[word] | (ext[word + 1] << np.uint64(32))      # bits may straddle two words
    mask = np.uint64((1 << bits) - 1)
    return ((two_words >> shift) & mask).astype(np.uint8)


def stream_words(n: int, bits: int) -> int:
    """32-bit words occupied by n indexes of `bits` bits (no per-index padding)."""
    if (n * bits) % 32:
        raise ValueError("stream must fill whole words")
    return n * bits // 32


def bf16_rne(x: np.ndarray) -> np.ndarray:
    """fp32 -> nearest bfloat16 (ties to even), returned as fp32 values."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    lsb = (u >> np.uint64(16)) & np.uint64(1)
    r = ((u + np.uint64(0x7FFF) + lsb) >> np.uint64(16)) << np.uint64(16)
    return r.astype(np.uint32).view(np.float32).reshape(np.shape(x))


# ----------------------------------------------------------------------------
# Section 4.2 / Section 6: dictionary lookup and outliers
# ----------------------------------------------------------------------------
def dequantize(codes: np.ndarray, centroids: np.ndarray,
               outlier_off: np.ndarray, outlier_val: np.ndarray) -> np.ndarray:
    """w_i = centroid[c_i]; then every outlier offset gets its preserved value (fp32, exact)."""
    w = np.asarray(centroids, dtype=np.float32)[np.asarray(codes, dtype=np.int64)]
    w = w.copy()
    if len(outlier_off):
        w[np.asarray(outlier_off, dtype=np.int64)] = np.asarray(outlier_val, dtype=np.float32)
    return w


def unit_matrix_shapes(hidden: int, head_dim: int, slice_width: int, kind: int):
    """Table 1: (name, (out_features, in_features)) of a vertical slice's matrices, blob order."""
    if kind == ATTN:
        return [("Q", (head_dim, hidden)), ("K", (head_dim, hidden)),
                ("V", (head_dim, hidden)), ("O", (hidden, head_dim))]
    return [("F1", (slice_width, hidden)), ("F2", (hidden, slice_width))]


def decode_unit(bits: int, words: np.ndarray, centroids: Optional[np.ndarray],
                outlier_off: np.ndarray, outlier_val: np.ndarray,
                hidden: int, head_dim: int, slice_width: int, kind: int,
                return_codes: bool = False):
    """All matrices of one shard unit as fp32 arrays (dict name -> [out, in])."""
    shapes = unit_matrix_shapes(hidden, head_dim, slice_width, kind)
    total = sum(r * c for _, (r, c) in shapes)
    words = np.ascontiguousarray(words, dtype=np.uint32)
    if bits == RAW_BITS:
        flat = words.view(np.float32)[:total].copy()
        codes_flat = None
    else:
        parts = []
        pos = 0
        for _, (r, c) in shapes:
            nw = stream_words(r * c, bits)
            parts.append(unpack_codes(words[pos:pos + nw], r * c, bits))
            pos += nw
            pos = (pos + 3) // 4 * 4                                  # next matrix starts 16-byte aligned
        codes_flat = np.concatenate(parts)
        flat = dequantize(codes_flat, centroids, outlier_off, outlier_val)
    out = {}
    codes = {}
    pos = 0
    for name, (r, c) in shapes:
        out[name] = flat[pos:pos + r * c].reshape(r, c)
        if codes_flat is not None:
            codes[name] = codes_flat[pos:pos + r * c].reshape(r, c)
        pos += r * c
    return (out, codes) if return_codes else out


# ----------------------------------------------------------------------------
# Section 2.1 / 4.2: one transformer layer over the kept shard units
# ----------------------------------------------------------------------------
def gelu_erf(v: np.ndarray) -> np.ndarray:
    """BERT's GELU: v * Phi(v), Phi the standard normal CDF, via the error function."""
    return 0.5 * v * (1.0 + _scipy_erf(v / math.sqrt(2.0)))


def layer_norm(v: np.ndarray, gamma: np.ndarray, beta: np.ndarray, eps: float) -> np.ndarray:
    mean = v.mean(axis=-1, keepdims=True)
    var = ((v - mean) ** 2).mean(axis=-1, keepdims=True)
    return (v - mean) / np.sqrt(var + eps) * gamma + beta


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def layer_forward(x: np.ndarray, dense: Dict[str, np.ndarray],
                  attn_units: Dict[int, Dict[str, np.ndarray]],
                  ffn_units: Dict[int, Dict[str, np.ndarray]],
                  eps: float = 1e-12, seq_lens: Optional[Sequence[int]] = None,
                  return_intermediates: bool = False):
    """y for x of shape [batch, seq, hidden].

    `attn_units[h]` holds Q,K,V ([head_dim, d]) and O ([d, head_dim]) of kept head h;
    `ffn_units[j]` holds F1 ([f, d]) and F2 ([d, f]) of kept FFN slice j.  Heads and
    slices that are absent contribute nothing.
    """
    x = np.asarray(x, dtype=np.float64)
    batch, seq, d = x.shape
    p = {k: np.asarray(v, dtype=np.float64) for k, v in dense.items()}
    y = np.empty_like(x)
    inter = {"h1": np.empty_like(x)}
    for b in range(batch):
        xb = x[b]
        valid = seq if seq_lens is None else int(seq_lens[b])
        attn = np.tile(p["bo"], (seq, 1))
        for h in sorted(attn_units):
            u = attn_units[h]
            wq, wk, wv, wo = (np.asarray(u[n], dtype=np.float64) for n in ("Q", "K", "V", "O"))
            q = xb @ wq.T + p["bq"][h]
            k = xb @ wk.T + p["bk"][h]
            v = xb @ wv.T + p["bv"][h]
            s = (q @ k.T) / math.sqrt(wq.shape[0])
            prob = np.zeros_like(s)
            prob[:, :valid] = softmax_rows(s[:, :valid])            # padded keys: probability 0
            a = prob @ v
            attn += a @ wo.T
        h1 = layer_norm(xb + attn, p["ln1_g"], p["ln1_b"], eps)
        ffn = np.tile(p["b2"], (seq, 1))
        for j in sorted(ffn_units):
            u = ffn_units[j]
            f1, f2 = np.asarray(u["F1"], dtype=np.float64), np.asarray(u["F2"], dtype=np.float64)
            act = gelu_erf(h1 @ f1.T + p["b1"][j])
            ffn += act @ f2.T
        y[b] = layer_norm(h1 + ffn, p["ln2_g"], p["ln2_b"], eps)
        inter["h1"][b] = h1
    return (y, inter) if return_intermediates else y


def model_forward(x: np.ndarray, layers: List[Tuple[Dict[str, np.ndarray],
                                                    Dict[int, Dict[str, np.ndarray]],
                                                    Dict[int, Dict[str, np.ndarray]]]],
                  eps: float = 1e-12, seq_lens: Optional[Sequence[int]] = None,
                  return_all: bool = False):
    """Layers in order, each output feeding the next (Section 5.5)."""
    outs = []
    h = np.asarray(x, dtype=np.float64)
    for dense, attn_units, ffn_units in layers:
        h = layer_forward(h, dense, attn_units, ffn_units, eps=eps, seq_lens=seq_lens)
        outs.append(h)
    return outs if return_all else h


# ----------------------------------------------------------------------------
# Convenience: run a whole synthetic workload (duck-typed: any object with the
# fields of workloads.Workload).  Decodes every kept unit from its blob.
# ----------------------------------------------------------------------------
def decode_layer(work, layer: int):
    sh = work.shape
    attn_units, ffn_units = {}, {}
    for (l, kind, idx), blob in work.blobs.items():
        if l != layer:
            continue
        mats = decode_unit(blob.bits, blob.codes, blob.centroids, blob.outlier_off, blob.outlier_val,
                           sh.hidden, sh.head_dim, sh.slice_width, kind)
        (attn_units if kind == ATTN else ffn_units)[idx] = mats
    return attn_units, ffn_units


def run_workload(work, layers: Optional[Sequence[int]] = None, x: Optional[np.ndarray] = None,
                 return_all: bool = False):
    ls = list(range(work.shape.n_layers)) if layers is None else list(layers)
    stack = []
    for l in ls:
        a, f = decode_layer(work, l)
        stack.append((work.dense[l], a, f))
    return model_forward(work.x if x is None else x, stack, eps=work.ln_eps,
                         seq_lens=work.seq_lens, return_all=return_all)
