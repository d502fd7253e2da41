"""Synthetic shard inputs: BERT-shaped weights, their quantized blobs, plans.

Everything here is input preparation for the execution path (Section 4.2 and
Section 6 of the paper describe how shards are produced offline):

* a layer is cut into M vertical slices (Table 1): attention head i with
  Q_i, K_i, V_i of shape [head_dim, d] and O_i of shape [d, head_dim], and FFN
  slice j with F1_j [f, d] and F2_j [d, f], f = d_ff / M_f.  All matrices are
  stored out-features x in-features, row-major (y = x W^T).  The attention
  part and the FFN part of a slice are handled as two independent shard
  units, each with its own keep flag and bitwidth; the paper's shard is the
  pair (head i, FFN slice i) with equal settings.
* each unit is dictionary-quantized (Section 6): a one-component Gaussian is
  fitted to the flat weight array, weights whose log-likelihood is below -4
  are outliers kept verbatim with their offsets, the others are sorted and cut
  into 2^k clusters of equal population whose arithmetic means are the
  centroids; every weight, outliers included, gets a k-bit index.
* the k-bit indexes are written as a bit stream: index i of a matrix (row-major
  flat order) occupies bits [i*k, i*k+k) of the stream, least-significant bit
  first, stored in little-endian 32-bit words.  A unit's blob is its matrices in
  the order Q,K,V,O or F1,F2, each starting on a 16-byte boundary.  The paper
  does not fix a bit order; this is the format of this library's upload call.

No unpacking, lookup or layer arithmetic lives here.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

ATTN = 0
FFN = 1
KIND_NAMES = ("attn", "ffn")
QUANT_BITS = (2, 3, 4, 5, 6)
RAW_BITS = 32
LOGLIK_OUTLIER_THRESHOLD = -4.0   # Section 6, following GOBO


@dataclass(frozen=True)
class ModelShape:
    n_layers: int
    hidden: int
    n_heads: int
    head_dim: int
    ffn: int
    n_ffn_slices: int

    @property
    def slice_width(self) -> int:
        return self.ffn // self.n_ffn_slices

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers)


BERT_BASE = ModelShape(n_layers=12, hidden=768, n_heads=12, head_dim=64, ffn=3072, n_ffn_slices=12)
BERT_LARGE = ModelShape(n_layers=24, hidden=1024, n_heads=16, head_dim=64, ffn=4096, n_ffn_slices=16)


def attn_matrix_shapes(shape: ModelShape) -> List[Tuple[str, Tuple[int, int]]]:
    d, hd = shape.hidden, shape.head_dim
    return [("Q", (hd, d)), ("K", (hd, d)), ("V", (hd, d)), ("O", (d, hd))]


def ffn_matrix_shapes(shape: ModelShape) -> List[Tuple[str, Tuple[int, int]]]:
    d, f = shape.hidden, shape.slice_width
    return [("F1", (f, d)), ("F2", (d, f))]


def unit_matrix_shapes(shape: ModelShape, kind: int) -> List[Tuple[str, Tuple[int, int]]]:
    return attn_matrix_shapes(shape) if kind == ATTN else ffn_matrix_shapes(shape)


def unit_weight_count(shape: ModelShape, kind: int) -> int:
    return sum(r * c for _, (r, c) in unit_matrix_shapes(shape, kind))


@dataclass
class ShardBlob:
    """One shard unit at one bitwidth, as handed to the upload call."""
    bits: int
    codes: np.ndarray                     # uint32 words; raw fp32 bit patterns when bits == 32
    centroids: Optional[np.ndarray]       # float32[2**bits]; None when bits == 32
    outlier_off: np.ndarray               # uint32, flat offsets within the unit, ascending
    outlier_val: np.ndarray               # float32

    @property
    def packed_bytes(self) -> int:
        n = self.codes.nbytes + self.outlier_off.nbytes + self.outlier_val.nbytes
        if self.centroids is not None:
            n += self.centroids.nbytes
        return n


@dataclass
class UnitPlan:
    keep: bool
    bits: int
    resident: bool


def _rng(seed: int, *path: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([int(seed), *[int(p) for p in path]]))


def make_unit_weights(shape: ModelShape, seed: int, layer: int, kind: int, index: int,
                      std: float = 0.02, outlier_stress: float = 0.0) -> List[np.ndarray]:
    """fp32 weights of one shard unit, N(0, std^2); optionally a fraction
    `outlier_stress` of them redrawn from N(0, (10 std)^2) to mimic the heavier
    tails (0.14-0.17 % outliers) the paper reports for trained models."""
    rng = _rng(seed, layer, kind, index, 0)
    mats = []
    for _, (r, c) in unit_matrix_shapes(shape, kind):
        w = rng.standard_normal((r, c), dtype=np.float32) * np.float32(std)
        mats.append(w)
    if outlier_stress > 0.0:
        for w in mats:
            flat = w.reshape(-1)
            n_out = max(1, int(round(outlier_stress * flat.size)))
            pos = rng.choice(flat.size, size=n_out, replace=False)
            flat[pos] = rng.standard_normal(n_out, dtype=np.float32) * np.float32(10.0 * std)
    return mats


def pack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """k-bit indexes -> 32-bit words, index i in stream bits [i*k, i*k+k), LSB first."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    if codes.size * bits % 32 != 0:
        raise ValueError("code count times bitwidth must fill whole 32-bit words")
    bitplane = (codes[:, None] >> np.arange(bits, dtype=np.uint8)[None, :]) & np.uint8(1)
    stream = np.packbits(bitplane.reshape(-1), bitorder="little")
    return stream.view("<u4").copy()


def quantize_unit(mats: Sequence[np.ndarray], bits: int) -> ShardBlob:
    """Gaussian outlier-aware dictionary quantization of one shard unit (Section 6)."""
    flat = np.concatenate([np.asarray(m, dtype=np.float32).reshape(-1) for m in mats])
    n = flat.size
    if bits == RAW_BITS:
        return ShardBlob(bits=RAW_BITS, codes=flat.view("<u4").copy(), centroids=None,
                         outlier_off=np.zeros(0, np.uint32), outlier_val=np.zeros(0, np.float32))
    if bits not in QUANT_BITS:
        raise ValueError(f"bitwidth {bits} not in {QUANT_BITS} or {RAW_BITS}")
    w64 = flat.astype(np.float64)
    mu = w64.mean()
    var = w64.var()                      # maximum-likelihood fit of one Gaussian component
    loglik = -0.5 * np.log(2.0 * np.pi * var) - (w64 - mu) ** 2 / (2.0 * var)
    is_out = loglik < LOGLIK_OUTLIER_THRESHOLD
    out_idx = np.flatnonzero(is_out)
    in_idx = np.flatnonzero(~is_out)
    order = in_idx[np.argsort(flat[in_idx], kind="stable")]    # ties keep original index order
    n_in = order.size
    n_clusters = 1 << bits
    bounds = (np.arange(n_clusters + 1, dtype=np.int64) * n_in) // n_clusters
    centroids = np.empty(n_clusters, dtype=np.float32)
    codes = np.empty(n, dtype=np.uint8)
    for c in range(n_clusters):
        members = order[bounds[c]:bounds[c + 1]]
        centroids[c] = np.float32(w64[members].mean()) if members.size else np.float32(0.0)
        codes[members] = c
    if out_idx.size:
        # an outlier's slot still holds a k-bit index: the nearest centroid, lower index on ties
        dist = np.abs(flat[out_idx, None].astype(np.float64) - centroids[None, :].astype(np.float64))
        codes[out_idx] = np.argmin(dist, axis=1).astype(np.uint8)
    words = []
    pos = 0
    for m in mats:
        cnt = int(np.asarray(m).size)
        words.append(pack_codes(codes[pos:pos + cnt], bits))
        pos += cnt
        if words[-1].nbytes % 16 != 0:
            raise ValueError("a matrix's bit stream must end on a 16-byte boundary")
    return ShardBlob(bits=bits, codes=np.concatenate(words), centroids=centroids,
                     outlier_off=out_idx.astype(np.uint32), outlier_val=flat[out_idx].copy())


def make_dense_params(shape: ModelShape, seed: int, layer: int) -> Dict[str, np.ndarray]:
    """Biases and LayerNorm parameters, kept in full precision (Section 6)."""
    rng = _rng(seed, layer, 2, 0, 0)
    d, hd, f = shape.hidden, shape.head_dim, shape.slice_width

    def n(*s):
        return (rng.standard_normal(s, dtype=np.float32) * np.float32(0.02))

    return {
        "bq": n(shape.n_heads, hd), "bk": n(shape.n_heads, hd), "bv": n(shape.n_heads, hd),
        "bo": n(d), "b1": n(shape.n_ffn_slices, f), "b2": n(d),
        "ln1_g": (1.0 + n(d)).astype(np.float32), "ln1_b": n(d),
        "ln2_g": (1.0 + n(d)).astype(np.float32), "ln2_b": n(d),
    }


def round_to_bf16(x: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Input preparation only: (uint16 bf16 bit patterns, the same values as fp32)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    bits16 = rounded.astype(np.uint16)
    back = (bits16.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return bits16, back


def make_activations(seed: int, batch: int, seq: int, hidden: int, act_dtype: str):
    """x ~ N(0,1).  Returns (x as fp32 values, device-format array)."""
    rng = _rng(seed, 0, 3, 0, 0)
    x = rng.standard_normal((batch, seq, hidden), dtype=np.float32)
    if act_dtype == "bf16":
        bits16, back = round_to_bf16(x)
        return back, bits16
    return x, x


@dataclass
class Workload:
    name: str
    shape: ModelShape
    batch: int
    seq: int
    act_dtype: str                                   # "f32" or "bf16"
    ln_eps: float
    ring_slots: int
    attn_plan: List[List[UnitPlan]]                  # [layer][head]
    ffn_plan: List[List[UnitPlan]]                   # [layer][slice]
    blobs: Dict[Tuple[int, int, int], ShardBlob]     # (layer, kind, index) -> blob, kept units only
    dense: List[Dict[str, np.ndarray]]               # per layer
    x: np.ndarray                                    # fp32 values [batch, seq, hidden]
    x_dev: np.ndarray                                # same in act_dtype storage (uint16 for bf16)
    seq_lens: Optional[np.ndarray] = None            # int32[batch] or None = all valid
    seed: int = 0
    originals: Dict[Tuple[int, int, int], List[np.ndarray]] = field(default_factory=dict)

    def kept(self, layer: int, kind: int) -> List[int]:
        plan = self.attn_plan if kind == ATTN else self.ffn_plan
        return [i for i, u in enumerate(plan[layer]) if u.keep]

    def packed_bytes(self, layers: Optional[Sequence[int]] = None) -> int:
        ls = range(self.shape.n_layers) if layers is None else layers
        return sum(b.packed_bytes for (l, _, _), b in self.blobs.items() if l in ls)

    def code_bytes(self) -> int:
        return sum(b.codes.nbytes for b in self.blobs.values())


def _layer_blobs(args):
    shape, seed, layer, attn_units, ffn_units, outlier_stress, keep_originals = args
    blobs, originals = {}, {}
    for kind, units in ((ATTN, attn_units), (FFN, ffn_units)):
        for idx, unit in enumerate(units):
            if not unit.keep:
                continue
            mats = make_unit_weights(shape, seed, layer, kind, idx, outlier_stress=outlier_stress)
            blobs[(layer, kind, idx)] = quantize_unit(mats, unit.bits)
            if keep_originals:
                originals[(layer, kind, idx)] = mats
    return blobs, originals


def build_workload(name: str, shape: ModelShape, batch: int, seq: int, act_dtype: str,
                   attn_plan: List[List[UnitPlan]], ffn_plan: List[List[UnitPlan]],
                   seed: int = 0, ring_slots: int = 2, ln_eps: float = 1e-12,
                   outlier_stress: float = 0.0, keep_originals: bool = False,
                   seq_lens: Optional[np.ndarray] = None, workers: int = 1) -> Workload:
    """`workers` > 1 quantizes layers in a pool of spawned processes (same result, faster)."""
    blobs: Dict[Tuple[int, int, int], ShardBlob] = {}
    originals: Dict[Tuple[int, int, int], List[np.ndarray]] = {}
    tasks = [(shape, seed, layer, attn_plan[layer], ffn_plan[layer], outlier_stress, keep_originals)
             for layer in range(shape.n_layers)]
    if workers > 1 and len(tasks) > 1:
        import concurrent.futures
        import multiprocessing
        ctx = multiprocessing.get_context("spawn")
        with concurrent.futures.ProcessPoolExecutor(max_workers=min(workers, len(tasks)), mp_context=ctx) as pool:
            results = list(pool.map(_layer_blobs, tasks))
    else:
        results = [_layer_blobs(t) for t in tasks]
    for b, o in results:
        blobs.update(b)
        originals.update(o)
    dense = [make_dense_params(shape, seed, layer) for layer in range(shape.n_layers)]
    x, x_dev = make_activations(seed, batch, seq, shape.hidden, act_dtype)
    return Workload(name=name, shape=shape, batch=batch, seq=seq, act_dtype=act_dtype, ln_eps=ln_eps,
                    ring_slots=ring_slots, attn_plan=attn_plan, ffn_plan=ffn_plan, blobs=blobs,
                    dense=dense, x=x, x_dev=x_dev, seq_lens=seq_lens, seed=seed, originals=originals)
