"""The five benchmark configurations as seeded synthetic workloads.

The paper evaluates on fine-tuned DynaBERT/DistilBERT weights and GLUE inputs;
neither is available offline, so weights are N(0, 0.02^2), activations N(0, 1),
quantized per shard unit with the paper's rule, and plans are drawn from the
distributions each configuration names.  The execution path is data-independent
(Section 5.2), so shapes, bitwidth mix, keep ratio and residency are what matter.
"""
from __future__ import annotations

from typing import List, Optional

import numpy as np

from .shards import (ATTN, FFN, BERT_BASE, BERT_LARGE, ModelShape, UnitPlan, Workload,
                     build_workload)

_SKEW3_BITS = np.array([2, 3, 4, 5, 6])
_SKEW3_P = np.array([0.15, 0.45, 0.20, 0.10, 0.10])


def _plan_rng(seed: int, tag: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([int(seed), 9, int(tag)]))


def _uniform_plan(shape: ModelShape, bits: int, resident_layers: int):
    attn = [[UnitPlan(True, bits, l < resident_layers) for _ in range(shape.n_heads)]
            for l in range(shape.n_layers)]
    ffn = [[UnitPlan(True, bits, l < resident_layers) for _ in range(shape.n_ffn_slices)]
           for l in range(shape.n_layers)]
    return attn, ffn


def _random_plan(shape: ModelShape, rng: np.random.Generator, resident_layers: int,
                 keep_heads: Optional[int] = None, keep_slices: Optional[int] = None,
                 keep_frac_range=None, bit_values=np.array([2, 3, 4, 5, 6]), bit_p=None):
    attn: List[List[UnitPlan]] = []
    ffn: List[List[UnitPlan]] = []
    for l in range(shape.n_layers):
        if keep_frac_range is not None:
            frac = rng.uniform(*keep_frac_range)
            kh = max(1, int(round(frac * shape.n_heads)))
            ks = max(1, int(round(frac * shape.n_ffn_slices)))
        else:
            kh = shape.n_heads if keep_heads is None else keep_heads
            ks = shape.n_ffn_slices if keep_slices is None else keep_slices
        heads = set(rng.choice(shape.n_heads, size=kh, replace=False).tolist())
        slices = set(rng.choice(shape.n_ffn_slices, size=ks, replace=False).tolist())
        res = l < resident_layers
        attn.append([UnitPlan(i in heads, int(rng.choice(bit_values, p=bit_p)), res)
                     for i in range(shape.n_heads)])
        ffn.append([UnitPlan(j in slices, int(rng.choice(bit_values, p=bit_p)), res)
                    for j in range(shape.n_ffn_slices)])
    return attn, ffn


def make_config(number: int, *, seed: int = 0, n_layers: Optional[int] = None,
                batch: Optional[int] = None, seq: Optional[int] = None,
                plan: str = "uniform3", resident: Optional[bool] = None,
                resident_layers: Optional[int] = None, keep_originals: bool = False,
                outlier_stress: float = 0.0, workers: int = 1) -> Workload:
    """Workload for configuration 1..5.

    1  one BERT-base layer, batch 1, seq 128, every unit kept at 4 bits, fp32 activations
    2  the same layer, bits ~ U{2..6} per unit, 8 of 12 heads and 9 of 12 FFN slices kept, bf16
    3  12-layer BERT-base, per-layer keep fraction ~ U[0.6, 1], bits ~ U{2..6},
       layers 0-2 in the preload buffer, the rest streamed, two ring slots
    4  24-layer BERT-large, seq 256, all kept, bits skewed toward 3, layers 0-1 preloaded
    5  BERT-large stack, batch/seq/plan given by the caller (`plan` is "uniform3" or "mixed"),
       bf16 activations, resident or streamed with a two-layer preload

    `n_layers` shortens the stack (tests); `resident_layers` overrides the preload depth;
    `workers` > 1 quantizes layers in parallel processes (same result).
    """
    if number == 1:
        shape = BERT_BASE.with_layers(n_layers or 1)
        attn, ffn = _uniform_plan(shape, 4, shape.n_layers if resident_layers is None else resident_layers)
        return build_workload("cfg1_base_layer_4bit", shape, batch or 1, seq or 128, "f32", attn, ffn,
                              seed=seed, keep_originals=keep_originals, outlier_stress=outlier_stress, workers=workers)
    if number == 2:
        shape = BERT_BASE.with_layers(n_layers or 1)
        attn, ffn = _random_plan(shape, _plan_rng(seed, 2),
                                 shape.n_layers if resident_layers is None else resident_layers,
                                 keep_heads=8, keep_slices=9)
        return build_workload("cfg2_base_layer_elastic", shape, batch or 1, seq or 128, "bf16", attn, ffn,
                              seed=seed, keep_originals=keep_originals, outlier_stress=outlier_stress, workers=workers)
    if number == 3:
        shape = BERT_BASE.with_layers(n_layers or 12)
        attn, ffn = _random_plan(shape, _plan_rng(seed, 3), 3 if resident_layers is None else resident_layers,
                                 keep_frac_range=(0.6, 1.0))
        return build_workload("cfg3_base_model_streamed", shape, batch or 1, seq or 128, "f32", attn, ffn,
                              seed=seed, ring_slots=2, keep_originals=keep_originals,
                              outlier_stress=outlier_stress, workers=workers)
    if number == 4:
        shape = BERT_LARGE.with_layers(n_layers or 24)
        attn, ffn = _random_plan(shape, _plan_rng(seed, 4), 2 if resident_layers is None else resident_layers,
                                 bit_values=_SKEW3_BITS, bit_p=_SKEW3_P)
        return build_workload("cfg4_large_model_streamed", shape, batch or 1, seq or 256, "f32", attn, ffn,
                              seed=seed, ring_slots=2, keep_originals=keep_originals,
                              outlier_stress=outlier_stress, workers=workers)
    if number == 5:
        shape = BERT_LARGE.with_layers(n_layers or 24)
        res_layers = resident_layers
        if res_layers is None:
            res_layers = shape.n_layers if (resident is None or resident) else 2
        if plan == "uniform3":
            attn, ffn = _uniform_plan(shape, 3, res_layers)
        elif plan == "mixed":
            attn, ffn = _random_plan(shape, _plan_rng(seed, 5), res_layers)
        else:
            raise ValueError("plan must be 'uniform3' or 'mixed'")
        b, s = batch or 1, seq or 128
        return build_workload(f"cfg5_large_b{b}_s{s}_{plan}_{'res' if res_layers >= shape.n_layers else 'str'}",
                              shape, b, s, "bf16", attn, ffn, seed=seed, ring_slots=2,
                              keep_originals=keep_originals, outlier_stress=outlier_stress, workers=workers)
    raise ValueError("configuration number must be 1..5")


def make_planned(keep, bits, preload, *, batch: int = 1, seq: int = 256, seed: int = 0,
                 act_dtype: str = "bf16", workers: int = 1, ring_slots: int = 4) -> Workload:
    """BERT-large workload for a planner result: `keep`, `bits`, `preload` are [n_layers][16] grids over
    the paper's shards; shard i of a layer is attention head i plus FFN slice i, which share the entry.
    Layers with no kept shard (beyond the submodel's depth) are left out.  `ring_slots` streamed-layer
    buffers let the copy engine run that many layers ahead of the computation."""
    keep = np.asarray(keep)
    depth = int(max(l + 1 for l in range(keep.shape[0]) if keep[l].any()))
    shape = BERT_LARGE.with_layers(depth)
    if keep.shape[1] != shape.n_heads or shape.n_ffn_slices != shape.n_heads:
        raise ValueError("planner grid must have one column per head / FFN slice")
    def grid():
        return [[UnitPlan(bool(keep[l][i]), int(bits[l][i]) if keep[l][i] else 2, bool(preload[l][i]))
                 for i in range(shape.n_heads)] for l in range(depth)]
    return build_workload(f"planned_large_b{batch}_s{seq}", shape, batch, seq, act_dtype, grid(), grid(),
                          seed=seed, ring_slots=ring_slots, workers=workers)
