"""Seeded synthetic inputs shared by the tests, the benchmark and the smoke run.

This package only *makes inputs*: random BERT-shaped weights, their
dictionary-quantized shard blobs in the canonical bit-stream format, dense
parameters, activations and shard plans.  It contains none of the execution
path's arithmetic (no unpacking, no lookup, no layer math) and imports neither
the CPU oracle nor the CUDA library.
"""
from .shards import (  # noqa: F401
    ModelShape, ShardBlob, UnitPlan, Workload,
    BERT_BASE, BERT_LARGE,
    attn_matrix_shapes, ffn_matrix_shapes, unit_matrix_shapes, unit_weight_count,
    quantize_unit, pack_codes, make_unit_weights, make_dense_params, make_activations,
    build_workload,
)
from .configs import make_config, make_planned  # noqa: F401
