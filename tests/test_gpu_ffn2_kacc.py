"""FFN2 through the K-accumulating kernel inside a whole layer: against the oracle layer and against the ordinary
path (one fp32 plane per K group, added up by LayerNorm), on token counts that give full blocks of four tile pairs,
a ragged last block, an odd number of token tiles and rows past the end of the last tile."""
import os

import numpy as np
import pytest
import torch

import workloads as W
from oracle import sti_oracle as O

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _work(batch, seq, act, seed, keep=lambda i: True):
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1536, n_ffn_slices=6)
    bits = [2, 3, 4, 5, 6, 32]
    attn = [[W.UnitPlan(True, bits[i % 5], True) for i in range(4)]]
    ffn = [[W.UnitPlan(keep(i), bits[(i + 1) % 6], True) for i in range(6)]]
    return W.build_workload("kacc", shape, batch, seq, act, attn, ffn, seed=seed, outlier_stress=0.0015)


def _run(work, tune):
    from gpu_util import run_layer
    old = os.environ.get("STI_TUNE")
    os.environ["STI_TUNE"] = tune
    try:
        with sti.Session(work) as s:
            y = run_layer(s, work, 0)
            launches = sti.sti_ctx_launch_count(s.ctx)
        return y, launches
    finally:
        if old is None:
            os.environ.pop("STI_TUNE", None)
        else:
            os.environ["STI_TUNE"] = old


@pytest.mark.parametrize("batch,seq,act,budget,kgroup,keep", [
    (16, 128, "bf16", 148, 256, lambda i: True),   # 2,048 tokens: 8 tile pairs over 8 CTA pairs per column pair
    (16, 128, "f32", 4, 256, lambda i: True),      # one CTA pair per column pair: two full blocks of four
    (11, 100, "bf16", 4, 512, lambda i: i != 4),   # 1,100 tokens: 9 tiles (odd), ragged rows, 5 slices (a 256-wide group)
    (24, 128, "bf16", 8, 256, lambda i: i % 2 == 0),    # 3,072 tokens: 12 tile pairs over two CTA pairs: blocks of 4 + 2
    (24, 128, "f32", 8, 512, lambda i: True),
    (16, 128, "bf16", 148, 512, lambda i: i == 3),      # one FFN slice kept: a single 256-wide K group
    (16, 128, "f32", 4, 256, lambda i: i in (0, 5)),    # two slices, one group each, two blocks per CTA pair
])
def test_layer_with_k_accumulating_ffn2(batch, seq, act, budget, kgroup, keep):
    from gpu_util import rel_err, REL_TOL
    work = _work(batch, seq, act, seed=batch * 100 + seq, keep=keep)
    a, f = O.decode_layer(work, 0)
    ref = O.layer_forward(work.x, work.dense[0], a, f, eps=work.ln_eps)
    y_k, _ = _run(work, f"f2_kacc_min_tokens=1024,f2_kacc_k={kgroup},cta_budget={budget}")
    y_p, _ = _run(work, f"f2_kacc_min_tokens=0,cta_budget={budget}")
    assert rel_err(y_k, ref) <= REL_TOL
    assert rel_err(y_p, ref) <= REL_TOL
    # same bf16 products, fp32 sums in a different order: the two paths agree far below the tolerance
    # (bf16 outputs may differ by one rounding step of 2^-8 relative)
    assert rel_err(y_k, y_p.astype(np.float64)) <= (1e-2 if act == "bf16" else 2e-3)
