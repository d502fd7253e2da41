"""The tensor-core attention kernel (tcgen05, one CTA per sequence and kept head) against the oracle layer, on
sequence lengths that are and are not multiples of its 128-row tiles, with and without padding masks, and against
the mma.sync kernel it replaces for many tokens."""
import os

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


def _work(batch, seq, act, seed, keep=lambda i: True):
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    bits = [2, 3, 4, 5, 6]
    attn = [[W.UnitPlan(keep(i), bits[i % 5], True) for i in range(4)]]
    ffn = [[W.UnitPlan(True, bits[(i + 2) % 5], True) for i in range(4)]]
    return W.build_workload("attn_tc", shape, batch, seq, act, attn, ffn, seed=seed)


def _run(work, lens, tune):
    from gpu_util import run_layer
    old = os.environ.get("STI_TUNE")
    os.environ["STI_TUNE"] = tune
    try:
        with sti.Session(work) as s:
            return run_layer(s, work, 0, lens=lens)
    finally:
        if old is None:
            os.environ.pop("STI_TUNE", None)
        else:
            os.environ["STI_TUNE"] = old


@pytest.mark.parametrize("batch,seq,lens,act", [
    (2, 128, None, "f32"),
    (3, 200, [200, 57, 130], "bf16"),          # ragged last tile, masks inside the first and the second chunk
    (2, 512, [512, 300], "bf16"),              # four chunks; a mask that cuts a whole chunk off
    (2, 384, [1, 129], "f32"),                 # a single valid key; one key into the second chunk
    (1, 130, None, "bf16"),                    # two rows into the second query tile
])
def test_tensor_core_attention_layer_matches_oracle_and_the_other_kernel(batch, seq, lens, act):
    from gpu_util import rel_err, REL_TOL
    work = _work(batch, seq, act, seed=batch * 1000 + seq, keep=lambda i: i != 1)
    a, f = O.decode_layer(work, 0)
    ref = O.layer_forward(work.x, work.dense[0], a, f, eps=work.ln_eps, seq_lens=lens)
    y_tc = _run(work, lens, "attn_tc_min_items=1")
    y_old = _run(work, lens, "attn_tc_min_items=0")
    assert np.isfinite(y_tc).all()
    assert rel_err(y_tc, ref) <= REL_TOL, rel_err(y_tc, ref)
    assert rel_err(y_old, ref) <= REL_TOL
    # same arithmetic, different order; with bf16 activations the LayerNorm output that feeds the FFN and the second
    # residual is bf16, so a one-step difference there can move an output by two bf16 steps (2 x 2^-8 of the maximum)
    assert rel_err(y_tc, y_old) <= (1e-2 if act == "bf16" else 5e-3)


def test_tensor_core_attention_is_the_default_for_many_sequences():
    # 24 sequences x 4 kept heads = 96 pairs of 256 tokens: the default rule picks the tensor-core kernel
    from gpu_util import rel_err, REL_TOL, run_layer
    work = _work(24, 256, "bf16", seed=77)
    a, f = O.decode_layer(work, 0)
    ref = O.layer_forward(work.x, work.dense[0], a, f, eps=work.ln_eps)
    with sti.Session(work) as s:
        y = run_layer(s, work, 0)
    assert rel_err(y, ref) <= REL_TOL
