"""sti_decode_rate_probe: one launch of the dequant-GEMM over the FFN1 tiles of every layer (Section 4.2 decompression
at its steady-state rate).  Its output must equal, bit for bit, what the per-layer probe of the same GEMM gives."""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import ATTN, FFN

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _work(shape, resident=True, drop=()):
    bits = [2, 3, 4, 5, 6, 32]
    attn = [[W.UnitPlan(True, 4, resident) for _ in range(shape.n_heads)] for _ in range(shape.n_layers)]
    ffn = [[W.UnitPlan((l, i) not in drop, bits[(l + i) % 6], resident) for i in range(shape.n_ffn_slices)]
           for l in range(shape.n_layers)]
    return W.build_workload("rate", shape, 1, 32, "bf16", attn, ffn, seed=21)


@pytest.mark.parametrize("tokens", [8, 32, 100])
def test_all_layers_in_one_launch_equal_the_per_layer_launches(tokens):
    shape = W.ModelShape(n_layers=3, hidden=512, n_heads=4, head_dim=64, ffn=2048, n_ffn_slices=8)
    drop = {(0, 3), (2, 0), (2, 7)}
    work = _work(shape, drop=drop)
    d, f, nl = shape.hidden, shape.slice_width, shape.n_layers
    g = torch.Generator(device="cpu").manual_seed(5)
    x = torch.randn(tokens, d, generator=g).to(torch.bfloat16).cuda()
    # rows padded to a multiple of 8 tokens keep every buffer 16-byte aligned
    with sti.Session(work) as s:
        out = torch.full((tokens, nl * shape.ffn), float("nan"), dtype=torch.bfloat16, device="cuda")
        packed, tiles = sti.sti_decode_rate_probe(s.plan, x.data_ptr(), tokens, out.data_ptr(), out.numel() * 2)
        sti.sti_sync(s.ctx)
        want_bytes = 0
        for l in range(nl):
            kept = work.kept(l, FFN)
            ns = len(kept)
            ref = torch.full((tokens, ns * f), float("nan"), dtype=torch.bfloat16, device="cuda")
            sti.sti_gemm_probe(s.plan, l, 2, x.data_ptr(), tokens, ref.data_ptr(), ref.numel() * 2)
            sti.sti_sync(s.ctx)
            got = out[:, l * shape.ffn:l * shape.ffn + ns * f]
            assert torch.equal(got.view(torch.int16), ref.view(torch.int16)), l
            assert not torch.isnan(ref.float()).any()
            for j in kept:
                b = work.blobs[(l, FFN, j)].bits
                want_bytes += f * d * b // 8 + (0 if b == 32 else 4 << b)
        assert packed == want_bytes
        assert tiles > 0
        with pytest.raises(sti.StiError) as e:
            sti.sti_decode_rate_probe(s.plan, x.data_ptr(), tokens, out.data_ptr(), out.numel() * 2 - 2)
        assert e.value.status == 4
        with pytest.raises(sti.StiError) as e:
            sti.sti_decode_rate_probe(s.plan, x.data_ptr(), 129, out.data_ptr(), out.numel() * 2)
        assert e.value.status == 3


def test_streamed_plan_is_refused():
    shape = W.ModelShape(n_layers=2, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    work = _work(shape, resident=False)
    x = torch.zeros(8, 256, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(8, 2 * 1024, dtype=torch.bfloat16, device="cuda")
    with sti.Session(work) as s:
        with pytest.raises(sti.StiError) as e:
            sti.sti_decode_rate_probe(s.plan, x.data_ptr(), 8, out.data_ptr(), out.numel() * 2)
        assert e.value.status == 5
