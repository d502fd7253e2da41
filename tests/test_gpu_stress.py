"""Forwards queued back to back with no host synchronisation and warm caches in between: the timing regime in which the
kernels of consecutive forwards follow each other most closely.  Every bounded device-side wait must still be met
(a timeout would surface as STI_ERR_TIMEOUT at the next sti_sync) and every forward must give the same bits."""
import numpy as np
import pytest
import torch

import workloads as W

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _bf16_act(work):
    return torch.from_numpy(work.x_dev.view(np.int16).copy()).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("batch,seq,resident", [
    (1, 256, True),          # the headline launch shapes (BERT-large layers, one 256-token sequence)
    (1, 256, False),
    (1, 512, True),          # three CTAs over four token tiles: two tiles on some CTAs
    (1, 512, False),
    (8, 128, True),          # 1024 tokens: the two-CTA kernel
    (1, 8, True),            # a handful of tokens
    (16, 512, False),        # 8192 tokens: K-accumulating FFN2, tensor-core attention, warp-per-row LayerNorm
])
def test_queued_forwards_meet_every_wait_and_repeat_bit_for_bit(batch, seq, resident):
    work = W.make_config(5, n_layers=3, plan="mixed", resident=resident, resident_layers=3 if resident else 1,
                         batch=batch, seq=seq, workers=3)
    x = _bf16_act(work)
    n = 300 if batch * seq <= 1024 else 40
    with sti.Session(work) as s:
        y0 = torch.empty_like(x)
        sti.sti_model_forward(s.plan, x.data_ptr(), y0.data_ptr(), batch, seq)
        sti.sti_sync(s.ctx)
        ys = [torch.empty_like(x) for _ in range(4)]
        for i in range(n):                                    # no synchronisation, no cache flush
            sti.sti_model_forward(s.plan, x.data_ptr(), ys[i % 4].data_ptr(), batch, seq)
        sti.sti_sync(s.ctx)                                   # raises if a device-side wait ran out
        for y in ys:
            assert torch.equal(y.view(torch.int16), y0.view(torch.int16))


@pytest.mark.parametrize("seq", [128, 256, 512])
def test_queued_forwards_bert_base_layers(seq):
    # hidden 768: 96 KB weight tiles, rings of four two-box stages, 12 K boxes per tile (a ragged last ring round)
    work = W.make_config(3, n_layers=4, seq=seq, workers=3)          # fp32 activations, layers 0-2 preloaded
    x = torch.from_numpy(work.x_dev).cuda()
    with sti.Session(work) as s:
        y0 = torch.empty_like(x)
        sti.sti_model_forward(s.plan, x.data_ptr(), y0.data_ptr(), work.batch, seq)
        sti.sti_sync(s.ctx)
        ys = [torch.empty_like(x) for _ in range(3)]
        for i in range(400):
            sti.sti_model_forward(s.plan, x.data_ptr(), ys[i % 3].data_ptr(), work.batch, seq)
        sti.sti_sync(s.ctx)
        for y in ys:
            assert torch.equal(y.view(torch.int32), y0.view(torch.int32))
