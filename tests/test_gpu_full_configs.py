"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (CUDA-graph replay,
programmatic dependent launch, streamed shards): configurations 3 and 4 whole, and one configuration-5 point
checked on sampled sequences (sequences of a batch are independent, so the oracle runs them one by one)."""
import dataclasses

import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import round_to_bf16
from oracle import sti_oracle as O

pytestmark = pytest.mark.gpu

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def test_config3_full_model_streamed():
    from gpu_util import run_model, rel_err, REL_TOL
    work = W.make_config(3, workers=4)                 # 12 layers, 0-2 preloaded, 3-11 streamed, 2 ring slots
    outs = O.run_workload(work, return_all=True)
    with sti.Session(work) as s:
        y = run_model(s, work)
        y2 = run_model(s, work)                         # graph replay
        yh = run_model(s, work, host=True)
    assert np.array_equal(y, y2) and np.array_equal(y, yh)
    e = rel_err(y, outs[-1])
    print("config 3 rel err after 12 layers: %.3e" % e)
    assert e <= REL_TOL


def test_config4_full_model_resident_and_streamed():
    from gpu_util import run_model, rel_err, REL_TOL
    work = W.make_config(4, workers=8)                 # 24 layers BERT-large, seq 256, layers 0-1 preloaded
    ref = O.run_workload(work)
    with sti.Session(work) as s:
        y_str = run_model(s, work)
        y_str2 = run_model(s, work)
    attn = [[W.UnitPlan(u.keep, u.bits, True) for u in layer] for layer in work.attn_plan]
    ffn = [[W.UnitPlan(u.keep, u.bits, True) for u in layer] for layer in work.ffn_plan]
    with sti.Session(dataclasses.replace(work, attn_plan=attn, ffn_plan=ffn)) as s:
        y_res = run_model(s, work)
    assert np.array_equal(y_str, y_str2) and np.array_equal(y_str, y_res)     # residency never changes results
    e = rel_err(y_res, ref)
    print("config 4 rel err after 24 layers: %.3e" % e)
    assert e <= REL_TOL


@pytest.mark.parametrize("plan", ["uniform3", "mixed"])
def test_config5_point_sampled_sequences(plan):
    from gpu_util import rel_err, REL_TOL
    B, L, n_layers = 8, 512, 3
    work = W.make_config(5, n_layers=n_layers, plan=plan, resident=False, resident_layers=1, batch=1, seq=L, workers=3)
    rng = np.random.default_rng(5)
    bits16, xv = round_to_bf16(rng.standard_normal((B, L, work.shape.hidden), dtype=np.float32))
    lens = [L, 300, L, 17, L, L, 512, 1]
    x = torch.from_numpy(bits16.view(np.int16)).cuda().view(torch.bfloat16)
    y = torch.empty_like(x)
    lens_dev = torch.tensor(lens, dtype=torch.int32).cuda()
    torch.cuda.synchronize()
    with sti.Session(work, max_batch=B, max_seq=L) as s:
        sti.sti_model_forward(s.plan, x.data_ptr(), y.data_ptr(), B, L, lens_dev.data_ptr())
        sti.sti_sync(s.ctx)
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    for b in (0, 1, 3, 7):                               # sampled sequences, incl. padded ones
        ref = O.run_workload(dataclasses.replace(work, seq_lens=[lens[b]]), x=xv[b:b + 1])
        e = rel_err(got[b:b + 1, :lens[b]], ref[:, :lens[b]])    # padded query rows carry no meaning
        assert e <= REL_TOL, (b, e)


def test_config5_largest_bench_point_sampled_sequences():
    # 32 x 512 = 16,384 tokens: the launch shapes bench.py times (two-CTA GEMMs, K-accumulating FFN2 with two
    # blocks of tile pairs per CTA pair, tensor-core attention, warp-per-row LayerNorm), two layers, streamed
    from gpu_util import rel_err, REL_TOL
    B, L, n_layers = 32, 512, 2
    work = W.make_config(5, n_layers=n_layers, plan="mixed", resident=False, resident_layers=1, batch=1, seq=L, workers=3)
    rng = np.random.default_rng(6)
    bits16, xv = round_to_bf16(rng.standard_normal((B, L, work.shape.hidden), dtype=np.float32))
    lens = [L] * B
    lens[5], lens[30] = 131, 400
    x = torch.from_numpy(bits16.view(np.int16)).cuda().view(torch.bfloat16)
    y = torch.empty_like(x)
    lens_dev = torch.tensor(lens, dtype=torch.int32).cuda()
    torch.cuda.synchronize()
    with sti.Session(work, max_batch=B, max_seq=L) as s:
        sti.sti_model_forward(s.plan, x.data_ptr(), y.data_ptr(), B, L, lens_dev.data_ptr())
        sti.sti_sync(s.ctx)
        y2 = torch.empty_like(x)
        sti.sti_model_forward(s.plan, x.data_ptr(), y2.data_ptr(), B, L, lens_dev.data_ptr())   # graph replay
        sti.sti_sync(s.ctx)
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    got = y.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    for b in (0, 5, 17, 30, 31):                         # first, last, middle and the padded sequences
        ref = O.run_workload(dataclasses.replace(work, seq_lens=[lens[b]]), x=xv[b:b + 1])
        e = rel_err(got[b:b + 1, :lens[b]], ref[:, :lens[b]])
        assert e <= REL_TOL, (b, e)
