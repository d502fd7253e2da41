"""GPU parity of the decode that lives INSIDE the dequant-GEMM (Section 4.2 decompression, Section 6 outliers).

sti_gemm_probe runs one of a layer's four GEMMs with the forward's own tile tables, decode routine and kernel.
With identity activations every output element is one exact product 1 * w, so the output is, bit for bit, the
bf16 weight tile the tensor cores were given; it must equal bf16_rne(oracle decode) for every kept unit.
"""
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


def _bf16_bits(a32: np.ndarray) -> np.ndarray:
    return (O.bf16_rne(a32).view(np.uint32) >> 16).astype(np.uint16)


def _identity_bf16(n: int) -> torch.Tensor:
    return torch.eye(n, dtype=torch.bfloat16, device="cuda")


def _plan(shape, bits_fn, keep_fn):
    attn = [[W.UnitPlan(keep_fn(ATTN, i), bits_fn(ATTN, i), True) for i in range(shape.n_heads)]]
    ffn = [[W.UnitPlan(keep_fn(FFN, i), bits_fn(FFN, i), True) for i in range(shape.n_ffn_slices)]]
    return attn, ffn


def _oracle_unit(work, kind, idx):
    sh = work.shape
    b = work.blobs[(0, kind, idx)]
    return O.decode_unit(b.bits, b.codes, b.centroids, b.outlier_off, b.outlier_val, sh.hidden, sh.head_dim,
                         sh.slice_width, kind)


def _probe(sess, gemm, K, out_shape, dtype, variant):
    x = _identity_bf16(K)
    out = torch.full(out_shape, float("nan"), dtype=dtype, device="cuda")
    torch.cuda.synchronize()
    n_part = sti.sti_gemm_probe(sess.plan, 0, gemm, x.data_ptr(), K, out.data_ptr(), out.numel() * out.element_size(),
                                variant)
    sti.sti_sync(sess.ctx)
    return out, n_part


def _check_all_gemms(work, sess, variant=0):
    """Every weight of every kept unit, through each of the four GEMMs, against the oracle's bf16 decode."""
    sh = work.shape
    d, f = sh.hidden, sh.slice_width
    heads, slices = work.kept(0, ATTN), work.kept(0, FFN)
    nh, ns = len(heads), len(slices)
    ref_a = {h: _oracle_unit(work, ATTN, h) for h in heads}
    ref_f = {j: _oracle_unit(work, FFN, j) for j in slices}
    max_parts = 16
    if nh:
        # QKV: out[(hi*3 + which)][t][r] = W_which,h[r][t]
        out, _ = _probe(sess, 0, d, (3 * nh, d, 64), torch.bfloat16, variant)
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        for hi, h in enumerate(heads):
            for which, name in enumerate("QKV"):
                want = _bf16_bits(ref_a[h][name]).T          # [d][64]
                assert np.array_equal(got[hi * 3 + which], want), ("QKV", h, name, variant)
        # O projection: sum over partials of out[sp][hi*64 + c][n] = O_h[n][c]
        out, n_part = _probe(sess, 1, nh * 64, (max_parts, nh * 64, d), torch.float32, variant)
        assert 1 <= n_part <= max_parts
        got = out[:n_part].cpu().numpy()
        assert np.isfinite(got).all()
        assert ((got != 0).sum(axis=0) <= 1).all()             # a weight comes from exactly one K group
        total = got.sum(axis=0)
        for hi, h in enumerate(heads):
            want = O.bf16_rne(ref_a[h]["O"]).T                # [64][d]
            assert np.array_equal(total[hi * 64:(hi + 1) * 64].view(np.uint32), want.view(np.uint32)), ("O", h, variant)
    if ns:
        out, _ = _probe(sess, 2, d, (d, ns * f), torch.bfloat16, variant)
        got = out.view(torch.int16).cpu().numpy().view(np.uint16)
        for ji, j in enumerate(slices):
            want = _bf16_bits(ref_f[j]["F1"]).T               # [d][f]
            assert np.array_equal(got[:, ji * f:(ji + 1) * f], want), ("FFN1", j, variant)
        out, n_part = _probe(sess, 3, ns * f, (max_parts, ns * f, d), torch.float32, variant)
        got = out[:n_part].cpu().numpy()
        assert np.isfinite(got).all()
        assert ((got != 0).sum(axis=0) <= 1).all()
        total = got.sum(axis=0)
        for ji, j in enumerate(slices):
            want = O.bf16_rne(ref_f[j]["F2"]).T               # [f][d]
            assert np.array_equal(total[ji * f:(ji + 1) * f].view(np.uint32), want.view(np.uint32)), ("FFN2", j, variant)


class _Tune:
    """STI_TUNE is read when a plan is created; set it around the session only."""
    def __init__(self, value):
        self.value = value

    def __enter__(self):
        self.old = os.environ.get("STI_TUNE")
        if self.value:
            os.environ["STI_TUNE"] = self.value
        return self

    def __exit__(self, *exc):
        if self.old is None:
            os.environ.pop("STI_TUNE", None)
        else:
            os.environ["STI_TUNE"] = self.old
        return False


BITS6 = [2, 3, 4, 5, 6, 32]


def _mixed_work(shape, seed, outlier_stress=0.0015, keep_fn=lambda k, i: True):
    attn, ffn = _plan(shape, lambda k, i: BITS6[(i + 2 * k) % 6], keep_fn)
    return W.build_workload("probe", shape, 1, 8, "bf16", attn, ffn, seed=seed, outlier_stress=outlier_stress)


@pytest.mark.parametrize("tune", ["", "qkv_n=32,f1_n=32,f2_n=32,o_group=1,f2_group=1",
                                  "qkv_n=64,f1_n=128,o_n=128,f2_n=128,o_group=3,f2_group=2"])
def test_fused_decode_small_shape_all_bitwidths_and_tilings(tune):
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=6, head_dim=64, ffn=1536, n_ffn_slices=6)
    work = _mixed_work(shape, seed=11)
    with _Tune(tune), sti.Session(work) as s:
        _check_all_gemms(work, s)


def test_fused_decode_bert_base_elastic_plan():
    # dropped units, every bitwidth, outliers at the paper's rate
    shape = W.BERT_BASE.with_layers(1)
    work = _mixed_work(shape, seed=12, keep_fn=lambda k, i: i not in ((1, 7) if k == ATTN else (0, 5, 10)))
    with sti.Session(work) as s:
        _check_all_gemms(work, s)


def test_fused_decode_bert_large_few_and_many_token_tilings():
    shape = W.BERT_LARGE.with_layers(1)
    work = _mixed_work(shape, seed=13)
    with sti.Session(work) as s:                              # tiling chosen for few tokens
        _check_all_gemms(work, s)
    with sti.Session(work, max_batch=8, max_seq=512) as s:    # tiling chosen for many tokens
        _check_all_gemms(work, s, variant=1)                  # one-CTA kernel
        _check_all_gemms(work, s, variant=2)                  # two-CTA (cta_group::2) kernel


def test_fused_decode_more_outliers_than_threads_in_a_tile():
    # 3 % of the weights redrawn with ten times the spread: a 64 x 1024 tile then holds more outliers than
    # the CTA has threads, which takes the decode's second outlier pass
    shape = W.ModelShape(n_layers=1, hidden=1024, n_heads=2, head_dim=64, ffn=512, n_ffn_slices=2)
    attn, ffn = _plan(shape, lambda k, i: 3 + i, lambda k, i: True)
    work = W.build_workload("probe", shape, 1, 8, "bf16", attn, ffn, seed=14, outlier_stress=0.03)
    off = work.blobs[(0, ATTN, 0)].outlier_off
    assert (off < 64 * 1024).sum() > 512                      # the Q matrix of head 0 is one tile
    with sti.Session(work) as s:
        _check_all_gemms(work, s)
        _check_all_gemms(work, s, variant=2)


def _check_ffn2_kacc(work, sess):
    """FFN2 through the K-accumulating kernel: one complete plane, every weight exactly once."""
    sh = work.shape
    f = sh.slice_width
    slices = work.kept(0, FFN)
    ns = len(slices)
    out, n_part = _probe(sess, 3, ns * f, (1, ns * f, sh.hidden), torch.float32, 3)
    assert n_part == 1
    got = out[0].cpu().numpy()
    assert np.isfinite(got).all()
    for ji, j in enumerate(slices):
        want = O.bf16_rne(_oracle_unit(work, FFN, j)["F2"]).T               # [f][d]
        assert np.array_equal(got[ji * f:(ji + 1) * f].view(np.uint32), want.view(np.uint32)), ("FFN2 kacc", j)


@pytest.mark.parametrize("tune,keep_ffn", [
    ("f2_kacc_min_tokens=1024", lambda i: True),                       # 6 K groups of 256, one tile pair per CTA pair
    ("f2_kacc_min_tokens=1024,cta_budget=4", lambda i: True),          # one CTA pair per column pair: 2 blocks (4 + 2 tiles)
    ("f2_kacc_min_tokens=1024,cta_budget=8", lambda i: i != 2),        # 5 slices kept
    ("f2_kacc_min_tokens=1024,f2_kacc_k=512", lambda i: True),         # K groups of two slices, whole decode tasks per warp
    ("f2_kacc_min_tokens=1024,f2_kacc_k=512,cta_budget=4", lambda i: i != 2),   # ... the last K group is 256 wide
])
def test_fused_decode_k_accumulating_ffn2_small_shape(tune, keep_ffn):
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1536, n_ffn_slices=6)
    work = _mixed_work(shape, seed=16, keep_fn=lambda k, i: True if k == ATTN else keep_ffn(i))
    with _Tune(tune), sti.Session(work, max_batch=8, max_seq=256) as s:
        _check_ffn2_kacc(work, s)


def test_fused_decode_k_accumulating_ffn2_bert_large():
    shape = W.BERT_LARGE.with_layers(1)
    work = _mixed_work(shape, seed=17)
    with sti.Session(work, max_batch=32, max_seq=512) as s:                # made for 16,384 tokens: the default rule applies
        _check_ffn2_kacc(work, s)
        _check_all_gemms(work, s, variant=2)
    with sti.Session(work, max_batch=4, max_seq=512) as s:                 # 2,048 tokens: no K-accumulating table
        x = _identity_bf16(64)
        out = torch.zeros(64 * 1024, dtype=torch.float32, device="cuda")
        with pytest.raises(sti.StiError) as e:
            sti.sti_gemm_probe(s.plan, 0, 3, x.data_ptr(), 64, out.data_ptr(), out.numel() * 4, 3)
        assert e.value.status == 5


def test_probe_argument_checks():
    shape = W.ModelShape(n_layers=1, hidden=256, n_heads=4, head_dim=64, ffn=1024, n_ffn_slices=4)
    attn, ffn = _plan(shape, lambda k, i: 4, lambda k, i: k == ATTN)      # no FFN slice kept
    work = W.build_workload("probe", shape, 1, 8, "bf16", attn, ffn, seed=15)
    x = _identity_bf16(256)
    out = torch.zeros(3 * 4 * 256 * 64, dtype=torch.bfloat16, device="cuda")
    with sti.Session(work) as s:
        with pytest.raises(sti.StiError) as e:
            sti.sti_gemm_probe(s.plan, 0, 2, x.data_ptr(), 256, out.data_ptr(), out.numel() * 2)
        assert e.value.status == 5                             # no kept unit feeds FFN1
        with pytest.raises(sti.StiError) as e:
            sti.sti_gemm_probe(s.plan, 0, 0, x.data_ptr(), 256, out.data_ptr(), out.numel() * 2 - 2)
        assert e.value.status == 4                             # output buffer too small
        with pytest.raises(sti.StiError) as e:
            sti.sti_gemm_probe(s.plan, 0, 7, x.data_ptr(), 256, out.data_ptr(), out.numel() * 2)
        assert e.value.status == 1
        sti.sti_gemm_probe(s.plan, 0, 0, x.data_ptr(), 256, out.data_ptr(), out.numel() * 2)
        sti.sti_sync(s.ctx)
