"""The allocation-free decode entry point against the plan-based one.

sti_matrix_decode_noalloc is for callers that cannot allocate device memory (a shard-file check inside a
serving process whose framework allocator owns the GPU's memory, code under an enforced memory budget):
it keeps its working copy of the shard in a fixed array inside the library instead of in a plan's arenas.
Here it must give, bit for bit, what sti_shard_decode gives for the same matrix and what the CPU oracle decodes,
on consecutive calls that reuse the array (larger matrix first, then smaller ones, so stale contents would show).
This file sorts last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import workloads as W
from workloads.shards import ATTN, FFN
from oracle import sti_oracle as O

sti = pytest.importorskip("paper_2207_05022_b200")


@pytest.fixture(scope="module", autouse=True)
def _built():
    from paper_2207_05022_b200 import build
    build.build_library()
    sti.load_library()


def _matrix_inputs(shape, kind, blob, m):
    """Canonical stream, table and outliers of matrix m alone (offsets rebased to the matrix)."""
    shapes = W.unit_matrix_shapes(shape, kind)
    word0 = sum(r * c * blob.bits // 32 for _, (r, c) in shapes[:m])
    flat0 = sum(r * c for _, (r, c) in shapes[:m])
    r, c = shapes[m][1]
    words = blob.codes[word0:word0 + r * c * blob.bits // 32]
    sel = (blob.outlier_off >= flat0) & (blob.outlier_off < flat0 + r * c)
    return r, c, words, (blob.outlier_off[sel] - flat0).astype(np.uint32), blob.outlier_val[sel]


@pytest.mark.gpu
def test_noalloc_decode_matches_plan_decode_on_consecutive_calls():
    shape = W.BERT_LARGE.with_layers(1)
    bits = [6, 3, 5, 2, 4]
    attn = [[W.UnitPlan(i < 3, bits[i % 5], True) for i in range(shape.n_heads)]]
    ffn = [[W.UnitPlan(i < 3, bits[(i + 2) % 5], True) for i in range(shape.n_ffn_slices)]]
    work = W.build_workload("noalloc", shape, 1, 8, "f32", attn, ffn, seed=7, outlier_stress=0.0015)
    # largest matrices first, then smaller ones: the shared array then still holds longer, older data
    order = [(FFN, 0, 0), (FFN, 0, 1), (ATTN, 0, 3), (ATTN, 1, 0), (FFN, 2, 1), (ATTN, 2, 2), (ATTN, 2, 3)]
    with sti.Session(work) as s:
        for kind, idx, m in order:
            blob = work.blobs[(0, kind, idx)]
            r, c, words, off, val = _matrix_inputs(shape, kind, blob, m)
            # the oracle's decode of the same matrix: indexes, fp32 values with outliers, bf16 operand bits
            o_w, o_codes = O.decode_unit(blob.bits, blob.codes, blob.centroids, blob.outlier_off, blob.outlier_val,
                                         shape.hidden, shape.head_dim, shape.slice_width, kind, return_codes=True)
            name = W.unit_matrix_shapes(shape, kind)[m][0]
            want_w = torch.from_numpy(o_w[name].reshape(-1).view(np.int32).copy())
            want_codes = torch.from_numpy(o_codes[name].reshape(-1).astype(np.uint8))
            want_bf16 = torch.from_numpy((O.bf16_rne(o_w[name]).reshape(-1).view(np.uint32) >> 16).astype(np.uint16)
                                         .view(np.int16).copy())
            ref = [torch.zeros(r * c, dtype=dt, device="cuda") for dt in (torch.float32, torch.uint8, torch.int16)]
            got = [torch.zeros(r * c, dtype=dt, device="cuda") for dt in (torch.float32, torch.uint8, torch.int16)]
            torch.cuda.synchronize()
            sti.sti_shard_decode(s.plan, 0, kind, idx, m, *[t.data_ptr() for t in ref])
            sti.sti_sync(s.ctx)
            for _ in range(2):                               # two calls in a row on the same inputs
                for t in got:
                    t.zero_()
                torch.cuda.synchronize()
                sti.sti_matrix_decode_noalloc(blob.bits, r, c, words, blob.centroids, off, val,
                                              *[t.data_ptr() for t in got])
                torch.cuda.synchronize()
                assert torch.equal(got[1], ref[1]), (kind, idx, m, "indexes")
                assert torch.equal(got[0].view(torch.int32), ref[0].view(torch.int32)), (kind, idx, m, "fp32")
                assert torch.equal(got[2], ref[2]), (kind, idx, m, "bf16")
                assert torch.equal(got[1].cpu(), want_codes), (kind, idx, m, "indexes vs oracle")
                assert torch.equal(got[0].view(torch.int32).cpu(), want_w), (kind, idx, m, "fp32 vs oracle")
                assert torch.equal(got[2].cpu(), want_bf16), (kind, idx, m, "bf16 vs oracle")
    assert torch.cuda.current_device() == 0                  # the call leaves the current device as it found it


def test_noalloc_rejects_what_the_fixed_array_cannot_hold():
    import ctypes as C
    lib = sti.load_library()
    words = np.zeros(1024 * 512 * 6 // 32, np.uint32)
    cent = np.zeros(64, np.float32)
    out = C.c_void_p(16)                                      # never dereferenced: the checks come first
    f = lib.sti_matrix_decode_noalloc
    ok_shape = (0, None, 6, 1024, 256)                        # 196,608 bytes: fits
    too_big = (0, None, 6, 1024, 512)                         # 393,216 bytes > 262,144
    assert f(*too_big, words.ctypes.data, cent.ctypes.data, None, None, 0, out, None, None) == 4      # STI_ERR_SIZE
    off = np.arange(5000, dtype=np.uint32)
    val = np.zeros(5000, np.float32)
    assert f(*ok_shape, words.ctypes.data, cent.ctypes.data, off.ctypes.data, val.ctypes.data, 5000,
             out, None, None) == 4                                                                    # too many outliers
    assert f(0, None, 7, 64, 128, words.ctypes.data, cent.ctypes.data, None, None, 0, out, None, None) == 2
    assert f(0, None, 4, 48, 128, words.ctypes.data, cent.ctypes.data, None, None, 0, out, None, None) == 3
    assert f(0, None, 4, 64, 128, words.ctypes.data, cent.ctypes.data, None, None, 0, None, None, None) == 1
