"""The C-ABI library builds, loads and exports every symbol the headers under include/ declare (no GPU needed)."""
import ctypes as C
import os
import re

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2207_05022_b200 import build, binding
    build.build_library()
    return binding.load_library()


def _declared_functions():
    text = "".join(open(os.path.join(ROOT, "include", h)).read()
                   for h in sorted(os.listdir(os.path.join(ROOT, "include"))) if h.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sti_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2207_05022_b200 import binding
    names = _declared_functions()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in a header but not exported"
    assert sorted(binding.EXPORTED) == names          # the binding wraps exactly the declared calls


def test_strerror_and_argument_checks(lib):
    import paper_2207_05022_b200 as sti
    assert sti.sti_strerror(0) == "ok"
    assert "upload" in sti.sti_strerror(6)
    out = C.c_void_p()
    assert lib.sti_ctx_create(None, 0, None, C.byref(out)) == 1          # STI_ERR_ARG
    bad = sti.StiModelDesc(n_layers=1, hidden=100, n_heads=2, head_dim=64, ffn=256, n_ffn_slices=2,
                           max_batch=1, max_seq=8, act_dtype=0, ln_eps=1e-12)
    assert lib.sti_ctx_create(C.byref(bad), 0, None, C.byref(out)) == 3  # STI_ERR_SHAPE: hidden % 128
    bad.hidden, bad.max_seq = 128, 1024
    assert lib.sti_ctx_create(C.byref(bad), 0, None, C.byref(out)) == 3  # max_seq > 512
    assert out.value is None                                             # untouched on error
    assert lib.sti_sync(None) == 1


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_fails_loudly(lib):
    import paper_2207_05022_b200 as sti
    good = sti.StiModelDesc(n_layers=1, hidden=128, n_heads=2, head_dim=64, ffn=256, n_ffn_slices=2,
                            max_batch=1, max_seq=8, act_dtype=0, ln_eps=1e-12)
    with pytest.raises(sti.StiError) as e:
        sti.sti_ctx_create(good, 0)
    assert e.value.status == 8                                           # STI_ERR_CUDA, no fallback path


def test_host_retile_rejects_bad_shapes(lib):
    src = np.zeros(64 * 128 * 3 // 8, np.uint8)
    dst = np.zeros_like(src)
    f = lib.sti_host_retile
    assert f(src.ctypes.data, dst.ctypes.data, 64, 128, 3) == 0
    assert f(src.ctypes.data, dst.ctypes.data, 64, 128, 7) == 2
    assert f(src.ctypes.data, dst.ctypes.data, 48, 128, 3) == 3
    assert f(src.ctypes.data, dst.ctypes.data, 96, 64, 3) == 3
    assert f(None, dst.ctypes.data, 64, 128, 3) == 1
