"""Host logic: the re-tiled index stream, read the way a warp reads it (plane p of lane l at
((g*J + j)*k + p)*512 + 16*l, index i of the lane's 128-index run at bits [i*k, i*k+k)), yields the
canonical row-major indexes.  Pure CPU; the reader below is a model of the kernels' access pattern."""
import numpy as np
import pytest

import workloads as W


def _read_like_a_warp(dev: np.ndarray, rows: int, cols: int, k: int) -> np.ndarray:
    out = np.zeros((rows, cols), dtype=np.int64)
    narrow = cols == 64
    J = 1 if narrow else cols // 128
    groups = rows // (64 if narrow else 32)
    for g in range(groups):
        for j in range(J):
            for lane in range(32):
                run = 0
                for p in range(k):
                    at = ((g * J + j) * k + p) * 512 + lane * 16
                    run |= int.from_bytes(dev[at:at + 16].tobytes(), "little") << (128 * p)
                for i in range(128):
                    c = (run >> (i * k)) & ((1 << k) - 1)
                    if narrow:
                        out[g * 64 + lane + 32 * (i // 64), i % 64] = c
                    else:
                        out[g * 32 + lane, j * 128 + i] = c
    return out


@pytest.mark.parametrize("k", [2, 3, 4, 5, 6])
@pytest.mark.parametrize("rows,cols", [(64, 128), (32, 256), (64, 384), (128, 64), (64, 64)])
def test_retile_matches_warp_reader(k, rows, cols):
    from paper_2207_05022_b200 import build, sti_host_retile
    build.build_library()
    rng = np.random.default_rng(rows * 1000 + cols + k)
    codes = rng.integers(0, 1 << k, size=(rows, cols))
    stream = W.pack_codes(codes.reshape(-1).astype(np.uint8), k)
    dev = sti_host_retile(stream, rows, cols, k)
    assert dev.nbytes == stream.nbytes == rows * cols * k // 8       # still k bits per weight
    assert np.array_equal(_read_like_a_warp(dev, rows, cols, k), codes)
    # it is a permutation of 8-byte pieces of the canonical stream: nothing lost or duplicated
    assert sorted(dev.view(np.uint64).tolist()) == sorted(stream.view(np.uint64).tolist())
