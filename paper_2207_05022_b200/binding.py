"""ctypes binding of include/sti.h: same names, argument marshalling only.

Device buffers are passed as integer addresses (e.g. `tensor.data_ptr()`); host arrays as
numpy arrays.  Nothing here computes: if the shared library is missing or cannot be loaded
the import of any entry point raises, there is no other execution path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

STI_OK = 0
STI_ATTN, STI_FFN = 0, 1
STI_F32, STI_BF16 = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libsti_b200.so"
_lib = None


class StiError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = sti_strerror(status) if _lib is not None else str(status)
        super().__init__(f"{where}: {msg} (status {status})")


class StiModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("n_ffn_slices", C.c_int32),
                ("max_batch", C.c_int32), ("max_seq", C.c_int32), ("act_dtype", C.c_int32),
                ("ln_eps", C.c_float)]


class StiShardCfg(C.Structure):
    _fields_ = [("keep", C.c_uint8), ("bits", C.c_uint8), ("resident", C.c_uint8)]


class StiShardBlob(C.Structure):
    _fields_ = [("bits", C.c_int32), ("codes", C.c_void_p), ("n_code_words", C.c_size_t),
                ("centroids", C.c_void_p), ("outlier_off", C.c_void_p), ("outlier_val", C.c_void_p),
                ("n_outliers", C.c_size_t)]


class StiStats(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("compute_us", C.c_float * 64), ("copy_us", C.c_float * 64),
                ("stall_us", C.c_float * 64), ("streamed_bytes", C.c_uint64 * 64),
                ("resident_bytes", C.c_uint64 * 64), ("total_us", C.c_float),
                ("gemm_us", C.c_float * 64), ("attn_us", C.c_float * 64), ("ln_us", C.c_float * 64),
                ("gemm_launches", C.c_int32)]


def library_path() -> str:
    return os.path.join(_HERE, _LIB_NAME)


def load_library():
    """Loads the C-ABI library built by `python -m paper_2207_05022_b200.build`."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2207_05022_b200.build` "
                           "(there is no fallback execution path)")
    lib = C.CDLL(path)
    vp, i32, u64p = C.c_void_p, C.c_int, C.POINTER(C.c_uint64)
    sigs = {
        "sti_ctx_create": ([C.POINTER(StiModelDesc), i32, vp, C.POINTER(vp)], i32),
        "sti_ctx_destroy": ([vp], None),
        "sti_ctx_set_layer_params": ([vp, i32] + [vp] * 10, i32),
        "sti_plan_create": ([vp, C.POINTER(StiShardCfg), C.POINTER(StiShardCfg), i32, C.POINTER(vp)], i32),
        "sti_plan_destroy": ([vp], None),
        "sti_shard_upload": ([vp, i32, i32, i32, C.POINTER(StiShardBlob)], i32),
        "sti_plan_finalize": ([vp], i32),
        "sti_layer_forward": ([vp, i32, vp, vp, i32, i32, vp], i32),
        "sti_model_forward": ([vp, vp, vp, i32, i32, vp], i32),
        "sti_model_forward_host": ([vp, vp, vp, i32, i32, vp], i32),
        "sti_sync": ([vp], i32),
        "sti_shard_decode": ([vp, i32, i32, i32, i32, vp, vp, vp], i32),
        "sti_gemm_probe": ([vp, i32, i32, vp, i32, vp, C.c_size_t, i32, C.POINTER(C.c_int32)], i32),
        "sti_decode_rate_probe": ([vp, vp, i32, vp, C.c_size_t, u64p, C.POINTER(C.c_int32)], i32),
        "sti_plan_set_profiling": ([vp, i32], i32),
        "sti_get_kernel_stamps": ([vp, vp, C.c_size_t, C.POINTER(C.c_int32)], i32),
        "sti_plan_set_overlap": ([vp, i32], i32),
        "sti_get_stats": ([vp, C.POINTER(StiStats)], i32),
        "sti_plan_memory": ([vp, u64p, u64p, u64p], i32),
        "sti_plan_check_guards": ([vp, C.POINTER(C.c_int32)], i32),
        "sti_plan_inject": ([vp, i32, i32, C.c_uint], i32),
        "sti_plan_retain": ([vp, vp, vp, u64p], i32),
        "sti_shard_adopt": ([vp, vp, i32, i32, i32], i32),
        "sti_plan_fill_stats": ([vp, u64p, u64p, u64p], i32),
        "sti_ctx_launch_count": ([vp], C.c_uint64),
        "sti_host_retile": ([vp, vp, C.c_uint32, C.c_uint32, C.c_uint32], i32),
        "sti_strerror": ([i32], C.c_char_p),
        "sti_matrix_decode_noalloc": ([i32, vp, i32, C.c_uint32, C.c_uint32, vp, vp, vp, vp, C.c_size_t, vp, vp, vp],
                                      i32),
    }
    for name, (argtypes, restype) in sigs.items():
        fn = getattr(lib, name)          # AttributeError if the library does not export it
        fn.argtypes = argtypes
        fn.restype = restype
    _lib = lib
    return lib


EXPORTED = ("sti_ctx_create", "sti_ctx_destroy", "sti_ctx_set_layer_params", "sti_plan_create",
            "sti_plan_destroy", "sti_shard_upload", "sti_plan_finalize", "sti_layer_forward",
            "sti_model_forward", "sti_model_forward_host", "sti_sync", "sti_shard_decode", "sti_gemm_probe", "sti_decode_rate_probe", "sti_get_kernel_stamps", "sti_plan_inject",
            "sti_plan_retain", "sti_shard_adopt", "sti_plan_fill_stats",
            "sti_plan_set_profiling", "sti_plan_set_overlap", "sti_get_stats", "sti_plan_memory", "sti_plan_check_guards", "sti_ctx_launch_count",
            "sti_host_retile", "sti_strerror", "sti_matrix_decode_noalloc", "sti_plan_auto",
            "sti_preload_after_run", "sti_quantize_units", "sti_quantize_units_by", "sti_quantize_workspace_bytes")


def _check(status: int, where: str):
    if status != STI_OK:
        raise StiError(status, where)


def _host(a: Optional[np.ndarray], dtype) -> Optional[np.ndarray]:
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=dtype)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def sti_strerror(status: int) -> str:
    return load_library().sti_strerror(int(status)).decode()


def sti_ctx_create(desc: StiModelDesc, device: int = 0, compute_stream: int = 0) -> int:
    out = C.c_void_p()
    _check(load_library().sti_ctx_create(C.byref(desc), device, C.c_void_p(compute_stream or None), C.byref(out)),
           "sti_ctx_create")
    return out.value


def sti_ctx_destroy(ctx: int):
    load_library().sti_ctx_destroy(C.c_void_p(ctx))


def sti_ctx_set_layer_params(ctx: int, layer: int, bq, bk, bv, bo, b1, b2, ln1_g, ln1_b, ln2_g, ln2_b):
    arrs = [_host(a, np.float32).reshape(-1) for a in (bq, bk, bv, bo, b1, b2, ln1_g, ln1_b, ln2_g, ln2_b)]
    _check(load_library().sti_ctx_set_layer_params(C.c_void_p(ctx), layer, *[_ptr(a) for a in arrs]),
           "sti_ctx_set_layer_params")


def _cfg_array(cfgs: Sequence[Sequence[int]]):
    arr = (StiShardCfg * len(cfgs))()
    for i, (keep, bits, resident) in enumerate(cfgs):
        arr[i].keep, arr[i].bits, arr[i].resident = int(bool(keep)), int(bits), int(bool(resident))
    return arr


def sti_plan_create(ctx: int, attn: Sequence[Sequence[int]], ffn: Sequence[Sequence[int]], ring_slots: int = 2) -> int:
    """attn/ffn: flat, layer-major sequences of (keep, bits, resident)."""
    out = C.c_void_p()
    _check(load_library().sti_plan_create(C.c_void_p(ctx), _cfg_array(attn), _cfg_array(ffn), ring_slots,
                                          C.byref(out)), "sti_plan_create")
    return out.value


def sti_plan_destroy(plan: int):
    load_library().sti_plan_destroy(C.c_void_p(plan))


def sti_shard_upload(plan: int, layer: int, kind: int, index: int, bits: int, codes: np.ndarray,
                     centroids: Optional[np.ndarray], outlier_off: Optional[np.ndarray] = None,
                     outlier_val: Optional[np.ndarray] = None):
    codes = _host(codes, np.uint32)
    cent = _host(centroids, np.float32)
    off = _host(outlier_off, np.uint32) if outlier_off is not None and len(outlier_off) else None
    val = _host(outlier_val, np.float32) if outlier_val is not None and len(outlier_val) else None
    blob = StiShardBlob(bits=int(bits), codes=_ptr(codes), n_code_words=codes.size, centroids=_ptr(cent),
                        outlier_off=_ptr(off), outlier_val=_ptr(val), n_outliers=0 if off is None else off.size)
    _check(load_library().sti_shard_upload(C.c_void_p(plan), layer, kind, index, C.byref(blob)), "sti_shard_upload")


def sti_plan_finalize(plan: int):
    _check(load_library().sti_plan_finalize(C.c_void_p(plan)), "sti_plan_finalize")


def sti_layer_forward(plan: int, layer: int, x_dev: int, y_dev: int, batch: int, seq: int, seq_lens_dev: int = 0):
    _check(load_library().sti_layer_forward(C.c_void_p(plan), layer, C.c_void_p(x_dev), C.c_void_p(y_dev), batch, seq,
                                            C.c_void_p(seq_lens_dev or None)), "sti_layer_forward")


def sti_model_forward(plan: int, x_dev: int, y_dev: int, batch: int, seq: int, seq_lens_dev: int = 0):
    _check(load_library().sti_model_forward(C.c_void_p(plan), C.c_void_p(x_dev), C.c_void_p(y_dev), batch, seq,
                                            C.c_void_p(seq_lens_dev or None)), "sti_model_forward")


def sti_model_forward_host(plan: int, x_host: int, y_host: int, batch: int, seq: int, seq_lens_host: int = 0):
    """x_host / y_host: host addresses (e.g. of pinned torch tensors or numpy arrays)."""
    _check(load_library().sti_model_forward_host(C.c_void_p(plan), C.c_void_p(x_host), C.c_void_p(y_host), batch, seq,
                                                 C.c_void_p(seq_lens_host or None)), "sti_model_forward_host")


def sti_sync(ctx: int):
    _check(load_library().sti_sync(C.c_void_p(ctx)), "sti_sync")


def sti_shard_decode(plan: int, layer: int, kind: int, index: int, matrix: int, w_dev: int = 0, codes_dev: int = 0,
                     wbf16_dev: int = 0):
    _check(load_library().sti_shard_decode(C.c_void_p(plan), layer, kind, index, matrix, C.c_void_p(w_dev or None),
                                           C.c_void_p(codes_dev or None), C.c_void_p(wbf16_dev or None)),
           "sti_shard_decode")


def sti_gemm_probe(plan: int, layer: int, gemm: int, x_bf16_dev: int, tokens: int, out_dev: int,
                   out_capacity_bytes: int, variant: int = 0) -> int:
    """One fused dequant-GEMM of a layer on the caller's activations (see sti.h); returns n_partials."""
    n = C.c_int32(0)
    _check(load_library().sti_gemm_probe(C.c_void_p(plan), layer, gemm, C.c_void_p(x_bf16_dev), tokens,
                                         C.c_void_p(out_dev), out_capacity_bytes, variant, C.byref(n)), "sti_gemm_probe")
    return int(n.value)


def sti_plan_set_profiling(plan: int, level: int):
    """0 = off, 1 = per-layer events, 2 = events around every kernel."""
    _check(load_library().sti_plan_set_profiling(C.c_void_p(plan), int(level)), "sti_plan_set_profiling")


def sti_decode_rate_probe(plan: int, x_bf16_dev: int, tokens: int, out_dev: int, out_capacity_bytes: int):
    """One launch over every layer's FFN1 tiles on few tokens (see sti.h); returns (packed bytes read, tiles)."""
    nb, nt = C.c_uint64(0), C.c_int32(0)
    _check(load_library().sti_decode_rate_probe(C.c_void_p(plan), C.c_void_p(x_bf16_dev), tokens, C.c_void_p(out_dev),
                                                out_capacity_bytes, C.byref(nb), C.byref(nt)), "sti_decode_rate_probe")
    return int(nb.value), int(nt.value)


STI_STAMP_KERNELS, STI_STAMP_WORDS = 8, 8
STAMP_KERNEL_NAMES = ("cast", "qkv", "attention", "o_proj", "layernorm1", "ffn1", "ffn2", "layernorm2")


def sti_get_kernel_stamps(plan: int, n_layers: int) -> np.ndarray:
    """uint64 [n_layers, STI_STAMP_KERNELS, STI_STAMP_WORDS] of the last forward run at profiling level 3 (see sti.h)."""
    out = np.zeros((n_layers, STI_STAMP_KERNELS, STI_STAMP_WORDS), np.uint64)
    n = C.c_int32(0)
    _check(load_library().sti_get_kernel_stamps(C.c_void_p(plan), _ptr(out), out.size, C.byref(n)), "sti_get_kernel_stamps")
    return out[:n.value]


def sti_plan_set_overlap(plan: int, overlap: bool):
    """False: load every streamed layer, then execute (the Load&Exec order); True: the layerwise pipeline."""
    _check(load_library().sti_plan_set_overlap(C.c_void_p(plan), int(bool(overlap))), "sti_plan_set_overlap")


def sti_get_stats(plan: int) -> StiStats:
    st = StiStats()
    _check(load_library().sti_get_stats(C.c_void_p(plan), C.byref(st)), "sti_get_stats")
    return st


def sti_plan_check_guards(plan: int) -> int:
    """Number of damaged guard regions around the preload buffer and the ring slots (0 = intact; see sti.h)."""
    n = C.c_int32(-1)
    _check(load_library().sti_plan_check_guards(C.c_void_p(plan), C.byref(n)), "sti_plan_check_guards")
    return int(n.value)


def sti_plan_memory(plan: int):
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    _check(load_library().sti_plan_memory(C.c_void_p(plan), C.byref(a), C.byref(b), C.byref(c)), "sti_plan_memory")
    return {"preload_bytes": a.value, "pinned_bytes": b.value, "ring_bytes": c.value}


STI_INJECT_NONE, STI_INJECT_SLOW_COPY, STI_INJECT_PINNED_ALLOC_FAILURE = 0, 1, 2


def sti_plan_inject(plan: int, what: int, layer: int = 0, value: int = 0):
    """Host-made faults for tests (see sti.h): a slow shard copy of one layer, a failing pinned allocation."""
    _check(load_library().sti_plan_inject(C.c_void_p(plan), what, layer, value), "sti_plan_inject")


def sti_plan_retain(plan: int, attn_keep, ffn_keep) -> int:
    """Marks kept units (flat, layer-major 0/1 arrays) to stay in device memory after the plan's next run (see sti.h);
    returns the bytes of the retained arena."""
    a, f = _host(attn_keep, np.uint8).reshape(-1), _host(ffn_keep, np.uint8).reshape(-1)
    n = C.c_uint64()
    _check(load_library().sti_plan_retain(C.c_void_p(plan), _ptr(a), _ptr(f), C.byref(n)), "sti_plan_retain")
    return int(n.value)


def sti_shard_adopt(plan: int, from_plan: int, layer: int, kind: int, index: int):
    """Takes a unit over from another plan's device memory instead of uploading it (see sti.h)."""
    _check(load_library().sti_shard_adopt(C.c_void_p(plan), C.c_void_p(from_plan), layer, kind, index), "sti_shard_adopt")


def sti_plan_fill_stats(plan: int):
    a, b, c = C.c_uint64(), C.c_uint64(), C.c_uint64()
    _check(load_library().sti_plan_fill_stats(C.c_void_p(plan), C.byref(a), C.byref(b), C.byref(c)), "sti_plan_fill_stats")
    return {"uploaded_bytes": a.value, "adopted_bytes": b.value, "retained_bytes": c.value}


def sti_ctx_launch_count(ctx: int) -> int:
    return int(load_library().sti_ctx_launch_count(C.c_void_p(ctx)))


def sti_host_retile(src: np.ndarray, rows: int, cols: int, bits: int) -> np.ndarray:
    src = np.ascontiguousarray(src).view(np.uint8).reshape(-1)
    dst = np.empty_like(src)
    _check(load_library().sti_host_retile(_ptr(src), _ptr(dst), rows, cols, bits), "sti_host_retile")
    return dst


def sti_matrix_decode_noalloc(bits: int, rows: int, cols: int, codes: np.ndarray, centroids: np.ndarray,
                              outlier_off: Optional[np.ndarray] = None, outlier_val: Optional[np.ndarray] = None,
                              w_dev: int = 0, codes_dev: int = 0, wbf16_dev: int = 0, device: int = 0, stream: int = 0):
    """Decode one shard matrix without a context, a plan or any allocation (see sti.h for who needs
    that and for the size limits).  codes/centroids/outliers are host arrays, outputs device addresses."""
    codes = _host(codes, np.uint32)
    cent = _host(centroids, np.float32)
    off = _host(outlier_off, np.uint32) if outlier_off is not None and len(outlier_off) else None
    val = _host(outlier_val, np.float32) if outlier_val is not None and len(outlier_val) else None
    _check(load_library().sti_matrix_decode_noalloc(
        device, C.c_void_p(stream or None), int(bits), rows, cols, _ptr(codes), _ptr(cent), _ptr(off), _ptr(val),
        0 if off is None else off.size, C.c_void_p(w_dev or None), C.c_void_p(codes_dev or None),
        C.c_void_p(wbf16_dev or None)), "sti_matrix_decode_noalloc")

class StiPlannerProfile(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_slices", C.c_int32), ("t_comp_us", C.POINTER(C.c_double)),
                ("t_io_us", C.c_double * 6), ("shard_bytes", C.c_uint64 * 6),
                ("importance", C.POINTER(C.c_float))]


class StiPlannerRequest(C.Structure):
    _fields_ = [("target_us", C.c_double), ("preload_bytes", C.c_uint64),
                ("preloaded_bits", C.POINTER(C.c_uint8))]


class StiPlannerResult(C.Structure):
    _fields_ = [("n", C.c_int32), ("m", C.c_int32), ("pass1_bits", C.c_int32), ("valid", C.c_int32),
                ("keep", C.POINTER(C.c_uint8)), ("bits", C.POINTER(C.c_uint8)),
                ("preload", C.POINTER(C.c_uint8)), ("aib_us", C.POINTER(C.c_double))]


def sti_plan_auto(target_us: float, n_layers: int, n_slices: int, t_comp_us, t_io_us, shard_bytes,
                  importance, preload_bytes: int, preloaded_bits=None) -> dict:
    """Two-stage planner (Section 5.3 and 5.4); marshals arrays, returns the result fields as numpy arrays."""
    lib = load_library()
    tc = _host(t_comp_us, np.float64)
    imp = _host(importance, np.float32).reshape(-1)
    if tc.size != n_slices + 1 or imp.size != n_layers * n_slices or len(t_io_us) != 6 or len(shard_bytes) != 6:
        raise ValueError("planner table sizes do not match n_layers / n_slices")
    pf = StiPlannerProfile(n_layers, n_slices, tc.ctypes.data_as(C.POINTER(C.c_double)),
                           (C.c_double * 6)(*[float(v) for v in t_io_us]),
                           (C.c_uint64 * 6)(*[int(v) for v in shard_bytes]),
                           imp.ctypes.data_as(C.POINTER(C.c_float)))
    pre = None if preloaded_bits is None else _host(preloaded_bits, np.uint8).reshape(-1)
    if pre is not None and pre.size != n_layers * n_slices:
        raise ValueError("preloaded_bits must have n_layers * n_slices entries")
    rq = StiPlannerRequest(float(target_us), int(preload_bytes),
                           None if pre is None else pre.ctypes.data_as(C.POINTER(C.c_uint8)))
    keep = np.zeros(n_layers * n_slices, np.uint8)
    bits = np.zeros_like(keep)
    preload = np.zeros_like(keep)
    aib = np.zeros(n_layers, np.float64)
    res = StiPlannerResult(0, 0, 0, 0, keep.ctypes.data_as(C.POINTER(C.c_uint8)),
                           bits.ctypes.data_as(C.POINTER(C.c_uint8)),
                           preload.ctypes.data_as(C.POINTER(C.c_uint8)),
                           aib.ctypes.data_as(C.POINTER(C.c_double)))
    lib.sti_plan_auto.restype = C.c_int
    lib.sti_plan_auto.argtypes = [C.POINTER(StiPlannerProfile), C.POINTER(StiPlannerRequest),
                                  C.POINTER(StiPlannerResult)]
    _check(lib.sti_plan_auto(C.byref(pf), C.byref(rq), C.byref(res)), "sti_plan_auto")
    shape = (n_layers, n_slices)
    return {"n": res.n, "m": res.m, "pass1_bits": res.pass1_bits, "valid": bool(res.valid),
            "keep": keep.reshape(shape), "bits": bits.reshape(shape), "preload": preload.reshape(shape),
            "aib_us": aib}


def sti_preload_after_run(keep, bits, shard_bytes, buffer_bytes: int):
    """Section 3.2 / 5.5: which loaded shards stay cached in a buffer of `buffer_bytes` after a run.
    Returns (preloaded_bits grid for the next sti_plan_auto call, bytes used)."""
    k = _host(keep, np.uint8)
    b = _host(bits, np.uint8)
    if k.ndim != 2 or k.shape != b.shape or len(shard_bytes) != 6:
        raise ValueError("keep and bits must be [n_layers, n_slices] grids; shard_bytes has 6 entries")
    out = np.zeros(k.shape, np.uint8)
    used = C.c_uint64()
    lib = load_library()
    lib.sti_preload_after_run.restype = C.c_int
    lib.sti_preload_after_run.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(C.c_uint64),
                                          C.c_uint64, C.c_void_p, C.POINTER(C.c_uint64)]
    _check(lib.sti_preload_after_run(k.shape[0], k.shape[1], _ptr(k), _ptr(b),
                                     (C.c_uint64 * 6)(*[int(v) for v in shard_bytes]), int(buffer_bytes),
                                     _ptr(out), C.byref(used)), "sti_preload_after_run")
    return out, int(used.value)


def sti_quantize_workspace_bytes(n_units: int, n_weights: int) -> int:
    lib = load_library()
    lib.sti_quantize_workspace_bytes.restype = C.c_size_t
    lib.sti_quantize_workspace_bytes.argtypes = [C.c_uint32, C.c_uint32]
    return int(lib.sti_quantize_workspace_bytes(n_units, n_weights))


def sti_quantize_units(w_dev: int, n_units: int, n_weights: int, bits: int, codes_dev: int, centroids_dev: int,
                       outlier_off_dev: int, outlier_val_dev: int, max_outliers: int, n_outliers_dev: int,
                       workspace_dev: int, workspace_bytes: int, device: int = 0, stream: int = 0):
    """Section 6 quantizer on the device; every buffer is a device address owned by the caller (see sti_quantize.h)."""
    lib = load_library()
    lib.sti_quantize_units.restype = C.c_int
    lib.sti_quantize_units.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_int, C.c_void_p,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p, C.c_size_t]
    _check(lib.sti_quantize_units(device, C.c_void_p(stream or None), C.c_void_p(w_dev), n_units, n_weights, int(bits),
                                  C.c_void_p(codes_dev), C.c_void_p(centroids_dev), C.c_void_p(outlier_off_dev),
                                  C.c_void_p(outlier_val_dev), max_outliers, C.c_void_p(n_outliers_dev),
                                  C.c_void_p(workspace_dev), workspace_bytes), "sti_quantize_units")


STI_QUANTIZE_SELECT, STI_QUANTIZE_SORT = 0, 1


def sti_quantize_units_by(w_dev: int, n_units: int, n_weights: int, bits: int, codes_dev: int, centroids_dev: int,
                          outlier_off_dev: int, outlier_val_dev: int, max_outliers: int, n_outliers_dev: int,
                          workspace_dev: int, workspace_bytes: int, method: int, sorted_units_dev: int = 0,
                          device: int = 0, stream: int = 0):
    """sti_quantize_units with the method named (STI_QUANTIZE_SELECT / STI_QUANTIZE_SORT); sorted_units_dev, when
    not 0, is a device array of n_units bytes that says which units the sort did (see sti_quantize.h)."""
    lib = load_library()
    lib.sti_quantize_units_by.restype = C.c_int
    lib.sti_quantize_units_by.argtypes = [C.c_int, C.c_void_p, C.c_void_p, C.c_uint32, C.c_uint32, C.c_int, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint32, C.c_void_p, C.c_void_p,
                                          C.c_size_t, C.c_int, C.c_void_p]
    _check(lib.sti_quantize_units_by(device, C.c_void_p(stream or None), C.c_void_p(w_dev), n_units, n_weights, int(bits),
                                     C.c_void_p(codes_dev), C.c_void_p(centroids_dev), C.c_void_p(outlier_off_dev),
                                     C.c_void_p(outlier_val_dev), max_outliers, C.c_void_p(n_outliers_dev),
                                     C.c_void_p(workspace_dev), workspace_bytes, int(method),
                                     C.c_void_p(sorted_units_dev or None)), "sti_quantize_units_by")


class Session:
    """Marshals a synthetic workload (any object with the fields of `workloads.Workload`) into a
    context and a plan: set dense parameters, create the plan, upload every kept unit."""

    def __init__(self, work, device: int = 0, compute_stream: int = 0, max_batch: Optional[int] = None,
                 max_seq: Optional[int] = None, ring_slots: Optional[int] = None, finalize: bool = True):
        sh = work.shape
        self.work = work
        self.desc = StiModelDesc(n_layers=sh.n_layers, hidden=sh.hidden, n_heads=sh.n_heads, head_dim=sh.head_dim,
                                 ffn=sh.ffn, n_ffn_slices=sh.n_ffn_slices, max_batch=max_batch or work.batch,
                                 max_seq=max_seq or work.seq,
                                 act_dtype=STI_BF16 if work.act_dtype == "bf16" else STI_F32, ln_eps=work.ln_eps)
        self.ctx = sti_ctx_create(self.desc, device, compute_stream)
        self.plan = 0
        try:
            for l, p in enumerate(work.dense):
                sti_ctx_set_layer_params(self.ctx, l, p["bq"], p["bk"], p["bv"], p["bo"], p["b1"], p["b2"],
                                         p["ln1_g"], p["ln1_b"], p["ln2_g"], p["ln2_b"])
            attn = [(u.keep, u.bits, u.resident) for layer in work.attn_plan for u in layer]
            ffn = [(u.keep, u.bits, u.resident) for layer in work.ffn_plan for u in layer]
            self.plan = sti_plan_create(self.ctx, attn, ffn, ring_slots or work.ring_slots)
            for (l, kind, idx), b in work.blobs.items():
                sti_shard_upload(self.plan, l, kind, idx, b.bits, b.codes, b.centroids, b.outlier_off, b.outlier_val)
            if finalize:
                sti_plan_finalize(self.plan)
        except Exception:
            self.close()
            raise

    def close(self):
        if self.plan:
            sti_plan_destroy(self.plan)
            self.plan = 0
        if self.ctx:
            sti_ctx_destroy(self.ctx)
            self.ctx = 0

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
        return False
