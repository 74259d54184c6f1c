"""ctypes binding of libsidco.so: argument marshalling only.

Every function has the name and the meaning of the C entry point declared in
``include/sidco.h``; tensors are passed as raw device (or host) pointers and
nothing is computed here.  Loading fails loudly if the library has not been
built (``python -m paper_2101_10761_b200.build``): there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
# SIDCO_LIB_VARIANT=profile|check selects a build of the same sources with device timestamps or with
# device-side bounds checks (see build.py); the default is the product library.
_VARIANT = os.environ.get("SIDCO_LIB_VARIANT", "")
LIB_PATH = os.path.join(_HERE, "libsidco%s.so" % ("_" + _VARIANT if _VARIANT else ""))

SID_EXP, SID_GAMMA, SID_GPD = 0, 1, 2
MAX_STAGES = 8

ST_NONFINITE, ST_DEGENERATE, ST_ALL_ZERO, ST_TIMEOUT, ST_BOUNDS = 1, 2, 4, 8, 16
BUILD_PROFILE, BUILD_BOUNDS_CHECK = 1, 2


class SegDebug(C.Structure):
    _fields_ = [
        ("M_used", C.c_int32),
        ("M_next", C.c_int32),
        ("status", C.c_int32),
        ("calls", C.c_int32),
        ("k_sum", C.c_int64),
        ("eta", C.c_double * MAX_STAGES),
        ("k_stage", C.c_int32 * MAX_STAGES),
    ]


EXPORTS = [
    "sidco_compress", "sidco_compress_host", "sidco_workspace_bytes", "sidco_set_workspace",
    "sidco_set_params", "sidco_reset_state", "sidco_get_debug", "sidco_state_save", "sidco_state_load",
    "sidco_release", "sidco_release_all", "sidco_launch_count", "sidco_error_string", "sidco_version",
    "sidco_get_phase_times", "sidco_get_cta_sweep_times", "sidco_compress_static",
    "sidco_reset_state_async", "sidco_set_test_hooks", "sidco_build_flags", "sidco_aggregate", "sidco_compress_bf16", "sidco_get_cta_selection_info",
    "sidco_reference_workspace_bytes", "sidco_topk", "sidco_dgc", "sidco_set_policy",
]

_lib = None


class SidcoError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().sidco_error_string(code).decode()
        super().__init__(f"{where} failed with code {code}: {msg}")


def lib() -> C.CDLL:
    """Load libsidco.so once.  Raises if it is missing: the CUDA path is the only path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} not found: build it with `python -m paper_2101_10761_b200.build` "
            "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, f32, i64, dbl = C.c_void_p, C.c_int, C.c_float, C.c_int64, C.c_double
    compress_sig = [vp, vp, C.POINTER(i64), i32, f32, i32, i32, vp, vp, vp, vp]
    L.sidco_compress.argtypes = compress_sig
    L.sidco_compress.restype = i32
    L.sidco_compress_host.argtypes = compress_sig
    L.sidco_compress_host.restype = i32
    L.sidco_compress_static.argtypes = compress_sig
    L.sidco_compress_static.restype = i32
    L.sidco_compress_bf16.argtypes = compress_sig
    L.sidco_compress_bf16.restype = i32
    L.sidco_workspace_bytes.argtypes = [i64, i32]
    L.sidco_workspace_bytes.restype = C.c_size_t
    L.sidco_set_workspace.argtypes = [vp, vp, C.c_size_t]
    L.sidco_set_workspace.restype = i32
    L.sidco_set_params.argtypes = [dbl, dbl, dbl, i32]
    L.sidco_set_params.restype = i32
    L.sidco_reset_state.argtypes = [vp]
    L.sidco_reset_state.restype = i32
    L.sidco_reset_state_async.argtypes = [vp, vp]
    L.sidco_reset_state_async.restype = i32
    L.sidco_get_debug.argtypes = [vp, C.POINTER(SegDebug), i32]
    L.sidco_get_debug.restype = i32
    L.sidco_get_phase_times.argtypes = [vp, C.POINTER(dbl)]
    L.sidco_get_phase_times.restype = i32
    L.sidco_get_cta_sweep_times.argtypes = [vp, C.POINTER(dbl), i32]
    L.sidco_get_cta_sweep_times.restype = i32
    L.sidco_state_save.argtypes = [vp, C.POINTER(i64), i32]
    L.sidco_state_save.restype = i32
    L.sidco_state_load.argtypes = [vp, C.POINTER(i64), i32]
    L.sidco_state_load.restype = i32
    L.sidco_release.argtypes = [vp]
    L.sidco_release.restype = i32
    L.sidco_release_all.argtypes = []
    L.sidco_release_all.restype = i32
    L.sidco_launch_count.argtypes = []
    L.sidco_launch_count.restype = i64
    L.sidco_error_string.argtypes = [i32]
    L.sidco_error_string.restype = C.c_char_p
    L.sidco_version.argtypes = []
    L.sidco_version.restype = i32
    L.sidco_set_test_hooks.argtypes = [i32, i32, C.c_longlong, i32]
    L.sidco_set_test_hooks.restype = i32
    L.sidco_build_flags.argtypes = []
    L.sidco_build_flags.restype = i32
    L.sidco_get_cta_selection_info.argtypes = [vp, C.POINTER(C.c_int32), i32]
    L.sidco_get_cta_selection_info.restype = i32
    L.sidco_reference_workspace_bytes.argtypes = [i64, i64]
    L.sidco_reference_workspace_bytes.restype = C.c_size_t
    L.sidco_topk.argtypes = [vp, vp, i64, i64, vp, vp, vp, vp, C.c_size_t, vp]
    L.sidco_topk.restype = i32
    L.sidco_dgc.argtypes = [vp, vp, i64, f32, vp, i64, vp, vp, vp, vp, C.c_size_t, vp]
    L.sidco_dgc.restype = i32
    L.sidco_set_policy.argtypes = [i32, i32, i32]
    L.sidco_set_policy.restype = i32
    L.sidco_aggregate.argtypes = [vp, vp, vp, i32, i64, i64, vp, vp, vp]
    L.sidco_aggregate.restype = i32
    _lib = L
    return L


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor, a numpy array or an int; None stays NULL."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    return x.data_ptr()


def _offsets(seg_offsets: Sequence[int]):
    arr = np.ascontiguousarray(np.asarray(seg_offsets, dtype=np.int64))
    return arr, arr.ctypes.data_as(C.POINTER(C.c_int64)), int(arr.size - 1)


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def sidco_compress(grad, residual, seg_offsets, delta: float, sid_type: int, max_stages: int,
                   out_idx, out_val, out_k, stream=None) -> None:
    """Device buffers (torch CUDA tensors or raw addresses); enqueues on `stream`
    (default: torch's current stream) and returns without synchronising."""
    arr, p, n = _offsets(seg_offsets)
    rc = lib().sidco_compress(_ptr(grad), _ptr(residual), p, n, delta, sid_type, max_stages,
                              _ptr(out_idx), _ptr(out_val), _ptr(out_k), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_compress")


def sidco_compress_bf16(grad_bf16, residual, seg_offsets, delta: float, sid_type: int, max_stages: int,
                        out_idx, out_val, out_k, stream=None) -> None:
    """sidco_compress with a bf16 gradient (torch.bfloat16 tensor, or uint16 bit patterns); fp32 residual."""
    arr, p, n = _offsets(seg_offsets)
    rc = lib().sidco_compress_bf16(_ptr(grad_bf16), _ptr(residual), p, n, delta, sid_type, max_stages,
                                   _ptr(out_idx), _ptr(out_val), _ptr(out_k), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_compress_bf16")


def sidco_compress_host(grad, residual, seg_offsets, delta: float, sid_type: int, max_stages: int,
                        out_idx, out_val, out_k, stream=None) -> None:
    """Host buffers (numpy arrays or pinned torch CPU tensors); copies in, compresses,
    copies back and synchronises."""
    arr, p, n = _offsets(seg_offsets)
    rc = lib().sidco_compress_host(_ptr(grad), _ptr(residual), p, n, delta, sid_type, max_stages,
                                   _ptr(out_idx), _ptr(out_val), _ptr(out_k), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_compress_host")


def sidco_workspace_bytes(d: int, n_segs: int) -> int:
    return int(lib().sidco_workspace_bytes(d, n_segs))


def sidco_set_workspace(residual, device_ptr, nbytes: int) -> None:
    rc = lib().sidco_set_workspace(_ptr(residual), _ptr(device_ptr), nbytes)
    if rc:
        raise SidcoError(rc, "sidco_set_workspace")


def sidco_set_params(delta1: float = 0.25, eps_H: float = 0.2, eps_L: float = 0.2, Q: int = 5) -> None:
    rc = lib().sidco_set_params(delta1, eps_H, eps_L, Q)
    if rc:
        raise SidcoError(rc, "sidco_set_params")


def sidco_set_policy(gamma_exact: bool = False, ratio_from_counts: bool = False, adapt_reversed: bool = False) -> None:
    """Variants the paper describes and replaces (see sidco.h); the defaults restore the method as evaluated."""
    rc = lib().sidco_set_policy(int(gamma_exact), int(ratio_from_counts), int(adapt_reversed))
    if rc:
        raise SidcoError(rc, "sidco_set_policy")


def sidco_reset_state(residual) -> None:
    rc = lib().sidco_reset_state(_ptr(residual))
    if rc:
        raise SidcoError(rc, "sidco_reset_state")


def sidco_get_debug(residual, n_segs: int):
    buf = (SegDebug * n_segs)()
    rc = lib().sidco_get_debug(_ptr(residual), buf, n_segs)
    if rc:
        raise SidcoError(rc, "sidco_get_debug")
    return list(buf)


def sidco_state_save(residual, n_segs: int) -> np.ndarray:
    blob = np.zeros(3 * n_segs, dtype=np.int64)
    rc = lib().sidco_state_save(_ptr(residual), blob.ctypes.data_as(C.POINTER(C.c_int64)), n_segs)
    if rc:
        raise SidcoError(rc, "sidco_state_save")
    return blob


def sidco_state_load(residual, blob: np.ndarray) -> None:
    blob = np.ascontiguousarray(blob, dtype=np.int64)
    rc = lib().sidco_state_load(_ptr(residual), blob.ctypes.data_as(C.POINTER(C.c_int64)), blob.size // 3)
    if rc:
        raise SidcoError(rc, "sidco_state_load")


def sidco_release(residual) -> None:
    rc = lib().sidco_release(_ptr(residual))
    if rc:
        raise SidcoError(rc, "sidco_release")


def sidco_release_all() -> None:
    lib().sidco_release_all()


def sidco_launch_count() -> int:
    return int(lib().sidco_launch_count())


def sidco_version() -> int:
    return int(lib().sidco_version())


AGG_MAX_WORKERS = 64
AGG_ST_COUNT, AGG_ST_ORDER = 1, 2


def sidco_aggregate(idx_all, val_all, counts, n_workers: int, stride: int, d: int, out_dense, status=None,
                    stream=None) -> None:
    """Dense mean of n_workers gathered sparse lists (device buffers; see sidco.h)."""
    rc = lib().sidco_aggregate(_ptr(idx_all), _ptr(val_all), _ptr(counts), n_workers, stride, d,
                               _ptr(out_dense), _ptr(status), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_aggregate")


def sidco_reference_workspace_bytes(d: int, n_sample: int = 0) -> int:
    return int(lib().sidco_reference_workspace_bytes(d, n_sample))


def sidco_topk(grad, residual, d: int, k: int, out_idx, out_val, out_k, workspace, workspace_bytes: int,
               stream=None) -> None:
    """Exact Top-k reference point (device buffers; see sidco.h)."""
    rc = lib().sidco_topk(_ptr(grad), _ptr(residual), d, k, _ptr(out_idx), _ptr(out_val), _ptr(out_k),
                          _ptr(workspace), workspace_bytes, _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_topk")


def sidco_dgc(grad, residual, d: int, delta: float, sample_idx, n_sample: int, out_idx, out_val, out_k,
              workspace, workspace_bytes: int, stream=None) -> None:
    """Sampled-threshold reference point (device buffers; see sidco.h)."""
    rc = lib().sidco_dgc(_ptr(grad), _ptr(residual), d, delta, _ptr(sample_idx), n_sample, _ptr(out_idx),
                         _ptr(out_val), _ptr(out_k), _ptr(workspace), workspace_bytes, _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_dgc")


def sidco_set_test_hooks(grid: int = 0, spec_enable: int = 1, spin_limit: int = 0,
                         drop_publication_seg: int = -1) -> None:
    """Test switches (see sidco.h); the defaults restore normal operation."""
    rc = lib().sidco_set_test_hooks(grid, spec_enable, spin_limit, drop_publication_seg)
    if rc:
        raise SidcoError(rc, "sidco_set_test_hooks")


def sidco_build_flags() -> int:
    return int(lib().sidco_build_flags())


def sidco_error_string(code: int) -> str:
    return lib().sidco_error_string(code).decode()


def sidco_get_phase_times(residual):
    """Microseconds of the last call: [P1, stage 2, stages 3..M, staging, placement, total] followed by
    six finer marks of CTA 0 (see sidco.h)."""
    buf = (C.c_double * 12)()
    rc = lib().sidco_get_phase_times(_ptr(residual), buf)
    if rc:
        raise SidcoError(rc, "sidco_get_phase_times")
    return list(buf)


def sidco_get_cta_sweep_times(residual, max_ctas: int = 1024) -> np.ndarray:
    """(n_ctas, 4) array: microseconds after kernel start at which each CTA finished its sweeps."""
    buf = (C.c_double * (4 * max_ctas))()
    rc = lib().sidco_get_cta_sweep_times(_ptr(residual), buf, max_ctas)
    if rc < 0:
        raise SidcoError(rc, "sidco_get_cta_sweep_times")
    return np.ctypeslib.as_array(buf)[: 4 * rc].reshape(rc, 4).copy()


def sidco_get_cta_selection_info(residual, max_ctas: int = 1024) -> np.ndarray:
    """(n_ctas, 8) int array, profile builds only: see sidco.h."""
    buf = (C.c_int32 * (8 * max_ctas))()
    rc = lib().sidco_get_cta_selection_info(_ptr(residual), buf, max_ctas)
    if rc < 0:
        raise SidcoError(rc, "sidco_get_cta_selection_info")
    return np.ctypeslib.as_array(buf)[: 8 * rc].reshape(rc, 8).copy()


STATIC_MAX_ELEMS = 1048576
STATIC_MAX_SEGS = 256


def sidco_compress_static(grad, residual, seg_offsets, delta: float, sid_type: int, max_stages: int,
                          out_idx, out_val, out_k, stream=None) -> None:
    """sidco_compress without any device allocation: the workspace is a fixed 18 MiB array inside the
    library, one per GPU, shared by all calls (do not overlap calls on one GPU).  For callers that
    cannot call cudaMalloc, e.g. under stream capture or inside a pool-managed allocator.  Limits:
    STATIC_MAX_ELEMS elements, STATIC_MAX_SEGS segments."""
    arr, p, n = _offsets(seg_offsets)
    rc = lib().sidco_compress_static(_ptr(grad), _ptr(residual), p, n, delta, sid_type, max_stages,
                                     _ptr(out_idx), _ptr(out_val), _ptr(out_k), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_compress_static")


def sidco_reset_state_async(residual, stream=None) -> None:
    """Reset the stage adaptation of `residual` on `stream` without synchronising."""
    rc = lib().sidco_reset_state_async(_ptr(residual), _stream(stream))
    if rc:
        raise SidcoError(rc, "sidco_reset_state_async")
