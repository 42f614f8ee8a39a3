"""Thin ctypes binding of librainfusion.so (same names as include/rainfusion.h).

Argument marshalling only: every step of the path runs in the CUDA kernels behind the C ABI.
torch supplies device memory and the current stream.  There is no fallback: if the shared
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

RF_SPATIAL, RF_TEMPORAL, RF_TEXTURAL, RF_DENSE = 0, 1, 2, 3
RF_SAMPLE_ALG1, RF_SAMPLE_GLOBAL = 0, 1
PARTIAL_BIT = 1 << 31

# RAINFUSION_LIBRARY selects another build of the same library (the bounds-checking build, say); there is still no
# fallback of any kind: the named file must exist and export every entry point.
_LIB_PATH = os.environ.get("RAINFUSION_LIBRARY") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "librainfusion.so")
_lib = None

EXPORTS = ["rf_status_string", "rf_schedule_dims", "rf_workspace_bytes", "rf_arm_classify",
           "rf_build_block_mask", "rf_reorder_tokens", "rf_sparse_attn_fwd", "rf_dense_attn_fwd",
           "rf_arm_classify_noalloc", "rf_selftest_wait_timeout", "rf_arm_classify_plus", "rf_build_block_mask_plus", "rf_sparse_attn_fwd_plus",
           "rf_sparse_attn_reordered", "rf_selftest_arm_abandoned", "rf_bounds_checked", "rf_host_pipeline_staging_bytes",
           "rf_host_pipeline_create", "rf_host_pipeline_run", "rf_host_pipeline_status", "rf_host_pipeline_destroy",
           "rf_host_pipeline_set_bandwidths", "rf_host_pipeline_head_class", "rf_host_pipeline_head_window"]


class rf_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("B", "H", "D", "T", "frame_h", "frame_w", "L_text")]


class rf_params(C.Structure):
    _fields_ = [("frame_window", C.c_int32), ("spatial_window", C.c_int32), ("textural_stride", C.c_int32),
                ("sample_mode", C.c_int32), ("sample_stride", C.c_int32), ("alpha", C.c_float),
                ("block_m", C.c_int32), ("block_n", C.c_int32), ("temporal_permute", C.c_int32),
                ("two_mask", C.c_int32), ("spatial_key_first_frame", C.c_int32), ("temporal_window_2d", C.c_int32),
                ("temporal_window_y", C.c_int32), ("temporal_window_x", C.c_int32)]


class rf_schedule(C.Structure):
    _fields_ = [("count", C.c_void_p), ("kv_tile", C.c_void_p), ("bitmap", C.c_void_p), ("kv_len", C.c_void_p),
                ("nQ", C.c_int32), ("nKmax", C.c_int32)]


class RainFusionError(RuntimeError):
    pass


def lib_path() -> str:
    return _LIB_PATH


def load():
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RainFusionError(f"{_LIB_PATH} is missing: build it with `python -m paper_2505_21036_b200.build`")
    lib = C.CDLL(_LIB_PATH)
    P, V, I, Z = C.POINTER, C.c_void_p, C.c_int, C.c_size_t
    lib.rf_host_pipeline_staging_bytes.restype = Z
    lib.rf_host_pipeline_staging_bytes.argtypes = [P(rf_shape), P(rf_params), C.c_int32]
    lib.rf_host_pipeline_create.restype = I
    lib.rf_host_pipeline_create.argtypes = [P(rf_shape), P(rf_params), C.c_int32, V, Z, P(V)]
    lib.rf_host_pipeline_run.restype = I
    lib.rf_host_pipeline_run.argtypes = [V, V, V, V, V, V]
    lib.rf_host_pipeline_status.restype = V
    lib.rf_host_pipeline_status.argtypes = [V]
    lib.rf_host_pipeline_set_bandwidths.restype = I
    lib.rf_host_pipeline_set_bandwidths.argtypes = [V, P(C.c_float), C.c_int32]
    lib.rf_host_pipeline_head_class.restype = V
    lib.rf_host_pipeline_head_class.argtypes = [V]
    lib.rf_host_pipeline_head_window.restype = V
    lib.rf_host_pipeline_head_window.argtypes = [V]
    lib.rf_host_pipeline_destroy.restype = None
    lib.rf_host_pipeline_destroy.argtypes = [V]
    lib.rf_bounds_checked.restype = C.c_int32
    lib.rf_bounds_checked.argtypes = []
    lib.rf_status_string.restype = C.c_char_p
    lib.rf_status_string.argtypes = [I]
    lib.rf_schedule_dims.restype = I
    lib.rf_schedule_dims.argtypes = [P(rf_shape), P(rf_params), P(C.c_int32), P(C.c_int32)]
    lib.rf_workspace_bytes.restype = Z
    lib.rf_workspace_bytes.argtypes = [P(rf_shape), P(rf_params)]
    lib.rf_arm_classify.restype = I
    lib.rf_arm_classify.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, V, Z, V, V]
    lib.rf_arm_classify_noalloc.restype = I
    lib.rf_arm_classify_noalloc.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, V, V]
    lib.rf_build_block_mask.restype = I
    lib.rf_build_block_mask.argtypes = [P(rf_shape), P(rf_params), V, P(rf_schedule), V, V]
    lib.rf_sparse_attn_fwd.restype = I
    lib.rf_sparse_attn_fwd.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, P(rf_schedule), V, V, V, Z, V, V]
    lib.rf_arm_classify_plus.restype = I
    lib.rf_arm_classify_plus.argtypes = [P(rf_shape), P(rf_params), P(C.c_float), C.c_int32, V, V, V, V, V, V, Z, V, V]
    lib.rf_build_block_mask_plus.restype = I
    lib.rf_build_block_mask_plus.argtypes = [P(rf_shape), P(rf_params), V, V, P(rf_schedule), V, V]
    lib.rf_sparse_attn_fwd_plus.restype = I
    lib.rf_sparse_attn_fwd_plus.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, V, P(rf_schedule), V, V, V, Z, V, V]
    lib.rf_sparse_attn_reordered.restype = I
    lib.rf_sparse_attn_reordered.argtypes = lib.rf_sparse_attn_fwd_plus.argtypes
    lib.rf_selftest_arm_abandoned.restype = I
    lib.rf_selftest_arm_abandoned.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, Z, V, V]
    lib.rf_selftest_wait_timeout.restype = I
    lib.rf_selftest_wait_timeout.argtypes = [V, C.c_int32, V, V]
    lib.rf_reorder_tokens.restype = I
    lib.rf_reorder_tokens.argtypes = [P(rf_shape), P(rf_params), V, V, V, V, V, Z, V]
    lib.rf_dense_attn_fwd.restype = I
    lib.rf_dense_attn_fwd.argtypes = [P(rf_shape), V, V, V, V, V, V, Z, V, V]
    _lib = lib
    return lib


def _check(code: int, what: str):
    if code != 0:
        raise RainFusionError(f"{what} failed: {load().rf_status_string(code).decode()} ({code})")


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> Optional[int]:
    import torch
    s = torch.cuda.current_stream().cuda_stream
    return s if s else None


def make_shape(B, H, D, T, frame_h, frame_w, L_text) -> rf_shape:
    return rf_shape(B, H, D, T, frame_h, frame_w, L_text)


def make_params(frame_window, spatial_window, textural_stride=2, sample_mode=RF_SAMPLE_ALG1, sample_stride=1,
                alpha=0.9, block_m=128, block_n=128, temporal_permute=1, two_mask=0, spatial_key_first_frame=0,
                temporal_window_2d=None) -> rf_params:
    """temporal_window_2d: None, or (w_y, w_x) for the 2-D in-frame window of Temporal heads."""
    t2 = (0, 0, 0) if temporal_window_2d is None else (1, int(temporal_window_2d[0]), int(temporal_window_2d[1]))
    return rf_params(frame_window, spatial_window, textural_stride, sample_mode, sample_stride, alpha,
                     block_m, block_n, temporal_permute, two_mask, spatial_key_first_frame, *t2)


def shape_of(wl) -> rf_shape:
    """rf_shape of a synth.Workload."""
    return rf_shape(wl.B, wl.H, wl.D, wl.T, wl.frame_h, wl.frame_w, wl.L_text)


def params_of(wl, block_m=128, block_n=128, temporal_permute=1, two_mask=0, spatial_key_first_frame=0,
              temporal_window_2d=None) -> rf_params:
    """rf_params of a synth.Workload."""
    return rf_params(wl.frame_window, wl.spatial_window, wl.textural_stride, wl.sample_mode, wl.sample_stride,
                     wl.alpha, block_m, block_n, temporal_permute, two_mask, spatial_key_first_frame,
                     *((0, 0, 0) if temporal_window_2d is None else (1, int(temporal_window_2d[0]), int(temporal_window_2d[1]))))


def rf_schedule_dims(shape: rf_shape, params: rf_params):
    nq, nk = C.c_int32(), C.c_int32()
    _check(load().rf_schedule_dims(C.byref(shape), C.byref(params), C.byref(nq), C.byref(nk)), "rf_schedule_dims")
    return nq.value, nk.value


def rf_workspace_bytes(shape: rf_shape, params: rf_params) -> int:
    n = load().rf_workspace_bytes(C.byref(shape), C.byref(params))
    if n == 0:
        raise RainFusionError("rf_workspace_bytes: invalid shape or parameters")
    return n


class Schedule:
    """Device arrays of a tile schedule plus the C struct that points at them."""

    def __init__(self, shape: rf_shape, params: rf_params, device, with_bitmap: bool = False):
        import torch
        self.nQ, self.nKmax = rf_schedule_dims(shape, params)
        BH = shape.B * shape.H
        self.count = torch.zeros((shape.B, shape.H, self.nQ), dtype=torch.int32, device=device)
        self.kv_tile = torch.zeros((shape.B, shape.H, self.nQ, self.nKmax), dtype=torch.int32, device=device)
        self.kv_len = torch.zeros((shape.B, shape.H), dtype=torch.int32, device=device)
        self.bitmap = (torch.zeros((BH, self.nQ, (self.nKmax + 31) // 32), dtype=torch.int32, device=device)
                       if with_bitmap else None)
        self.c = rf_schedule(self.count.data_ptr(), self.kv_tile.data_ptr(), _ptr(self.bitmap),
                             self.kv_len.data_ptr(), self.nQ, self.nKmax)


def alloc_workspace(shape: rf_shape, params: rf_params, device):
    import torch
    return torch.empty(rf_workspace_bytes(shape, params), dtype=torch.uint8, device=device)


def rf_arm_classify(shape, params, q, k, head_class, recall, ws, dev_status=None):
    _check(load().rf_arm_classify(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(), head_class.data_ptr(),
                                  _ptr(recall), ws.data_ptr(), ws.numel(), _ptr(dev_status), _stream()), "rf_arm_classify")


def rf_arm_classify_noalloc(shape, params, q, k, head_class, recall, dev_status=None):
    """rf_arm_classify without a workspace: for callers that may not allocate device memory (a frozen
    serving pool, a plug-in that must not re-enter the framework allocator).  The scratch is a fixed
    4 MiB array inside the library; problems that need more raise RainFusionError.  Calls that overlap
    on the GPU share that array and race; run them one after the other."""
    _check(load().rf_arm_classify_noalloc(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(),
                                          head_class.data_ptr(), _ptr(recall), _ptr(dev_status), _stream()),
           "rf_arm_classify_noalloc")


def rf_build_block_mask(shape, params, head_class, sched: Schedule, dev_status=None):
    _check(load().rf_build_block_mask(C.byref(shape), C.byref(params), head_class.data_ptr(), C.byref(sched.c),
                                      _ptr(dev_status), _stream()), "rf_build_block_mask")


def rf_sparse_attn_fwd(shape, params, q, k, v, head_class, sched: Schedule, o, lse, ws, dev_status=None):
    _check(load().rf_sparse_attn_fwd(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                     head_class.data_ptr(), C.byref(sched.c), o.data_ptr(), _ptr(lse), ws.data_ptr(),
                                     ws.numel(), _ptr(dev_status), _stream()), "rf_sparse_attn_fwd")


def rf_arm_classify_plus(shape, params, bandwidths, q, k, head_class, head_window, recall, ws, dev_status=None):
    arr = (C.c_float * len(bandwidths))(*bandwidths)
    _check(load().rf_arm_classify_plus(C.byref(shape), C.byref(params), arr, len(bandwidths), q.data_ptr(), k.data_ptr(),
                                       head_class.data_ptr(), head_window.data_ptr(), _ptr(recall), ws.data_ptr(),
                                       ws.numel(), _ptr(dev_status), _stream()), "rf_arm_classify_plus")


def rf_build_block_mask_plus(shape, params, head_class, head_window, sched: Schedule, dev_status=None):
    _check(load().rf_build_block_mask_plus(C.byref(shape), C.byref(params), head_class.data_ptr(), _ptr(head_window),
                                           C.byref(sched.c), _ptr(dev_status), _stream()), "rf_build_block_mask_plus")


def rf_sparse_attn_fwd_plus(shape, params, q, k, v, head_class, head_window, sched: Schedule, o, lse, ws, dev_status=None):
    _check(load().rf_sparse_attn_fwd_plus(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                          head_class.data_ptr(), _ptr(head_window), C.byref(sched.c), o.data_ptr(),
                                          _ptr(lse), ws.data_ptr(), ws.numel(), _ptr(dev_status), _stream()),
           "rf_sparse_attn_fwd_plus")


def rf_sparse_attn_reordered(shape, params, q, k, v, head_class, head_window, sched: Schedule, o, lse, ws, dev_status=None):
    _check(load().rf_sparse_attn_reordered(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                           head_class.data_ptr(), _ptr(head_window), C.byref(sched.c), o.data_ptr(),
                                           _ptr(lse), ws.data_ptr(), ws.numel(), _ptr(dev_status), _stream()),
           "rf_sparse_attn_reordered")


def rf_selftest_wait_timeout(dev_status, limit_ms, waits_returned):
    _check(load().rf_selftest_wait_timeout(dev_status.data_ptr(), limit_ms, waits_returned.data_ptr(), _stream()),
           "rf_selftest_wait_timeout")


def rf_selftest_arm_abandoned(shape, params, q, k, head_class, ws, dev_status):
    _check(load().rf_selftest_arm_abandoned(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(),
                                            head_class.data_ptr(), ws.data_ptr(), ws.numel(), _ptr(dev_status), _stream()),
           "rf_selftest_arm_abandoned")


class HostPipeline:
    """rf_host_pipeline_*: the whole path with Q, K, V, O in (pinned) host memory, pipelined over groups of heads.
    torch supplies the staging block; everything else happens behind the C ABI."""

    def __init__(self, shape: rf_shape, params: rf_params, device, head_groups: int):
        import torch
        lib = load()
        n = lib.rf_host_pipeline_staging_bytes(C.byref(shape), C.byref(params), head_groups)
        if n == 0:
            raise RainFusionError("rf_host_pipeline_staging_bytes: invalid shape, parameters or head_groups")
        self.staging = torch.empty(n, dtype=torch.uint8, device=device)
        h = C.c_void_p()
        _check(lib.rf_host_pipeline_create(C.byref(shape), C.byref(params), head_groups, self.staging.data_ptr(), n,
                                           C.byref(h)), "rf_host_pipeline_create")
        self._h = h
        self._status_ptr = lib.rf_host_pipeline_status(h)
        self._heads = shape.B * shape.H

    def set_bandwidths(self, bandwidths):
        """Candidate bandwidths of the dynamic-bandwidth variant (empty: back to the fixed windows)."""
        bw = list(bandwidths)
        arr = (C.c_float * max(len(bw), 1))(*bw)
        _check(load().rf_host_pipeline_set_bandwidths(self._h, arr, len(bw)), "rf_host_pipeline_set_bandwidths")

    def _ints(self, ptr):
        import torch
        torch.cuda.synchronize()
        off = ptr - self.staging.data_ptr()
        return self.staging[off:off + 4 * self._heads].view(torch.int32).cpu().numpy()

    def head_class(self):
        """ARM's classes of the last run, [B*H] (synchronises)."""
        return self._ints(load().rf_host_pipeline_head_class(self._h))

    def head_window(self):
        """The per-head windows of the last run with bandwidths set, [B*H] (synchronises)."""
        return self._ints(load().rf_host_pipeline_head_window(self._h))

    def run(self, qh, kh, vh, oh):
        _check(load().rf_host_pipeline_run(self._h, qh.data_ptr(), kh.data_ptr(), vh.data_ptr(), oh.data_ptr(), _stream()),
               "rf_host_pipeline_run")

    def status(self) -> int:
        """The device status word, read back (synchronises)."""
        import torch
        torch.cuda.synchronize()
        off = self._status_ptr - self.staging.data_ptr()
        return int(self.staging[off:off + 4].view(torch.int32).item())

    def close(self):
        if self._h is not None:
            load().rf_host_pipeline_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def rf_reorder_tokens(shape, params, q, k, v, head_class, ws):
    _check(load().rf_reorder_tokens(C.byref(shape), C.byref(params), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                    head_class.data_ptr(), ws.data_ptr(), ws.numel(), _stream()), "rf_reorder_tokens")


def rf_dense_attn_fwd(shape, q, k, v, o, lse, dev_status=None):
    _check(load().rf_dense_attn_fwd(C.byref(shape), q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), _ptr(lse),
                                    None, 0, _ptr(dev_status), _stream()), "rf_dense_attn_fwd")
