"""ctypes binding of libexcp.so (include/excp.h).  Argument marshalling only:
every step of compression and decompression runs in the library's CUDA kernels.
PyTorch supplies device memory and the stream.  There is no CPU fallback: if
the library cannot be loaded the import of this module's handle fails loudly."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

from . import build as _build

MEDIAN_ABS_WEIGHT = 0
MEDIAN_ABS_RESIDUAL = 1

STATUS = {0: "OK", -1: "INVALID_ARG", -2: "UNSUPPORTED", -3: "BUFFER_TOO_SMALL", -4: "CUDA",
          -5: "CORRUPT_BLOB", -6: "NONFINITE_INPUT", -7: "TIMEOUT"}

EXPORTS = ["excp_create", "excp_destroy", "excp_record_bytes", "excp_compress_bound",
           "excp_status_string", "excp_last_cuda_error", "excp_compress_tensor",
           "excp_compress_checkpoint", "excp_compress_checkpoint_indexed", "excp_compress_checkpoint_w16", "excp_decompress_checkpoint_w16",
           "excp_compress_checkpoint_host", "excp_decompress_tensor", "excp_decompress_checkpoint",
           "excp_decompress_tensor_noalloc", "excp_dense_bytes", "excp_record_to_dense", "excp_checkpoint_to_dense",
           "excp_decompress_dense_tensor", "excp_decompress_dense_checkpoint", "excp_profile_enable", "excp_profile_stage_count", "excp_profile_stage_name", "excp_profile_read",
           "excp_set_kmeans_margin", "excp_set_wait_limit", "excp_selftest_wait_timeout", "excp_set_report_sse"]


class ExcpError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: EXCP_ERR_{STATUS.get(status, status)}")
        self.status = status


class CParams(C.Structure):
    _fields_ = [("alpha", C.c_float), ("beta", C.c_float), ("bits", C.c_int), ("kmeans_iters", C.c_int),
                ("seed", C.c_ulonglong), ("median_source", C.c_int), ("flags", C.c_uint)]


class CStats(C.Structure):
    _fields_ = [("numel", C.c_ulonglong), ("nnz_w", C.c_ulonglong), ("nnz_o", C.c_ulonglong),
                ("blob_bytes", C.c_ulonglong), ("median", C.c_float), ("mean_abs_ea", C.c_float),
                ("thr_w", C.c_float), ("thr_o", C.c_float),
                ("sse_w", C.c_double), ("sse_ea", C.c_double), ("sse_eas", C.c_double)]


FLAG_NO_W2M, FLAG_NO_M2W, FLAG_NO_RESIDUAL, FLAG_NO_PRUNE, FLAG_NO_QUANT = 1, 2, 4, 8, 16


@dataclass
class Params:
    alpha: float = 5e-5
    beta: float = 2.0
    bits: int = 4
    kmeans_iters: int = 10
    seed: int = 0
    median_source: int = MEDIAN_ABS_WEIGHT
    flags: int = 0          # FLAG_NO_*: the ablation switches; 0 = the full method

    def to_c(self) -> CParams:
        return CParams(self.alpha, self.beta, self.bits, self.kmeans_iters, self.seed, self.median_source,
                       self.flags)


_lib = None


def load_library() -> C.CDLL:
    """Loads (building first if the sources are newer) libexcp.so and declares the prototypes."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    lib = C.CDLL(path)
    vp, sz = C.c_void_p, C.c_size_t
    lib.excp_create.argtypes = [C.POINTER(vp), C.c_int, sz]
    lib.excp_destroy.argtypes = [vp]
    lib.excp_record_bytes.argtypes = [sz, sz, sz, C.c_int]
    lib.excp_record_bytes.restype = sz
    lib.excp_compress_bound.argtypes = [sz, C.c_int]
    lib.excp_compress_bound.restype = sz
    lib.excp_status_string.argtypes = [C.c_int]
    lib.excp_status_string.restype = C.c_char_p
    lib.excp_last_cuda_error.argtypes = [vp, C.POINTER(C.c_int)]
    lib.excp_compress_tensor.argtypes = [vp, C.POINTER(CParams), vp, vp, vp, vp, sz, vp, sz,
                                         C.POINTER(sz), C.POINTER(CStats), vp]
    lib.excp_compress_checkpoint.argtypes = [vp, C.POINTER(CParams), sz, C.POINTER(vp), C.POINTER(vp),
                                             C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), vp, sz,
                                             C.POINTER(sz), C.POINTER(CStats), vp]
    lib.excp_compress_checkpoint_host.argtypes = lib.excp_compress_checkpoint.argtypes
    lib.excp_compress_checkpoint_indexed.argtypes = [vp, C.POINTER(CParams), sz, C.POINTER(vp), C.POINTER(vp),
                                                     C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), C.POINTER(sz), vp, sz,
                                                     C.POINTER(sz), C.POINTER(CStats), vp]
    lib.excp_compress_checkpoint_w16.argtypes = [vp, C.POINTER(CParams), sz, C.POINTER(vp), C.POINTER(vp),
                                                 C.POINTER(vp), C.POINTER(vp), C.POINTER(sz), C.c_int, vp, sz,
                                                 C.POINTER(sz), C.POINTER(CStats), vp]
    lib.excp_decompress_checkpoint_w16.argtypes = [vp, vp, C.POINTER(sz), sz, C.POINTER(vp), C.POINTER(sz), C.c_int,
                                                   C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp]
    lib.excp_decompress_tensor.argtypes = [vp, vp, sz, vp, sz, vp, vp, vp, vp]
    lib.excp_decompress_checkpoint.argtypes = [vp, vp, C.POINTER(sz), sz, C.POINTER(vp), C.POINTER(sz),
                                               C.POINTER(vp), C.POINTER(vp), C.POINTER(vp), vp]
    lib.excp_decompress_tensor_noalloc.argtypes = [vp, sz, vp, sz, vp, vp, vp, vp]
    lib.excp_dense_bytes.argtypes = [sz, C.c_int]
    lib.excp_dense_bytes.restype = sz
    lib.excp_record_to_dense.argtypes = [vp, vp, sz, sz, vp, sz, C.POINTER(sz), vp]
    lib.excp_checkpoint_to_dense.argtypes = [vp, vp, C.POINTER(sz), sz, C.POINTER(sz), vp, sz, C.POINTER(sz), vp]
    lib.excp_decompress_dense_tensor.argtypes = lib.excp_decompress_tensor.argtypes
    lib.excp_decompress_dense_checkpoint.argtypes = lib.excp_decompress_checkpoint.argtypes
    lib.excp_profile_enable.argtypes = [vp, C.c_int]
    lib.excp_set_kmeans_margin.argtypes = [vp, C.c_int]
    lib.excp_set_wait_limit.argtypes = [vp, C.c_ulonglong]
    lib.excp_set_report_sse.argtypes = [vp, C.c_int]
    lib.excp_selftest_wait_timeout.argtypes = [vp, C.c_ulonglong, vp]
    lib.excp_profile_stage_count.argtypes = []
    lib.excp_profile_stage_name.argtypes = [C.c_int]
    lib.excp_profile_stage_name.restype = C.c_char_p
    lib.excp_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_ulonglong)]
    for name in EXPORTS:
        if getattr(lib, name).restype is C.c_int:
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(t: torch.Tensor | None) -> int:
    return 0 if t is None or t.numel() == 0 else t.data_ptr()


def _check_f32_cuda(*ts: torch.Tensor) -> None:
    for t in ts:
        if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()):
            raise TypeError("expected contiguous float32 CUDA tensors")


WEIGHTS_F32, WEIGHTS_F16, WEIGHTS_BF16 = 0, 1, 2
_WEIGHT_DTYPE = {WEIGHTS_F32: torch.float32, WEIGHTS_F16: torch.float16, WEIGHTS_BF16: torch.bfloat16}


def _check_weights(weight_format: int, *ts: torch.Tensor) -> None:
    for t in ts:
        if not (t.is_cuda and t.dtype == _WEIGHT_DTYPE[weight_format] and t.is_contiguous()):
            raise TypeError(f"expected contiguous {_WEIGHT_DTYPE[weight_format]} CUDA tensors")


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def record_bytes(numel: int, nnz_w: int, nnz_o: int, bits: int = 4) -> int:
    return load_library().excp_record_bytes(numel, nnz_w, nnz_o, bits)


def dense_bytes(numel: int, bits: int = 4) -> int:
    return load_library().excp_dense_bytes(numel, bits)


def compress_bound(numel: int, bits: int = 4) -> int:
    return load_library().excp_compress_bound(numel, bits)


NOALLOC_MAX_NUMEL = 1 << 24


def decompress_tensor_noalloc(blob: torch.Tensor, blob_bytes: int, w_prev, w_out, ea_out, eas_out) -> None:
    """excp_decompress_tensor_noalloc: decode one record on the current device without a handle
    and without any allocation by the library (for restore paths that cannot allocate: the
    device is fully reserved by the framework's allocator, or cudaMalloc's device-wide
    synchronisation is not acceptable).  Tensors of more than NOALLOC_MAX_NUMEL elements are
    refused; calls must not overlap on the GPU."""
    _check_f32_cuda(w_prev, w_out, ea_out, eas_out)
    st = load_library().excp_decompress_tensor_noalloc(blob.data_ptr(), blob_bytes, _ptr(w_prev), w_prev.numel(),
                                                       _ptr(w_out), _ptr(ea_out), _ptr(eas_out), _stream())
    if st != 0:
        raise ExcpError(st, "excp_decompress_tensor_noalloc")


class Handle:
    """Owns the library's scratch workspace on one device (excp_create / excp_destroy)."""

    def __init__(self, workspace_numel: int, device: int | None = None):
        self.lib = load_library()
        self.device = torch.cuda.current_device() if device is None else device
        self._h = C.c_void_p()
        st = self.lib.excp_create(C.byref(self._h), self.device, workspace_numel)
        if st != 0:
            raise ExcpError(st, "excp_create")

    def close(self) -> None:
        if self._h:
            self.lib.excp_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def last_cuda_error(self) -> int:
        e = C.c_int(0)
        self.lib.excp_last_cuda_error(self._h, C.byref(e))
        return e.value

    def set_kmeans_margin(self, margin: int) -> None:
        """excp_set_kmeans_margin: a tuning knob; the centres do not depend on it."""
        st = self.lib.excp_set_kmeans_margin(self._h, int(margin))
        if st != 0:
            raise ExcpError(st, "excp_set_kmeans_margin")

    def set_report_sse(self, on: bool = True) -> None:
        """excp_set_report_sse: fill sse_w, sse_ea, sse_eas of the statistics (off by default)."""
        st = self.lib.excp_set_report_sse(self._h, int(on))
        if st != 0:
            raise ExcpError(st, "excp_set_report_sse")

    def set_wait_limit(self, nanoseconds: int) -> None:
        """excp_set_wait_limit: how long a warp waits for an asynchronous copy before the call gives up."""
        st = self.lib.excp_set_wait_limit(self._h, int(nanoseconds))
        if st != 0:
            raise ExcpError(st, "excp_set_wait_limit")

    def selftest_wait_timeout(self, nanoseconds: int) -> int:
        """excp_selftest_wait_timeout: returns the status (EXCP_ERR_TIMEOUT = -7 is the expected one)."""
        return self.lib.excp_selftest_wait_timeout(self._h, int(nanoseconds), _stream())

    def profile_enable(self, on: bool = True) -> None:
        st = self.lib.excp_profile_enable(self._h, int(on))
        if st != 0:
            raise ExcpError(st, "excp_profile_enable")

    def profile_read(self):
        """(dict stage name -> ms of the last call, kernel launches of the last call)."""
        n = self.lib.excp_profile_stage_count()
        ms = (C.c_double * n)()
        launches = C.c_ulonglong(0)
        self.lib.excp_profile_read(self._h, ms, C.byref(launches))
        return {self.lib.excp_profile_stage_name(i).decode(): ms[i] for i in range(n)}, launches.value

    # ---- Algorithm 1 -----------------------------------------------------
    def compress_tensor(self, p: Params, w_t, w_prev, ea, eas, blob_out: torch.Tensor):
        """excp_compress_tensor.  Returns (record bytes, stats)."""
        _check_f32_cuda(w_t, w_prev, ea, eas)
        cp, nbytes, stats = p.to_c(), C.c_size_t(0), CStats()
        st = self.lib.excp_compress_tensor(self._h, C.byref(cp), _ptr(w_t), _ptr(w_prev), _ptr(ea), _ptr(eas),
                                           w_t.numel(), blob_out.data_ptr(), blob_out.numel() * blob_out.element_size(),
                                           C.byref(nbytes), C.byref(stats), _stream())
        if st != 0:
            raise ExcpError(st, "excp_compress_tensor")
        return nbytes.value, stats

    def compress_checkpoint(self, p: Params, tensors, blob_out: torch.Tensor, want_stats: bool = True,
                            weight_format: int = WEIGHTS_F32, tensor_indices=None):
        """excp_compress_checkpoint (or, for 16-bit weights, excp_compress_checkpoint_w16) over a list of
        (w_t, w_prev, ea, eas).  Returns (offsets list of len n+1, list of stats or None).  With
        `tensor_indices` (the tensors' places in the whole checkpoint, for a rank that compresses a share of
        it) the call is excp_compress_checkpoint_indexed."""
        n = len(tensors)
        for q in tensors:
            _check_weights(weight_format, q[0], q[1])
            _check_f32_cuda(q[2], q[3])
        arr = lambda k: (C.c_void_p * n)(*[_ptr(q[k]) for q in tensors])
        numel = (C.c_size_t * n)(*[q[0].numel() for q in tensors])
        offs = (C.c_size_t * (n + 1))()
        stats = (CStats * n)() if want_stats else None
        cp = p.to_c()
        cap = blob_out.numel() * blob_out.element_size()
        if tensor_indices is not None:
            if weight_format != WEIGHTS_F32 or len(tensor_indices) != n:
                raise ValueError("tensor_indices: one per tensor, fp32 weights only")
            idx = (C.c_size_t * n)(*[int(i) for i in tensor_indices])
            st = self.lib.excp_compress_checkpoint_indexed(self._h, C.byref(cp), n, arr(0), arr(1), arr(2), arr(3), numel, idx,
                                                           blob_out.data_ptr(), cap, offs, stats, _stream())
        elif weight_format == WEIGHTS_F32:
            st = self.lib.excp_compress_checkpoint(self._h, C.byref(cp), n, arr(0), arr(1), arr(2), arr(3), numel,
                                                   blob_out.data_ptr(), cap, offs, stats, _stream())
        else:
            st = self.lib.excp_compress_checkpoint_w16(self._h, C.byref(cp), n, arr(0), arr(1), arr(2), arr(3), numel,
                                                       weight_format, blob_out.data_ptr(), cap, offs, stats, _stream())
        if st != 0:
            raise ExcpError(st, "excp_compress_checkpoint" + ("" if weight_format == WEIGHTS_F32 else "_w16"))
        return list(offs), (list(stats) if want_stats else None)

    def compress_checkpoint_host(self, p: Params, tensors, blob_out: torch.Tensor, want_stats: bool = True):
        """excp_compress_checkpoint_host: `tensors` and `blob_out` are HOST tensors
        (page-locked for the copies to overlap the kernels)."""
        n = len(tensors)
        for q in tensors:
            for t in q:
                if t.is_cuda or t.dtype != torch.float32 or not t.is_contiguous():
                    raise TypeError("expected contiguous float32 host tensors")
        if blob_out.is_cuda:
            raise TypeError("blob_out must be a host tensor")
        arr = lambda k: (C.c_void_p * n)(*[_ptr(q[k]) for q in tensors])
        numel = (C.c_size_t * n)(*[q[0].numel() for q in tensors])
        offs = (C.c_size_t * (n + 1))()
        stats = (CStats * n)() if want_stats else None
        cp = p.to_c()
        st = self.lib.excp_compress_checkpoint_host(self._h, C.byref(cp), n, arr(0), arr(1), arr(2), arr(3), numel,
                                                    blob_out.data_ptr(), blob_out.numel() * blob_out.element_size(),
                                                    offs, stats, _stream())
        if st != 0:
            raise ExcpError(st, "excp_compress_checkpoint_host")
        return list(offs), (list(stats) if want_stats else None)

    # ---- Algorithm 2 -----------------------------------------------------
    def decompress_tensor(self, blob: torch.Tensor, blob_bytes: int, w_prev, w_out, ea_out, eas_out) -> None:
        _check_f32_cuda(w_prev, w_out, ea_out, eas_out)
        st = self.lib.excp_decompress_tensor(self._h, blob.data_ptr(), blob_bytes, _ptr(w_prev), w_prev.numel(),
                                             _ptr(w_out), _ptr(ea_out), _ptr(eas_out), _stream())
        if st != 0:
            raise ExcpError(st, "excp_decompress_tensor")

    def decompress_checkpoint(self, blob: torch.Tensor, offsets, w_prev, w_out, ea_out, eas_out,
                              dense: bool = False, weight_format: int = WEIGHTS_F32) -> None:
        n = len(w_prev)
        _check_weights(weight_format, *w_prev, *w_out)
        _check_f32_cuda(*ea_out, *eas_out)
        arr = lambda ts: (C.c_void_p * n)(*[_ptr(t) for t in ts])
        numel = (C.c_size_t * n)(*[t.numel() for t in w_prev])
        offs = (C.c_size_t * (n + 1))(*offsets)
        if weight_format != WEIGHTS_F32:
            if dense:
                raise ValueError("the dense layout decodes to fp32 weights only")
            st = self.lib.excp_decompress_checkpoint_w16(self._h, blob.data_ptr(), offs, n, arr(w_prev), numel,
                                                         weight_format, arr(w_out), arr(ea_out), arr(eas_out), _stream())
            if st != 0:
                raise ExcpError(st, "excp_decompress_checkpoint_w16")
            return
        fn = self.lib.excp_decompress_dense_checkpoint if dense else self.lib.excp_decompress_checkpoint
        st = fn(self._h, blob.data_ptr(), offs, n, arr(w_prev), numel, arr(w_out), arr(ea_out), arr(eas_out),
                _stream())
        if st != 0:
            raise ExcpError(st, "excp_decompress_dense_checkpoint" if dense else "excp_decompress_checkpoint")

    # ---- the dense index layout (Sections 3.3 / 4.2) ----------------------
    def record_to_dense(self, record: torch.Tensor, record_bytes: int, numel: int, dense_out: torch.Tensor) -> int:
        out = C.c_size_t(0)
        st = self.lib.excp_record_to_dense(self._h, record.data_ptr(), record_bytes, numel, dense_out.data_ptr(),
                                           dense_out.numel(), C.byref(out), _stream())
        if st != 0:
            raise ExcpError(st, "excp_record_to_dense")
        return out.value

    def checkpoint_to_dense(self, blob: torch.Tensor, offsets, numels, dense_out: torch.Tensor) -> list[int]:
        n = len(numels)
        offs = (C.c_size_t * (n + 1))(*offsets)
        numel = (C.c_size_t * n)(*numels)
        douts = (C.c_size_t * (n + 1))()
        st = self.lib.excp_checkpoint_to_dense(self._h, blob.data_ptr(), offs, n, numel, dense_out.data_ptr(),
                                               dense_out.numel(), douts, _stream())
        if st != 0:
            raise ExcpError(st, "excp_checkpoint_to_dense")
        return list(douts)

    def decompress_dense_tensor(self, dense: torch.Tensor, dense_bytes_: int, w_prev, w_out, ea_out, eas_out) -> None:
        _check_f32_cuda(w_prev, w_out, ea_out, eas_out)
        st = self.lib.excp_decompress_dense_tensor(self._h, dense.data_ptr(), dense_bytes_, _ptr(w_prev),
                                                   w_prev.numel(), _ptr(w_out), _ptr(ea_out), _ptr(eas_out), _stream())
        if st != 0:
            raise ExcpError(st, "excp_decompress_dense_tensor")
