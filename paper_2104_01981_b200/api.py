"""Thin ctypes binding of libgc.so: the same names as the C ABI, argument marshalling only.

Every step of the path runs inside the library's CUDA kernels.  PyTorch appears here only as
the owner of device memory and streams (``tensor.data_ptr()``, ``torch.cuda.current_stream``).
If the shared library is missing or cannot be loaded, importing a compute entry point raises:
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.environ.get("GC_LIBRARY_PATH") or os.path.join(_HERE, "libgc.so")

GC_OK, GC_E_INVALID, GC_E_UNSUPPORTED, GC_E_CUDA, GC_E_TOO_LARGE, GC_E_TIMEOUT = 0, -1, -2, -3, -4, -5
GC_W_TRUNCATED = 1
GC_TOPK, GC_THRESHOLD = 0, 1
GC_MAX_WORKERS = 64
GC_K_COUNT = 16
(GC_Q_N_TENSORS, GC_Q_TOTAL_N, GC_Q_TOTAL_CAP, GC_Q_WORKSPACE_BYTES, GC_Q_TENSOR_N, GC_Q_TENSOR_K,
 GC_Q_TENSOR_CAP, GC_Q_TENSOR_OFFSET, GC_Q_TENSOR_OUT_OFFSET, GC_Q_TENSOR_STRIDE, GC_Q_MODE,
 GC_Q_KERNEL_LAUNCHES, GC_Q_CANDIDATE_CAPACITY, GC_Q_COMPRESS_ROUTE) = range(14)
(GC_ROUTE_NONE, GC_ROUTE_TOPK_ONE, GC_ROUTE_TOPK_MANY, GC_ROUTE_TOPK_GENERAL, GC_ROUTE_TOPK_STAGED, GC_ROUTE_EXACT,
 GC_ROUTE_THRESHOLD_ONE, GC_ROUTE_THRESHOLD_MANY, GC_ROUTE_THRESHOLD_STAGED) = range(9)
GC_OPT_PATH, GC_OPT_SAMPLE_RANK_PERMILLE, GC_OPT_CANDIDATE_CAPACITY, GC_OPT_DECODE_ROUTE = 0, 1, 2, 3
GC_DECODE_AUTO, GC_DECODE_NARROW, GC_DECODE_WIDE = 0, 1, 2
GC_OPT_DECODE_ORDER = 4
GC_OPT_WORKSPACE_PRIVATE = 5
GC_ORDER_FIXED, GC_ORDER_ANY = 0, 1
GC_PATH_AUTO, GC_PATH_EXACT, GC_PATH_STAGED = 0, 1, 2

_ERR = {GC_E_INVALID: "GC_E_INVALID", GC_E_UNSUPPORTED: "GC_E_UNSUPPORTED", GC_E_CUDA: "GC_E_CUDA",
        GC_E_TOO_LARGE: "GC_E_TOO_LARGE", GC_E_TIMEOUT: "GC_E_TIMEOUT"}

_lib: Optional[ctypes.CDLL] = None


class GcError(RuntimeError):
    def __init__(self, where: str, code: int):
        super().__init__(f"{where} failed: {_ERR.get(code, code)}")
        self.code = code


def lib() -> ctypes.CDLL:
    """Loads libgc.so (built in-tree by ``build.py``); raises if it is not there."""
    global _lib
    if _lib is None:
        if not os.path.exists(_SO):
            raise RuntimeError(f"{_SO} not found: build it with paper_2104_01981_b200.build.build(); "
                               "there is no fallback path")
        L = ctypes.CDLL(_SO)
        vp, u32, u64, i32, f64 = (ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int,
                                  ctypes.c_double)
        L.gc_version.restype = u32
        L.gc_version.argtypes = []
        L.gc_plan.restype = i32
        L.gc_plan.argtypes = [ctypes.POINTER(vp), i32, u32, vp, f64, i32, u32, f64]
        L.gc_plan_set_option.restype = i32
        L.gc_plan_set_option.argtypes = [vp, i32, u64]
        L.gc_plan_query.restype = i32
        L.gc_plan_query.argtypes = [vp, i32, u32, ctypes.POINTER(u64)]
        L.gc_compress.restype = i32
        L.gc_compress.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.gc_compress_bf16.restype = i32
        L.gc_compress_bf16.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.gc_compress_workers.restype = i32
        L.gc_compress_workers.argtypes = [vp, u32, vp, vp, vp, vp, vp, vp, vp]
        L.gc_decompress_accumulate.restype = i32
        L.gc_decompress_accumulate.argtypes = [vp, u32, vp, vp, vp, vp, i32, vp, vp]
        L.gc_last_status.restype = i32
        L.gc_last_status.argtypes = [vp, vp, vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(u64)]
        L.gc_decompress_apply_momentum.restype = i32
        L.gc_decompress_apply_momentum.argtypes = [vp, u32, vp, vp, vp, vp, vp, ctypes.c_float, ctypes.c_float,
                                                   ctypes.c_float, vp, vp]
        L.gc_compress_host.restype = i32
        L.gc_compress_host.argtypes = [vp] * 11
        L.gc_profile_enable.restype = i32
        L.gc_profile_enable.argtypes = [vp, u32]
        L.gc_profile_read.restype = i32
        L.gc_profile_read.argtypes = [vp, vp, vp]
        L.gc_kernel_name.restype = ctypes.c_char_p
        L.gc_kernel_name.argtypes = [i32]
        L.gc_compress_noalloc.restype = i32
        L.gc_compress_noalloc.argtypes = [vp, vp, u32, u32, vp, vp, vp, vp]
        L.gc_last_counters.restype = i32
        L.gc_last_counters.argtypes = [vp, vp, vp, vp]
        L.gc_last_phase_times.restype = i32
        L.gc_last_phase_times.argtypes = [vp, vp, vp, vp, vp]
        L.gc_last_cuda_error.restype = i32
        L.gc_last_cuda_error.argtypes = [vp]
        L.gc_destroy.restype = i32
        L.gc_destroy.argtypes = [vp]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


GC_NOALLOC_MAX_N = 1 << 24


def compress_noalloc(grad: torch.Tensor, residual: torch.Tensor, n: int, k: int, out_idx: torch.Tensor,
                     out_val: torch.Tensor, device_status: Optional[torch.Tensor] = None, stream=None) -> int:
    """gc_compress_noalloc: one tensor, scratch inside the library, no plan and no allocation.
    Returns the status code (negative codes are returned, not raised, so callers can test them)."""
    return lib().gc_compress_noalloc(_ptr(grad), _ptr(residual), n, k, _ptr(out_idx), _ptr(out_val),
                                     _ptr(device_status), _stream_handle(stream))


class Plan:
    """Owns one ``gc_plan_t``.  ``device=-1`` gives a host-only plan (queries only)."""

    def __init__(self, sizes: Sequence[int], density: float, mode: int = GC_TOPK, device: int = 0,
                 sample_stride: int = 0, cap_factor: float = 0.0):
        self._h = ctypes.c_void_p()
        arr = (ctypes.c_uint64 * max(len(sizes), 1))(*[int(s) for s in sizes])
        rc = lib().gc_plan(ctypes.byref(self._h), device, len(sizes), ctypes.cast(arr, ctypes.c_void_p),
                           float(density), mode, sample_stride, float(cap_factor))
        if rc != GC_OK:
            self._h = ctypes.c_void_p()
            raise GcError("gc_plan", rc)
        self.device = device
        self.mode = mode
        self.n_tensors = len(sizes)
        self.total_n = self.query(GC_Q_TOTAL_N)
        self.total_cap = self.query(GC_Q_TOTAL_CAP)
        self.workspace_bytes = self.query(GC_Q_WORKSPACE_BYTES)

    # --- gc_plan_query
    def query(self, what: int, tensor: int = 0) -> int:
        v = ctypes.c_uint64(0)
        rc = lib().gc_plan_query(self._h, what, tensor, ctypes.byref(v))
        if rc != GC_OK:
            raise GcError("gc_plan_query", rc)
        return int(v.value)

    # --- gc_plan_set_option
    def set_option(self, option: int, value: int) -> None:
        rc = lib().gc_plan_set_option(self._h, option, value)
        if rc != GC_OK:
            raise GcError("gc_plan_set_option", rc)
        self.workspace_bytes = self.query(GC_Q_WORKSPACE_BYTES)

    def tensor_k(self) -> List[int]:
        return [self.query(GC_Q_TENSOR_K, t) for t in range(self.n_tensors)]

    def tensor_cap(self) -> List[int]:
        return [self.query(GC_Q_TENSOR_CAP, t) for t in range(self.n_tensors)]

    def tensor_out_offset(self) -> List[int]:
        return [self.query(GC_Q_TENSOR_OUT_OFFSET, t) for t in range(self.n_tensors)]

    # --- buffers (PyTorch as the allocator)
    def alloc_workspace(self) -> torch.Tensor:
        return torch.zeros(max(self.workspace_bytes, 256), dtype=torch.uint8, device=f"cuda:{self.device}")

    def alloc_outputs(self):
        dev = f"cuda:{self.device}"
        return (torch.empty(max(self.total_cap, 1), dtype=torch.int32, device=dev),     # uint32 bit patterns
                torch.empty(max(self.total_cap, 1), dtype=torch.float32, device=dev),
                torch.zeros(max(2 * self.n_tensors, 1), dtype=torch.int32, device=dev))

    # --- gc_compress
    def compress(self, grad: torch.Tensor, residual: torch.Tensor, out_idx: torch.Tensor,
                 out_val: torch.Tensor, out_count: Optional[torch.Tensor], workspace: torch.Tensor,
                 stream=None) -> int:
        rc = lib().gc_compress(self._h, _ptr(grad), _ptr(residual), _ptr(out_idx), _ptr(out_val),
                               _ptr(out_count), _ptr(workspace), _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_compress", rc)
        return rc

    # --- gc_compress_workers
    def compress_workers(self, grads: Sequence[torch.Tensor], residuals: Sequence[torch.Tensor],
                         out_idx: Sequence[torch.Tensor], out_val: Sequence[torch.Tensor],
                         out_count: Optional[Sequence[torch.Tensor]], workspaces: Sequence[torch.Tensor],
                         stream=None) -> int:
        """All workers of one step in one call (one workspace, residual and output set per worker)."""
        W = len(grads)
        arr = lambda ts: (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in ts])
        rc = lib().gc_compress_workers(self._h, W, arr(grads), arr(residuals), arr(out_idx), arr(out_val),
                                       arr(out_count) if out_count is not None else None, arr(workspaces),
                                       _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_compress_workers", rc)
        return rc

    def compress_bf16(self, grad_bf16: torch.Tensor, residual: torch.Tensor, out_idx: torch.Tensor,
                      out_val: torch.Tensor, out_count: Optional[torch.Tensor], workspace: torch.Tensor,
                      stream=None) -> int:
        """``compress`` for a gradient stored as torch.bfloat16."""
        assert grad_bf16.dtype == torch.bfloat16
        rc = lib().gc_compress_bf16(self._h, _ptr(grad_bf16), _ptr(residual), _ptr(out_idx), _ptr(out_val),
                                    _ptr(out_count), _ptr(workspace), _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_compress_bf16", rc)
        return rc

    def compress_ptr(self, grad: int, residual: int, out_idx: int, out_val: int, out_count: Optional[int],
                     workspace: int, stream: int) -> int:
        """Raw-address form of ``compress`` (host or device addresses are passed through as is)."""
        return lib().gc_compress(self._h, grad, residual, out_idx, out_val, out_count, workspace, stream)

    # --- gc_compress_host
    def compress_host(self, host_grad: torch.Tensor, grad_staging: torch.Tensor, residual: torch.Tensor,
                      out_idx: torch.Tensor, out_val: torch.Tensor, out_count: Optional[torch.Tensor],
                      host_idx: torch.Tensor, host_val: torch.Tensor, workspace: torch.Tensor,
                      stream=None) -> int:
        assert not host_grad.is_cuda and not host_idx.is_cuda and not host_val.is_cuda
        rc = lib().gc_compress_host(self._h, _ptr(host_grad), _ptr(grad_staging), _ptr(residual),
                                    _ptr(out_idx), _ptr(out_val), _ptr(out_count), _ptr(host_idx),
                                    _ptr(host_val), _ptr(workspace), _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_compress_host", rc)
        return rc

    # --- gc_profile_enable / gc_profile_read
    def profile_enable(self, max_records: int) -> None:
        rc = lib().gc_profile_enable(self._h, max_records)
        if rc < 0:
            raise GcError("gc_profile_enable", rc)

    def profile_read(self):
        """{kernel name: (total ms, launches)} since the last read; synchronises the device."""
        ms = (ctypes.c_float * GC_K_COUNT)()
        cnt = (ctypes.c_uint32 * GC_K_COUNT)()
        rc = lib().gc_profile_read(self._h, ms, cnt)
        if rc < 0:
            raise GcError("gc_profile_read", rc)
        out = {}
        for i in range(GC_K_COUNT):
            if cnt[i]:
                out[lib().gc_kernel_name(i).decode()] = (float(ms[i]), int(cnt[i]))
        return out

    # --- gc_decompress_accumulate
    def decompress_accumulate(self, idx: Sequence[torch.Tensor], val: Sequence[torch.Tensor],
                              count: Optional[Sequence[torch.Tensor]], dense_out: torch.Tensor,
                              zero_first: bool, workspace: torch.Tensor, stream=None) -> int:
        W = len(idx)
        ip = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in idx])
        vp = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in val])
        cp = None
        if count is not None:
            cp = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in count])
        rc = lib().gc_decompress_accumulate(self._h, W, ip, vp, cp, _ptr(dense_out), 1 if zero_first else 0,
                                            _ptr(workspace), _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_decompress_accumulate", rc)
        return rc

    # --- gc_decompress_apply_momentum
    def decompress_apply_momentum(self, idx: Sequence[torch.Tensor], val: Sequence[torch.Tensor],
                                  count: Optional[Sequence[torch.Tensor]], param: torch.Tensor,
                                  velocity: torch.Tensor, lr: float, momentum: float, scale: float,
                                  workspace: torch.Tensor, stream=None) -> int:
        W = len(idx)
        ip = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in idx])
        vp = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in val])
        cp = None
        if count is not None:
            cp = (ctypes.c_void_p * max(W, 1))(*[t.data_ptr() for t in count])
        rc = lib().gc_decompress_apply_momentum(self._h, W, ip, vp, cp, _ptr(param), _ptr(velocity), lr, momentum,
                                                scale, _ptr(workspace), _stream_handle(stream))
        if rc < 0:
            raise GcError("gc_decompress_apply_momentum", rc)
        return rc

    # --- gc_last_status (synchronises the stream)
    def last_status(self, workspace: torch.Tensor, stream=None):
        st = ctypes.c_int32(0)
        det = ctypes.c_uint64(0)
        rc = lib().gc_last_status(self._h, _ptr(workspace), _stream_handle(stream), ctypes.byref(st),
                                  ctypes.byref(det))
        if rc < 0:
            raise GcError("gc_last_status", rc)
        return int(st.value), int(det.value)

    def last_counters(self, workspace: torch.Tensor, stream=None):
        """(candidates, overflowed, failed tensors) of the last compress; synchronises."""
        c = (ctypes.c_uint32 * 3)()
        rc = lib().gc_last_counters(self._h, _ptr(workspace), _stream_handle(stream), c)
        if rc < 0:
            raise GcError("gc_last_counters", rc)
        return int(c[0]), int(c[1]), int(c[2])

    def last_phase_times(self, workspace: torch.Tensor, stream=None):
        """Phase durations (microseconds) of the last fused top-k launch; synchronises."""
        ns = (ctypes.c_uint64 * 20)()
        n = ctypes.c_uint32(0)
        rc = lib().gc_last_phase_times(self._h, _ptr(workspace), _stream_handle(stream), ns, ctypes.byref(n))
        if rc < 0:
            raise GcError("gc_last_phase_times", rc)
        return [ns[i] / 1e3 for i in range(n.value)]

    def launches(self) -> int:
        return self.query(GC_Q_KERNEL_LAUNCHES)

    # --- gc_destroy
    def destroy(self) -> None:
        if self._h:
            lib().gc_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
