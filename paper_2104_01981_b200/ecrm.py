"""ctypes binding of include/ecrm.h (argument marshalling only; all arithmetic runs in the
CUDA kernels of csrc/ecrm.cu).  PyTorch provides device memory and streams."""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

import torch

from . import api

ECRM_OK, ECRM_E_INVALID, ECRM_E_CUDA = 0, -1, -3
ECRM_ADAGRAD, ECRM_MOMENTUM = 0, 1
ECRM_MAX_K = 32


class EcrmError(RuntimeError):
    def __init__(self, fn: str, rc: int):
        super().__init__(f"{fn} failed with status {rc}")
        self.rc = rc


_configured = False


def lib() -> ctypes.CDLL:
    global _configured
    l = api.lib()                       # fails loudly if the CUDA library is missing
    if not _configured:
        vp, u32, u64, f32 = ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_float
        pp = ctypes.POINTER(ctypes.c_void_p)
        l.ecrm_encode.argtypes = [u32, pp, vp, u64, vp]
        l.ecrm_decode.argtypes = [u32, pp, vp, vp, u64, vp]
        l.ecrm_rows_step.argtypes = [ctypes.c_int, u32, vp, vp, vp, vp, u64, u32, f32, f32, vp, vp, vp, vp]
        l.ecrm_parity_add.argtypes = [u32, vp, vp, vp, vp, vp, u64, u32, vp, vp]
        l.ecrm_rows_step_parity.argtypes = [ctypes.c_int, u32, vp, vp, vp, vp, vp, u64, vp, vp, u64, u32, f32, f32, vp, vp]
        l.ecrm_degraded_read.argtypes = [u32, u32, vp, pp, pp, vp, u64, u32, vp, vp, vp]
        l.ecrm_placement.argtypes = [u32, u64, ctypes.POINTER(u32), ctypes.POINTER(u32)]
        for f in (l.ecrm_encode, l.ecrm_decode, l.ecrm_rows_step, l.ecrm_parity_add, l.ecrm_degraded_read,
                  l.ecrm_placement, l.ecrm_rows_step_parity):
            f.restype = ctypes.c_int
        _configured = True
    return l


def _ptr(t: Optional[torch.Tensor]):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def _table(ts: Sequence[Optional[torch.Tensor]]):
    arr = (ctypes.c_void_p * max(len(ts), 1))(*[(t.data_ptr() if t is not None else 0) for t in ts])
    return ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)), arr


def _stream(stream):
    return api._stream_handle(stream)


def _check(fn: str, rc: int) -> int:
    if rc < 0:
        raise EcrmError(fn, rc)
    return rc


def encode(shards: Sequence[torch.Tensor], parity: torch.Tensor, stream=None) -> int:
    tab, keep = _table(shards)
    return _check("ecrm_encode", lib().ecrm_encode(len(shards), tab, _ptr(parity), parity.numel(), _stream(stream)))


def decode(survivors: Sequence[torch.Tensor], parity: torch.Tensor, out: torch.Tensor, stream=None) -> int:
    tab, keep = _table(survivors)
    return _check("ecrm_decode", lib().ecrm_decode(len(survivors), tab, _ptr(parity), _ptr(out), out.numel(),
                                                   _stream(stream)))


def rows_step(optimizer: int, rows: torch.Tensor, grad: torch.Tensor, entry: torch.Tensor, state: torch.Tensor,
              lr: float, hyper: float, d_entry: torch.Tensor, d_state: torch.Tensor,
              bad_rows: Optional[torch.Tensor] = None, stream=None) -> int:
    n_rows, dim = entry.shape
    return _check("ecrm_rows_step", lib().ecrm_rows_step(optimizer, rows.numel(), _ptr(rows), _ptr(grad), _ptr(entry),
                                                         _ptr(state), n_rows, dim, lr, hyper, _ptr(d_entry),
                                                         _ptr(d_state), _ptr(bad_rows), _stream(stream)))


def parity_add(prow: torch.Tensor, d_entry: torch.Tensor, d_state: Optional[torch.Tensor], p_entry: torch.Tensor,
               p_state: Optional[torch.Tensor], bad_rows: Optional[torch.Tensor] = None, stream=None) -> int:
    n_prows, dim = p_entry.shape
    return _check("ecrm_parity_add", lib().ecrm_parity_add(prow.numel(), _ptr(prow), _ptr(d_entry), _ptr(d_state),
                                                           _ptr(p_entry), _ptr(p_state), n_prows, dim,
                                                           _ptr(bad_rows), _stream(stream)))


def rows_step_parity(optimizer: int, rows: torch.Tensor, prow: torch.Tensor, grad: torch.Tensor, entry: torch.Tensor,
                     state: torch.Tensor, p_entry: torch.Tensor, p_state: torch.Tensor, lr: float, hyper: float,
                     bad_rows: Optional[torch.Tensor] = None, stream=None) -> int:
    n_rows, dim = entry.shape
    return _check("ecrm_rows_step_parity",
                  lib().ecrm_rows_step_parity(optimizer, rows.numel(), _ptr(rows), _ptr(prow), _ptr(grad), _ptr(entry),
                                              _ptr(state), n_rows, _ptr(p_entry), _ptr(p_state), p_entry.shape[0], dim,
                                              lr, hyper, _ptr(bad_rows), _stream(stream)))


def degraded_read(prow: torch.Tensor, srows: Optional[Sequence[Optional[torch.Tensor]]],
                  shards: Sequence[torch.Tensor], parity: torch.Tensor, out: torch.Tensor,
                  bad_rows: Optional[torch.Tensor] = None, stream=None) -> int:
    n_rows, dim = parity.shape
    stab, keep1 = _table(shards)
    rtab, keep2 = _table(list(srows) if srows is not None else [None] * len(shards))
    return _check("ecrm_degraded_read", lib().ecrm_degraded_read(len(shards), prow.numel(), _ptr(prow), rtab, stab,
                                                                 _ptr(parity), n_rows, dim, _ptr(out),
                                                                 _ptr(bad_rows), _stream(stream)))


def placement(k: int, group: int):
    ps = ctypes.c_uint32(0)
    ds = (ctypes.c_uint32 * k)()
    _check("ecrm_placement", lib().ecrm_placement(k, group, ctypes.byref(ps), ds))
    return ps.value, list(ds)
