"""ctypes access to the CPU oracle (test infrastructure only).

Only the tests, the smoke check and the benchmark's CPU-baseline leg import this package;
the CUDA product path never does.  ``build()`` compiles ``gc_oracle.cpp`` with g++ into
``liboracle.so`` next to this file; ``lib()`` loads it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_SRC = os.path.join(_HERE, "gc_oracle.cpp")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(_SO) and os.path.getmtime(_SO) >= os.path.getmtime(_SRC):
        return _SO
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
           "-Wall", "-o", _SO, _SRC]
    subprocess.run(cmd, check=True)
    return _SO


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_SO)
        u64, u32, f64, vp = ctypes.c_uint64, ctypes.c_uint32, ctypes.c_double, ctypes.c_void_p
        L.oracle_k_from_density.restype = u64
        L.oracle_k_from_density.argtypes = [u64, f64]
        L.oracle_effective_stride.restype = u32
        L.oracle_effective_stride.argtypes = [u64, u32]
        L.oracle_sample_count.restype = u64
        L.oracle_sample_count.argtypes = [u64, u32]
        L.oracle_topk_compress.restype = ctypes.c_int
        L.oracle_topk_compress.argtypes = [vp, vp, u64, u64, u64, vp, vp]
        L.oracle_topk_compress_tensors.restype = ctypes.c_int
        L.oracle_topk_compress_tensors.argtypes = [u32, vp, vp, vp, vp, vp, vp]
        L.oracle_threshold_compress.restype = ctypes.c_int
        L.oracle_threshold_compress.argtypes = [vp, vp, u64, f64, u32, u64, u64, vp, vp, vp, vp, vp]
        L.oracle_decode_accumulate.restype = ctypes.c_int
        L.oracle_decode_accumulate.argtypes = [u32, vp, vp, vp, vp, u64, ctypes.c_int]
        _lib = L
    return _lib


def _f32(x) -> np.ndarray:
    a = np.ascontiguousarray(x, dtype=np.float32)
    return a


def k_from_density(n: int, density: float) -> int:
    return int(lib().oracle_k_from_density(n, density))


def effective_stride(n: int, stride: int) -> int:
    return int(lib().oracle_effective_stride(n, stride))


def sample_count(n: int, stride: int) -> int:
    return int(lib().oracle_sample_count(n, stride))


def topk_compress(g: np.ndarray, r: np.ndarray, k: int, index_base: int = 0
                  ) -> Tuple[np.ndarray, np.ndarray]:
    """One tensor, one step.  ``r`` (float32, contiguous) is updated in place."""
    g = _f32(g)
    assert r.dtype == np.float32 and r.flags.c_contiguous and r.shape == g.shape
    idx = np.empty(k, dtype=np.uint32)
    val = np.empty(k, dtype=np.float32)
    rc = lib().oracle_topk_compress(g.ctypes.data, r.ctypes.data, g.size, k, index_base,
                                    idx.ctypes.data, val.ctypes.data)
    if rc:
        raise ValueError(f"oracle_topk_compress failed: {rc}")
    return idx, val


def topk_compress_tensors(sizes: Sequence[int], ks: Sequence[int], g: np.ndarray, r: np.ndarray
                          ) -> Tuple[np.ndarray, np.ndarray]:
    """Layer-wise top-k over tensors laid back to back in flat ``g`` / ``r`` (r in place)."""
    g = _f32(g)
    assert r.dtype == np.float32 and r.flags.c_contiguous and r.size == g.size == sum(sizes)
    sz = np.asarray(sizes, dtype=np.uint64)
    kk = np.asarray(ks, dtype=np.uint64)
    tot = int(kk.sum())
    idx = np.empty(tot, dtype=np.uint32)
    val = np.empty(tot, dtype=np.float32)
    rc = lib().oracle_topk_compress_tensors(len(sizes), sz.ctypes.data, kk.ctypes.data,
                                            g.ctypes.data, r.ctypes.data,
                                            idx.ctypes.data, val.ctypes.data)
    if rc:
        raise ValueError(f"oracle_topk_compress_tensors failed: {rc}")
    return idx, val


def threshold_compress(g: np.ndarray, r: np.ndarray, density: float, stride: int, cap: int,
                       index_base: int = 0):
    """Returns (idx[:sent], val[:sent], n_hits, tau_key); ``r`` is updated in place."""
    g = _f32(g)
    assert r.dtype == np.float32 and r.flags.c_contiguous and r.shape == g.shape
    idx = np.empty(max(cap, 1), dtype=np.uint32)
    val = np.empty(max(cap, 1), dtype=np.float32)
    sent, hits = ctypes.c_uint64(0), ctypes.c_uint64(0)
    tau = ctypes.c_uint32(0)
    rc = lib().oracle_threshold_compress(g.ctypes.data, r.ctypes.data, g.size, density, stride, cap,
                                         index_base, idx.ctypes.data, val.ctypes.data,
                                         ctypes.addressof(sent), ctypes.addressof(hits),
                                         ctypes.addressof(tau))
    if rc:
        raise ValueError(f"oracle_threshold_compress failed: {rc}")
    return idx[:sent.value].copy(), val[:sent.value].copy(), int(hits.value), int(tau.value)


def decode_accumulate(pairs: List[Tuple[np.ndarray, np.ndarray]], out: np.ndarray,
                      zero_first: bool = True) -> np.ndarray:
    """Adds W sparse sets into dense float32 ``out`` (in place), worker order 0..W-1."""
    assert out.dtype == np.float32 and out.flags.c_contiguous
    W = len(pairs)
    idxs = [np.ascontiguousarray(p[0], dtype=np.uint32) for p in pairs]
    vals = [np.ascontiguousarray(p[1], dtype=np.float32) for p in pairs]
    ip = (ctypes.c_void_p * max(W, 1))(*[a.ctypes.data for a in idxs])
    vp = (ctypes.c_void_p * max(W, 1))(*[a.ctypes.data for a in vals])
    cnt = np.asarray([a.size for a in idxs], dtype=np.uint64)
    rc = lib().oracle_decode_accumulate(W, ip, vp, cnt.ctypes.data, out.ctypes.data, out.size,
                                        1 if zero_first else 0)
    if rc:
        raise ValueError(f"oracle_decode_accumulate failed: {rc}")
    return out


def decode_apply_momentum(pairs: List[Tuple[np.ndarray, np.ndarray]], param: np.ndarray, vel: np.ndarray,
                          lr: float, momentum: float, scale: float) -> None:
    """The decode followed by momentum SGD, in place on float32 ``param`` and ``vel``:
    s = worker-ordered sum of the sparse sets (+0 where nothing was sent),
    v' = fl(fl(momentum v) + fl(scale s)), p' = fl(p - fl(lr v')): one rounding per operation.
    Written as the plain definition: the dense sum first, then three elementwise numpy steps."""
    assert param.dtype == np.float32 and vel.dtype == np.float32
    f = np.float32
    s = decode_accumulate(pairs, np.empty(param.size, np.float32), True)
    vn = ((f(momentum) * vel).astype(f) + (f(scale) * s).astype(f)).astype(f)
    param[:] = (param - (f(lr) * vn).astype(f)).astype(f)
    vel[:] = vn
