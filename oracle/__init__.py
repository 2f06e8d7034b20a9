"""CPU oracle for Benes routing -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper around ``benes_oracle.c`` (plain sequential C).  Nothing in
the product package may import this module; only the tests, the smoke check and
the benchmark's CPU-baseline leg do.  It shares no code with the CUDA path.

Conventions (gather form ``out[j] = in[pi[j]]``, canonical colouring "smallest
output index of every loop goes up", stage-major bit layout) are written out in
the header comment of ``benes_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "benes_oracle.c")
_LIB = os.path.join(_HERE, "libbenes_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no optimisation tricks: plain -O2)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u32p = ctypes.POINTER(ctypes.c_uint32)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        lib.oracle_route_trace.argtypes = [u32p, ctypes.c_int, u32p, u32p, u8p]
        lib.oracle_route_batch.argtypes = [u32p, ctypes.c_int, ctypes.c_int, u32p]
        lib.oracle_apply_batch.argtypes = [u32p, ctypes.c_void_p, ctypes.c_void_p,
                                           ctypes.c_int, ctypes.c_int, ctypes.c_int]
        for f in (lib.oracle_route_trace, lib.oracle_route_batch, lib.oracle_apply_batch):
            f.restype = ctypes.c_int
        _lib = lib
    return _lib


def stage_words(log2n: int) -> int:
    return max(1, (1 << log2n) // 64)


def _u32(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32))


def route(perm: np.ndarray, log2n: int) -> np.ndarray:
    """Switch bits for ``perm`` of shape (N,) or (batch, N); returns
    (2n-1, W) or (batch, 2n-1, W) uint32 words."""
    perm = np.ascontiguousarray(perm, dtype=np.uint32)
    N = 1 << log2n
    single = perm.ndim == 1
    p2 = perm.reshape(-1, N)
    bits = np.empty((p2.shape[0], 2 * log2n - 1, stage_words(log2n)), dtype=np.uint32)
    rc = _load().oracle_route_batch(_u32(p2), log2n, p2.shape[0], _u32(bits))
    if rc != 0:
        raise RuntimeError("oracle_route_batch failed (%d)" % rc)
    return bits[0] if single else bits


def route_trace(perm: np.ndarray, log2n: int):
    """Single permutation; also returns every level's block-local
    sub-permutations (n, N) and colours (n, N; last row unused)."""
    perm = np.ascontiguousarray(perm, dtype=np.uint32)
    N = 1 << log2n
    assert perm.shape == (N,)
    bits = np.empty((2 * log2n - 1, stage_words(log2n)), dtype=np.uint32)
    tp = np.zeros((log2n, N), dtype=np.uint32)
    tc = np.zeros((log2n, N), dtype=np.uint8)
    rc = _load().oracle_route_trace(_u32(perm), log2n, _u32(bits), _u32(tp),
                                    tc.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)))
    if rc != 0:
        raise RuntimeError("oracle_route_trace failed (%d)" % rc)
    return bits, tp, tc


def apply(bits: np.ndarray, x: np.ndarray, log2n: int) -> np.ndarray:
    """Push payload ``x`` of shape (N,) or (batch, N) (any 1/2/4/8-byte dtype)
    through the network described by ``bits``; returns the routed payload."""
    N = 1 << log2n
    x = np.ascontiguousarray(x)
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    x2 = x.reshape(-1, N)
    batch = x2.shape[0]
    assert bits.size == batch * (2 * log2n - 1) * stage_words(log2n)
    out = np.empty_like(x2)
    rc = _load().oracle_apply_batch(_u32(bits), x2.ctypes.data, out.ctypes.data,
                                    x.dtype.itemsize, log2n, batch)
    if rc != 0:
        raise RuntimeError("oracle_apply_batch failed (%d)" % rc)
    return out.reshape(x.shape)
