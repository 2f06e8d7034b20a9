"""Seeded synthetic inputs (permutations and payloads) for tests and benchmarks.

A module of its own: it holds no routing arithmetic and depends on neither the
CUDA library nor the CPU oracle, so both sides can be fed the very same arrays.

Random permutations come from ``gen.c`` (Fisher-Yates / Sattolo driven by
SplitMix64, built with gcc on first use); the structured ones are closed-form
numpy expressions.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libbenes_inputs.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64 = ctypes.c_uint64
        vp = ctypes.c_void_p
        lib.gen_fisher_yates.argtypes = [vp, u64, u64]
        lib.gen_fisher_yates_batch.argtypes = [vp, u64, u64, u64]
        lib.gen_sattolo.argtypes = [vp, u64, u64]
        lib.gen_payload_f32.argtypes = [vp, u64, u64]
        lib.gen_payload_u64.argtypes = [vp, u64, u64]
        for f in (lib.gen_fisher_yates, lib.gen_fisher_yates_batch, lib.gen_sattolo,
                  lib.gen_payload_f32, lib.gen_payload_u64):
            f.restype = None
        _lib = lib
    return _lib


def random_perm(log2n: int, seed: int) -> np.ndarray:
    """Uniform random permutation of 2^log2n (Fisher-Yates, given seed)."""
    N = 1 << log2n
    p = np.empty(N, dtype=np.uint32)
    _load().gen_fisher_yates(p.ctypes.data, N, seed)
    return p


def random_perm_any(n_elems: int, batch: int, seed0: int = 0) -> np.ndarray:
    """(batch, n_elems) uniform permutations of [0, n_elems) for any n_elems >= 1
    (the same Fisher-Yates generator; seeds seed0 .. seed0+batch-1)."""
    p = np.empty((batch, n_elems), dtype=np.uint32)
    for b in range(batch):
        _load().gen_fisher_yates(p[b].ctypes.data, n_elems, seed0 + b)
    return p


def pad_with_fixed_points(perm: np.ndarray, log2n: int) -> np.ndarray:
    """Rows of n_elems values -> rows of 2^log2n values, pi[j] = j beyond n_elems."""
    perm = np.atleast_2d(perm)
    N = 1 << log2n
    out = np.tile(np.arange(N, dtype=np.uint32), (perm.shape[0], 1))
    out[:, :perm.shape[1]] = perm
    return out


def random_perm_batch(log2n: int, batch: int, seed0: int = 0) -> np.ndarray:
    """(batch, N) independent uniform permutations, seeds seed0 .. seed0+batch-1."""
    N = 1 << log2n
    p = np.empty((batch, N), dtype=np.uint32)
    _load().gen_fisher_yates_batch(p.ctypes.data, N, batch, seed0)
    return p


def sattolo_perm(log2n: int, seed: int) -> np.ndarray:
    """Uniform random permutation consisting of one N-cycle (Sattolo)."""
    N = 1 << log2n
    p = np.empty(N, dtype=np.uint32)
    _load().gen_sattolo(p.ctypes.data, N, seed)
    return p


def identity_perm(log2n: int) -> np.ndarray:
    return np.arange(1 << log2n, dtype=np.uint32)


def shift_perm(log2n: int, k: int = 1) -> np.ndarray:
    """Cyclic shift: pi[j] = (j + k) mod N."""
    N = 1 << log2n
    return ((np.arange(N, dtype=np.uint64) + (k % N)) % N).astype(np.uint32)


def bit_reversal_perm(log2n: int) -> np.ndarray:
    """pi[j] = j with its log2n-bit binary representation reversed."""
    j = np.arange(1 << log2n, dtype=np.uint32)
    r = np.zeros_like(j)
    for b in range(log2n):
        r |= ((j >> np.uint32(b)) & np.uint32(1)) << np.uint32(log2n - 1 - b)
    return r


def transpose_perm(log2n: int) -> np.ndarray:
    """Index map of a matrix transpose: pi[r*C + c] = c*R + r for an R x C matrix,
    R = 2^floor(log2n/2), C = N/R (square when log2n is even)."""
    R = 1 << (log2n // 2)
    C = (1 << log2n) // R
    j = np.arange(1 << log2n, dtype=np.uint32)
    return ((j % C) * R + j // C).astype(np.uint32)


def payload_f32(n_elems: int, seed: int) -> np.ndarray:
    """fp32 values uniform in [0, 1)."""
    x = np.empty(n_elems, dtype=np.float32)
    _load().gen_payload_f32(x.ctypes.data, n_elems, seed)
    return x


def payload_u64(n_elems: int, seed: int) -> np.ndarray:
    """uint64 values: element index in the low 32 bits, random high 32 bits."""
    x = np.empty(n_elems, dtype=np.uint64)
    _load().gen_payload_u64(x.ctypes.data, n_elems, seed)
    return x


def structured_perms(log2n: int, sattolo_seed: int = 3) -> dict:
    """The five structured cases: identity, shift by one, bit reversal,
    square transpose map, random single cycle."""
    return {
        "identity": identity_perm(log2n),
        "shift1": shift_perm(log2n, 1),
        "bitrev": bit_reversal_perm(log2n),
        "transpose": transpose_perm(log2n),
        "sattolo": sattolo_perm(log2n, sattolo_seed),
    }
