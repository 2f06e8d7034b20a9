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
        lib.oracle_route_part.argtypes = [u32p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_size_t,
                                          ctypes.c_size_t, u32p, u32p]
        lib.oracle_apply_part.argtypes = [u32p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int,
                                          ctypes.c_int, ctypes.c_int, ctypes.c_size_t, ctypes.c_size_t]
        for f in (lib.oracle_route_trace, lib.oracle_route_batch, lib.oracle_apply_batch,
                  lib.oracle_route_part, lib.oracle_apply_part):
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


def _split_level(log2n: int, threads: int) -> int:
    """First level whose sub-networks are handed to `threads` host threads: the
    smallest level with at least `threads` sub-networks, each of 64 outputs or more."""
    level = 0
    while (1 << level) < threads and log2n - (level + 1) >= 6:
        level += 1
    return level


def _run_parts(threads: int, jobs):
    from concurrent.futures import ThreadPoolExecutor
    with ThreadPoolExecutor(max_workers=threads) as pool:      # ctypes releases the GIL
        for rc in pool.map(lambda job: job(), jobs):
            if rc != 0:
                raise RuntimeError("oracle part failed (%d)" % rc)


def route_parallel(perm: np.ndarray, log2n: int, threads: int) -> np.ndarray:
    """Same result as ``route``.  A batch: permutations are spread over `threads` host
    threads.  One permutation: the levels above ``_split_level`` run on one thread, the
    independent sub-networks below them on `threads` threads (same C routine, by range)."""
    perm = np.ascontiguousarray(perm, dtype=np.uint32)
    n, N, lib = log2n, 1 << log2n, _load()
    p2 = perm.reshape(-1, N)
    bits = np.zeros((p2.shape[0], 2 * n - 1, stage_words(n)), dtype=np.uint32)
    if p2.shape[0] > 1:
        step = -(-p2.shape[0] // threads)
        _run_parts(threads, [
            (lambda a=a: lib.oracle_route_batch(_u32(p2[a:a + step]), n, len(p2[a:a + step]), _u32(bits[a:a + step])))
            for a in range(0, p2.shape[0], step)])
    else:
        split = _split_level(n, threads)
        mid = np.empty(N, dtype=np.uint32)
        rc = lib.oracle_route_part(_u32(p2[0]), n, 0, split, 0, N, _u32(bits[0]), _u32(mid))
        if rc != 0:
            raise RuntimeError("oracle_route_part failed (%d)" % rc)
        M = N >> split
        _run_parts(threads, [
            (lambda lo=lo: lib.oracle_route_part(_u32(mid), n, split, n, lo, lo + M, _u32(bits[0]), None))
            for lo in range(0, N, M)])
    return bits[0] if perm.ndim == 1 else bits


def apply_parallel(bits: np.ndarray, x: np.ndarray, log2n: int, threads: int) -> np.ndarray:
    """Same result as ``apply``; the stages strictly inside ``_split_level`` form
    independent sub-networks and run on `threads` host threads."""
    n, N, lib = log2n, 1 << log2n, _load()
    x = np.ascontiguousarray(x)
    bits = np.ascontiguousarray(bits, dtype=np.uint32)
    x2 = x.reshape(-1, N)
    batch, e = x2.shape[0], x.dtype.itemsize
    b2 = bits.reshape(batch, 2 * n - 1, stage_words(n))
    out = x2.copy()
    tmp = np.empty_like(out)
    if batch > 1:
        _run_parts(threads, [
            (lambda b=b: lib.oracle_apply_part(_u32(b2[b]), out[b].ctypes.data, tmp[b].ctypes.data, e, n,
                                               0, 2 * n - 1, 0, N))
            for b in range(batch)])
    else:
        split = _split_level(n, threads)
        M = N >> split
        args = (_u32(b2[0]), out[0].ctypes.data, tmp[0].ctypes.data, e, n)
        if lib.oracle_apply_part(*args, 0, split, 0, N) != 0:
            raise RuntimeError("oracle_apply_part failed")
        _run_parts(threads, [
            (lambda lo=lo: lib.oracle_apply_part(*args, split, 2 * n - 1 - split, lo, lo + M))
            for lo in range(0, N, M)])
        if lib.oracle_apply_part(*args, 2 * n - 1 - split, 2 * n - 1, 0, N) != 0:
            raise RuntimeError("oracle_apply_part failed")
    return out.reshape(x.shape)


def _stage_bits(bits_row: np.ndarray, count: int) -> np.ndarray:
    """First `count` bits of one stage row (LSB-first 32-bit words) as a 0/1 array."""
    words = np.ascontiguousarray(bits_row, dtype=np.uint32)
    return np.unpackbits(words.view(np.uint8), bitorder="little")[:count]


def export_butterfly(bits: np.ndarray, log2n: int) -> np.ndarray:
    """The settings of one permutation, (2n-1, W) words, re-indexed for the network drawn
    in place (data never moves between stages; stage row r pairs positions that differ in
    bit i, i = r up to the middle and 2n-2-r after it; pair p = the position with bit i
    taken out).  Done by pushing position labels through the wiring of the recursive
    network with every switch straight: the two labels that meet in a switch are the two
    in-place positions that switch acts on (they must differ in exactly bit i)."""
    n, N = log2n, 1 << log2n
    W = stage_words(n)
    bits = np.ascontiguousarray(bits, dtype=np.uint32).reshape(2 * n - 1, W)
    out_bits = np.zeros((2 * n - 1, N // 2 if N >= 2 else 1), dtype=np.uint8)
    label = np.arange(N, dtype=np.int64)          # label[q] = in-place position of what sits at q
    per_level = []
    for level in range(n):                        # input side, then the middle (level n-1)
        a, b = label[0::2], label[1::2]           # switch w takes positions 2w, 2w+1 of the flat array
        assert np.array_equal(a ^ b, np.full(N // 2, 1 << level)) and not (a & (1 << level)).any()
        pair = ((a >> (level + 1)) << level) | (a & ((1 << level) - 1))
        out_bits[level, pair] = _stage_bits(bits[level], N // 2)
        per_level.append(pair)
        if level < n - 1:                         # wiring: switch s of a block -> position s of each half
            M = N >> level
            blk = label.reshape(-1, M)
            label = np.concatenate([blk[:, 0::2], blk[:, 1::2]], axis=1).reshape(-1)
    for level in range(n - 2, -1, -1):            # output side mirrors the input side
        out_bits[2 * n - 2 - level, per_level[level]] = _stage_bits(bits[2 * n - 2 - level], N // 2)
    packed = np.zeros((2 * n - 1, W * 32), dtype=np.uint8)
    packed[:, :out_bits.shape[1]] = out_bits[:, :W * 32]
    return np.packbits(packed, axis=1, bitorder="little").view(np.uint32).reshape(2 * n - 1, W)


def apply_butterfly(bfly: np.ndarray, x: np.ndarray, log2n: int) -> np.ndarray:
    """Run the in-place network on a copy of x: row r swaps x[u] and x[u | 2^i] where bit p is set."""
    n, N = log2n, 1 << log2n
    W = stage_words(n)
    bfly = np.ascontiguousarray(bfly, dtype=np.uint32).reshape(2 * n - 1, W)
    y = np.array(x, copy=True)
    for r in range(2 * n - 1):
        i = r if r <= n - 1 else 2 * n - 2 - r
        p = np.nonzero(_stage_bits(bfly[r], N // 2))[0].astype(np.int64)
        u = ((p >> i) << (i + 1)) | (p & ((1 << i) - 1))
        v = u | (1 << i)
        y[u], y[v] = y[v].copy(), y[u].copy()
    return y
