"""ctypes binding of ``libbenes.so`` -- argument marshalling only.

Function names and argument orders are those of ``include/benes.h``.  Device
buffers are ``torch`` CUDA tensors (PyTorch is used for device memory and
streams, nothing else); every step of the path runs inside the library's CUDA
kernels.  There is no CPU fallback: if the library has not been built, loading
raises ``RuntimeError``.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbenes.so")

BENES_OK = 0
BENES_ERR_BADARG = -1
BENES_ERR_CUDA = -2
BENES_ERR_NOMEM = -3
BENES_ERR_NOT_PERMUTATION = -4
BENES_ERR_TOO_LARGE = -5
STATIC_SCRATCH_BYTES = 4 << 20

# every symbol include/benes.h declares: name -> (restype, argtypes)
_vp, _i, _sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
SYMBOLS = {
    "benes_route": (_i, [_vp, _i, _i, _vp, _vp]),
    "benes_apply": (_i, [_vp, _vp, _vp, _i, _i, _vp]),
    "benes_apply_ex": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp]),
    "benes_apply_static": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp]),
    "benes_export_butterfly": (_i, [_vp, _vp, _i, _i, _vp]),
    "benes_padded_log2n": (_i, [_sz]),
    "benes_route_padded": (_i, [_vp, _sz, _i, _vp, _vp]),
    "benes_apply_padded": (_i, [_vp, _vp, _vp, _i, _sz, _i, _vp]),
    "benes_route_host": (_i, [_vp, _i, _i, _vp, _vp]),
    "benes_apply_host": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp]),
    "benes_route_apply_host": (_i, [_vp, _vp, _vp, _i, _i, _i, _vp, _vp]),
    "benes_switch_words": (_sz, [_i, _i]),
    "benes_route_workspace_bytes": (_sz, [_i, _i]),
    "benes_apply_workspace_bytes": (_sz, [_i, _i, _i]),
    "benes_set_workspace": (_i, [_vp, _sz]),
    "benes_release_workspace": (_i, []),
    "benes_validate_perm": (_i, [_vp, _i, _i, _vp]),
    "benes_set_option": (_i, [_i, _i]),
    "benes_get_option": (_i, [_i]),
    "benes_launch_count": (ctypes.c_ulonglong, []),
    "benes_plan_create": (_i, [ctypes.POINTER(_vp), _vp, _i, _i, _vp, _vp, _vp, _i]),
    "benes_plan_launch": (_i, [_vp, _vp]),
    "benes_plan_destroy": (_i, [_vp]),
    "benes_profile_enabled": (_i, []),
    "benes_profile_enable": (_i, [_i]),
    "benes_profile_reset": (_i, []),
    "benes_profile_read": (_i, [_i, ctypes.POINTER(ctypes.c_ulonglong), ctypes.POINTER(ctypes.c_double)]),
    "benes_profile_span": (_i, [_i, ctypes.POINTER(_i), ctypes.POINTER(ctypes.c_ulonglong),
                                ctypes.POINTER(ctypes.c_double)]),
    "benes_profile_kind_name": (ctypes.c_char_p, [_i]),
    "benes_shard_batch": (_i, [_i, _i, _i, ctypes.POINTER(_i), ctypes.POINTER(_i)]),
    "benes_probe_random_access": (_i, [_vp, _i, _i, _i, _sz, _vp, _vp]),
    "benes_debug_build": (_i, []),
    "benes_debug_guard_hits": (_i, [ctypes.POINTER(ctypes.c_ulonglong), ctypes.c_char_p, _sz, _i]),
    "benes_fused_log2m": (_i, []),
    "benes_status_string": (ctypes.c_char_p, [_i]),
}

_lib = None


class BenesError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__("%s failed: %s (%d)" % (what, status_string(status), status))


def _open(path: str) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise RuntimeError(
            "%s is not built (%s); run `python -m paper_1912_04050_b200.build`. "
            "There is no CPU fallback." % (os.path.basename(path), path))
    lib = ctypes.CDLL(path)
    for name, (res, args) in SYMBOLS.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


def load() -> ctypes.CDLL:
    """Load the CUDA library; fails loudly if it is not built."""
    global _lib
    if _lib is None:
        _lib = _open(LIB_PATH)
    return _lib


def use_library(path: str = None) -> None:
    """Route every call of this module through another build of the library with the same
    ABI (the checked build, libbenes_debug.so); None switches back to libbenes.so."""
    global _lib
    _lib = _open(path or LIB_PATH)


def status_string(status: int) -> str:
    return load().benes_status_string(status).decode()


def _check(status: int, what: str) -> None:
    if status != BENES_OK:
        raise BenesError(status, what)


def _dev_ptr(t: torch.Tensor, what: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError("%s must be a contiguous CUDA tensor" % what)
    return t.data_ptr()


def _host_ptr(t, what: str) -> int:
    if isinstance(t, torch.Tensor):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError("%s must be a contiguous host tensor" % what)
        return t.data_ptr()
    return t.ctypes.data        # numpy array


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def benes_switch_words(log2n: int, batch: int) -> int:
    return load().benes_switch_words(log2n, batch)


def benes_route_workspace_bytes(log2n: int, batch: int) -> int:
    return load().benes_route_workspace_bytes(log2n, batch)


def benes_apply_workspace_bytes(elem_bytes: int, log2n: int, batch: int) -> int:
    return load().benes_apply_workspace_bytes(elem_bytes, log2n, batch)


def benes_route(perm: torch.Tensor, log2n: int, batch: int, switch_bits: torch.Tensor, stream=None) -> None:
    _check(load().benes_route(_dev_ptr(perm, "perm"), log2n, batch,
                              _dev_ptr(switch_bits, "switch_bits"), _stream(stream)), "benes_route")


def benes_apply(switch_bits: torch.Tensor, inp: torch.Tensor, out: torch.Tensor, log2n: int, batch: int,
                stream=None) -> None:
    _check(load().benes_apply(_dev_ptr(switch_bits, "switch_bits"), _dev_ptr(inp, "in"),
                              _dev_ptr(out, "out"), log2n, batch, _stream(stream)), "benes_apply")


def benes_apply_ex(switch_bits: torch.Tensor, inp: torch.Tensor, out: torch.Tensor, elem_bytes: int,
                   log2n: int, batch: int, stream=None) -> None:
    _check(load().benes_apply_ex(_dev_ptr(switch_bits, "switch_bits"), _dev_ptr(inp, "in"),
                                 _dev_ptr(out, "out"), elem_bytes, log2n, batch, _stream(stream)),
           "benes_apply_ex")


def benes_apply_static(switch_bits: torch.Tensor, inp: torch.Tensor, out: torch.Tensor, elem_bytes: int,
                       log2n: int, batch: int, stream=None) -> None:
    """benes_apply_ex without any allocation: the scratch is a fixed 4 MiB array inside the
    library, so batch * N * elem_bytes must fit in it (BenesError with BENES_ERR_TOO_LARGE if not)."""
    _check(load().benes_apply_static(_dev_ptr(switch_bits, "switch_bits"), _dev_ptr(inp, "in"),
                                     _dev_ptr(out, "out"), elem_bytes, log2n, batch, _stream(stream)),
           "benes_apply_static")


def benes_export_butterfly(switch_bits: torch.Tensor, butterfly_bits: torch.Tensor, log2n: int, batch: int,
                           stream=None) -> None:
    _check(load().benes_export_butterfly(_dev_ptr(switch_bits, "switch_bits"),
                                         _dev_ptr(butterfly_bits, "butterfly_bits"), log2n, batch,
                                         _stream(stream)), "benes_export_butterfly")


def benes_padded_log2n(n_elems: int) -> int:
    return load().benes_padded_log2n(n_elems)


def benes_route_padded(perm: torch.Tensor, n_elems: int, batch: int, switch_bits: torch.Tensor, stream=None) -> None:
    _check(load().benes_route_padded(_dev_ptr(perm, "perm"), n_elems, batch,
                                     _dev_ptr(switch_bits, "switch_bits"), _stream(stream)),
           "benes_route_padded")


def benes_apply_padded(switch_bits: torch.Tensor, inp: torch.Tensor, out: torch.Tensor, elem_bytes: int,
                       n_elems: int, batch: int, stream=None) -> None:
    _check(load().benes_apply_padded(_dev_ptr(switch_bits, "switch_bits"), _dev_ptr(inp, "in"),
                                     _dev_ptr(out, "out"), elem_bytes, n_elems, batch, _stream(stream)),
           "benes_apply_padded")


def benes_route_host(perm_host, log2n: int, batch: int, switch_bits_host, stream=None) -> None:
    _check(load().benes_route_host(_host_ptr(perm_host, "perm_host"), log2n, batch,
                                   _host_ptr(switch_bits_host, "switch_bits_host"), _stream(stream)),
           "benes_route_host")


def benes_apply_host(switch_bits_host, in_host, out_host, elem_bytes: int, log2n: int, batch: int,
                     stream=None) -> None:
    _check(load().benes_apply_host(_host_ptr(switch_bits_host, "switch_bits_host"),
                                   _host_ptr(in_host, "in_host"), _host_ptr(out_host, "out_host"),
                                   elem_bytes, log2n, batch, _stream(stream)), "benes_apply_host")


def benes_route_apply_host(perm_host, in_host, out_host, elem_bytes: int, log2n: int, batch: int,
                           switch_bits_host=None, stream=None) -> None:
    bits = None if switch_bits_host is None else _host_ptr(switch_bits_host, "switch_bits_host")
    _check(load().benes_route_apply_host(_host_ptr(perm_host, "perm_host"), _host_ptr(in_host, "in_host"),
                                         _host_ptr(out_host, "out_host"), elem_bytes, log2n, batch, bits,
                                         _stream(stream)), "benes_route_apply_host")


class Plan:
    """A captured route (+ apply) on fixed buffers; launch() replays it with one call."""

    def __init__(self, perm: torch.Tensor, log2n: int, batch: int, switch_bits: torch.Tensor,
                 inp: torch.Tensor = None, out: torch.Tensor = None, elem_bytes: int = 0):
        self._h = _vp(None)
        self._keep = (perm, switch_bits, inp, out)          # the plan points into these
        _check(load().benes_plan_create(ctypes.byref(self._h), _dev_ptr(perm, "perm"), log2n, batch,
                                        _dev_ptr(switch_bits, "switch_bits"),
                                        None if inp is None else _dev_ptr(inp, "in"),
                                        None if out is None else _dev_ptr(out, "out"), elem_bytes),
               "benes_plan_create")

    def launch(self, stream=None) -> None:
        _check(load().benes_plan_launch(self._h, _stream(stream)), "benes_plan_launch")

    def destroy(self) -> None:
        if self._h:
            load().benes_plan_destroy(self._h)
            self._h = _vp(None)

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def benes_set_workspace(buf, nbytes: int = 0) -> None:
    if buf is None:
        _check(load().benes_set_workspace(None, 0), "benes_set_workspace")
    else:
        _check(load().benes_set_workspace(_dev_ptr(buf, "workspace"),
                                          nbytes or buf.numel() * buf.element_size()),
               "benes_set_workspace")


def benes_release_workspace() -> None:
    _check(load().benes_release_workspace(), "benes_release_workspace")


def benes_validate_perm(perm: torch.Tensor, log2n: int, batch: int, stream=None) -> bool:
    """True if every row is a permutation; False if not; raises on other errors."""
    rc = load().benes_validate_perm(_dev_ptr(perm, "perm"), log2n, batch, _stream(stream))
    if rc == BENES_ERR_NOT_PERMUTATION:
        return False
    _check(rc, "benes_validate_perm")
    return True


def benes_launch_count() -> int:
    return load().benes_launch_count()


PROFILE_KINDS = 12
OPT_SAMPLE_LOG2K = 0
OPT_WALK_CAP = 1
OPT_APPLY_FUSED = 2
OPT_INVERSE_PARTITIONED = 3
OPT_CHUNK_LOG2 = 4
OPT_CLUSTER = 5
OPT_WALK_PAIRS = 6


def benes_set_option(key: int, value: int) -> None:
    _check(load().benes_set_option(key, value), "benes_set_option")


def benes_get_option(key: int) -> int:
    v = load().benes_get_option(key)
    if v < 0:
        _check(v, "benes_get_option")
    return v


def benes_profile_enable(on: bool) -> None:
    _check(load().benes_profile_enable(1 if on else 0), "benes_profile_enable")


def benes_profile_reset() -> None:
    _check(load().benes_profile_reset(), "benes_profile_reset")


def benes_profile_read(kind: int):
    """(launches, milliseconds) of one kernel kind since the last reset."""
    n, ms = ctypes.c_ulonglong(0), ctypes.c_double(0.0)
    _check(load().benes_profile_read(kind, ctypes.byref(n), ctypes.byref(ms)), "benes_profile_read")
    return n.value, ms.value


def benes_profile_spans():
    """[(kind name, launches, milliseconds), ...] of every timed group since the last reset."""
    out, i = [], 0
    k, n, ms = ctypes.c_int(0), ctypes.c_ulonglong(0), ctypes.c_double(0.0)
    while load().benes_profile_span(i, ctypes.byref(k), ctypes.byref(n), ctypes.byref(ms)) == BENES_OK:
        out.append((benes_profile_kind_name(k.value), n.value, ms.value))
        i += 1
    return out


def benes_profile_kind_name(kind: int) -> str:
    return load().benes_profile_kind_name(kind).decode()


def benes_shard_batch(batch: int, world: int, rank: int):
    """(first, count): the contiguous slice of a batch that rank `rank` of `world` routes."""
    first, count = _i(0), _i(0)
    _check(load().benes_shard_batch(batch, world, rank, ctypes.byref(first), ctypes.byref(count)),
           "benes_shard_batch")
    return first.value, count.value


def benes_probe_random_access(table: torch.Tensor, log2_records: int, record_bytes: int, mode: int, ops: int,
                              sink: torch.Tensor, stream=None) -> None:
    _check(load().benes_probe_random_access(_dev_ptr(table, "table"), log2_records, record_bytes, mode, ops,
                                            _dev_ptr(sink, "sink"), _stream(stream)), "benes_probe_random_access")


def benes_debug_build() -> bool:
    return bool(load().benes_debug_build())


def benes_debug_guard_hits(clear: bool = True):
    """(events, "file:line" of one of them): index guards that had to change a value."""
    hits = ctypes.c_ulonglong(0)
    where = ctypes.create_string_buffer(128)
    _check(load().benes_debug_guard_hits(ctypes.byref(hits), where, 128, 1 if clear else 0),
           "benes_debug_guard_hits")
    return hits.value, where.value.decode()


def benes_fused_log2m() -> int:
    return load().benes_fused_log2m()


# ---- small conveniences that only allocate outputs -------------------------------------------
def route(perm: torch.Tensor, stream=None) -> torch.Tensor:
    """perm: (N,) or (batch, N) CUDA tensor holding uint32 values (dtype int32 or uint32).
    Returns the switch bits as an int32 tensor of shape ([batch,] 2n-1, W)."""
    N = perm.shape[-1]
    log2n = N.bit_length() - 1
    if N < 2 or (1 << log2n) != N:
        raise ValueError("N must be a power of two >= 2")
    batch = perm.numel() // N
    W = max(1, N // 64)
    bits = torch.empty(perm.shape[:-1] + (2 * log2n - 1, W), dtype=torch.int32, device=perm.device)
    benes_route(perm, log2n, batch, bits, stream)
    return bits


def apply(switch_bits: torch.Tensor, x: torch.Tensor, stream=None) -> torch.Tensor:
    """Push payload x ((N,) or (batch, N), 4- or 8-byte dtype) through the network."""
    N = x.shape[-1]
    log2n = N.bit_length() - 1
    batch = x.numel() // N
    out = torch.empty_like(x)
    benes_apply_ex(switch_bits, x, out, x.element_size(), log2n, batch, stream)
    return out
