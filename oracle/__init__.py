"""Python face of the CPU oracle — TEST INFRASTRUCTURE ONLY.

Loads ``tm_oracle.cpp`` (plain single-threaded C++, see that file's header for the definitions
it writes out) through ctypes and wraps it for numpy byte arrays.  Only tests, the smoke check
and the CPU-baseline legs of the benchmark may import this package; the CUDA library and its
Python binding never do, and this package never imports them.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tm_oracle.cpp")
_LIB = os.path.join(_HERE, "libtm_oracle.so")

_u64 = ctypes.c_uint64
_u32 = ctypes.c_uint32
_p = ctypes.c_void_p
_lib = None


class OracleError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"oracle {what} failed with status {code}")
        self.code = code


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (seconds).  Building the checker is not using it."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-o", tmp, _SRC], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _configure(L: ctypes.CDLL) -> ctypes.CDLL:
    L.oracle_layout.argtypes = [_p, _u64, _u64, _p, _p, _p]
    L.oracle_checksum.argtypes = [_p, _u64, _u64, _p]
    L.oracle_pack.argtypes = [_p, _p, _u64, _u64, _p, _u64, _p]
    L.oracle_pack_range.argtypes = [_p, _p, _u64, _u64, _u64, _p]
    L.oracle_unpack.argtypes = [_p, _p, _u64, _p, _u64]
    L.oracle_shard_bounds.argtypes = [_u64, _u32, _u32, _p, _p]
    L.oracle_shard.argtypes = [_p, _p, _u64, _u32, _u32, _u32, _p, _u64, _p]
    L.oracle_shard_insert.argtypes = [_p, _p, _u64, _u32, _u32, _u32, _p, _u64, _p]
    for name in ("oracle_layout", "oracle_checksum", "oracle_pack", "oracle_pack_range",
                 "oracle_unpack", "oracle_shard_bounds", "oracle_shard", "oracle_shard_insert"):
        getattr(L, name).restype = ctypes.c_int
    return L


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = _configure(ctypes.CDLL(build()))
    return _lib


class use_library:
    """Context manager that makes every function of this module call another build of the oracle
    (used by the mutation test, which plants mistakes in copies of tm_oracle.cpp to show that the
    pins catch them)."""

    def __init__(self, path: str):
        self.path = path

    def __enter__(self):
        global _lib
        self._saved = lib()
        _lib = _configure(ctypes.CDLL(self.path))
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self._saved
        return False


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise OracleError(rc, what)


def _as_bytes(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a)
    return a.reshape(-1).view(np.uint8)


def _ptr_table(arrays: Sequence[Optional[np.ndarray]]):
    n = len(arrays)
    ptrs = (ctypes.c_void_p * n)()
    for k, a in enumerate(arrays):
        ptrs[k] = None if a is None else a.ctypes.data
    return ptrs


def _sizes(nbytes: Sequence[int]) -> np.ndarray:
    return np.asarray(list(nbytes), dtype=np.uint64)


def layout(nbytes: Sequence[int], bucket_bytes: int) -> Tuple[np.ndarray, int, int]:
    """(offsets off_k, total T, n_buckets) of the packed stream."""
    sz = _sizes(nbytes)
    off = np.zeros(len(sz), dtype=np.uint64)
    total, nb = _u64(0), _u64(0)
    _check(lib().oracle_layout(sz.ctypes.data, len(sz), bucket_bytes, off.ctypes.data,
                               ctypes.addressof(total), ctypes.addressof(nb)), "layout")
    return off, int(total.value), int(nb.value)


def checksum(data: np.ndarray, bucket_bytes: int) -> np.ndarray:
    """One checksum per bucket of `bucket_bytes` over the bytes of `data`."""
    b = _as_bytes(data)
    nb = (b.size + bucket_bytes - 1) // bucket_bytes if bucket_bytes > 0 else 0
    out = np.zeros(nb, dtype=np.uint64)
    _check(lib().oracle_checksum(b.ctypes.data if b.size else None, b.size, bucket_bytes,
                                 out.ctypes.data if nb else None), "checksum")
    return out


def pack(tensors: Sequence[np.ndarray], bucket_bytes: int,
         out: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """(packed stream bytes, per-bucket checksums) for tensors given as byte arrays."""
    tb = [_as_bytes(t) for t in tensors]
    sz = _sizes([t.size for t in tb])
    _, total, nb = layout(sz, bucket_bytes)
    if out is None:
        out = np.empty(total, dtype=np.uint8)
    cks = np.zeros(nb, dtype=np.uint64)
    ptrs = _ptr_table(tb)
    _check(lib().oracle_pack(ptrs, sz.ctypes.data, len(tb), bucket_bytes, out.ctypes.data,
                             out.size, cks.ctypes.data), "pack")
    return out[:total], cks


def pack_range(tensors: Sequence[Optional[np.ndarray]], nbytes: Sequence[int], lo: int,
               hi: int) -> np.ndarray:
    """Stream bytes [lo, hi); tensors that do not intersect the range may be None."""
    tb = [None if t is None else _as_bytes(t) for t in tensors]
    sz = _sizes(nbytes)
    out = np.empty(hi - lo, dtype=np.uint8)
    ptrs = _ptr_table(tb)
    _check(lib().oracle_pack_range(ptrs, sz.ctypes.data, len(tb), lo, hi,
                                   out.ctypes.data if out.size else None), "pack_range")
    return out


def unpack(stream: np.ndarray, nbytes: Sequence[int]) -> List[np.ndarray]:
    """Tensors (as byte arrays) cut back out of a packed stream."""
    s = _as_bytes(stream)
    sz = _sizes(nbytes)
    outs = [np.empty(int(n), dtype=np.uint8) for n in sz]
    ptrs = _ptr_table(outs)
    _check(lib().oracle_unpack(ptrs, sz.ctypes.data, len(outs), s.ctypes.data, s.size), "unpack")
    return outs


def shard_bounds(n_elems: int, r: int, D: int) -> Tuple[int, int]:
    lo, hi = _u64(0), _u64(0)
    _check(lib().oracle_shard_bounds(n_elems, r, D, ctypes.addressof(lo), ctypes.addressof(hi)),
           "shard_bounds")
    return int(lo.value), int(hi.value)


def shard(tensors: Sequence[Optional[np.ndarray]], nbytes: Sequence[int], elem_size: int, r: int,
          D: int) -> np.ndarray:
    """Bytes of shard r of D of the plane; tensors outside the shard may be None."""
    tb = [None if t is None else _as_bytes(t) for t in tensors]
    sz = _sizes(nbytes)
    n_elems = int(sz.sum()) // elem_size if elem_size in (2, 4, 8) else 0
    cap = 0
    if elem_size in (2, 4, 8) and D > 0 and r < D:
        lo, hi = (r * n_elems) // D, ((r + 1) * n_elems) // D  # capacity only; bounds come from C++
        cap = (hi - lo) * elem_size
    out = np.empty(cap, dtype=np.uint8)
    got = _u64(0)
    ptrs = _ptr_table(tb)
    _check(lib().oracle_shard(ptrs, sz.ctypes.data, len(tb), elem_size, r, D,
                              out.ctypes.data if cap else None, cap, ctypes.addressof(got)),
           "shard")
    return out[: int(got.value) * elem_size]


def shard_insert(tensors: Sequence[Optional[np.ndarray]], nbytes: Sequence[int], elem_size: int, r: int,
                 D: int, data: np.ndarray) -> int:
    """Writes `data` (shard r of D) into the plane's tensors IN PLACE (uint8 arrays); tensors the
    shard does not touch may be None.  Returns the number of elements written."""
    for t in tensors:
        assert t is None or (t.dtype == np.uint8 and t.flags.c_contiguous and t.flags.writeable)
    sz = _sizes(nbytes)
    d = _as_bytes(data)
    got = _u64(0)
    ptrs = _ptr_table(tensors)
    _check(lib().oracle_shard_insert(ptrs, sz.ctypes.data, len(tensors), elem_size, r, D,
                                     d.ctypes.data if d.size else None, d.size, ctypes.addressof(got)),
           "shard_insert")
    return int(got.value)
