"""ctypes front end of the plain-C ZVC oracle (``zvc_oracle.c``).

TEST INFRASTRUCTURE -- see the package docstring.  Marshals numpy arrays to
the C routines; holds no arithmetic of the method itself.

The shared object is built with gcc on first use (and by ``build()``), next to
the source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "zvc_oracle.c")
_LIB = os.path.join(_HERE, "libzvc_oracle.so")
_lock = threading.Lock()
_lib = None

ERR_BAD_ARG = -1
ERR_TOO_SMALL = -5
ERR_MALFORMED = -6


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object beside its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-shared", "-fPIC",
                 "-pthread", "-o", tmp, _SRC])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        u64, u32, vp = ctypes.c_uint64, ctypes.c_uint, ctypes.c_void_p
        lib.zvc_oracle_closed_form_bytes.restype = u64
        lib.zvc_oracle_closed_form_bytes.argtypes = [u64, u64, u32]
        lib.zvc_oracle_table_entries.restype = u64
        lib.zvc_oracle_table_entries.argtypes = [u64]
        lib.zvc_oracle_compress.restype = ctypes.c_int64
        lib.zvc_oracle_compress.argtypes = [vp, u64, u32, vp, u64, vp]
        lib.zvc_oracle_decompress.restype = ctypes.c_int64
        lib.zvc_oracle_decompress.argtypes = [vp, u64, u64, u32, vp]
        lib.zvc_oracle_check_table.restype = ctypes.c_int
        lib.zvc_oracle_check_table.argtypes = [vp, u64, u64, u32, vp]
        lib.zvc_oracle_compress_mt.restype = ctypes.c_int64
        lib.zvc_oracle_compress_mt.argtypes = [vp, u64, u32, vp, u64, vp, u32]
        lib.zvc_oracle_decompress_mt.restype = ctypes.c_int64
        lib.zvc_oracle_decompress_mt.argtypes = [vp, u64, vp, u64, u32, vp, u32]
        _lib = lib
    return _lib


def _as_bytes_view(x: np.ndarray) -> np.ndarray:
    """Flat uint8 view of a C-contiguous array (no copy)."""
    if not x.flags["C_CONTIGUOUS"]:
        raise ValueError("the oracle takes tensors dense in their memory order")
    return x.reshape(-1).view(np.uint8)


def _ptr(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data) if a.size else ctypes.c_void_p(0)


def table_entries(n: int) -> int:
    return int(_load().zvc_oracle_table_entries(n))


def closed_form_bytes(n: int, nnz: int, s: int) -> int:
    return int(_load().zvc_oracle_closed_form_bytes(n, nnz, s))


def compress(x: np.ndarray, capacity: int | None = None, threads: int = 1):
    """Compress ``x`` (any dtype of 1, 2 or 4 bytes per element, memory order).

    Returns ``(payload uint8[C], table uint64[K+1])``.  With ``capacity`` given
    the destination is that many bytes and a too-small one raises
    ``BufferError``.
    """
    lib = _load()
    s = x.dtype.itemsize
    n = x.size
    raw = _as_bytes_view(x)
    cap = 4 * ((n + 31) // 32) + s * n if capacity is None else int(capacity)
    dst = np.zeros(cap, dtype=np.uint8)
    table = np.zeros(table_entries(n), dtype=np.uint64)
    if threads <= 1:
        r = lib.zvc_oracle_compress(_ptr(raw), n, s, _ptr(dst), cap, _ptr(table))
    else:
        r = lib.zvc_oracle_compress_mt(_ptr(raw), n, s, _ptr(dst), cap, _ptr(table), threads)
    if r == ERR_TOO_SMALL:
        raise BufferError("destination too small")
    if r < 0:
        raise ValueError("oracle compress failed: %d" % r)
    return dst[:r], table


def decompress(payload: np.ndarray, n: int, dtype, table: np.ndarray | None = None,
               threads: int = 1) -> np.ndarray:
    """Expand a payload back into ``n`` elements of ``dtype`` (flat array).

    The single-thread walk ignores ``table``; the threaded driver needs it.
    Raises ``ValueError`` on a malformed stream.
    """
    lib = _load()
    dtype = np.dtype(dtype)
    s = dtype.itemsize
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    out = np.empty(n, dtype=dtype)
    outb = out.view(np.uint8)
    if threads <= 1:
        r = lib.zvc_oracle_decompress(_ptr(payload), payload.size, n, s, _ptr(outb))
    else:
        if table is None:
            raise ValueError("the threaded driver needs the offset table")
        table = np.ascontiguousarray(table, dtype=np.uint64)
        r = lib.zvc_oracle_decompress_mt(_ptr(payload), payload.size, _ptr(table), n, s,
                                         _ptr(outb), threads)
    if r < 0:
        raise ValueError("malformed stream (%d)" % r)
    return out


def check_table(payload: np.ndarray, n: int, s: int, table: np.ndarray) -> bool:
    lib = _load()
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    table = np.ascontiguousarray(table, dtype=np.uint64)
    if table.size != table_entries(n):
        return False
    return lib.zvc_oracle_check_table(_ptr(payload), payload.size, n, s, _ptr(table)) == 0


def compress_into(x: np.ndarray, dst: np.ndarray, table: np.ndarray, threads: int = 1) -> int:
    """Compress into caller-provided buffers (no allocation inside the timed call).
    Returns the payload size or a negative error code."""
    lib = _load()
    raw = _as_bytes_view(x)
    s = x.dtype.itemsize
    if threads <= 1:
        return int(lib.zvc_oracle_compress(_ptr(raw), x.size, s, _ptr(dst), dst.size, _ptr(table)))
    return int(lib.zvc_oracle_compress_mt(_ptr(raw), x.size, s, _ptr(dst), dst.size, _ptr(table), threads))


def decompress_into(payload: np.ndarray, table: np.ndarray, out: np.ndarray, threads: int = 1) -> int:
    """Expand into a caller-provided array.  Returns bytes written or a negative error."""
    lib = _load()
    s = out.dtype.itemsize
    outb = out.reshape(-1).view(np.uint8)
    if threads <= 1:
        return int(lib.zvc_oracle_decompress(_ptr(payload), payload.size, out.size, s, _ptr(outb)))
    return int(lib.zvc_oracle_decompress_mt(_ptr(payload), payload.size, _ptr(table), out.size, s,
                                            _ptr(outb), threads))
