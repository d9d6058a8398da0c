"""Thin ctypes binding of ``libcdma.so``: same names as the C ABI, argument
marshalling only.  Every step of the codec runs in the library's CUDA kernels.

Tensors are passed as raw device pointers (``tensor.data_ptr()``), streams as
the integer handle of a ``torch.cuda.Stream`` (``stream.cuda_stream``).  There
is no CPU implementation behind these calls: if the library cannot be loaded
(or built with nvcc) the import of this module's functions fails loudly.
"""
from __future__ import annotations

import ctypes
from ctypes import POINTER, c_char_p, c_int, c_int64, c_uint32, c_uint64, c_void_p

from . import _build

OK = 0
ERR_INVALID_ARG = 1
ERR_UNSUPPORTED_DTYPE = 2
ERR_UNSUPPORTED_LAYOUT = 3
ERR_ALIGNMENT = 4
ERR_BUFFER_TOO_SMALL = 5
ERR_CORRUPT_STREAM = 6
ERR_TIMEOUT = 7
ERR_CUDA = 8
ERR_OUT_OF_MEMORY = 9
ERR_BAD_TICKET = 10

F32, F16, BF16, U8 = 0, 1, 2, 3
NCHW, NHWC, CHWN = 0, 1, 2
LAYOUT_CODES = {"NCHW": NCHW, "NHWC": NHWC, "CHWN": CHWN}

WINDOW = 32
CHUNK = 1024


class cdma_ticket(ctypes.Structure):
    _fields_ = [("id", c_uint64)]


class CdmaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s failed: %s (status %d)" % (where, status_string(status), status))


_SIGNATURES = {
    "cdma_status_string": (c_char_p, [c_int]),
    "cdma_dtype_size": (c_uint32, [c_int]),
    "cdma_zvc_max_compressed_bytes": (c_uint64, [c_uint64, c_int]),
    "cdma_zvc_table_entries": (c_uint64, [c_uint64]),
    "cdma_zvc_workspace_bytes": (c_uint64, [c_uint64, c_int]),
    "cdma_zvc_compress": (c_int64, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64, c_void_p,
                                    c_void_p, c_uint64, c_void_p]),
    "cdma_zvc_compress_async": (c_int, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64, c_void_p,
                                        c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_zvc_relu_compress": (c_int64, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_void_p, c_uint64, c_void_p,
                                         c_void_p, c_uint64, c_void_p]),
    "cdma_zvc_relu_compress_async": (c_int, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_void_p, c_uint64, c_void_p,
                                             c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_zvc_compress_static_ws": (c_int64, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64, c_void_p,
                                              c_void_p]),
    "cdma_zvc_decompress": (c_int64, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p,
                                      c_void_p, c_uint64, c_void_p]),
    "cdma_zvc_decompress_async": (c_int, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p,
                                          c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_zvc_relu_backward": (c_int64, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p, c_void_p,
                                         c_void_p, c_uint64, c_void_p]),
    "cdma_zvc_relu_backward_async": (c_int, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p, c_void_p,
                                             c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_rle_compress": (c_int64, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64, c_void_p,
                                    c_void_p, c_uint64, c_void_p]),
    "cdma_rle_compress_async": (c_int, [c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64, c_void_p,
                                        c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_rle_decompress": (c_int64, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p,
                                      c_void_p, c_uint64, c_void_p]),
    "cdma_rle_decompress_async": (c_int, [c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int, c_void_p,
                                          c_void_p, c_uint64, c_void_p, c_void_p]),
    "cdma_ctx_create": (c_int, [c_uint64, c_uint64, POINTER(c_void_p)]),
    "cdma_ctx_destroy": (c_int, [c_void_p]),
    "cdma_offload": (c_int64, [c_void_p, c_void_p, c_uint64, c_int, c_int, c_void_p, POINTER(cdma_ticket)]),
    "cdma_offload_async": (c_int, [c_void_p, c_void_p, c_uint64, c_int, c_int, c_void_p, POINTER(cdma_ticket)]),
    "cdma_prefetch": (c_int64, [c_void_p, cdma_ticket, c_void_p, c_void_p]),
    "cdma_prefetch_async": (c_int, [c_void_p, cdma_ticket, c_void_p, c_void_p]),
    "cdma_offload_direct": (c_int64, [c_void_p, c_void_p, c_uint64, c_int, c_int, c_void_p, POINTER(cdma_ticket)]),
    "cdma_prefetch_direct": (c_int64, [c_void_p, cdma_ticket, c_void_p, c_void_p]),
    "cdma_ctx_synchronize": (c_int, [c_void_p]),
    "cdma_ticket_info": (c_int, [c_void_p, cdma_ticket, POINTER(c_uint64), POINTER(c_uint64)]),
    "cdma_ticket_host_view": (c_int, [c_void_p, cdma_ticket, POINTER(c_void_p), POINTER(c_void_p)]),
    "cdma_zvc_compress_host": (c_int64, [c_void_p, c_void_p, c_uint64, c_int, c_int, c_void_p, c_uint64,
                                         c_void_p]),
    "cdma_zvc_decompress_host": (c_int64, [c_void_p, c_void_p, c_uint64, c_void_p, c_uint64, c_int, c_int,
                                           c_void_p]),
    "cdma_time_next_kernel": (None, [c_void_p, c_void_p]),
    "cdma_kernel_launch_count": (c_uint64, []),
}

_lib = None


def exported_names():
    return sorted(_SIGNATURES)


def library_path() -> str:
    return _build.LIB_PATH


def lib():
    """Load (building first if the sources are newer) the CUDA library."""
    global _lib
    if _lib is None:
        path = _build.ensure_built()
        handle = ctypes.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)      # AttributeError if the library lacks a symbol
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().cdma_status_string(int(status)).decode()


def _vp(x):
    return c_void_p(int(x)) if x else c_void_p(0)


def cdma_dtype_size(dtype: int) -> int:
    return int(lib().cdma_dtype_size(dtype))


def cdma_zvc_max_compressed_bytes(n: int, dtype: int) -> int:
    return int(lib().cdma_zvc_max_compressed_bytes(n, dtype))


def cdma_zvc_table_entries(n: int) -> int:
    return int(lib().cdma_zvc_table_entries(n))


def cdma_zvc_workspace_bytes(n: int, dtype: int) -> int:
    return int(lib().cdma_zvc_workspace_bytes(n, dtype))


def cdma_zvc_compress(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, d_workspace,
                      workspace_bytes, cuda_stream=0) -> int:
    """Returns the payload size C, or a negative status."""
    return int(lib().cdma_zvc_compress(_vp(d_src), n, dtype, layout, _vp(d_dst), dst_capacity,
                                       _vp(d_table), _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_zvc_compress_async(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, d_workspace,
                            workspace_bytes, cuda_stream, h_result) -> int:
    return int(lib().cdma_zvc_compress_async(_vp(d_src), n, dtype, layout, _vp(d_dst), dst_capacity,
                                             _vp(d_table), _vp(d_workspace), workspace_bytes,
                                             _vp(cuda_stream), _vp(h_result)))


def cdma_rle_compress(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, d_workspace,
                      workspace_bytes, cuda_stream=0) -> int:
    """Run-length comparison codec (4-byte elements).  Returns the payload size C, or a negative status."""
    return int(lib().cdma_rle_compress(_vp(d_src), n, dtype, layout, _vp(d_dst), dst_capacity, _vp(d_table),
                                       _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_rle_compress_async(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, d_workspace,
                            workspace_bytes, cuda_stream, h_result) -> int:
    return int(lib().cdma_rle_compress_async(_vp(d_src), n, dtype, layout, _vp(d_dst), dst_capacity,
                                             _vp(d_table), _vp(d_workspace), workspace_bytes,
                                             _vp(cuda_stream), _vp(h_result)))


def cdma_rle_decompress(d_src, src_bytes, d_table, n, dtype, layout, d_dst, d_workspace,
                        workspace_bytes, cuda_stream=0) -> int:
    return int(lib().cdma_rle_decompress(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout, _vp(d_dst),
                                         _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_rle_decompress_async(d_src, src_bytes, d_table, n, dtype, layout, d_dst, d_workspace,
                              workspace_bytes, cuda_stream, h_result) -> int:
    return int(lib().cdma_rle_decompress_async(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout,
                                               _vp(d_dst), _vp(d_workspace), workspace_bytes,
                                               _vp(cuda_stream), _vp(h_result)))


def cdma_zvc_relu_compress(d_src, n, dtype, layout, d_relu_out, d_dst, dst_capacity, d_table, d_workspace,
                           workspace_bytes, cuda_stream=0) -> int:
    """y = max(x, 0) and its compression in one pass; d_relu_out (may be 0) receives the dense y.
    Returns the payload size C, or a negative status."""
    return int(lib().cdma_zvc_relu_compress(_vp(d_src), n, dtype, layout, _vp(d_relu_out), _vp(d_dst), dst_capacity,
                                            _vp(d_table), _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_zvc_relu_compress_async(d_src, n, dtype, layout, d_relu_out, d_dst, dst_capacity, d_table, d_workspace,
                                 workspace_bytes, cuda_stream, h_result) -> int:
    return int(lib().cdma_zvc_relu_compress_async(_vp(d_src), n, dtype, layout, _vp(d_relu_out), _vp(d_dst),
                                                  dst_capacity, _vp(d_table), _vp(d_workspace), workspace_bytes,
                                                  _vp(cuda_stream), _vp(h_result)))


def cdma_zvc_compress_static_ws(d_src, n, dtype, layout, d_dst, dst_capacity, d_table, cuda_stream=0) -> int:
    """Compression without a caller-provided workspace, for callers that cannot
    allocate device memory (an eviction path, a plug-in that owns no buffers).
    Uses the library's built-in fixed workspace: at most 2**28 elements, and
    calls on one device must not overlap in time.  Returns C or a negative status."""
    return int(lib().cdma_zvc_compress_static_ws(_vp(d_src), n, dtype, layout, _vp(d_dst), dst_capacity,
                                                 _vp(d_table), _vp(cuda_stream)))


def cdma_zvc_decompress(d_src, src_bytes, d_table, n, dtype, layout, d_dst, d_workspace,
                        workspace_bytes, cuda_stream=0) -> int:
    """Returns n*s, or a negative status."""
    return int(lib().cdma_zvc_decompress(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout,
                                         _vp(d_dst), _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_zvc_decompress_async(d_src, src_bytes, d_table, n, dtype, layout, d_dst, d_workspace,
                              workspace_bytes, cuda_stream, h_result) -> int:
    return int(lib().cdma_zvc_decompress_async(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout,
                                               _vp(d_dst), _vp(d_workspace), workspace_bytes,
                                               _vp(cuda_stream), _vp(h_result)))


def cdma_zvc_relu_backward(d_src, src_bytes, d_table, n, dtype, layout, d_dy, d_dx, d_workspace, workspace_bytes,
                           cuda_stream=0) -> int:
    """dx = dy where the compressed tensor's element is non-zero, else 0, from the masks alone.
    Returns n*s, or a negative status."""
    return int(lib().cdma_zvc_relu_backward(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout, _vp(d_dy), _vp(d_dx),
                                            _vp(d_workspace), workspace_bytes, _vp(cuda_stream)))


def cdma_zvc_relu_backward_async(d_src, src_bytes, d_table, n, dtype, layout, d_dy, d_dx, d_workspace, workspace_bytes,
                                 cuda_stream, h_result) -> int:
    return int(lib().cdma_zvc_relu_backward_async(_vp(d_src), src_bytes, _vp(d_table), n, dtype, layout, _vp(d_dy),
                                                  _vp(d_dx), _vp(d_workspace), workspace_bytes, _vp(cuda_stream),
                                                  _vp(h_result)))


def cdma_ctx_create(pinned_bytes: int, device_staging_bytes: int):
    """Returns an opaque context handle; raises CdmaError on failure."""
    out = c_void_p(0)
    st = lib().cdma_ctx_create(pinned_bytes, device_staging_bytes, ctypes.byref(out))
    if st != OK:
        raise CdmaError(st, "cdma_ctx_create")
    return out


def cdma_ctx_destroy(ctx) -> int:
    return int(lib().cdma_ctx_destroy(ctx))


def cdma_offload(ctx, d_src, n, dtype, layout, compute_stream=0):
    """Returns (C or negative status, ticket)."""
    t = cdma_ticket(0)
    r = lib().cdma_offload(ctx, _vp(d_src), n, dtype, layout, _vp(compute_stream), ctypes.byref(t))
    return int(r), t


def cdma_offload_async(ctx, d_src, n, dtype, layout, compute_stream=0):
    """Enqueue compression and the copy to the pinned pool without waiting.  Returns (status, ticket)."""
    t = cdma_ticket(0)
    st = lib().cdma_offload_async(ctx, _vp(d_src), n, dtype, layout, _vp(compute_stream), ctypes.byref(t))
    return int(st), t


def cdma_prefetch(ctx, ticket, d_dst, compute_stream=0) -> int:
    return int(lib().cdma_prefetch(ctx, ticket, _vp(d_dst), _vp(compute_stream)))


def cdma_prefetch_async(ctx, ticket, d_dst, compute_stream=0) -> int:
    return int(lib().cdma_prefetch_async(ctx, ticket, _vp(d_dst), _vp(compute_stream)))


def cdma_offload_direct(ctx, d_src, n, dtype, layout, compute_stream=0):
    """Compress straight into the pinned pool (no staging, no second copy).  Returns (C or negative status, ticket)."""
    t = cdma_ticket(0)
    r = lib().cdma_offload_direct(ctx, _vp(d_src), n, dtype, layout, _vp(compute_stream), ctypes.byref(t))
    return int(r), t


def cdma_prefetch_direct(ctx, ticket, d_dst, compute_stream=0) -> int:
    """Decompress straight from the pinned pool.  Returns n*s or a negative status."""
    return int(lib().cdma_prefetch_direct(ctx, ticket, _vp(d_dst), _vp(compute_stream)))


def cdma_ctx_synchronize(ctx) -> int:
    return int(lib().cdma_ctx_synchronize(ctx))


def cdma_ticket_info(ctx, ticket):
    """Returns (status, payload_bytes, n)."""
    c, n = c_uint64(0), c_uint64(0)
    st = lib().cdma_ticket_info(ctx, ticket, ctypes.byref(c), ctypes.byref(n))
    return int(st), int(c.value), int(n.value)


def cdma_ticket_host_view(ctx, ticket):
    """Returns (status, host address of the payload, host address of the table)."""
    hp, ht = c_void_p(0), c_void_p(0)
    st = lib().cdma_ticket_host_view(ctx, ticket, ctypes.byref(hp), ctypes.byref(ht))
    return int(st), hp.value or 0, ht.value or 0


def cdma_zvc_compress_host(ctx, h_src, n, dtype, layout, h_dst, dst_capacity, h_table) -> int:
    return int(lib().cdma_zvc_compress_host(ctx, _vp(h_src), n, dtype, layout, _vp(h_dst), dst_capacity,
                                            _vp(h_table)))


def cdma_zvc_decompress_host(ctx, h_src, src_bytes, h_table, n, dtype, layout, h_dst) -> int:
    return int(lib().cdma_zvc_decompress_host(ctx, _vp(h_src), src_bytes, _vp(h_table), n, dtype, layout,
                                              _vp(h_dst)))


def cdma_time_next_kernel(start_event, stop_event) -> None:
    """Bracket the next codec kernel launch of this thread with the two cudaEvent_t handles
    (e.g. ``torch.cuda.Event(enable_timing=True).cuda_event`` after a first ``record()``)."""
    lib().cdma_time_next_kernel(_vp(start_event), _vp(stop_event))


def cdma_kernel_launch_count() -> int:
    return int(lib().cdma_kernel_launch_count())
