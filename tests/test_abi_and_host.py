"""CPU-only checks of the C-ABI library: every symbol the header declares is
exported, and the host-side size arithmetic and argument validation behave as
documented.  No kernel is launched here."""
import ctypes
import os
import re

import pytest

from paper_1705_01626_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cdma.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cdma_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_primary_entry_points():
    names = declared_functions()
    for must in ("cdma_zvc_compress", "cdma_zvc_decompress", "cdma_offload", "cdma_prefetch"):
        assert must in names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(B._build.ensure_built())
    for name in declared_functions():
        assert hasattr(lib, name), "libcdma.so lacks %s" % name


def test_binding_covers_every_declared_symbol():
    assert set(B.exported_names()) == set(declared_functions())
    B.lib()      # resolves all of them with their signatures


def test_size_arithmetic():
    assert B.cdma_dtype_size(B.F32) == 4 and B.cdma_dtype_size(B.F16) == 2 and B.cdma_dtype_size(B.BF16) == 2
    assert B.cdma_dtype_size(7) == 0
    # worst case: one mask per window and every element kept, rounded up to 16
    for n in (0, 1, 31, 32, 33, 1024, 1025, 205520896, 1 << 29):
        for dt, s in ((B.F32, 4), (B.F16, 2)):
            raw = 4 * ((n + 31) // 32) + s * n
            got = B.cdma_zvc_max_compressed_bytes(n, dt)
            assert got == (raw + 15) // 16 * 16
        assert B.cdma_zvc_table_entries(n) == (n + 1023) // 1024 + 1
        w = B.cdma_zvc_workspace_bytes(n, B.F32)
        assert w % 256 == 0 and w >= 32
    assert B.cdma_zvc_max_compressed_bytes(10, 9) == 0
    # a full window of non-zeros costs 132 bytes: 3.125 % more than the 128 it held
    assert 4 * 1 + 4 * 32 == 132


def test_status_strings():
    assert B.status_string(0) == "ok"
    assert "corrupt" in B.status_string(-B.ERR_CORRUPT_STREAM)
    assert "unknown" in B.status_string(99)


def test_argument_validation_needs_no_device():
    buf = (ctypes.c_uint8 * 4096)()
    base = (ctypes.addressof(buf) + 255) // 256 * 256          # host memory stands in: nothing is launched
    args = dict(d_src=base, n=64, dtype=B.F32, layout=B.NCHW, d_dst=base + 1024, dst_capacity=512,
                d_table=base + 2048, d_workspace=base + 2560, workspace_bytes=256)
    assert B.cdma_zvc_compress(**{**args, "dtype": 5}) == -B.ERR_UNSUPPORTED_DTYPE
    assert B.cdma_zvc_compress(**{**args, "layout": 3}) == -B.ERR_UNSUPPORTED_LAYOUT
    assert B.cdma_zvc_compress(**{**args, "d_src": base + 2}) == -B.ERR_ALIGNMENT
    assert B.cdma_zvc_compress(**{**args, "d_table": base + 2052}) == -B.ERR_ALIGNMENT
    assert B.cdma_zvc_compress(**{**args, "workspace_bytes": 8}) == -B.ERR_BUFFER_TOO_SMALL
    assert B.cdma_zvc_compress(**{**args, "d_workspace": 0}) == -B.ERR_INVALID_ARG
    assert B.cdma_zvc_compress(**{**args, "d_dst": base + 128}) == -B.ERR_INVALID_ARG      # overlaps the source
    assert B.cdma_zvc_compress(**{**args, "n": 1 << 41}) == -B.ERR_INVALID_ARG
    dargs = dict(d_src=base + 1024, src_bytes=8 + 4 * 64, d_table=base + 2048, n=64, dtype=B.F32, layout=B.NCHW,
                 d_dst=base, d_workspace=base + 2560, workspace_bytes=256)
    # payload sizes the format cannot produce are refused up front
    assert B.cdma_zvc_decompress(**{**dargs, "src_bytes": 4}) == -B.ERR_CORRUPT_STREAM
    assert B.cdma_zvc_decompress(**{**dargs, "src_bytes": 8 + 4 * 64 + 4}) == -B.ERR_CORRUPT_STREAM
    assert B.cdma_zvc_decompress(**{**dargs, "src_bytes": 10}) == -B.ERR_CORRUPT_STREAM
    assert B.cdma_zvc_decompress(**{**dargs, "dtype": -1}) == -B.ERR_UNSUPPORTED_DTYPE
    assert B.cdma_offload(None, base, 64, B.F32, B.NCHW, 0)[0] == -B.ERR_INVALID_ARG
    assert B.cdma_ctx_synchronize(None) == B.ERR_INVALID_ARG
