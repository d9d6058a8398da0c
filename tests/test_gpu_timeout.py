"""GPU: the bounded look-back wait.  A compression tile that never publishes its
descriptor makes the tiles behind it wait; the wait is bounded, so the kernel
returns normally with CDMA_ERR_TIMEOUT, having written nothing beyond its buffers,
and the next ordinary call works.  The silent tile comes from a test hook of the
library (exported, not part of the public header); nothing here faults, traps or
spins without limit."""
import ctypes
import time

import numpy as np
import pytest
import torch

from oracle import zvc_c
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu


def stalled(codec, x, stall_tile, limit_ns):
    fn = B.lib().cdma_test_compress_stalled
    fn.restype = ctypes.c_int64
    fn.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p,
                   ctypes.c_void_p, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_uint32, ctypes.c_uint64]
    return int(fn(x.data_ptr(), x.numel(), codec.code, codec.payload.data_ptr(), codec.cap, codec.table.data_ptr(),
                  codec.ws.data_ptr(), codec.ws_bytes, None, stall_tile, limit_ns))


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
@pytest.mark.parametrize("stall_tile", [0, 3, 57])
def test_a_silent_tile_ends_in_timeout_not_in_a_hang(dtype, stall_tile):
    n = 100 * 16384 + 123                                    # about 100 tiles (200 of 4-byte elements)
    x = wl.iid_relu_like((n,), 0.4, seed=900 + stall_tile, device="cuda", dtype=dtype, floor=2.0 ** -10)
    codec = DeviceCodec(n, dtype)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    r = stalled(codec, x, stall_tile, 1_000_000)             # waits give up after 1 ms
    dt = time.perf_counter() - t0
    assert r == -B.ERR_TIMEOUT, B.status_string(r)
    assert dt < 1.0                                          # nothing waited anywhere near the default 2 s
    assert codec.canaries_intact()
    # the same buffers, workspace included, serve an ordinary call right away
    c = codec.compress(x)
    want, want_table = zvc_c.compress(raw_numpy(x))
    assert c == len(want)
    assert codec.payload_numpy(c).tobytes() == want.tobytes()
    assert np.array_equal(codec.table_numpy(), want_table)
    assert codec.canaries_intact()


def test_the_hook_without_a_silent_tile_is_an_ordinary_compression():
    n = 20 * 8192 + 5
    x = wl.iid_relu_like((n,), 0.25, seed=950, device="cuda")
    codec = DeviceCodec(n, torch.float32)
    r = stalled(codec, x, 0xFFFFFFFF, 1_000_000)
    want, _ = zvc_c.compress(raw_numpy(x))
    assert r == len(want)
    assert codec.payload_numpy(r).tobytes() == want.tobytes()
    # a silent last tile is nobody's predecessor: the call still succeeds
    last = (n + 8191) // 8192 - 1
    assert stalled(codec, x, last, 1_000_000) == len(want)
