"""GPU parity of the run-length comparison codec against its numpy oracle: payload bytes,
offset table and round trip, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import rle_numpy
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import CANARY, DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu


def make(n, density, seed, run=1):
    """Random bit patterns; zeros in runs of `run` elements (run = 1: independent)."""
    rng = np.random.default_rng(seed)
    raw = rng.integers(1, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32)
    keep = np.repeat(rng.random((n + run - 1) // run) < density, run)[:n]
    raw[~keep] = 0
    return torch.from_numpy(raw.view(np.int32)).cuda().view(torch.float32), raw


def rle_compress(codec, x):
    return B.cdma_rle_compress(x.data_ptr() if codec.n else 0, codec.n, B.F32, B.NCHW, codec.payload.data_ptr(),
                               codec.cap, codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0)


def rle_decompress(codec, out, nbytes):
    return B.cdma_rle_decompress(codec.payload.data_ptr(), nbytes, codec.table.data_ptr(), codec.n, B.F32, B.NCHW,
                                 out.data_ptr() if codec.n else 0, codec.ws.data_ptr(), codec.ws_bytes, 0)


def check(x, raw):
    n = x.numel()
    codec = DeviceCodec(n, torch.float32)
    c = rle_compress(codec, x)
    assert c >= 0, B.status_string(c)
    want, want_table = rle_numpy.compress(raw)
    assert c == len(want)
    assert codec.payload_numpy(c).tobytes() == want.tobytes()
    assert np.array_equal(codec.table_numpy(), want_table)
    assert codec.canaries_intact()
    out = torch.full((n + 32,), 3.5, device="cuda")
    r = rle_decompress(codec, out, c)
    assert r == 4 * n, B.status_string(r)
    assert raw_numpy(out[:n]).tobytes() == raw.tobytes()
    assert bool((out[n:] == 3.5).all())
    return c


@pytest.mark.parametrize("n", [0, 1, 31, 32, 33, 1023, 1024, 1025, 8191, 8192, 8193, 5 * 8192 + 1024 + 17, 300_000])
def test_sizes_and_tails(n):
    for seed, (density, run) in enumerate([(0.1, 1), (0.5, 1), (0.93, 1), (0.4, 7), (0.3, 64)]):
        x, raw = make(n, density, 100 * seed + n, run)
        check(x, raw)


def test_limits_and_special_values():
    n = 3 * 8192 + 100
    check(torch.zeros(n, device="cuda"), np.zeros(n, dtype=np.uint32))                    # one token per chunk
    x, raw = make(n, 1.0, 1)
    assert check(x, raw) == 4 * n + 4 * ((n + 1023) // 1024)                                # one token + the chunk
    alt = np.zeros(n, dtype=np.uint32); alt[0::2] = 5                                       # shortest runs: 1025 words per chunk
    check(torch.from_numpy(alt.view(np.int32)).cuda().view(torch.float32), alt)
    alt = np.zeros(n, dtype=np.uint32); alt[1::2] = 5
    check(torch.from_numpy(alt.view(np.int32)).cuda().view(torch.float32), alt)
    sp = wl.special_values(5000, 9, torch.float32, device="cuda")
    check(sp, raw_numpy(sp))                                                                # -0.0, NaN, denormals are literals


def test_layout_dependence_on_clustered_activations():
    """Same elements, three memory layouts (Section VI-A, Fig. 11): the zero-value codec gives one
    size, run-length encoding does not."""
    x = wl.correlated_relu((8, 32, 28, 28), 0.3, 11, "cuda")
    sizes = {}
    for layout in ("NCHW", "NHWC", "CHWN"):
        t = wl.to_layout(x, layout).reshape(-1)
        sizes[layout] = check(t, raw_numpy(t))
    assert len(set(sizes.values())) > 1
    assert sizes["NCHW"] < sizes["NHWC"]          # zeros cluster in the image plane, not across channels


def test_errors():
    x, raw = make(4 * 8192 + 300, 0.4, 5, 3)
    n = x.numel()
    want, table = rle_numpy.compress(raw)
    # capacity
    codec = DeviceCodec(n, torch.float32, capacity=(len(want) // 2) & ~15)
    assert rle_compress(codec, x) == -B.ERR_BUFFER_TOO_SMALL
    assert codec.canaries_intact()
    assert codec.payload_numpy(codec.cap).tobytes() == want[:codec.cap].tobytes()
    # dtype
    codec = DeviceCodec(n, torch.float32)
    assert B.cdma_rle_compress(x.data_ptr(), n, B.F16, B.NCHW, codec.payload.data_ptr(), codec.cap,
                               codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0) == -B.ERR_UNSUPPORTED_DTYPE
    out = torch.zeros(n, device="cuda")

    def run(p, t, nbytes=None):
        codec = DeviceCodec(n, torch.float32)
        codec.load(p, t)
        r = rle_decompress(codec, out, len(p) if nbytes is None else nbytes)
        assert codec.canaries_intact()
        return r

    assert run(want, table) == 4 * n
    t = table.copy(); t[2] += 4
    assert run(want, t) == -B.ERR_CORRUPT_STREAM
    t = table.copy(); t[3] = t[2] - 4
    assert run(want, t) == -B.ERR_CORRUPT_STREAM
    p = want.copy(); p.view(np.uint32)[int(table[1]) // 4] += 1          # one zero too many in chunk 1's first token
    assert run(p, table) == -B.ERR_CORRUPT_STREAM
    p = want.copy(); p.view(np.uint32)[int(table[1]) // 4] = 0           # an empty token
    assert run(p, table) == -B.ERR_CORRUPT_STREAM
    assert run(want, table, nbytes=len(want) - 4) == -B.ERR_CORRUPT_STREAM
    # garbage behind a plausible table
    rng = np.random.default_rng(3)
    junk = rng.integers(0, 256, size=len(want), dtype=np.uint8)
    assert run(junk, table) in (-B.ERR_CORRUPT_STREAM, 4 * n)
