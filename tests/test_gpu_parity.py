"""GPU parity: the CUDA codec, called through the C ABI, against the CPU oracle.

Integer / byte work throughout, so the bar is bit-exact (tolerance 0): payload
bytes, offset table and the decompressed tensor, -0.0 and NaN patterns included.
"""
import os

import numpy as np
import pytest
import torch

from oracle import zvc_c, zvc_numpy
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import CANARY, DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu

TILE = 8 * 1024      # elements one CTA compresses (4-byte elements; twice that for 2-byte)
SIZES = [0, 1, 31, 32, 33, 63, 64, 65, 1023, 1024, 1025, 2047, 2048, 2049,
         3072, 4095, 4096, 4097, 5120,        # around the four-chunk groups of the narrow-element decoder
         TILE - 1, TILE, TILE + 1, 32 * 1024 - 1, 32 * 1024 + 1,
         5 * TILE + 1024 + 17, 40 * TILE + 999]


def make(n, density, seed, dtype):
    it = {torch.float32: np.uint32, torch.float16: np.uint16, torch.uint8: np.uint8}[dtype]
    rng = np.random.default_rng(seed)
    raw = rng.integers(1, np.iinfo(it).max, size=n, dtype=it, endpoint=True)
    raw[rng.random(n) >= density] = 0
    t = torch.from_numpy(raw.view({np.uint32: np.int32, np.uint16: np.int16, np.uint8: np.uint8}[it])).cuda()
    return t.view(dtype), raw


def check_against_oracle(x: torch.Tensor, raw: np.ndarray):
    n = x.numel()
    codec = DeviceCodec(n, x.dtype)
    c = codec.compress(x)
    assert c >= 0, B.status_string(c)
    want_payload, want_table = zvc_c.compress(raw)
    assert c == len(want_payload)
    assert codec.payload_numpy(c).tobytes() == want_payload.tobytes()
    assert np.array_equal(codec.table_numpy(), want_table)
    assert codec.canaries_intact()
    out = torch.full_like(x.view(-1), 77 if x.dtype == torch.uint8 else (1.25 if x.dtype != torch.float32 else 3.5))
    r = codec.decompress(out, c)
    assert r == n * x.element_size(), B.status_string(r)
    assert raw_numpy(out).tobytes() == raw.tobytes()
    # and the GPU decoder accepts the oracle's own stream
    codec.load(want_payload, want_table)
    out.fill_(7)
    assert codec.decompress(out, len(want_payload)) == n * x.element_size()
    assert raw_numpy(out).tobytes() == raw.tobytes()
    return c


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.uint8])
@pytest.mark.parametrize("n", SIZES + [4 * TILE - 1, 4 * TILE + 1, 9 * TILE + 77])
def test_sizes_and_tails(n, dtype):
    for seed, density in enumerate([0.1, 0.5, 0.93]):
        x, raw = make(n, density, 1000 * seed + n, dtype)
        check_against_oracle(x, raw)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16, torch.uint8])
def test_all_zero_and_all_dense(dtype):
    n = 3 * TILE + 100 if dtype != torch.uint8 else 9 * TILE + 100
    z = torch.zeros(n, dtype=dtype, device="cuda")
    c = check_against_oracle(z, raw_numpy(z))
    assert c == 4 * ((n + 31) // 32)
    d = torch.full((n,), 1.0, dtype=dtype, device="cuda")
    c = check_against_oracle(d, raw_numpy(d))
    assert c == 4 * ((n + 31) // 32) + n * d.element_size()


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
def test_negative_zero_nan_denormals_are_kept(dtype):
    x = wl.special_values(70_000, seed=5, dtype=dtype, device="cuda")
    check_against_oracle(x, raw_numpy(x))


def test_every_16bit_mask_pattern_in_both_halves():
    pats = np.arange(1 << 16, dtype=np.uint32)
    bits16 = ((pats[:, None] >> np.arange(16)[None, :]) & 1).astype(bool)
    lo = np.zeros((1 << 16, 32), dtype=bool); lo[:, :16] = bits16
    hi = np.zeros((1 << 16, 32), dtype=bool); hi[:, 16:] = bits16
    pattern = np.concatenate([lo, hi]).reshape(-1)
    for it, dt in ((np.uint32, torch.float32), (np.uint16, torch.float16), (np.uint8, torch.uint8)):
        raw = np.where(pattern, (np.arange(pattern.size) % 251 + 1), 0).astype(it)
        x = torch.from_numpy(raw.view({np.uint32: np.int32, np.uint16: np.int16, np.uint8: np.uint8}[it])).cuda().view(dt)
        check_against_oracle(x, raw)


def test_alexnet_conv1_workload_full_size():
    x = wl.alexnet_conv1(device="cuda")
    assert x.numel() == 32 * 96 * 55 * 55
    check_against_oracle(x, raw_numpy(x))


def test_layouts_give_equal_size_and_round_trip():
    x = wl.correlated_relu((8, 32, 28, 28), 0.25, seed=9, device="cuda")
    sizes = set()
    for name in wl.LAYOUTS:
        y = wl.to_layout(x, name)
        codec = DeviceCodec(y.numel(), y.dtype)
        c = codec.compress(y, layout=B.LAYOUT_CODES[name])
        want, table = zvc_c.compress(raw_numpy(y))
        assert codec.payload_numpy(c).tobytes() == want.tobytes()
        sizes.add(c)
        out = torch.empty_like(y)
        assert codec.decompress(out, c, layout=B.LAYOUT_CODES[name]) == y.numel() * 4
        assert torch.equal(out, y)
    assert len(sizes) == 1


def test_capacity_too_small_is_reported_without_overrun():
    x, raw = make(6 * TILE + 77, 0.5, 3, torch.float32)
    want, _ = zvc_c.compress(raw)
    for cap in (len(want) - 4, (len(want) // 2) & ~15, 16, 0):
        codec = DeviceCodec(x.numel(), x.dtype, capacity=cap)
        r = codec.compress(x)
        assert r == -B.ERR_BUFFER_TOO_SMALL
        assert codec.canaries_intact()
        # what was written below the capacity is the true prefix of the stream
        assert codec.payload_numpy(cap).tobytes() == want[:cap].tobytes()
    codec = DeviceCodec(x.numel(), x.dtype, capacity=(len(want) + 15) & ~15)
    assert codec.compress(x) == len(want)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.uint8])
def test_capacity_at_tile_and_line_boundaries(dtype):
    """Capacities that end on, just before and just after the places where the copy-out
    changes row or tile: everything below the capacity is the stream's prefix, nothing
    above it is touched."""
    x, raw = make((5 * TILE + 3 * 1024) * (4 if dtype == torch.uint8 else 1) + 41, 0.45, 17, dtype)
    want, table = zvc_c.compress(raw)
    s = x.element_size()
    tile_starts = [int(table[k]) for k in range(0, len(table) - 1, 8)]      # first chunk of every 8th
    caps = set()
    for t in tile_starts[1:4]:
        line = (t + 127) // 128 * 128                                       # first full line of the tile
        for c in (t - s, t, t + s, line - s, line, line + s, line + 128 * 8 + 4 * s, t + 10):
            if 0 <= c < len(want):
                caps.add(c)
    for cap in sorted(caps):
        codec = DeviceCodec(x.numel(), x.dtype, capacity=cap)
        assert codec.compress(x) == -B.ERR_BUFFER_TOO_SMALL
        assert codec.canaries_intact()
        whole = cap // s * s                                                # whole elements below the capacity
        assert codec.payload_numpy(whole).tobytes() == want[:whole].tobytes(), cap
        assert (codec.payload_numpy(cap)[whole:] == CANARY).all(), cap


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.uint8])
def test_corrupt_table_and_stream_are_rejected_without_faulting(dtype):
    x, raw = make(4 * TILE + 300, 0.4, 11, dtype)
    n = x.numel()
    payload, table = zvc_c.compress(raw)
    out = torch.zeros(n, dtype=dtype, device="cuda")

    def run(p, t, nbytes=None):
        codec = DeviceCodec(n, dtype)
        codec.load(p, t)
        r = codec.decompress(out, len(p) if nbytes is None else nbytes)
        assert codec.canaries_intact()
        return r

    assert run(payload, table) == x.element_size() * n
    t = table.copy(); t[3] += 4
    assert run(payload, t) == -B.ERR_CORRUPT_STREAM
    t = table.copy(); t[5] = t[4] - 4                       # decreasing offsets
    assert run(payload, t) == -B.ERR_CORRUPT_STREAM
    t = table.copy(); t[2] = np.uint64(1) << np.uint64(60)  # far outside the payload
    assert run(payload, t) == -B.ERR_CORRUPT_STREAM
    t = table.copy(); t[-1] -= 4                            # total disagrees with src_bytes
    assert run(payload, t) == -B.ERR_CORRUPT_STREAM
    # flip a bit in the mask of the last window of chunk 1: the chunk's length
    # then disagrees with the table (an earlier window could re-synchronise)
    p = payload.copy()
    last_mask = int(zvc_numpy.window_offsets(raw)[2 * 32 - 1])
    p[last_mask] ^= 0x10
    assert run(p, table) == -B.ERR_CORRUPT_STREAM
    if dtype == torch.float32:     # (the table-less serial walk of the oracle can fall back into step on 2-byte data)
        with pytest.raises(ValueError):
            zvc_c.decompress(p, n, np.float32)
    assert run(payload, table, nbytes=len(payload) - 4) == -B.ERR_CORRUPT_STREAM
    if dtype != torch.float32:
        return
    # a mask naming an element beyond n (short last window)
    y, rawy = make(40, 1.0, 1, torch.float32)
    py, ty = zvc_c.compress(rawy)
    bad = py.copy(); bad[4 + 32 * 4 + 1] |= 0x01             # bit 8 of the second mask, element 40
    codec = DeviceCodec(40, torch.float32)
    codec.load(bad, ty)
    assert codec.decompress(torch.zeros(40, device="cuda"), len(bad)) == -B.ERR_CORRUPT_STREAM


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.uint8])
def test_garbage_streams_never_fault(dtype):
    """Streams that are not streams: random bytes, all-ones masks (records as long as they get),
    zeros, behind tables whose chunk sizes are possible.  The answer is CORRUPT_STREAM (or, by
    luck, success); nothing is read outside the payload or written outside the tensor."""
    n = 6 * 1024 + 500
    s = torch.empty(0, dtype=dtype).element_size()
    k = (n + 1023) // 1024
    rng = np.random.default_rng(170501626)
    guard = 64
    for trial in range(16):
        sizes = []
        for c in range(k):
            nelem = min(1024, n - 1024 * c)
            nwin = (nelem + 31) // 32
            lo, hi = 4 * nwin, 4 * nwin + s * nelem
            pick = [lo, hi, (lo + hi) // 2, int(rng.integers(lo, hi + 1))][trial % 4]
            sizes.append(pick // s * s)
        table = np.concatenate([[0], np.cumsum(sizes)]).astype(np.uint64)
        total = int(table[-1])
        kind = (trial // 4) % 4
        if kind == 0:
            payload = rng.integers(0, 256, size=total, dtype=np.uint8)
        elif kind == 1:
            payload = np.full(total, 0xFF, dtype=np.uint8)
        elif kind == 2:
            payload = np.zeros(total, dtype=np.uint8)
        else:
            payload = rng.integers(0, 2, size=total, dtype=np.uint8) * 0xFF
        codec = DeviceCodec(n, dtype)
        codec.load(payload, table)
        out = torch.full((n + guard,), 7, dtype=dtype, device="cuda")
        r = codec.decompress(out, total)
        assert r in (-B.ERR_CORRUPT_STREAM, n * s), B.status_string(r)
        assert codec.canaries_intact()
        assert bool((out[n:] == 7).all())
    # the library still works afterwards
    x, raw = make(n, 0.3, 2, dtype)
    check_against_oracle(x, raw)


def test_argument_checks():
    x = torch.ones(2048, device="cuda")
    codec = DeviceCodec(2048, torch.float32)
    args = dict(d_src=x.data_ptr(), n=2048, dtype=B.F32, layout=B.NCHW, d_dst=codec.payload.data_ptr(),
                dst_capacity=codec.cap, d_table=codec.table.data_ptr(), d_workspace=codec.ws.data_ptr(),
                workspace_bytes=codec.ws_bytes)
    assert B.cdma_zvc_compress(**args) == 4 * 64 + 4 * 2048
    assert B.cdma_zvc_compress(**{**args, "dtype": 9}) == -B.ERR_UNSUPPORTED_DTYPE
    assert B.cdma_zvc_compress(**{**args, "layout": 5}) == -B.ERR_UNSUPPORTED_LAYOUT
    assert B.cdma_zvc_compress(**{**args, "d_src": x.data_ptr() + 4}) == -B.ERR_ALIGNMENT
    assert B.cdma_zvc_compress(**{**args, "d_dst": codec.payload.data_ptr() + 8}) == -B.ERR_ALIGNMENT
    assert B.cdma_zvc_compress(**{**args, "workspace_bytes": 16}) == -B.ERR_BUFFER_TOO_SMALL
    assert B.cdma_zvc_compress(**{**args, "d_table": 0}) == -B.ERR_INVALID_ARG
    assert B.cdma_zvc_compress(**{**args, "d_dst": x.data_ptr(), "dst_capacity": 64}) == -B.ERR_INVALID_ARG
    # the library is still usable afterwards
    assert B.cdma_zvc_compress(**args) == 4 * 64 + 4 * 2048


def test_runs_on_a_side_stream_and_async_result():
    x, raw = make(9 * TILE + 5, 0.3, 21, torch.float32)
    want, want_table = zvc_c.compress(raw)
    codec = DeviceCodec(x.numel(), x.dtype)
    stream = torch.cuda.Stream()
    res = torch.zeros(2, dtype=torch.int64).pin_memory()
    torch.cuda.synchronize()
    st = B.cdma_zvc_compress_async(x.data_ptr(), x.numel(), B.F32, B.NCHW, codec.payload.data_ptr(),
                                   codec.cap, codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes,
                                   stream.cuda_stream, res.data_ptr())
    assert st == B.OK
    stream.synchronize()
    assert int(res[0]) == len(want) and int(res[1]) == 0
    assert codec.payload_numpy(len(want)).tobytes() == want.tobytes()
    out = torch.empty_like(x)
    st = B.cdma_zvc_decompress_async(codec.payload.data_ptr(), len(want), codec.table.data_ptr(), x.numel(),
                                     B.F32, B.NCHW, out.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes,
                                     stream.cuda_stream, res.data_ptr())
    assert st == B.OK
    stream.synchronize()
    assert int(res[0]) == 4 * x.numel() and int(res[1]) == 0
    assert torch.equal(out.view(torch.int32), x.view(torch.int32))


def test_repeated_calls_share_a_workspace():
    codec = DeviceCodec(20 * TILE, torch.float32)
    for seed in range(4):
        x, raw = make(20 * TILE, 0.2 + 0.2 * seed, seed, torch.float32)
        want, table = zvc_c.compress(raw)
        assert codec.compress(x) == len(want)
        assert codec.payload_numpy(len(want)).tobytes() == want.tobytes()
        assert np.array_equal(codec.table_numpy(), table)
