"""Pins of the CPU oracle against what the paper and the arithmetic fix.

None of these tests touches the CUDA path.  Each is chosen so that a plausible
slip in the oracle (wrong bit order, wrong byte order, values before the mask,
descending order, a float compare instead of a bit compare, a dropped tail, a
table off by one chunk) fails at least one of them.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import zvc_c, zvc_numpy

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "zvc_paper_examples.txt")


def u32(vals):
    return np.array(vals, dtype=np.uint32)


def u16(vals):
    return np.array(vals, dtype=np.uint16)


def u8(vals):
    return np.array(vals, dtype=np.uint8)


# --------------------------------------------------------------------------- #
# hand-written byte vectors (typed out, not computed)
# --------------------------------------------------------------------------- #
HAND_VECTORS = [
    # fp32, n=3: only element 1 (1.0f) is non-zero -> mask 0b010
    (u32([0, 0x3F800000, 0]),
     "02000000" "0000803f"),
    # fp32, n=33: element 0, element 31 and element 32 non-zero.
    # window 0 mask = bit0|bit31 = 0x80000001, stored LSB first; values ascending;
    # window 1 (short) mask = 1.
    (u32([0x11223344] + [0] * 30 + [0xAABBCCDD] + [0x00000100]),
     "01000080" "44332211" "ddccbbaa" "01000000" "00010000"),
    # fp32, n=4: -0.0 and a NaN are non-zero by bit pattern; +0.0 is zero
    (u32([0x80000000, 0x00000000, 0x7FC00001, 0x00000000]),
     "05000000" "00000080" "0100c07f"),
    # fp32, n=32 all zero: just the zero mask
    (u32([0] * 32), "00000000"),
    # fp32, n=64: second window only, element 40 (bit 8 -> second mask byte)
    (u32([0] * 40 + [0xDEADBEEF] + [0] * 23),
     "00000000" "00010000" "efbeadde"),
    # fp16, n=5: elements 0, 2 (-0.0) and 4 (NaN) non-zero -> mask 0b10101
    (u16([0x0001, 0x0000, 0x8000, 0x0000, 0x7E00]),
     "15000000" "0100" "0080" "007e"),
    # fp16, n=34: one value in window 0 makes window 1's mask start at byte 6
    (u16([0] * 7 + [0xBEEF] + [0] * 24 + [0x1234, 0x0000]),
     "80000000" "efbe" "01000000" "3412"),
    # 1-byte elements (fp8 / int8), n=6: elements 1, 2 (0x80: -0.0 in fp8) and 5 non-zero -> mask 0b100110
    (u8([0x00, 0x7F, 0x80, 0x00, 0x00, 0x01]),
     "26000000" "7f" "80" "01"),
    # 1-byte elements, n=35: three values in window 0 make window 1's mask start at byte 7 (odd address)
    (u8([0xAA] + [0] * 15 + [0xBB] + [0] * 14 + [0xCC] + [0x00, 0xDD, 0xEE]),
     "01000180" "aa" "bb" "cc" "06000000" "dd" "ee"),
]


@pytest.mark.parametrize("x,hexbytes", HAND_VECTORS)
def test_hand_vectors(x, hexbytes):
    payload, table = zvc_c.compress(x)
    assert payload.tobytes().hex() == hexbytes
    assert table[0] == 0 and table[-1] == len(payload)
    back = zvc_c.decompress(payload, x.size, x.dtype)
    assert back.tobytes() == x.tobytes()
    # the independent numpy statement must give the same bytes
    assert zvc_numpy.build_stream(x).tobytes().hex() == hexbytes


# --------------------------------------------------------------------------- #
# the paper's printed micro-examples (Section V-A)
# --------------------------------------------------------------------------- #
def _golden_cases():
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, n, zeros, expected, quantity = line.split()
            yield name, int(n), int(zeros), float(expected), quantity


@pytest.mark.parametrize("name,n,zeros,expected,quantity", list(_golden_cases()))
def test_paper_examples(name, n, zeros, expected, quantity):
    x = np.zeros(n, dtype=np.float32)
    # spread the non-zeros evenly; their position must not matter to the size
    nz = n - zeros
    if nz:
        x[np.linspace(0, n - 1, nz).round().astype(int)] = 1.5
    assert np.count_nonzero(x) == nz
    payload, _ = zvc_c.compress(x)
    if quantity == "stream_bytes":
        assert len(payload) == expected
    elif quantity == "ratio":
        assert x.nbytes / len(payload) == expected
    elif quantity == "metadata_percent":
        masks = len(payload) - 4 * nz
        assert round(100.0 * masks / x.nbytes, 1) == expected
    elif quantity == "value_ratio":
        assert x.nbytes / (4 * nz) == expected
        # with the masks counted the ratio is 1/(0.4 + 1/32)
        assert x.nbytes / len(payload) == pytest.approx(1.0 / (0.4 + 1.0 / 32.0), rel=1e-12)
    else:
        raise AssertionError(quantity)


# --------------------------------------------------------------------------- #
# closed form, all-zero, all-dense
# --------------------------------------------------------------------------- #
BOUNDARY_N = [0, 1, 31, 32, 33, 63, 64, 65, 1023, 1024, 1025, 2047, 2048, 2049,
              32 * 1024 - 1, 32 * 1024, 32 * 1024 + 1]


def random_sparse(n, density, seed, dtype):
    rng = np.random.default_rng(seed)
    it = {4: np.uint32, 2: np.uint16, 1: np.uint8}[np.dtype(dtype).itemsize]
    raw = rng.integers(1, np.iinfo(it).max, size=n, dtype=it, endpoint=True)
    raw[rng.random(n) >= density] = 0
    return raw.view(dtype)


@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
@pytest.mark.parametrize("n", BOUNDARY_N)
def test_closed_form_size_and_round_trip(n, dtype):
    s = np.dtype(dtype).itemsize
    for seed in range(3):
        x = random_sparse(n, [0.1, 0.5, 0.9][seed], 100 + seed, dtype)
        nnz = int(np.count_nonzero(x.view({4: np.uint32, 2: np.uint16, 1: np.uint8}[s])))
        payload, table = zvc_c.compress(x)
        assert len(payload) == 4 * ((n + 31) // 32) + s * nnz
        assert len(payload) == zvc_c.closed_form_bytes(n, nnz, s)
        assert zvc_c.decompress(payload, n, dtype).tobytes() == x.tobytes()
        assert zvc_c.check_table(payload, n, s, table)
        # independent closed-form construction gives the same bytes and table
        assert zvc_numpy.build_stream(x).tobytes() == payload.tobytes()
        assert np.array_equal(zvc_numpy.table(x), table)


@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
@pytest.mark.parametrize("n", [1, 32, 33, 1024, 1025, 5000])
def test_all_zero(n, dtype):
    x = np.zeros(n, dtype=dtype)
    payload, table = zvc_c.compress(x)
    w = (n + 31) // 32
    assert len(payload) == 4 * w
    assert not payload.any()
    # a full window of zeros shrinks 32x for 4-byte elements (Section V-A)
    if n % 32 == 0 and dtype == np.float32:
        assert x.nbytes / len(payload) == 32
    assert np.array_equal(table[:-1], 128 * np.arange(len(table) - 1, dtype=np.uint64))


@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
@pytest.mark.parametrize("n", [1, 31, 32, 33, 1024, 1030, 4099])
def test_all_dense(n, dtype):
    s = np.dtype(dtype).itemsize
    it = {4: np.uint32, 2: np.uint16, 1: np.uint8}[s]
    x = (np.arange(n, dtype=np.uint64) % (255 if s == 1 else 65535) + 1).astype(it).view(dtype)
    payload, _ = zvc_c.compress(x)
    w = (n + 31) // 32
    assert len(payload) == 4 * w + s * n
    masks, vals, end = zvc_numpy.split_stream(payload, n, s)
    assert end == len(payload)
    full = n // 32
    assert (masks[:full] == 0xFFFFFFFF).all()
    if n % 32:
        assert masks[-1] == (1 << (n % 32)) - 1
    assert np.array_equal(vals, x.view(it))
    if n % 32 == 0 and s == 4:
        # mask overhead of an all-dense window: 4 bytes on 128 (3.125 %)
        assert (len(payload) - x.nbytes) / x.nbytes == 1 / 32


# --------------------------------------------------------------------------- #
# every zero/non-zero pattern on tiny inputs, checked by properties of the
# stream (sentinel values reveal which element each stored value came from)
# --------------------------------------------------------------------------- #
def _check_stream_by_properties(payload, pattern, s):
    """pattern[j] True = element j was non-zero and held sentinel j+1."""
    n = len(pattern)
    pos = 0
    for w0 in range(0, n, 32):
        mask = int.from_bytes(payload[pos:pos + 4].tobytes(), "little")
        pos += 4
        for i in range(32):
            bit = (mask >> i) & 1
            j = w0 + i
            if j >= n:
                assert bit == 0
                continue
            assert bit == int(pattern[j])
            if bit:
                v = int.from_bytes(payload[pos:pos + s].tobytes(), "little")
                assert v == sentinel(j, s)
                pos += s
    assert pos == len(payload)


def sentinel(j, s):
    # non-zero in every byte, distinct per position
    return {4: 0xA5C30000 | (j + 1), 2: 0xA500 | (j + 1), 1: 0xC0 | (j + 1)}[s]


@pytest.mark.parametrize("s", [4, 2, 1])
def test_every_pattern_of_tiny_inputs(s):
    # every zero / non-zero pattern of every length up to 16 (4-byte elements; up to 12 for 2-byte ones)
    it = {4: np.uint32, 2: np.uint16, 1: np.uint8}[s]
    for n in range(1, 17 if s == 4 else 13):
        for bits in itertools.product([False, True], repeat=n):
            x = np.array([sentinel(j, s) if b else 0 for j, b in enumerate(bits)], dtype=it)
            payload, _ = zvc_c.compress(x)
            _check_stream_by_properties(payload, bits, s)


@pytest.mark.parametrize("s", [4, 2])
def test_all_16bit_patterns_in_both_window_halves(s):
    it = {4: np.uint32, 2: np.uint16, 1: np.uint8}[s]
    pats = np.arange(1 << 16, dtype=np.uint32)
    bits16 = ((pats[:, None] >> np.arange(16)[None, :]) & 1).astype(bool)       # [65536,16]
    lo = np.zeros((1 << 16, 32), dtype=bool)
    lo[:, :16] = bits16
    hi = np.zeros((1 << 16, 32), dtype=bool)
    hi[:, 16:] = bits16
    pattern = np.concatenate([lo, hi]).reshape(-1)
    n = pattern.size
    x = np.where(pattern, ((np.arange(n) % 200) + 1).astype(it) | it(0x4000), it(0)).astype(it)
    payload, table = zvc_c.compress(x)
    masks, vals, end = zvc_numpy.split_stream(payload, n, s)
    assert end == len(payload)
    assert np.array_equal(masks[: 1 << 16], pats)
    assert np.array_equal(masks[1 << 16:], pats << 16)
    assert np.array_equal(vals, x[pattern])
    assert zvc_c.check_table(payload, n, s, table)
    assert zvc_c.decompress(payload, n, it).tobytes() == x.tobytes()


@pytest.mark.parametrize("s", [4, 2])
def test_walking_one_and_walking_zero(s):
    it = {4: np.uint32, 2: np.uint16, 1: np.uint8}[s]
    for i in range(32):
        one = np.zeros(32, dtype=it)
        one[i] = 0x7B
        p, _ = zvc_c.compress(one)
        assert p.tobytes() == (1 << i).to_bytes(4, "little") + (0x7B).to_bytes(s, "little")
        zero = np.arange(1, 33, dtype=it)
        zero[i] = 0
        p, _ = zvc_c.compress(zero)
        assert p[:4].tobytes() == (0xFFFFFFFF ^ (1 << i)).to_bytes(4, "little")
        kept = np.delete(np.arange(1, 33, dtype=it), i)
        assert p[4:].tobytes() == kept.astype("<u%d" % s).tobytes()


def test_every_byte_pattern_in_each_mask_byte():
    for byte_index in range(4):
        for pat in range(256):
            x = np.zeros(32, dtype=np.uint32)
            for b in range(8):
                if (pat >> b) & 1:
                    x[8 * byte_index + b] = 0x01010101 * (b + 1)
            p, _ = zvc_c.compress(x)
            expect_mask = bytearray(4)
            expect_mask[byte_index] = pat
            assert p[:4].tobytes() == bytes(expect_mask)
            assert len(p) == 4 + 4 * bin(pat).count("1")


# --------------------------------------------------------------------------- #
# structure: self-delimiting walk, packbits masks, table, layouts
# --------------------------------------------------------------------------- #
@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
def test_masks_and_values_match_packbits(dtype):
    s = np.dtype(dtype).itemsize
    x = random_sparse(50_000 + 7, 0.37, 5, dtype)
    payload, _ = zvc_c.compress(x)
    masks, vals, end = zvc_numpy.split_stream(payload, x.size, s)
    assert end == len(payload)                     # walk visits W masks and ends at C
    assert len(masks) == (x.size + 31) // 32
    assert np.array_equal(masks, zvc_numpy.masks(x))
    assert np.array_equal(vals, zvc_numpy.values(x))


@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
def test_table_from_independent_chunk_counts(dtype):
    s = np.dtype(dtype).itemsize
    n = 10 * 1024 + 77
    x = random_sparse(n, 0.3, 9, dtype)
    payload, table = zvc_c.compress(x)
    raw = x.view({4: np.uint32, 2: np.uint16, 1: np.uint8}[s])
    k = (n + 1023) // 1024
    assert len(table) == k + 1 == zvc_c.table_entries(n)
    assert table[0] == 0
    for c in range(k):
        part = raw[c * 1024:(c + 1) * 1024]
        windows = (len(part) + 31) // 32
        assert int(table[c + 1] - table[c]) == 4 * windows + s * int(np.count_nonzero(part))
    assert table[k] == len(payload)
    # a table shifted by one entry, or with a wrong total, is rejected
    bad = table.copy()
    bad[1] += s
    assert not zvc_c.check_table(payload, n, s, bad)
    bad = table.copy()
    bad[-1] -= 1
    assert not zvc_c.check_table(payload, n, s, bad)


def test_special_values_survive():
    pats = np.array([0x00000000, 0x80000000, 0x7FC00000, 0x7F800001, 0xFFC12345,
                     0x00000001, 0x807FFFFF, 0x7F800000, 0xFF800000, 0x3F800000] * 13,
                    dtype=np.uint32)
    payload, _ = zvc_c.compress(pats.view(np.float32))
    nnz = int((pats != 0).sum())
    assert len(payload) == 4 * ((pats.size + 31) // 32) + 4 * nnz
    back = zvc_c.decompress(payload, pats.size, np.float32)
    assert back.view(np.uint32).tobytes() == pats.tobytes()
    # a float comparison would have dropped -0.0: make sure it is counted
    assert (pats == 0x80000000).sum() > 0
    h = np.array([0x0000, 0x8000, 0x7E00, 0x7C01, 0xFE00, 0x0001, 0x83FF, 0x7C00, 0xFC00, 0x3C00] * 7,
                 dtype=np.uint16)
    payload, _ = zvc_c.compress(h.view(np.float16))
    assert len(payload) == 4 * ((h.size + 31) // 32) + 2 * int((h != 0).sum())
    assert zvc_c.decompress(payload, h.size, np.float16).view(np.uint16).tobytes() == h.tobytes()


def test_size_is_layout_independent_but_bytes_are_not():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((4, 6, 10, 12)).astype(np.float32)
    x[rng.random(x.shape) < 0.6] = 0
    nchw = np.ascontiguousarray(x)
    nhwc = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    chwn = np.ascontiguousarray(x.transpose(1, 2, 3, 0))
    sizes = {len(zvc_c.compress(t)[0]) for t in (nchw, nhwc, chwn)}
    assert len(sizes) == 1
    assert zvc_c.compress(nchw)[0].tobytes() != zvc_c.compress(nhwc)[0].tobytes()
    back = zvc_c.decompress(zvc_c.compress(nhwc)[0], x.size, np.float32).reshape(nhwc.shape)
    assert np.array_equal(back.transpose(0, 3, 1, 2), x)


# --------------------------------------------------------------------------- #
# failure behaviour
# --------------------------------------------------------------------------- #
def test_malformed_streams_are_rejected():
    x = random_sparse(300, 0.5, 1, np.float32)
    payload, _ = zvc_c.compress(x)
    with pytest.raises(ValueError):
        zvc_c.decompress(payload[:-1], 300, np.float32)          # truncated
    with pytest.raises(ValueError):
        zvc_c.decompress(np.concatenate([payload, payload[:4]]), 300, np.float32)  # trailing bytes
    with pytest.raises(ValueError):
        zvc_c.decompress(payload, 299 - 32, np.float32)          # fewer windows than the stream has
    # a mask bit naming an element beyond n
    y = np.ones(5, dtype=np.uint32)
    p, _ = zvc_c.compress(y)
    bad = np.concatenate([p, np.array([1, 0, 0, 0], dtype=np.uint8)])
    bad[0] |= 0x20
    with pytest.raises(ValueError):
        zvc_c.decompress(bad, 5, np.uint32)


def test_too_small_destination_is_reported_and_not_overrun():
    x = random_sparse(1000, 0.5, 2, np.float32)
    full, _ = zvc_c.compress(x)
    with pytest.raises(BufferError):
        zvc_c.compress(x, capacity=len(full) - 1)
    payload, _ = zvc_c.compress(x, capacity=len(full))
    assert payload.tobytes() == full.tobytes()


@pytest.mark.parametrize("dtype", [np.float32, np.float16, np.uint8])
@pytest.mark.parametrize("threads", [2, 3, 8])
def test_threaded_driver_equals_single_thread(dtype, threads):
    for n in (1, 1024, 5 * 1024 + 3, 40_000):
        x = random_sparse(n, 0.4, n, dtype)
        p1, t1 = zvc_c.compress(x)
        pm, tm = zvc_c.compress(x, threads=threads)
        assert p1.tobytes() == pm.tobytes()
        assert np.array_equal(t1, tm)
        back = zvc_c.decompress(pm, n, dtype, table=tm, threads=threads)
        assert back.tobytes() == x.tobytes()
