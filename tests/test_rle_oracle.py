"""Pins of the run-length comparison codec's oracle.  The paper gives no format for it
(Section V-A names the scheme, Section VI-A reports its layout sensitivity), so what can be
pinned is: hand-worked streams of the stated format, the size formula against brute-force
run counting, exact round trips, the limits, and the qualitative claim of the paper that
run-length encoding -- unlike zero-value compression -- depends on where the zeros lie."""
import numpy as np
import pytest

from oracle import rle_numpy, zvc_c


def words(payload):
    return payload.view(np.uint32).tolist()


def test_hand_worked_streams():
    # 3 zeros, 2 values, 1 zero, 1 value, 2 zeros (9 elements)
    x = np.array([0, 0, 0, 7, 9, 0, 5, 0, 0], dtype=np.uint32)
    payload, table = rle_numpy.compress(x)
    assert words(payload) == [3 | (2 << 16), 7, 9, 1 | (1 << 16), 5, 2]
    assert table.tolist() == [0, 24]
    # starts with a value, ends with a value
    x = np.array([4, 0, 0, 8], dtype=np.uint32)
    assert words(rle_numpy.compress(x)[0]) == [0 | (1 << 16), 4, 2 | (1 << 16), 8]
    # all zeros: one record per chunk, 32 zeros -> 4 bytes as in the paper's example for its mask scheme
    assert words(rle_numpy.compress(np.zeros(32, dtype=np.uint32))[0]) == [32]
    # all non-zero: one token in front of the whole chunk
    x = np.arange(1, 1025, dtype=np.uint32)
    assert words(rle_numpy.compress(x)[0]) == [1024 << 16] + x.tolist()
    # two chunks: runs do not cross the chunk boundary
    x = np.zeros(2048, dtype=np.uint32); x[1020:1030] = 3
    payload, table = rle_numpy.compress(x)
    assert words(payload) == [1020 | (4 << 16), 3, 3, 3, 3, 0 | (6 << 16), 3, 3, 3, 3, 3, 3, 1018]
    assert table.tolist() == [0, 20, 52]


def brute_force_records(x):
    """Count records chunk by chunk with a plain loop."""
    total = 0
    for c in range(0, len(x), 1024):
        chunk = x[c:c + 1024]
        prev = 0
        for v in chunk:
            if v != 0 and prev == 0:
                total += 1
            prev = v
        if chunk[-1] == 0:
            total += 1
    return total


@pytest.mark.parametrize("n,density,seed", [(1, 1.0, 0), (1, 0.0, 1), (1023, 0.5, 2), (1024, 0.3, 3), (1025, 0.9, 4),
                                            (5000, 0.05, 5), (40000, 0.5, 6)])
def test_size_formula_round_trip_and_table(n, density, seed):
    rng = np.random.default_rng(seed)
    x = rng.integers(1, 2 ** 32, size=n, dtype=np.uint64).astype(np.uint32)
    x[rng.random(n) >= density] = 0
    payload, table = rle_numpy.compress(x)
    assert payload.size == 4 * brute_force_records(x) + 4 * int(np.count_nonzero(x))
    assert payload.size == rle_numpy.compressed_bytes(x)
    assert int(table[-1]) == payload.size and np.all(np.diff(table.astype(np.int64)) >= 4)
    assert np.array_equal(rle_numpy.decompress(payload, n), x)
    # every chunk decodes on its own from its table entry
    for c in range(len(table) - 1):
        part = payload[int(table[c]):int(table[c + 1])]
        size = min(1024, n - 1024 * c)
        assert np.array_equal(rle_numpy.decompress(part, size), x[1024 * c:1024 * c + size])


def test_special_bit_patterns_are_literals():
    x = np.array([0x80000000, 0x7FC00000, 0x00000001, 0, 0xFF800000], dtype=np.uint32)   # -0.0, NaN, denormal, 0, -inf
    payload, _ = rle_numpy.compress(x)
    assert words(payload) == [0 | (3 << 16), 0x80000000, 0x7FC00000, 1, 1 | (1 << 16), 0xFF800000]
    assert np.array_equal(rle_numpy.decompress(payload, 5), x)


def test_malformed_streams_are_refused():
    x = np.array([0, 0, 5, 6, 0], dtype=np.uint32)
    payload, _ = rle_numpy.compress(x)
    w = payload.view(np.uint32).copy()
    for bad in ([w[0] + 1] + w[1:].tolist(),             # one zero too many: overruns the chunk
                w[:-1].tolist(),                         # truncated
                w.tolist() + [1],                        # bytes left over
                [0] + w[1:].tolist()):                   # literal placed over a zero... then sizes disagree
        with pytest.raises(ValueError):
            rle_numpy.decompress(np.array(bad, dtype=np.uint32).view(np.uint8), 5)


def test_run_length_depends_on_where_the_zeros_lie_and_zero_value_compression_does_not():
    # the same multiset of elements, clustered and scattered (Section V-A / Fig. 11)
    n = 64 * 1024
    clustered = np.zeros(n, dtype=np.uint32)
    clustered.reshape(-1, 256)[:, :64] = 9                      # 64 values, 192 zeros, repeating
    rng = np.random.default_rng(1)
    scattered = clustered.copy(); rng.shuffle(scattered)
    assert rle_numpy.compressed_bytes(clustered) < 0.6 * rle_numpy.compressed_bytes(scattered)
    zc, _ = zvc_c.compress(clustered); zs, _ = zvc_c.compress(scattered)
    assert len(zc) == len(zs)
    # clustered zeros: run-length beats the per-window masks; scattered: it loses
    assert rle_numpy.compressed_bytes(clustered) < len(zc) < rle_numpy.compressed_bytes(scattered)
