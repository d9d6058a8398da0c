"""Plain numpy statement of the run-length comparison codec (Section V-A,
"Run-length encoding compression").

TEST INFRASTRUCTURE -- see the package docstring.  PARITY UNPINNED against the
paper: it prints no format and no worked example for this scheme, so this file
is pinned only by hand-worked streams of the format stated below, the size
formula against brute-force run counting, round trips and invariants.

The paper names run-length
encoding as the first scheme it tried and reports how its ratio depends on the
activation layout (Section VI-A, Fig. 11), but gives no format.  The format
below is this build's own; what the paper fixes
is only the idea: runs of zeros are replaced by their length, so the scheme
pays off for consecutive zeros and is sensitive to the memory layout.

Format, 4-byte elements only, on the same framing as the zero-value codec
(independent chunks of 1024 elements, a table of ceil(n/1024)+1 byte offsets
outside the payload):

    chunk   := record*
    record  := token literals
    token   := uint32, little endian: zeros | (count << 16)
               zeros = number of zero elements in front of the literals (0..1024)
               count = number of literal (non-zero) elements that follow (0..1024)
    literals:= count raw elements

A record is written for every maximal run of non-zero elements, carrying the
zero run in front of it; a chunk that ends in zeros gets a last record with
count = 0.  An empty chunk cannot occur (the last chunk has at least one
element).  "Zero" is bitwise, as in the zero-value codec.  Chunk size in bytes:
4 * (number of records) + 4 * (number of non-zero elements).
"""
from __future__ import annotations

import numpy as np

CHUNK = 1024


def _chunk_records(x: np.ndarray) -> np.ndarray:
    """The records of one chunk (uint32 words) from its elements (uint32 bit patterns)."""
    nz = (x != 0).astype(np.int8)
    edges = np.flatnonzero(np.diff(np.concatenate(([0], nz, [0]))))   # run starts and ends, alternating
    starts, ends = edges[0::2], edges[1::2]
    words = []
    prev_end = 0
    for s, e in zip(starts.tolist(), ends.tolist()):
        words.append(np.uint32((s - prev_end) | ((e - s) << 16)))
        words.extend(x[s:e].tolist())
        prev_end = e
    if prev_end < x.size:
        words.append(np.uint32(x.size - prev_end))
    return np.array(words, dtype=np.uint32)


def compress(raw: np.ndarray):
    """(payload as uint8, table as uint64) for a flat array of uint32 bit patterns."""
    raw = np.ascontiguousarray(raw, dtype=np.uint32).reshape(-1)
    n = raw.size
    k = (n + CHUNK - 1) // CHUNK
    parts, table = [], np.zeros(k + 1, dtype=np.uint64)
    for c in range(k):
        rec = _chunk_records(raw[c * CHUNK:(c + 1) * CHUNK])
        parts.append(rec)
        table[c + 1] = table[c] + np.uint64(4 * rec.size)
    payload = np.concatenate(parts).view(np.uint8) if parts else np.zeros(0, dtype=np.uint8)
    return payload, table


def decompress(payload: np.ndarray, n: int) -> np.ndarray:
    """Walk the records serially (the table is not needed) and rebuild n elements.
    Raises ValueError on a malformed stream."""
    words = np.ascontiguousarray(payload, dtype=np.uint8).view(np.uint32)
    out = np.zeros(n, dtype=np.uint32)
    p = 0
    for c in range((n + CHUNK - 1) // CHUNK):
        base, size = c * CHUNK, min(CHUNK, n - c * CHUNK)
        pos = 0
        while pos < size:
            if p >= words.size:
                raise ValueError("stream ends inside a chunk")
            token = int(words[p]); p += 1
            zeros, count = token & 0xFFFF, token >> 16
            if pos + zeros + count > size or p + count > words.size or (zeros == 0 and count == 0):
                raise ValueError("record does not fit its chunk")
            lits = words[p:p + count]
            if np.any(lits == 0):
                raise ValueError("a literal is zero")
            out[base + pos + zeros: base + pos + zeros + count] = lits
            p += count
            pos += zeros + count
    if p != words.size:
        raise ValueError("bytes left over")
    return out


def compressed_bytes(raw: np.ndarray) -> int:
    """Payload size without building the stream: 4 bytes per record and per non-zero
    element, records counted chunk by chunk with array operations only."""
    raw = np.ascontiguousarray(raw, dtype=np.uint32).reshape(-1)
    n = raw.size
    k = (n + CHUNK - 1) // CHUNK
    pad = k * CHUNK - n
    nz = np.concatenate([raw != 0, np.zeros(pad, dtype=bool)]).reshape(k, CHUNK)
    prev = np.concatenate([np.zeros((k, 1), dtype=bool), nz[:, :-1]], axis=1)
    run_starts = int(np.count_nonzero(nz & ~prev))
    sizes = np.full(k, CHUNK)
    if pad:
        sizes[-1] = CHUNK - pad
    last = nz[np.arange(k), sizes - 1]
    trailing = int(np.count_nonzero(~last))
    return 4 * (run_starts + trailing) + 4 * int(np.count_nonzero(nz))
