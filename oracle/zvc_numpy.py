"""A second, independent statement of ZVC in numpy, used to cross-check the C oracle.

TEST INFRASTRUCTURE -- see the package docstring.

Where the C oracle appends records one after another, this module states the
same stream in closed form (paper Section V-A):

* the masks are the non-zero indicator bits of the tensor, 32 per word, bit i
  of window w being element 32w+i  (``numpy.packbits(..., bitorder="little")``
  is that textbook packing);
* the packed values are the non-zero elements in memory order (``x[bits]``);
* window w's record starts ``4*w + s*(non-zeros before window w)`` bytes into
  the stream, because every earlier window contributed one mask and its own
  non-zeros -- the "pop-count gives the offset of the next mask" rule summed up.

``split_stream`` goes the other way: it walks a stream using pop-counts only
and returns the masks and values it meets.
"""
from __future__ import annotations

import numpy as np

WINDOW = 32
CHUNK = 1024


def _raw(x: np.ndarray) -> np.ndarray:
    """Flat unsigned-integer view of the element bit patterns."""
    x = np.ascontiguousarray(x).reshape(-1)
    if x.dtype.itemsize == 4:
        return x.view(np.uint32)
    if x.dtype.itemsize == 2:
        return x.view(np.uint16)
    if x.dtype.itemsize == 1:
        return x.view(np.uint8)
    raise ValueError("elements must be 1, 2 or 4 bytes")


def nonzero_bits(x: np.ndarray) -> np.ndarray:
    """Boolean per element: is its bit pattern different from all-zero."""
    return _raw(x) != 0


def masks(x: np.ndarray) -> np.ndarray:
    """uint32[ceil(n/32)]: bit i of word w set iff element 32w+i is non-zero."""
    bits = nonzero_bits(x)
    n = bits.size
    w = (n + WINDOW - 1) // WINDOW
    padded = np.zeros(w * WINDOW, dtype=np.uint8)
    padded[:n] = bits
    packed = np.packbits(padded, bitorder="little")
    return packed.view("<u4").astype(np.uint32)


def values(x: np.ndarray) -> np.ndarray:
    """The non-zero elements' bit patterns in memory order."""
    r = _raw(x)
    return r[r != 0]


def payload_bytes(x: np.ndarray) -> int:
    n = x.size
    return 4 * ((n + WINDOW - 1) // WINDOW) + x.dtype.itemsize * int(np.count_nonzero(_raw(x)))


def window_offsets(x: np.ndarray) -> np.ndarray:
    """uint64[W+1]: byte offset of every window's record; last = payload size."""
    bits = nonzero_bits(x)
    n = bits.size
    s = x.dtype.itemsize
    w = (n + WINDOW - 1) // WINDOW
    padded = np.zeros(w * WINDOW, dtype=np.int64)
    padded[:n] = bits
    per_window = padded.reshape(w, WINDOW).sum(axis=1) if w else np.zeros(0, dtype=np.int64)
    off = np.zeros(w + 1, dtype=np.int64)
    np.cumsum(4 + s * per_window, out=off[1:])
    return off.astype(np.uint64)


def table(x: np.ndarray) -> np.ndarray:
    """uint64[ceil(n/1024)+1]: offsets of windows 0, 32, 64, ... and the total."""
    off = window_offsets(x)
    k = (x.size + CHUNK - 1) // CHUNK
    out = np.empty(k + 1, dtype=np.uint64)
    out[:k] = off[:-1:CHUNK // WINDOW][:k]
    out[k] = off[-1]
    return out


def build_stream(x: np.ndarray) -> np.ndarray:
    """The whole payload as uint8, placed by closed-form offsets (no appending)."""
    r = _raw(x)
    s = r.dtype.itemsize
    n = r.size
    off = window_offsets(x).astype(np.int64)
    out = np.zeros(int(off[-1]), dtype=np.uint8)
    m = masks(x)
    w = m.size
    if w == 0:
        return out
    # masks: 4 bytes, least-significant first, at each record's start
    mb = m.astype("<u4").view(np.uint8).reshape(w, 4)
    out[(off[:-1, None] + np.arange(4)[None, :]).reshape(-1)] = mb.reshape(-1)
    # values: element j (non-zero) sits after its window's mask, behind the
    # non-zeros of the same window that come before it
    idx = np.flatnonzero(r != 0)
    if idx.size:
        win = idx // WINDOW
        before = np.arange(idx.size, dtype=np.int64)          # non-zeros before j overall
        first_of_window = np.searchsorted(win, win, side="left")  # non-zeros before j's window
        rank = before - first_of_window
        pos = off[win] + 4 + s * rank
        vb = r[idx].astype(r.dtype.newbyteorder("<")).view(np.uint8).reshape(idx.size, s)
        out[(pos[:, None] + np.arange(s)[None, :]).reshape(-1)] = vb.reshape(-1)
    return out


def split_stream(payload: np.ndarray, n: int, s: int):
    """Walk a stream by pop-counts.  Returns (masks uint32[W], values uintN[nnz], end).

    ``end`` is the position reached after the last window; a well-formed
    stream has ``end == len(payload)``.
    """
    payload = np.ascontiguousarray(payload, dtype=np.uint8)
    w = (n + WINDOW - 1) // WINDOW
    out_masks = np.zeros(w, dtype=np.uint32)
    chunks = []
    pos = 0
    vt = {4: np.dtype("<u4"), 2: np.dtype("<u2"), 1: np.dtype("u1")}[s]
    for i in range(w):
        if pos + 4 > payload.size:
            raise ValueError("stream ends inside a mask")
        mask = int.from_bytes(payload[pos:pos + 4].tobytes(), "little")
        out_masks[i] = mask
        cnt = bin(mask).count("1")
        pos += 4
        if pos + s * cnt > payload.size:
            raise ValueError("stream ends inside a record")
        chunks.append(payload[pos:pos + s * cnt])
        pos += s * cnt
    vals = np.concatenate(chunks).view(vt) if chunks else np.zeros(0, dtype=vt)
    return out_masks, vals.astype({4: np.uint32, 2: np.uint16, 1: np.uint8}[s]), pos
