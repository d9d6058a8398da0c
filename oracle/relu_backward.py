"""Plain CPU statement of the activation function's backward pass computed from a
compressed activation map.

TEST INFRASTRUCTURE -- see the package docstring.  Nothing in the CUDA package
imports this module.

What is computed (paper Section II-B: the backward pass of a layer reuses the
activation map the forward pass produced; Section V-A: a window's mask has bit i
set when element i is non-zero): for the map y held by a compressed stream and
an incoming gradient dy of the same shape,

    dx[j] = dy[j]   if element j of y is non-zero (as a bit pattern)
    dx[j] = +0      otherwise

taken as a selection of bit patterns: nothing is multiplied, so the result is exact.
The definition is written out on the dense y that the byte-wise C oracle
(``zvc_c.decompress``) rebuilds from the stream; the masks of the stream are not
looked at here.  For y = max(x, 0) this is the textbook ReLU backward, which is what
the tests pin it to.
"""
from __future__ import annotations

import numpy as np

from . import zvc_c


def _raw(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a).reshape(-1)
    return a.view({4: np.uint32, 2: np.uint16, 1: np.uint8}[a.dtype.itemsize])


def relu_backward(payload: np.ndarray, n: int, dy: np.ndarray) -> np.ndarray:
    """dx (same dtype as dy, flat) for the map of n elements held by ``payload``."""
    dy = np.ascontiguousarray(dy).reshape(-1)
    if dy.size != n:
        raise ValueError("dy must have n elements")
    y = zvc_c.decompress(payload, n, dy.dtype)          # serial pop-count walk, element by element
    keep = _raw(y) != 0
    out = np.where(keep, _raw(dy), 0).astype(_raw(dy).dtype)
    return out.view(dy.dtype)
