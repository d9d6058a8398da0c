"""CPU pins of the backward-pass oracle (``oracle/relu_backward.py``): for y = max(x, 0)
it must be the ReLU backward of a library (torch autograd on the CPU), bit for bit,
special values included; and it must follow the non-zero pattern, nothing else."""
import numpy as np
import pytest
import torch

from oracle import relu_backward as rb
from oracle import zvc_c


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("n", [1, 31, 32, 33, 1023, 1024, 1025, 5000])
def test_equals_autograd_relu_backward(dtype, n):
    g = torch.Generator().manual_seed(n)
    x = torch.randn(n, generator=g).to(dtype).requires_grad_(True)
    dy = torch.randn(n, generator=g).to(dtype)
    y = torch.relu(x)
    y.backward(dy)
    want = x.grad
    it = torch.int32 if dtype == torch.float32 else torch.int16
    np_t = np.uint32 if dtype == torch.float32 else np.uint16
    y_raw = y.detach().view(it).numpy().view(np_t)
    payload, _ = zvc_c.compress(y_raw)
    got = rb.relu_backward(payload, n, dy.view(it).numpy().view(np_t))
    assert got.tobytes() == want.view(it).numpy().tobytes()


def test_nan_and_negative_zero_in_the_gradient_pass_through_unchanged():
    y = np.array([0.0, 1.0, 0.0, 2.0, 3.0], dtype=np.float32)
    dy = np.array([np.nan, -0.0, 5.0, np.inf, -7.5], dtype=np.float32)
    payload, _ = zvc_c.compress(y)
    got = rb.relu_backward(payload, 5, dy)
    assert got.view(np.uint32).tolist() == [0, 0x80000000, 0, 0x7F800000, np.float32(-7.5).view(np.uint32)]


def test_follows_the_bit_pattern_of_y_not_its_value():
    # -0.0 and a NaN in y are non-zero patterns: the gradient passes (a ReLU output never holds -0.0;
    # a NaN passes the gradient in the usual "y <= 0 ? 0 : dy" formulation too)
    y = np.array([0x80000000, 0x7FC00000, 0x00000000, 0x00000001], dtype=np.uint32)
    dy = np.array([1.5, 2.5, 3.5, 4.5], dtype=np.float32)
    payload, _ = zvc_c.compress(y)
    got = rb.relu_backward(payload, 4, dy)
    assert got.tolist() == [1.5, 2.5, 0.0, 4.5]
    t = torch.tensor([float("nan")], requires_grad=True)
    torch.relu(t).backward(torch.tensor([2.5]))
    assert float(t.grad[0]) == 2.5
