"""GPU: cdma_zvc_relu_backward (gradient gated by the masks of a compressed map) against the
CPU oracle, bit for bit (a selection of bit patterns: tolerance 0)."""
import numpy as np
import pytest
import torch

from oracle import relu_backward as rb
from oracle import zvc_c, zvc_numpy
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import DT, DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu


def run(x, dy, in_place=False):
    n = x.numel()
    codec = DeviceCodec(n, x.dtype)
    c = codec.compress(x)
    assert c >= 0, B.status_string(c)
    dx = dy if in_place else torch.full_like(dy, 9.0)
    dy_raw = raw_numpy(dy).copy()
    r = B.cdma_zvc_relu_backward(codec.payload.data_ptr(), c, codec.table.data_ptr(), n, codec.code, B.NCHW,
                                 dy.data_ptr() if n else 0, dx.data_ptr() if n else 0, codec.ws.data_ptr(),
                                 codec.ws_bytes, 0)
    assert r == n * x.element_size(), B.status_string(r)
    want = rb.relu_backward(zvc_c.compress(raw_numpy(x))[0], n, dy_raw)
    assert raw_numpy(dx).tobytes() == want.tobytes()
    return codec, c


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("n", [1, 31, 33, 1023, 1024, 1025, 8 * 1024 + 5, 300_000 + 77])
def test_matches_the_oracle(dtype, n):
    for i, density in enumerate([0.05, 0.5, 1.0]):
        x = wl.iid_relu_like((n,), density, seed=4000 + n + i, device="cuda", dtype=dtype, floor=2.0 ** -10)
        dy = torch.randn(n, device="cuda").to(dtype)
        run(x, dy)


def test_one_byte_elements():
    for n, density in [(5, 1.0), (1024, 0.5), (70_000 + 3, 0.2)]:
        raw = np.random.default_rng(n).integers(1, 255, size=n, dtype=np.uint8)
        raw[np.random.default_rng(n + 1).random(n) >= density] = 0
        x = torch.from_numpy(raw).cuda()
        dy = torch.from_numpy(np.random.default_rng(n + 2).integers(0, 255, size=n, dtype=np.uint8)).cuda()
        run(x, dy)


def test_is_the_relu_backward_of_the_framework_on_a_fused_forward():
    n = 1_000_000 + 3
    x = torch.randn(n, device="cuda", requires_grad=True)
    dy = torch.randn(n, device="cuda")
    torch.relu(x).backward(dy)
    codec = DeviceCodec(n, torch.float32)
    c = B.cdma_zvc_relu_compress(x.data_ptr(), n, B.F32, B.NCHW, 0, codec.payload.data_ptr(), codec.cap,
                                 codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0)
    assert c > 0
    dx = torch.empty_like(dy)
    assert B.cdma_zvc_relu_backward(codec.payload.data_ptr(), c, codec.table.data_ptr(), n, B.F32, B.NCHW,
                                    dy.data_ptr(), dx.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0) == 4 * n
    assert torch.equal(dx.view(torch.int32), x.grad.view(torch.int32))


def test_in_place_and_special_values():
    x = wl.special_values(70_000, seed=6, dtype=torch.float32, device="cuda")
    dy = wl.special_values(70_000, seed=7, dtype=torch.float32, device="cuda")
    run(x, dy.clone(), in_place=True)
    h = wl.special_values(70_001, seed=8, dtype=torch.float16, device="cuda")
    run(h, wl.special_values(70_001, seed=9, dtype=torch.float16, device="cuda"))


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.uint8])
def test_corrupt_streams_and_bad_arguments_are_refused(dtype):
    n = 20_000
    s = torch.empty(0, dtype=dtype).element_size()
    if dtype == torch.uint8:
        raw = np.random.default_rng(5).integers(1, 255, size=n, dtype=np.uint8)
        raw[np.random.default_rng(6).random(n) >= 0.4] = 0
        x = torch.from_numpy(raw).cuda()
        dy = torch.from_numpy(np.random.default_rng(7).integers(0, 255, size=n, dtype=np.uint8)).cuda()
    else:
        x = wl.iid_relu_like((n,), 0.4, seed=77, device="cuda", dtype=dtype, floor=2.0 ** -10)
        dy = torch.randn(n, device="cuda").to(dtype)
    dx = torch.empty_like(dy)
    codec = DeviceCodec(n, dtype)
    c = codec.compress(x)
    args = lambda payload_bytes=c, table=codec.table: (codec.payload.data_ptr(), payload_bytes, table.data_ptr(), n,
                                                       codec.code, B.NCHW, dy.data_ptr(), dx.data_ptr(),
                                                       codec.ws.data_ptr(), codec.ws_bytes, 0)
    bad = codec.table.clone()
    bad[3] += 4
    assert B.cdma_zvc_relu_backward(*args(table=bad)) == -B.ERR_CORRUPT_STREAM
    assert B.cdma_zvc_relu_backward(*args(payload_bytes=c - 4)) == -B.ERR_CORRUPT_STREAM
    payload = codec.payload.clone()
    # one bit flipped in the mask of a chunk's last window: the walk misses the chunk's end
    # (an earlier window could fall back into step on narrow elements)
    last_mask = int(zvc_numpy.window_offsets(raw_numpy(x))[3 * 32 - 1])
    codec.payload[last_mask] ^= 0x10
    assert B.cdma_zvc_relu_backward(*args()) == -B.ERR_CORRUPT_STREAM
    codec.payload.copy_(payload)
    assert B.cdma_zvc_relu_backward(*args()) == s * n                  # and the intact stream still works
    assert codec.canaries_intact()
    # overlap of dx with the payload
    assert B.cdma_zvc_relu_backward(codec.payload.data_ptr(), c, codec.table.data_ptr(), n, codec.code, B.NCHW,
                                    dy.data_ptr(), codec.payload.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes,
                                    0) == -B.ERR_INVALID_ARG
