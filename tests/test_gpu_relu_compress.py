"""GPU: activation function + compression in one pass (cdma_zvc_relu_compress).

The expected result is written out from the definition with plain PyTorch CPU
ops -- y = x where x > 0 or x is NaN, else +0 -- followed by the CPU oracle's
compression of y; the kernel decides the same thing on bit patterns.  Bit-exact
bar: payload, table, and the dense y it optionally writes."""
import numpy as np
import pytest
import torch

from oracle import zvc_c
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import DT, DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu


def relu_reference(x_cpu: torch.Tensor) -> torch.Tensor:
    keep = torch.isnan(x_cpu) | (x_cpu > 0)
    return torch.where(keep, x_cpu, torch.zeros_like(x_cpu))


def pre_activations(n, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    x = (torch.randn(n, generator=g) - 0.4).to(dtype)
    # sprinkle special values: +-0, +-NaN with payloads, +-Inf, denormals
    sp = wl.special_values(max(1, n // 7), seed=seed + 1, dtype=torch.float32 if dtype == torch.float32 else torch.float16)
    if dtype == torch.bfloat16:
        sp = sp.view(torch.int16).view(torch.bfloat16)
    idx = torch.randperm(n, generator=g)[: sp.numel()]
    x[idx] = sp.to(dtype) if sp.dtype != dtype else sp
    return x


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("n", [1, 33, 1024, 12 * 1024 + 5, 24 * 1024 * 3 + 1000, 400_000 + 3])
def test_relu_compress_matches_relu_then_oracle(n, dtype):
    x_cpu = pre_activations(n, dtype, 100 + n % 97)
    y_cpu = relu_reference(x_cpu)
    want, want_table = zvc_c.compress(raw_numpy(y_cpu))
    x = x_cpu.cuda()
    codec = DeviceCodec(n, dtype)
    y = torch.full_like(x, 7.0)
    c = B.cdma_zvc_relu_compress(x.data_ptr(), n, DT[dtype], B.NCHW, y.data_ptr(), codec.payload.data_ptr(), codec.cap,
                                 codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0)
    assert c == len(want), B.status_string(c)
    assert codec.payload_numpy(c).tobytes() == want.tobytes()
    assert np.array_equal(codec.table_numpy(), want_table)
    assert raw_numpy(y).tobytes() == raw_numpy(y_cpu).tobytes()
    assert codec.canaries_intact()
    # decompressing gives y back
    out = torch.empty_like(x)
    assert codec.decompress(out, c) == n * x.element_size()
    assert raw_numpy(out).tobytes() == raw_numpy(y_cpu).tobytes()
    # without the dense output, and in place
    codec2 = DeviceCodec(n, dtype)
    assert B.cdma_zvc_relu_compress(x.data_ptr(), n, DT[dtype], B.NCHW, 0, codec2.payload.data_ptr(), codec2.cap,
                                    codec2.table.data_ptr(), codec2.ws.data_ptr(), codec2.ws_bytes, 0) == c
    assert codec2.payload_numpy(c).tobytes() == want.tobytes()
    assert raw_numpy(x).tobytes() == raw_numpy(x_cpu).tobytes()            # the input was not touched
    codec3 = DeviceCodec(n, dtype)
    assert B.cdma_zvc_relu_compress(x.data_ptr(), n, DT[dtype], B.NCHW, x.data_ptr(), codec3.payload.data_ptr(),
                                    codec3.cap, codec3.table.data_ptr(), codec3.ws.data_ptr(), codec3.ws_bytes, 0) == c
    assert codec3.payload_numpy(c).tobytes() == want.tobytes()
    assert raw_numpy(x).tobytes() == raw_numpy(y_cpu).tobytes()            # in-place activation


def test_relu_rule_on_special_values():
    # +0, -0, +tiny, -tiny, +Inf, -Inf, +qNaN, -qNaN, +sNaN payload, -sNaN payload, 1.0, -1.0
    bits = np.array([0x00000000, 0x80000000, 0x00000001, 0x80000001, 0x7F800000, 0xFF800000,
                     0x7FC00000, 0xFFC00000, 0x7F800123, 0xFF800123, 0x3F800000, 0xBF800000], dtype=np.uint32)
    keep = np.array([0, 0, 1, 0, 1, 0, 1, 1, 1, 1, 1, 0], dtype=bool)
    x = torch.from_numpy(bits.view(np.int32)).cuda().view(torch.float32)
    codec = DeviceCodec(12, torch.float32)
    y = torch.empty_like(x)
    c = B.cdma_zvc_relu_compress(x.data_ptr(), 12, B.F32, B.NCHW, y.data_ptr(), codec.payload.data_ptr(), codec.cap,
                                 codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0)
    assert c == 4 + 4 * int(keep.sum())
    assert np.array_equal(raw_numpy(y), np.where(keep, bits, 0).astype(np.uint32))
    # and plain PyTorch agrees with that table
    ref = relu_reference(torch.from_numpy(bits.view(np.int32)).view(torch.float32))
    assert np.array_equal(raw_numpy(ref), np.where(keep, bits, 0).astype(np.uint32))


def test_relu_compress_argument_checks():
    x = torch.randn(4096, device="cuda")
    codec = DeviceCodec(4096, torch.float32)
    args = (B.F32, B.NCHW)
    tail = (codec.payload.data_ptr(), codec.cap, codec.table.data_ptr(), codec.ws.data_ptr(), codec.ws_bytes, 0)
    assert B.cdma_zvc_relu_compress(x.data_ptr(), 4096, *args, x.data_ptr() + 4, *tail) == -B.ERR_ALIGNMENT
    assert B.cdma_zvc_relu_compress(x.data_ptr(), 4096, *args, x.data_ptr() + 1024, *tail) == -B.ERR_INVALID_ARG
    assert B.cdma_zvc_relu_compress(x.data_ptr(), 4096, *args, codec.payload.data_ptr(), *tail) == -B.ERR_INVALID_ARG
    assert B.cdma_zvc_relu_compress(x.data_ptr(), 4096, *args, 0, *tail) > 0
