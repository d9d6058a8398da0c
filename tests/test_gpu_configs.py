"""GPU parity at the benchmark's full sizes, in the launch configuration the
benchmark times.  The whole payload and table are compared with the CPU oracle
(run on all host cores), the 2^29-element tensors and the 13-tensor offload set
included; sizes are also checked against the closed form and every round trip
bit for bit."""
import ctypes
import os

import numpy as np
import pytest
import torch

from oracle import zvc_c
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import DeviceCodec, raw_numpy

pytestmark = pytest.mark.gpu

CORES = len(os.sched_getaffinity(0))


def bits(x):
    return x.view(-1).view({4: torch.int32, 2: torch.int16, 1: torch.uint8}[x.element_size()])


def full_compare(x):
    n = x.numel()
    codec = DeviceCodec(n, x.dtype)
    c = codec.compress(x)
    assert c >= 0, B.status_string(c)
    raw = raw_numpy(x)
    want, want_table = zvc_c.compress(raw, threads=CORES)
    assert c == len(want)
    assert codec.payload_numpy(c).tobytes() == want.tobytes()
    assert np.array_equal(codec.table_numpy(), want_table)
    out = torch.empty_like(x)
    assert codec.decompress(out, c) == n * x.element_size()
    assert torch.equal(bits(out), bits(x))
    assert codec.canaries_intact()
    return c


def test_config2_vgg_conv1_2_full_size():
    x = wl.per_channel_beta(device="cuda")
    assert x.numel() == 64 * 64 * 224 * 224
    c = full_compare(x)
    assert 2.0 < x.numel() * 4 / c < 4.0


def test_config4_layout_and_density_sweep():
    sizes = {}
    for d, layout, x in wl.layout_density_sweep(device="cuda"):
        codec = DeviceCodec(x.numel(), x.dtype)
        c = codec.compress(x, layout=B.LAYOUT_CODES[layout])
        nnz = int(torch.count_nonzero(bits(x)))
        assert c == 4 * (x.numel() // 32) + 4 * nnz
        out = torch.empty_like(x)
        assert codec.decompress(out, c, layout=B.LAYOUT_CODES[layout]) == 4 * x.numel()
        assert torch.equal(bits(out), bits(x))
        sizes.setdefault(d, set()).add(c)
        if layout == "NHWC" and d in (0.05, 1.0):           # whole-stream parity on two points
            want, table = zvc_c.compress(raw_numpy(x), threads=CORES)
            assert codec.payload_numpy(c).tobytes() == want.tobytes()
            assert np.array_equal(codec.table_numpy(), table)
    # the compressed size does not depend on the layout (Section V-A)
    assert all(len(s) == 1 for s in sizes.values())
    # all-dense: the mask is pure overhead, 1/32 of the input
    (c_dense,) = sizes[1.0]
    assert c_dense == 128 * 256 * 28 * 28 * 4 * 33 // 32


@pytest.mark.parametrize("which", ["a", "b", "c"])
def test_config5_large_extremes(which):
    x = wl.large_extremes(which, device="cuda")
    n, s = x.numel(), x.element_size()
    assert n == 1 << 29
    codec = DeviceCodec(n, x.dtype)
    c = codec.compress(x)
    assert c >= 0, B.status_string(c)
    nnz = int(torch.count_nonzero(bits(x)))
    assert c == 4 * (n // 32) + s * nnz                      # closed form, 64-bit offsets (c > 2^31 for b)
    if which == "b":
        assert c == 2_214_592_512
    table = codec.table_numpy()
    assert table[0] == 0 and table[-1] == c and (np.diff(table.astype(np.int64)) >= 128).all()
    out = torch.empty_like(x)
    assert codec.decompress(out, c) == n * s
    assert torch.equal(bits(out), bits(x))
    assert codec.canaries_intact()
    del out
    # the whole stream and table, byte for byte against the oracle (all host cores)
    want, want_table = zvc_c.compress(raw_numpy(x), threads=CORES)
    assert c == len(want)
    assert np.array_equal(table, want_table)
    step = 1 << 28                                           # compare in pieces: bounded host copies
    for lo in range(0, c, step):
        hi = min(c, lo + step)
        assert codec.payload[lo:hi].cpu().numpy().tobytes() == want[lo:hi].tobytes()
    del want, want_table
    del codec, x
    torch.cuda.empty_cache()


def _ticket_bytes(ctx, ticket):
    st, c, n = B.cdma_ticket_info(ctx, ticket)
    assert st == 0
    st, hp, ht = B.cdma_ticket_host_view(ctx, ticket)
    assert st == 0
    payload = np.ctypeslib.as_array((ctypes.c_uint8 * c).from_address(hp)) if c else np.zeros(0, np.uint8)
    table = np.ctypeslib.as_array((ctypes.c_uint64 * (n // 1024 + 1)).from_address(ht))
    return c, payload, table


@pytest.mark.parametrize("mode", ["staged", "direct", "async"])
def test_config3_offload_set_full_size(mode):
    """The 13 conv outputs of the VGG-16-shaped network at batch 64 (3.47 GB): every tensor offloaded
    (OFF in forward order), each ticket's bytes in the pinned pool compared with the oracle, then
    prefetched in reverse order (PRE in backward order) and compared bit for bit."""
    tensors = [t for t, _ in wl.vgg16_offload_set(device="cuda")]
    assert len(tensors) == 13 and sum(t.numel() for t in tensors) == 867_041_280
    worst = max(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32) + 8 * B.cdma_zvc_table_entries(t.numel())
                + B.cdma_zvc_workspace_bytes(t.numel(), B.F32) + 4096 for t in tensors)
    pinned = sum(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32) // 2 + 8 * B.cdma_zvc_table_entries(t.numel())
                 + 4096 for t in tensors) + worst
    ctx = B.cdma_ctx_create(pinned, 2 * worst)
    stream = torch.cuda.Stream()
    try:
        tickets = []
        with torch.cuda.stream(stream):
            for t in tensors:
                if mode == "async":
                    st, tk = B.cdma_offload_async(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, stream.cuda_stream)
                    assert st == 0, B.status_string(st)
                else:
                    off = B.cdma_offload if mode == "staged" else B.cdma_offload_direct
                    c, tk = off(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, stream.cuda_stream)
                    assert c > 0, B.status_string(c)
                tickets.append(tk)
            assert B.cdma_ctx_synchronize(ctx) == 0
            total = 0
            for t, tk in zip(tensors, tickets):
                c, payload, table = _ticket_bytes(ctx, tk)
                want, want_table = zvc_c.compress(raw_numpy(t), threads=CORES)
                assert c == len(want)
                assert payload.tobytes() == want.tobytes()
                assert np.array_equal(table, want_table)
                total += c
            assert 2.0 < sum(t.numel() * 4 for t in tensors) / total < 2.6     # size-weighted ratio
            outs = [torch.empty_like(t) for t in tensors]
            for i in reversed(range(len(tensors))):
                if mode == "direct":
                    r = B.cdma_prefetch_direct(ctx, tickets[i], outs[i].data_ptr(), stream.cuda_stream)
                    assert r == tensors[i].numel() * 4, B.status_string(r)
                else:
                    st = B.cdma_prefetch_async(ctx, tickets[i], outs[i].data_ptr(), stream.cuda_stream)
                    assert st == 0, B.status_string(st)
            assert B.cdma_ctx_synchronize(ctx) == 0
        stream.synchronize()
        for t, o in zip(tensors, outs):
            assert torch.equal(bits(o), bits(t))
    finally:
        B.cdma_ctx_destroy(ctx)
        del tensors
        torch.cuda.empty_cache()


def test_more_than_two_to_the_32_elements():
    """Element indices beyond 32 bits: 2^32 + 70,001 one-byte elements (4 GiB; ragged chunk, group and tile),
    the whole payload and table against the oracle, and the round trip."""
    n = (1 << 32) + 70_001
    g = torch.Generator(device="cuda").manual_seed(170501626 + 5900)
    x = torch.randint(1, 256, (n,), dtype=torch.uint8, device="cuda", generator=g)
    # zeros in runs of 1 .. 4096 elements so that chunks differ widely in size
    keep = torch.rand((n + 4095) // 4096, device="cuda", generator=g) < 0.3
    x *= keep.repeat_interleave(4096)[:n].to(torch.uint8)
    x *= (torch.rand(n, device="cuda", generator=g) < 0.8).to(torch.uint8)
    del keep
    c = full_compare(x)
    assert c == 4 * ((n + 31) // 32) + int(torch.count_nonzero(x))
