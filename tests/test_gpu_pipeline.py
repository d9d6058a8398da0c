"""GPU: the offload / prefetch context and the host-buffer calls, checked
against the CPU oracle and bit-exact round trips."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import zvc_c
from paper_1705_01626_b200 import binding as B
from paper_1705_01626_b200 import workloads as wl
from tests.gpu_helpers import raw_numpy

pytestmark = pytest.mark.gpu


def bits(x):
    return x.view(-1).view(torch.int32 if x.element_size() == 4 else torch.int16)


def make_ctx(tensors, slack=1 << 16):
    worst = max(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32 if t.element_size() == 4 else B.F16)
                + 8 * B.cdma_zvc_table_entries(t.numel())
                + B.cdma_zvc_workspace_bytes(t.numel(), B.F32) + 4096 for t in tensors)
    pinned = sum(B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32 if t.element_size() == 4 else B.F16)
                 + 8 * B.cdma_zvc_table_entries(t.numel()) + 512 for t in tensors) + slack
    return B.cdma_ctx_create(pinned, 2 * worst)


def small_offload_set():
    shapes = ((8, 56, 56), (8, 56, 56), (16, 28, 28), (16, 28, 28), (32, 14, 14), (32, 7, 7))
    return [t for t, _ in wl.vgg16_offload_set(batch=4, device="cuda", shapes=shapes)]


def test_offload_all_then_prefetch_in_reverse_order():
    tensors = small_offload_set()
    ctx = make_ctx(tensors)
    stream = torch.cuda.Stream()
    try:
        tickets, sizes = [], []
        with torch.cuda.stream(stream):
            for t in tensors:
                c, ticket = B.cdma_offload(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, stream.cuda_stream)
                assert c >= 0, B.status_string(c)
                want, _ = zvc_c.compress(raw_numpy(t))
                assert c == len(want)                       # the call returns the compressed size
                st, payload_bytes, n = B.cdma_ticket_info(ctx, ticket)
                assert (st, payload_bytes, n) == (0, c, t.numel())
                tickets.append(ticket)
                sizes.append(c)
            assert B.cdma_ctx_synchronize(ctx) == 0
            outs = [torch.full_like(t, -1.0) for t in tensors]
            for i in reversed(range(len(tensors))):        # backward pass order
                st = B.cdma_prefetch_async(ctx, tickets[i], outs[i].data_ptr(), stream.cuda_stream)
                assert st == 0, B.status_string(st)
            assert B.cdma_ctx_synchronize(ctx) == 0
        stream.synchronize()
        for t, o in zip(tensors, outs):
            assert torch.equal(bits(o), bits(t))
        # tickets are consumed
        assert B.cdma_prefetch(ctx, tickets[0], outs[0].data_ptr(), stream.cuda_stream) == -B.ERR_BAD_TICKET
        ratio = sum(t.numel() * 4 for t in tensors) / sum(sizes)
        assert 1.5 < ratio < 8
    finally:
        B.cdma_ctx_destroy(ctx)


def test_blocking_prefetch_and_pool_reuse():
    tensors = small_offload_set()[:3]
    ctx = make_ctx(tensors)
    try:
        for rounds in range(3):                             # the pinned pool is recycled
            tickets = []
            for t in tensors:
                c, ticket = B.cdma_offload(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, 0)
                assert c > 0
                tickets.append(ticket)
            for t, ticket in zip(tensors, tickets):
                out = torch.zeros_like(t)
                r = B.cdma_prefetch(ctx, ticket, out.data_ptr(), 0)
                assert r == t.numel() * 4, B.status_string(r)
                assert torch.equal(bits(out), bits(t))
    finally:
        B.cdma_ctx_destroy(ctx)


def test_pool_exhaustion_and_small_staging_are_reported():
    t = wl.iid_relu_like((64 * 1024,), 0.9, seed=3, device="cuda")
    need = B.cdma_zvc_max_compressed_bytes(t.numel(), B.F32)
    ctx = B.cdma_ctx_create(4096, 2 * (need + 65536))       # pinned pool far too small
    try:
        c, _ = B.cdma_offload(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, 0)
        assert c == -B.ERR_OUT_OF_MEMORY
    finally:
        B.cdma_ctx_destroy(ctx)
    ctx = B.cdma_ctx_create(1 << 20, 2 * 65536)             # staging slot smaller than the payload
    try:
        c, _ = B.cdma_offload(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, 0)
        assert c == -B.ERR_BUFFER_TOO_SMALL
        # the context still works for a tensor that fits
        s = wl.iid_relu_like((8 * 1024,), 0.1, seed=4, device="cuda")
        c, ticket = B.cdma_offload(ctx, s.data_ptr(), s.numel(), B.F32, B.NCHW, 0)
        assert c > 0
        out = torch.zeros_like(s)
        assert B.cdma_prefetch(ctx, ticket, out.data_ptr(), 0) == 4 * s.numel()
        assert torch.equal(bits(out), bits(s))
    finally:
        B.cdma_ctx_destroy(ctx)


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
def test_host_buffer_calls_match_the_oracle(dtype, pinned):
    """Page-locked buffers take the one-kernel path (the kernel reads and writes host
    memory directly); pageable ones are staged through device memory."""
    n = 300_000 + 77
    code = B.F32 if dtype == torch.float32 else B.F16
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t)
    x = pin(wl.iid_relu_like((n,), 0.3, seed=8, device="cpu", dtype=dtype, floor=2.0 ** -10))
    cap = B.cdma_zvc_max_compressed_bytes(n, code)
    entries = B.cdma_zvc_table_entries(n)
    h_p = pin(torch.zeros(cap, dtype=torch.uint8))
    h_t = pin(torch.zeros(entries, dtype=torch.int64))
    h_y = pin(torch.zeros(n, dtype=dtype))
    ctx = B.cdma_ctx_create(1 << 16, 2 * (cap + 8 * entries + B.cdma_zvc_workspace_bytes(n, code) + 4096))
    try:
        c = B.cdma_zvc_compress_host(ctx, x.data_ptr(), n, code, B.NCHW, h_p.data_ptr(), cap, h_t.data_ptr())
        want, want_table = zvc_c.compress(x.numpy().view(np.uint32 if dtype == torch.float32 else np.uint16))
        assert c == len(want), B.status_string(c)
        assert h_p[:c].numpy().tobytes() == want.tobytes()
        assert np.array_equal(h_t.numpy().view(np.uint64), want_table)
        r = B.cdma_zvc_decompress_host(ctx, h_p.data_ptr(), c, h_t.data_ptr(), n, code, B.NCHW, h_y.data_ptr())
        assert r == n * x.element_size(), B.status_string(r)
        assert torch.equal(bits(h_y), bits(x))
        # too small a host destination is refused
        assert B.cdma_zvc_compress_host(ctx, x.data_ptr(), n, code, B.NCHW, h_p.data_ptr(), c - 4,
                                        h_t.data_ptr()) == -B.ERR_BUFFER_TOO_SMALL
        # a corrupted table is reported, not followed
        bad = pin(h_t.clone())
        bad[1] += 4
        assert B.cdma_zvc_decompress_host(ctx, h_p.data_ptr(), c, bad.data_ptr(), n, code, B.NCHW,
                                          h_y.data_ptr()) == -B.ERR_CORRUPT_STREAM
    finally:
        B.cdma_ctx_destroy(ctx)


def test_one_byte_elements_through_the_pipeline_and_the_host_buffer_calls():
    """1-byte elements: staged offload / prefetch, direct offload / prefetch, and the page-locked
    host-buffer calls (kernels reading and writing host memory), all against the oracle."""
    n = 900_000 + 41
    raw = np.random.default_rng(12).integers(1, 255, size=n, dtype=np.uint8)
    raw[np.random.default_rng(13).random(n) >= 0.35] = 0
    x = torch.from_numpy(raw).cuda()
    want, want_table = zvc_c.compress(raw)
    cap = B.cdma_zvc_max_compressed_bytes(n, B.U8)
    entries = B.cdma_zvc_table_entries(n)
    ctx = B.cdma_ctx_create(4 * (cap + 8 * entries + 4096), 2 * (cap + 8 * entries + B.cdma_zvc_workspace_bytes(n, B.U8) + 4096))
    try:
        for offload, prefetch in ((B.cdma_offload, B.cdma_prefetch), (B.cdma_offload_direct, B.cdma_prefetch_direct)):
            c, ticket = offload(ctx, x.data_ptr(), n, B.U8, B.NCHW, 0)
            assert c == len(want), B.status_string(c)
            assert B.cdma_ctx_synchronize(ctx) == 0
            payload, table = host_view(ctx, ticket, c, entries)
            assert payload.tobytes() == want.tobytes()
            assert np.array_equal(table, want_table)
            out = torch.full_like(x, 7)
            assert prefetch(ctx, ticket, out.data_ptr(), 0) == n
            assert torch.equal(out, x)
        h_x = torch.from_numpy(raw).pin_memory()
        h_p = torch.zeros(cap, dtype=torch.uint8).pin_memory()
        h_t = torch.zeros(entries, dtype=torch.int64).pin_memory()
        h_y = torch.zeros(n, dtype=torch.uint8).pin_memory()
        c = B.cdma_zvc_compress_host(ctx, h_x.data_ptr(), n, B.U8, B.NCHW, h_p.data_ptr(), cap, h_t.data_ptr())
        assert c == len(want), B.status_string(c)
        assert h_p[:c].numpy().tobytes() == want.tobytes()
        assert np.array_equal(h_t.numpy().view(np.uint64), want_table)
        assert B.cdma_zvc_decompress_host(ctx, h_p.data_ptr(), c, h_t.data_ptr(), n, B.U8, B.NCHW, h_y.data_ptr()) == n
        assert torch.equal(h_y, h_x)
    finally:
        B.cdma_ctx_destroy(ctx)


def host_view(ctx, ticket, nbytes, entries):
    st, hp, ht = B.cdma_ticket_host_view(ctx, ticket)
    assert st == 0
    payload = np.frombuffer(ctypes.string_at(hp, nbytes), dtype=np.uint8)
    table = np.frombuffer(ctypes.string_at(ht, 8 * entries), dtype=np.uint64)
    return payload, table


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
def test_direct_offload_writes_the_oracle_stream_into_the_pinned_pool(dtype):
    code = B.F32 if dtype == torch.float32 else B.F16
    tensors = [wl.iid_relu_like((n,), d, seed=31 + i, device="cuda", dtype=dtype, floor=2.0 ** -10)
               for i, (n, d) in enumerate([(700_000 + 13, 0.3), (12 * 1024 * 5, 0.9), (1000, 0.0), (333_333, 0.05)])]
    worst = max(B.cdma_zvc_max_compressed_bytes(t.numel(), code) + 8 * B.cdma_zvc_table_entries(t.numel()) + 4096
                for t in tensors)
    ctx = B.cdma_ctx_create(len(tensors) * worst + (1 << 16), 2 * (worst + (1 << 20)))
    try:
        tickets = []
        for t in tensors:                                    # direct: kernel stores into host memory
            c, tk = B.cdma_offload_direct(ctx, t.data_ptr(), t.numel(), code, B.NCHW, 0)
            assert c >= 0, B.status_string(c)
            want, want_table = zvc_c.compress(raw_numpy(t))
            assert c == len(want)
            got, got_table = host_view(ctx, tk, c, B.cdma_zvc_table_entries(t.numel()))
            assert got.tobytes() == want.tobytes()
            assert np.array_equal(got_table, want_table)
            tickets.append(tk)
        # staged tickets hold the same bytes
        c2, tk2 = B.cdma_offload(ctx, tensors[0].data_ptr(), tensors[0].numel(), code, B.NCHW, 0)
        got, got_table = host_view(ctx, tk2, c2, B.cdma_zvc_table_entries(tensors[0].numel()))
        want, want_table = zvc_c.compress(raw_numpy(tensors[0]))
        assert got.tobytes() == want.tobytes() and np.array_equal(got_table, want_table)
        # either kind of ticket can come back either way
        outs = [torch.full_like(t, 3.0) for t in tensors]
        for i in reversed(range(len(tensors))):
            if i % 2 == 0:
                r = B.cdma_prefetch_direct(ctx, tickets[i], outs[i].data_ptr(), 0)
            else:
                r = B.cdma_prefetch(ctx, tickets[i], outs[i].data_ptr(), 0)
            assert r == tensors[i].numel() * tensors[i].element_size(), B.status_string(r)
            assert torch.equal(bits(outs[i]), bits(tensors[i]))
        out = torch.zeros_like(tensors[0])
        assert B.cdma_prefetch_direct(ctx, tk2, out.data_ptr(), 0) == out.numel() * out.element_size()
        assert torch.equal(bits(out), bits(tensors[0]))
        assert B.cdma_prefetch_direct(ctx, tk2, out.data_ptr(), 0) == -B.ERR_BAD_TICKET
        # the worst-case reservation was given back: the pool takes the same set again
        for t in tensors:
            c, tk = B.cdma_offload_direct(ctx, t.data_ptr(), t.numel(), code, B.NCHW, 0)
            assert c >= 0
        assert B.cdma_ctx_synchronize(ctx) == 0
    finally:
        B.cdma_ctx_destroy(ctx)


def test_offload_async_returns_before_the_compute_stream_has_caught_up():
    """OFF must not make the host wait for the layer that produces the map (Fig. 2b): with a long-running
    operation queued on the compute stream in front of it, the call comes back while that operation is
    still running; the ticket later yields the oracle's bytes."""
    t = wl.correlated_relu((8, 32, 56, 56), 0.3, seed=77, device="cuda")
    n = t.numel()
    ctx = make_ctx([t], slack=1 << 20)
    stream = torch.cuda.Stream()
    a = torch.randn(8192, 8192, device="cuda")
    busy = torch.cuda.Event()
    try:
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            for _ in range(40):                              # tens of milliseconds of work in front of the offload
                a = torch.mm(a, a).clamp_(-1.0, 1.0)
            busy.record(stream)
            st, ticket = B.cdma_offload_async(ctx, t.data_ptr(), n, B.F32, B.NCHW, stream.cuda_stream)
            still_running = not busy.query()                 # looked at right after the call returned
        assert st == 0, B.status_string(st)
        assert still_running, "cdma_offload_async waited for the compute stream"
        want, want_table = zvc_c.compress(raw_numpy(t))
        st, c, n_back = B.cdma_ticket_info(ctx, ticket)      # settles the ticket (waits for its bytes)
        assert (st, c, n_back) == (0, len(want), n)
        got, got_table = host_view(ctx, ticket, c, B.cdma_zvc_table_entries(n))
        assert got.tobytes() == want.tobytes()
        assert np.array_equal(got_table, want_table)
        out = torch.zeros_like(t)
        assert B.cdma_prefetch(ctx, ticket, out.data_ptr(), stream.cuda_stream) == 4 * n
        assert torch.equal(bits(out), bits(t))
        assert B.cdma_ctx_synchronize(ctx) == 0
    finally:
        B.cdma_ctx_destroy(ctx)


def test_offload_async_reports_a_slot_too_small_through_synchronize():
    t = wl.iid_relu_like((64 * 1024,), 0.9, seed=3, device="cuda")
    ctx = B.cdma_ctx_create(1 << 20, 2 * 65536)             # staging slot smaller than the payload
    try:
        st, ticket = B.cdma_offload_async(ctx, t.data_ptr(), t.numel(), B.F32, B.NCHW, 0)
        assert st == 0
        assert B.cdma_ctx_synchronize(ctx) == B.ERR_BUFFER_TOO_SMALL
        assert B.cdma_ticket_info(ctx, ticket)[0] == B.ERR_BAD_TICKET      # the ticket was dropped
        assert B.cdma_ctx_synchronize(ctx) == 0
        s = wl.iid_relu_like((8 * 1024,), 0.1, seed=4, device="cuda")      # the context still works
        st, ticket = B.cdma_offload_async(ctx, s.data_ptr(), s.numel(), B.F32, B.NCHW, 0)
        assert st == 0
        out = torch.zeros_like(s)
        assert B.cdma_prefetch(ctx, ticket, out.data_ptr(), 0) == 4 * s.numel()
        assert torch.equal(bits(out), bits(s))
    finally:
        B.cdma_ctx_destroy(ctx)


def test_prefetch_async_then_direct_offload_into_the_recycled_region():
    """The end of a backward pass followed by the next forward pass: a prefetch whose host-to-device copy
    is still in flight gives its pinned region back, and a direct offload (a kernel that writes the pool
    from the caller's stream) is handed that very region.  Both tensors must come out bit-exact."""
    a = wl.iid_relu_like((6_000_000,), 0.6, seed=41, device="cuda")      # ~15 MB payload: a copy that takes a while
    b = wl.iid_relu_like((6_000_000,), 0.6, seed=42, device="cuda")
    need = B.cdma_zvc_max_compressed_bytes(a.numel(), B.F32) + 8 * B.cdma_zvc_table_entries(a.numel()) + 4096
    ws = B.cdma_zvc_workspace_bytes(a.numel(), B.F32)
    ctx = B.cdma_ctx_create(need + 8192, 2 * (need + ws + 4096))          # room for exactly one ticket
    stream = torch.cuda.Stream()
    try:
        for _ in range(4):
            c, tk_a = B.cdma_offload_direct(ctx, a.data_ptr(), a.numel(), B.F32, B.NCHW, stream.cuda_stream)
            assert c > 0, B.status_string(c)
            out_a = torch.zeros_like(a)
            assert B.cdma_prefetch_async(ctx, tk_a, out_a.data_ptr(), stream.cuda_stream) == 0
            # no synchronisation here: the copy of a's payload out of the pool may still be running
            c, tk_b = B.cdma_offload_direct(ctx, b.data_ptr(), b.numel(), B.F32, B.NCHW, stream.cuda_stream)
            assert c > 0, B.status_string(c)
            out_b = torch.zeros_like(b)
            assert B.cdma_prefetch(ctx, tk_b, out_b.data_ptr(), stream.cuda_stream) == 4 * b.numel()
            assert B.cdma_ctx_synchronize(ctx) == 0
            stream.synchronize()
            assert torch.equal(bits(out_a), bits(a))
            assert torch.equal(bits(out_b), bits(b))
    finally:
        B.cdma_ctx_destroy(ctx)
