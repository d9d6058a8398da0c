"""The N > 1 path on CPU: two gloo ranks each compress a chunk-aligned range of
one tensor; concatenating their payloads and globalising their tables must give
exactly the stream and table of the whole tensor.  (On GPUs every rank would
call the CUDA library; here the CPU oracle stands in for it, the host logic
under test is the partition and the offset exchange.)"""
import os
import socket
import tempfile

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_1705_01626_b200 import shard


def test_partition_is_chunk_aligned_and_covers():
    for n in (0, 1, 1023, 1024, 1025, 10_000, 1 << 20, (1 << 20) + 5):
        for world in (1, 2, 3, 8):
            parts = shard.partition(n, world)
            assert len(parts) == world
            assert parts[0][0] == 0 and parts[-1][1] == n
            for (a, b), (c, d) in zip(parts, parts[1:]):
                assert b == c
            for lo, hi in parts:
                assert lo <= hi and (lo % 1024 == 0 or lo == n)
            sizes = [((hi - lo) + 1023) // 1024 for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1
    assert shard.exclusive_offsets([5, 0, 7]) == [0, 5, 5]


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, n, outdir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import zvc_c
        rng = np.random.default_rng(1234)                  # same tensor on every rank
        x = rng.standard_normal(n).astype(np.float32)
        x[rng.random(n) < 0.6] = 0
        lo, hi = shard.partition(n, world)[rank]
        payload, table = zvc_c.compress(x[lo:hi])
        sizes = shard.gather_payload_sizes(len(payload))
        offs = shard.exclusive_offsets(sizes)
        gtab = shard.globalize_table(table, offs[rank], rank == world - 1)
        np.save(os.path.join(outdir, "payload%d.npy" % rank), payload)
        np.save(os.path.join(outdir, "table%d.npy" % rank), gtab)
        # every rank also learns the global size without moving payload bytes
        total = torch.tensor([len(payload)], dtype=torch.int64)
        dist.all_reduce(total)
        assert int(total) == sum(sizes)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n", [5 * 1024 + 300, 64 * 1024])
def test_two_ranks_reproduce_the_single_stream(n):
    from oracle import zvc_c
    world = 2
    with tempfile.TemporaryDirectory() as d:
        mp.spawn(_worker, args=(world, _free_port(), n, d), nprocs=world, join=True)
        payload = np.concatenate([np.load(os.path.join(d, "payload%d.npy" % r)) for r in range(world)])
        table = np.concatenate([np.load(os.path.join(d, "table%d.npy" % r)) for r in range(world)])
    rng = np.random.default_rng(1234)
    x = rng.standard_normal(n).astype(np.float32)
    x[rng.random(n) < 0.6] = 0
    want_payload, want_table = zvc_c.compress(x)
    assert payload.tobytes() == want_payload.tobytes()
    assert np.array_equal(table, want_table)
    assert zvc_c.decompress(payload, n, np.float32).tobytes() == x.tobytes()
