"""CPU: the descriptor protocol behind the single-pass compression (decoupled
look-back) as a host-thread simulation.  The simulated tiles run the functions the
kernels themselves use for packing descriptors and for reading a round of 32
predecessors (``csrc/lookback_protocol.h``), in random publication order, with
leftovers of another launch in the workspace, and with one tile that never
publishes: every tile behind it must end with the error state and nobody may wait
for ever."""
import ctypes
import os
import subprocess

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
NO_TILE = 0xFFFFFFFF


@pytest.fixture(scope="module")
def sim(tmp_path_factory):
    out = tmp_path_factory.mktemp("lookback") / "liblookback_sim.so"
    subprocess.check_call(["g++", "-O2", "-std=c++17", "-shared", "-fPIC", "-pthread",
                           "-I", os.path.join(ROOT, "paper_1705_01626_b200", "csrc"),
                           os.path.join(ROOT, "tests", "lookback_sim.cpp"), "-o", str(out)])
    lib = ctypes.CDLL(str(out))
    lib.lookback_sim_run.restype = ctypes.c_int
    lib.lookback_sim_run.argtypes = [ctypes.c_uint32, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_uint64,
                                     ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64,
                                     ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.lookback_sim_head.restype = ctypes.c_uint64
    lib.lookback_sim_head.argtypes = [ctypes.c_uint32, ctypes.c_uint64]
    lib.lookback_sim_state.restype = ctypes.c_uint32
    lib.lookback_sim_state.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
    lib.lookback_sim_plan.restype = None
    lib.lookback_sim_plan.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p]
    return lib


def run(sim, sizes, delays, tag, stall=NO_TILE, poll_limit=200000, garbage=(0, 0)):
    tiles = len(sizes)
    sizes = np.asarray(sizes, dtype=np.uint64)
    delays = np.asarray(delays, dtype=np.uint32)
    excl = np.zeros(tiles, dtype=np.uint64)
    failed = np.zeros(tiles, dtype=np.uint32)
    polls = np.zeros(tiles, dtype=np.uint32)
    assert sim.lookback_sim_run(tiles, sizes.ctypes.data, delays.ctypes.data, tag, stall, poll_limit,
                                garbage[0], garbage[1], excl.ctypes.data, failed.ctypes.data, polls.ctypes.data) == 0
    return excl, failed, polls


def test_packing_keeps_every_bit_of_state_tag_and_value(sim):
    tags = [1, 2, 0x123456789ABCDEF, (1 << 62) - 1, (1 << 61) + 5]
    for tag in tags:
        for state in range(4):
            head = sim.lookback_sim_head(state, tag)
            assert head >> 62 == state and head & ((1 << 62) - 1) == tag
            assert sim.lookback_sim_state(head, tag) == state
            for other in tags:                               # another launch's descriptor is "not published"
                if other != tag:
                    assert sim.lookback_sim_state(head, other) == 0
    assert sim.lookback_sim_state(0xFFFFFFFFFFFFFFFF, 12345) == 0      # a workspace filled with 0xFF
    assert sim.lookback_sim_state(0, 12345) == 0


def plan(sim, m_prefix, m_invalid, m_error):
    out = (ctypes.c_uint32 * 3)()
    sim.lookback_sim_plan(m_prefix, m_invalid, m_error, out)
    return tuple(out)


def test_round_decisions(sim):
    WAIT, FAIL, CONTINUE, DONE = 0, 1, 2, 3
    assert plan(sim, 0, 0, 0) == (CONTINUE, 0xFFFFFFFF, 0)             # 32 sizes, no prefix yet: keep walking
    assert plan(sim, 1, 0, 0) == (DONE, 0, 0)                          # the nearest tile already knows its prefix
    assert plan(sim, 0b1000, 0, 0) == (DONE, 0b0111, 3)                # three sizes, then a prefix
    assert plan(sim, 0b1000, 0b10000, 0b100000)[0] == DONE             # whatever lies beyond the prefix is ignored
    assert plan(sim, 0b1000, 0b0010, 0)[0] == WAIT                     # a tile in front of the prefix is silent
    assert plan(sim, 0b1000, 0b0010, 0b0001)[0] == FAIL                # ... but an error in front decides first
    assert plan(sim, 0, 1 << 31, 0)[0] == WAIT
    assert plan(sim, 1 << 31, 0, 0) == (DONE, 0x7FFFFFFF, 31)


@pytest.mark.parametrize("tiles", [1, 2, 33, 100])
def test_random_publication_order_gives_exact_prefixes(sim, tiles):
    rng = np.random.default_rng(tiles)
    sizes = rng.integers(128, 33792, tiles).astype(np.uint64)
    if tiles > 2:
        sizes[1] = (1 << 40) + 12345                          # values well beyond 32 bits survive the walk
    delays = rng.integers(0, 3000, tiles)
    # descriptors of an earlier launch (different tag, plausible states) are lying around
    garbage = ((2 << 62) | 0x777, 999999)
    excl, failed, _ = run(sim, sizes, delays, tag=0x1234567, garbage=garbage)
    assert not failed.any()
    want = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.uint64)
    assert np.array_equal(excl, want)


@pytest.mark.parametrize("stall", [0, 5, 40])
def test_a_tile_that_never_publishes_fails_every_tile_behind_it(sim, stall):
    tiles = 70
    rng = np.random.default_rng(stall)
    sizes = rng.integers(128, 33792, tiles).astype(np.uint64)
    delays = rng.integers(0, 2000, tiles)
    excl, failed, polls = run(sim, sizes, delays, tag=99, stall=stall, poll_limit=300)
    want = np.concatenate([[0], np.cumsum(sizes)[:-1]]).astype(np.uint64)
    # tiles up to and including the silent one are unaffected (it still finds its own place)
    assert not failed[: stall + 1].any()
    assert np.array_equal(excl[: stall + 1], want[: stall + 1])
    # everybody behind it ends with the error state, after a bounded number of polls
    assert failed[stall + 1:].all()
    assert polls.max() <= 301
    # only tiles that still had the silent tile inside their look-back window had to wait for the limit;
    # the others met the error mark of a tile in front of them
    assert (polls[stall + 1:] > 300).sum() >= 1
