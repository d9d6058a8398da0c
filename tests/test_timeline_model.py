"""The step-time model against what the paper prints (Section VI) and against a
brute-force event simulation of the Fig. 2b schedule written out here."""
import math
import random

import pytest

from paper_1705_01626_b200 import timeline as tl


def test_paper_bandwidth_figures():
    # Section VI / Section V-B: PCIe gen3 at 16 GB/s, maximum per-layer ratio 13.8, average 2.6
    assert tl.comp_bw(13.8, 16.0) == pytest.approx(220.8)           # "16 x 13.8 = 220.8 GB/s"
    assert tl.comp_bw(2.6, 16.0) == pytest.approx(41.6)             # printed as 41.3: 16 x 2.6 is 41.6
    leftover = 336.0 - 100.0                                        # "336 - 100 = 236 GB/sec"
    assert leftover == 236.0
    assert tl.copy_inflation(13.8, 16.0, leftover) == 1.0           # 220.8 < 236: link stays saturated
    assert tl.copy_inflation(13.8, 16.0, 200.0) == pytest.approx(220.8 / 200.0)   # the conservative cap
    assert tl.copy_inflation(2.6, 16.0, 200.0) == 1.0


def test_copy_time_is_bytes_over_ratio_over_link():
    # 32 zeros -> 4 bytes (32x), 128-byte window of non-zeros -> 132 bytes (Section V-A)
    assert tl.copy_seconds(128.0, 32.0, 16.0) == pytest.approx(4.0 / 16e9)
    assert tl.copy_seconds(128.0, 128.0 / 132.0, 16.0) == pytest.approx(132.0 / 16e9)
    # a copy that needs more DRAM bandwidth than allowed is stretched by COMP_BW / DRAM_BW
    assert tl.copy_seconds(1e9, 13.8, 16.0, 200.0) == pytest.approx(1e9 / 13.8 / 16e9 * 1.104)


def simulate(layers, pcie_gbs, dram, compressed):
    """Event simulation: one compute engine, one copy engine, the dependencies of Fig. 2b."""
    def copy(l):
        r = l.ratio if compressed else 1.0
        t = l.act_bytes / r / (pcie_gbs * 1e9)
        if compressed and r * pcie_gbs > dram:
            t *= r * pcie_gbs / dram
        return t
    now = 0.0
    for l in layers:                       # layer and its offload start together; next layer waits for both
        compute_done = now + l.fwd_s
        copy_done = now + copy(l)
        now = max(compute_done, copy_done)
    for i in reversed(range(len(layers))):
        compute_done = now + layers[i].bwd_s
        copy_done = now + (copy(layers[i - 1]) if i > 0 else 0.0)
        now = max(compute_done, copy_done)
    return now


def test_closed_form_equals_event_simulation():
    rng = random.Random(170501626)
    for _ in range(200):
        layers = [tl.Layer(rng.uniform(1e-4, 5e-3), rng.uniform(1e-4, 1e-2), rng.uniform(1e6, 1e9),
                           rng.uniform(0.97, 13.8)) for _ in range(rng.randint(1, 16))]
        pcie = rng.choice([12.8, 16.0, 55.0])
        dram = rng.choice([50.0, 200.0, math.inf])
        for compressed in (False, True):
            assert tl.step_seconds(layers, pcie, dram, compressed) == pytest.approx(
                simulate(layers, pcie, dram, compressed), rel=1e-12)


def test_limits():
    layers = [tl.Layer(2e-3, 4e-3, 8e8, 2.6), tl.Layer(1e-3, 2e-3, 4e8, 5.0), tl.Layer(5e-4, 1e-3, 1e8, 13.8)]
    s = tl.summary(layers, 16.0, 200.0)
    assert s["oracle_s"] == pytest.approx(10.5e-3)
    assert s["oracle_s"] <= s["cdma_s"] <= s["vdnn_s"]
    # ratio 1 everywhere: compressed copies are plain copies
    plain = [tl.Layer(l.fwd_s, l.bwd_s, l.act_bytes, 1.0) for l in layers]
    assert tl.step_seconds(plain, 16.0, 200.0, True) == tl.step_seconds(plain, 16.0, compressed=False)
    # an infinitely fast link: no stall, every variant equals the oracle
    assert tl.step_seconds(layers, 1e12, compressed=False) == pytest.approx(s["oracle_s"])
    # compute-bound layers: copies are hidden, compression buys nothing
    slow = [tl.Layer(1.0, 1.0, l.act_bytes, l.ratio) for l in layers]
    assert tl.summary(slow, 16.0)["cdma_speedup_over_vdnn"] == 1.0
    # a higher ratio never makes the step longer while the DRAM cap is not hit
    better = [tl.Layer(l.fwd_s, l.bwd_s, l.act_bytes, l.ratio * 1.5) for l in layers]
    assert tl.step_seconds(better, 16.0) <= tl.step_seconds(layers, 16.0)
    assert s["traffic_reduction"] == pytest.approx(1.3e9 / (8e8 / 2.6 + 4e8 / 5.0 + 1e8 / 13.8))
    with pytest.raises(ValueError):
        tl.copy_seconds(1.0, 0.0, 16.0)
