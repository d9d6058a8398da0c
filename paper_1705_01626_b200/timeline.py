"""Analytical model of one vDNN training step with plain and with compressed
activation copies (Section VI, "Effect of cDMA on memory bandwidth"; the
offload / prefetch timeline of Section II-B, Fig. 2b).

Host arithmetic only: it takes measured layer times, activation sizes,
compression ratios and link rates and returns step times.  Nothing here touches
the GPU; `bench.py --workload timeline` feeds it with numbers measured on the
device.

What the paper fixes and this module restates:

* COMP_BW = compression ratio x PCIe rate is the DRAM read rate the codec needs
  to keep the link saturated with compressed data;
* when COMP_BW exceeds the DRAM bandwidth the codec may use (DRAM_BW, the
  paper caps it at 200 GB/s of the 336 - 100 = 236 GB/s left over by cuDNN),
  the copy of that layer takes COMP_BW / DRAM_BW times longer;
* vDNN stalls a layer whenever its copy takes longer than its computation.

The paper prints no equations for the timeline itself.  Reading used here (the
double-buffered schedule of Fig. 2b, offload-all policy): during forward
propagation the input activation map of layer i is offloaded while layer i
computes and layer i+1 starts when both are done; during backward propagation
the activation map that layer i-1 needs is prefetched while layer i computes.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Iterable, Sequence


@dataclass(frozen=True)
class Layer:
    """One layer whose input activation map is offloaded."""
    fwd_s: float          # forward computation time, seconds
    bwd_s: float          # backward computation time, seconds
    act_bytes: float      # size of the offloaded activation map, bytes
    ratio: float = 1.0    # compression ratio of that map (dense bytes / compressed bytes)


def comp_bw(ratio: float, pcie_gbs: float) -> float:
    """DRAM read rate (GB/s) that produces compressed data at the link's rate."""
    return ratio * pcie_gbs


def copy_inflation(ratio: float, pcie_gbs: float, dram_bw_gbs: float = math.inf) -> float:
    """Factor by which a layer's compressed copy is slowed down when the codec
    cannot read DRAM fast enough to saturate the link (never below 1)."""
    if dram_bw_gbs <= 0:
        raise ValueError("dram_bw_gbs must be positive")
    return max(1.0, comp_bw(ratio, pcie_gbs) / dram_bw_gbs)


def copy_seconds(act_bytes: float, ratio: float, pcie_gbs: float, dram_bw_gbs: float = math.inf) -> float:
    """Time on the link for one activation map stored at `ratio`."""
    if ratio <= 0 or pcie_gbs <= 0:
        raise ValueError("ratio and pcie_gbs must be positive")
    return act_bytes / ratio / (pcie_gbs * 1e9) * copy_inflation(ratio, pcie_gbs, dram_bw_gbs)


def step_seconds(layers: Sequence[Layer], pcie_gbs: float, dram_bw_gbs: float = math.inf,
                 compressed: bool = True) -> float:
    """One training step (forward + backward) under the Fig. 2b schedule."""
    def copy(layer: Layer) -> float:
        r = layer.ratio if compressed else 1.0
        return copy_seconds(layer.act_bytes, r, pcie_gbs, dram_bw_gbs if compressed else math.inf)

    total = 0.0
    for layer in layers:                                   # forward: offload overlaps the layer itself
        total += max(layer.fwd_s, copy(layer))
    for i in range(len(layers) - 1, -1, -1):               # backward: prefetch for the layer below
        below = copy(layers[i - 1]) if i > 0 else 0.0
        total += max(layers[i].bwd_s, below)
    return total


def oracle_seconds(layers: Iterable[Layer]) -> float:
    """The same step on a GPU with enough memory: no copies at all."""
    return sum(l.fwd_s + l.bwd_s for l in layers)


def summary(layers: Sequence[Layer], pcie_gbs: float, dram_bw_gbs: float = math.inf) -> dict:
    """Step times and the ratios the paper reports (Fig. 13: performance normalised
    to the oracle; speed-up of compressed over plain copies)."""
    t_oracle = oracle_seconds(layers)
    t_vdnn = step_seconds(layers, pcie_gbs, compressed=False)
    t_cdma = step_seconds(layers, pcie_gbs, dram_bw_gbs, compressed=True)
    dense = sum(l.act_bytes for l in layers)
    packed = sum(l.act_bytes / l.ratio for l in layers)
    return {
        "oracle_s": t_oracle, "vdnn_s": t_vdnn, "cdma_s": t_cdma,
        "vdnn_vs_oracle": t_oracle / t_vdnn if t_vdnn else 1.0,
        "cdma_vs_oracle": t_oracle / t_cdma if t_cdma else 1.0,
        "cdma_speedup_over_vdnn": t_vdnn / t_cdma if t_cdma else 1.0,
        "traffic_reduction": dense / packed if packed else 1.0,
        "max_comp_bw_gbs": max((comp_bw(l.ratio, pcie_gbs) for l in layers), default=0.0),
        "avg_comp_bw_gbs": comp_bw(dense / packed, pcie_gbs) if packed else 0.0,
    }
