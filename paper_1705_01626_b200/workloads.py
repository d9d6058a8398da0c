"""Seeded synthetic activation maps shaped like the paper's CNN workloads.

These generators only produce inputs.  They contain nothing of the codec (no
masks, no sizes, no offsets) and are the one module the CPU checker's tests and
the CUDA path's tests both use.

The paper measures on activations of ImageNet-trained CNNs (Section IV,
Figs. 4-7), which are not available here; these tensors stand in for them with
the same shapes, element type, density range (about 50 % dense in the first
layer falling to about 10 % in deep layers, Section IV-A/B) and, where asked,
the spatial clustering of zeros visible in the paper's activation pictures
(Fig. 5).  Values never change the compressed size or speed of zero-value
compression -- only the zero pattern does -- but they are kept plausible
(non-negative, ReLU-like).

Every generator takes a seed and a torch device and is deterministic for a
given (seed, device type, torch build).
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import torch

BASE_SEED = 170501626

LAYOUTS = ("NCHW", "NHWC", "CHWN")

# conv+ReLU outputs of a VGG-16-shaped network at batch 64: (channels, height, width)
VGG16_CONV_SHAPES: Tuple[Tuple[int, int, int], ...] = (
    (64, 224, 224), (64, 224, 224),
    (128, 112, 112), (128, 112, 112),
    (256, 56, 56), (256, 56, 56), (256, 56, 56),
    (512, 28, 28), (512, 28, 28), (512, 28, 28),
    (512, 14, 14), (512, 14, 14), (512, 14, 14),
)


def seed_for(config: int, index: int = 0) -> int:
    return BASE_SEED + 1000 * config + index


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def iid_relu_like(shape: Sequence[int], density: float, seed: int, device="cpu",
                  dtype=torch.float32, floor: float = 0.0) -> torch.Tensor:
    """Each element independently non-zero with probability ``density``; non-zero
    values are |N(0,1)| + floor (``floor`` > 0 guarantees no accidental zero
    after rounding to a narrow type)."""
    g = _gen(seed, device)
    n = int(math.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    step = 1 << 26
    for lo in range(0, n, step):
        m = min(step, n - lo)
        v = torch.randn(m, generator=g, device=device, dtype=torch.float32).abs_()
        if floor:
            v += floor
        if density < 1.0:
            keep = torch.rand(m, generator=g, device=device) < density
            v *= keep
        out[lo:lo + m] = v.to(dtype)
    return out.view(*shape)


def alexnet_conv1(seed: int | None = None, device="cpu", shape=(32, 96, 55, 55)) -> torch.Tensor:
    """Workload 1: AlexNet conv1-shaped fp32 NCHW map, i.i.d. density 0.5."""
    return iid_relu_like(shape, 0.5, seed_for(1) if seed is None else seed, device)


def per_channel_beta(shape=(64, 64, 224, 224), seed: int | None = None, device="cpu") -> torch.Tensor:
    """Workload 2: VGG-16 conv1_2-shaped fp32 NCHW map.

    One density per channel c (shared by the whole batch) drawn from
    Beta(2, 4) (mean 1/3); zeros i.i.d. inside a channel; non-zero values are a
    normal N(0.5, 1) conditioned on being positive (inverse-CDF sampling).
    """
    seed = seed_for(2) if seed is None else seed
    g = _gen(seed, device)
    nb, c, h, w = shape
    # Beta(2,4) = G2 / (G2 + G4) with Gk a Gamma(k,1) = -log of a product of k uniforms
    u = torch.rand(6, c, generator=g, device=device, dtype=torch.float64).clamp_(min=1e-300)
    g2 = -(u[:2].log().sum(0))
    g4 = -(u[2:].log().sum(0))
    d_c = (g2 / (g2 + g4)).to(torch.float32)
    out = torch.empty(shape, dtype=torch.float32, device=device)
    a = 0.5 * (1.0 + math.erf(-0.5 / math.sqrt(2.0)))       # P[N(0.5,1) <= 0]
    tiny = torch.finfo(torch.float32).tiny
    for b in range(nb):
        keep = torch.rand(c, h, w, generator=g, device=device) < d_c.view(c, 1, 1)
        q = torch.rand(c, h, w, generator=g, device=device, dtype=torch.float32)
        q = (a + q * (1.0 - a)).clamp_(max=1.0 - 1e-7)
        v = (0.5 + torch.special.ndtri(q)).clamp_(min=tiny)
        out[b] = v * keep
    return out


def _gaussian_kernel1d(sigma: float, radius: int, device) -> torch.Tensor:
    x = torch.arange(-radius, radius + 1, device=device, dtype=torch.float32)
    k = torch.exp(-0.5 * (x / sigma) ** 2)
    return k / k.sum()


def correlated_relu(shape: Sequence[int], density: float, seed: int, device="cpu",
                    sigma: float = 2.0) -> torch.Tensor:
    """fp32 NCHW map whose zeros are spatially clustered.

    Every (n, c) plane is an N(0,1) field blurred with a separable Gaussian
    (sigma = 2 px, radius 6, reflect padding); the tensor is the ReLU of that
    field shifted by the threshold that leaves a fraction ``density`` positive
    (threshold = empirical quantile over a subsample).  density >= 1 gives
    |field| + 2^-20 (no zeros).
    """
    g = _gen(seed, device)
    nb, c, h, w = shape
    radius = 6
    k = _gaussian_kernel1d(sigma, radius, device)
    out = torch.empty(shape, dtype=torch.float32, device=device)
    pad = min(radius, h - 1, w - 1)
    for b in range(nb):
        z = torch.randn(c, 1, h, w, generator=g, device=device)
        zp = torch.nn.functional.pad(z, (pad, pad, pad, pad), mode="reflect") if pad > 0 else z
        kk = k[radius - pad: radius + pad + 1]
        kk = kk / kk.sum()
        zp = torch.nn.functional.conv2d(zp, kk.view(1, 1, 1, -1))
        zp = torch.nn.functional.conv2d(zp, kk.view(1, 1, -1, 1))
        out[b] = zp.view(c, h, w)
    out /= out.std()
    if density >= 1.0:
        return out.abs_().add_(2.0 ** -20)
    flat = out.view(-1)
    sub = flat[:: max(1, flat.numel() // (1 << 22))][: 1 << 22]   # torch.quantile caps its input size
    t = torch.quantile(sub, 1.0 - density)
    return out.sub_(t).clamp_(min=0.0)


def vgg16_offload_set(batch: int = 64, seed: int | None = None, device="cpu",
                      shapes: Sequence[Tuple[int, int, int]] = VGG16_CONV_SHAPES
                      ) -> List[Tuple[torch.Tensor, float]]:
    """Workload 3: the 13 conv+ReLU outputs of a VGG-16-shaped CNN, density
    falling linearly from 0.5 (first) to 0.1 (last), clustered zeros.
    Returns [(tensor, nominal density)]."""
    out = []
    last = max(1, len(shapes) - 1)
    for i, (c, h, w) in enumerate(shapes):
        d = 0.5 - 0.4 * i / last
        s = seed_for(3, i) if seed is None else seed + i
        out.append((correlated_relu((batch, c, h, w), d, s, device), d))
    return out


def to_layout(x_nchw: torch.Tensor, layout: str) -> torch.Tensor:
    """Physical copy of a logical NCHW tensor in the named memory layout
    (Section II-C): NCHW as is, NHWC channels innermost, CHWN batch innermost."""
    if layout == "NCHW":
        return x_nchw.contiguous()
    if layout == "NHWC":
        return x_nchw.permute(0, 2, 3, 1).contiguous()
    if layout == "CHWN":
        return x_nchw.permute(1, 2, 3, 0).contiguous()
    raise ValueError(layout)


SWEEP_DENSITIES = (0.05, 0.1, 0.25, 0.5, 0.75, 0.95, 1.0)


def layout_density_sweep(shape=(128, 256, 28, 28), device="cpu", seed: int | None = None):
    """Workload 4: yields (density, layout, tensor) for 7 densities x 3 layouts."""
    for i, d in enumerate(SWEEP_DENSITIES):
        s = seed_for(4, i) if seed is None else seed + i
        x = correlated_relu(shape, d, s, device)
        for layout in LAYOUTS:
            yield d, layout, to_layout(x, layout)


def large_extremes(which: str, n: int = 1 << 29, device="cpu", seed: int | None = None) -> torch.Tensor:
    """Workload 5: 'a' fp32 density 0.05; 'b' fp32 all non-zero; 'c' fp16 density 0.3."""
    idx = "abc".index(which)
    s = seed_for(5, idx) if seed is None else seed
    if which == "a":
        return iid_relu_like((n,), 0.05, s, device)
    if which == "b":
        return iid_relu_like((n,), 1.0, s, device, floor=2.0 ** -20)
    return iid_relu_like((n,), 0.3, s, device, dtype=torch.float16, floor=2.0 ** -10)


def special_values(n: int, seed: int, dtype=torch.float32, device="cpu") -> torch.Tensor:
    """A tensor mixing +0, -0, NaNs with payloads, denormals, infinities and
    ordinary values, as raw bit patterns (returned as the float dtype)."""
    g = _gen(seed, "cpu")
    if dtype == torch.float32:
        it, pats = torch.int32, [0x00000000, -0x80000000, 0x7fc00000, 0x7f800001, -0x00400001,
                                 0x00000001, -0x7fffffff, 0x7f800000, -0x00800000, 0x3f800000]
    else:
        it, pats = torch.int16, [0x0000, -0x8000, 0x7e00, 0x7c01, -0x0200,
                                 0x0001, -0x7fff, 0x7c00, -0x0400, 0x3c00]
    table = torch.tensor(pats, dtype=it)
    pick = torch.randint(0, len(pats), (n,), generator=g)
    return table[pick].view(dtype).to(device)
