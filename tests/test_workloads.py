"""The seeded input generators: determinism, shapes, densities, layouts."""
import numpy as np
import torch

from oracle import zvc_c
from paper_1705_01626_b200 import workloads as wl


def density(x):
    return float((x != 0).float().mean())


def test_alexnet_conv1_small_is_deterministic_and_half_dense():
    a = wl.alexnet_conv1(shape=(2, 8, 55, 55))
    b = wl.alexnet_conv1(shape=(2, 8, 55, 55))
    assert torch.equal(a, b)
    assert a.dtype == torch.float32 and (a >= 0).all()
    assert abs(density(a) - 0.5) < 0.02


def test_per_channel_beta_has_per_channel_densities():
    x = wl.per_channel_beta(shape=(2, 16, 32, 32))
    assert x.shape == (2, 16, 32, 32) and (x >= 0).all()
    per_c = (x != 0).float().mean(dim=(0, 2, 3))
    assert per_c.std() > 0.05            # channels differ
    assert 0.15 < float(per_c.mean()) < 0.55
    assert torch.equal(x, wl.per_channel_beta(shape=(2, 16, 32, 32)))


def test_correlated_relu_hits_density_and_clusters_zeros():
    for d in (0.1, 0.5, 0.95):
        x = wl.correlated_relu((2, 4, 56, 56), d, seed=7)
        assert abs(density(x) - d) < 0.03
    x = wl.correlated_relu((2, 4, 56, 56), 0.5, seed=7)
    z = (x == 0)
    same_as_right = (z[..., :, 1:] == z[..., :, :-1]).float().mean()
    assert same_as_right > 0.8           # i.i.d. zeros would give about 0.5
    assert density(wl.correlated_relu((1, 2, 28, 28), 1.0, seed=1)) == 1.0


def test_offload_set_shapes_and_density_ramp():
    shapes = ((4, 16, 16), (8, 8, 8), (8, 8, 8))
    ts = wl.vgg16_offload_set(batch=2, shapes=shapes)
    assert [tuple(t.shape) for t, _ in ts] == [(2, 4, 16, 16), (2, 8, 8, 8), (2, 8, 8, 8)]
    assert [round(d, 3) for _, d in ts] == [0.5, 0.3, 0.1]
    assert len(wl.VGG16_CONV_SHAPES) == 13
    assert sum(64 * c * h * w for c, h, w in wl.VGG16_CONV_SHAPES) == 867_041_280


def test_layouts_permute_the_same_values_and_keep_the_compressed_size():
    x = wl.correlated_relu((3, 5, 8, 8), 0.4, seed=11)
    sizes = set()
    for layout in wl.LAYOUTS:
        y = wl.to_layout(x, layout)
        assert y.is_contiguous() and y.numel() == x.numel()
        assert torch.equal(y.reshape(-1).sort().values[-5:], x.reshape(-1).sort().values[-5:])
        sizes.add(len(zvc_c.compress(y.numpy())[0]))
    assert len(sizes) == 1
    assert torch.equal(wl.to_layout(x, "NHWC"), x.permute(0, 2, 3, 1).contiguous())
    assert torch.equal(wl.to_layout(x, "CHWN"), x.permute(1, 2, 3, 0).contiguous())


def test_large_extremes_small_instances():
    a = wl.large_extremes("a", n=1 << 16)
    b = wl.large_extremes("b", n=1 << 16)
    c = wl.large_extremes("c", n=1 << 16)
    assert abs(density(a) - 0.05) < 0.01
    assert density(b) == 1.0
    assert c.dtype == torch.float16 and abs(density(c) - 0.3) < 0.02
    assert (c[c != 0] > 0).all()


def test_special_values_contain_negative_zero_and_nan():
    x = wl.special_values(4096, seed=3)
    bits = x.view(torch.int32)
    assert (bits == -0x80000000).any() and torch.isnan(x).any()
    h = wl.special_values(4096, seed=3, dtype=torch.float16)
    assert (h.view(torch.int16) == -0x8000).any()
    payload, _ = zvc_c.compress(x.numpy())
    assert zvc_c.decompress(payload, x.numel(), np.float32).tobytes() == x.numpy().tobytes()
