"""Seeded random small layers through every convolution path, against the fp64 oracle (Eq. 1).

The fixed cases of test_gpu_parity.py pin known tile/tail situations; this sweep looks for the
ones nobody thought of: odd combinations of kernel size, stride, padding, channel counts and
image sizes (tiles that cross several images, strips shorter than the kernel's boxes, one-channel
layers, wide output-channel tails)."""
import numpy as np
import pytest
import torch

from paper_2608_20725_b200 import workloads
from gpu_helpers import check_conv, check_fused, gpu_conv, gpu_conv_nhwc, gpu_transform, gpu_transform_nhwc, oracle, oracle_inputs

pytestmark = pytest.mark.gpu


def random_layers(seed, count):
    rng = np.random.default_rng(seed)
    layers = []
    while len(layers) < count:
        kh = int(rng.choice([1, 2, 3, 3, 3, 4, 5, 7]))
        kw = int(rng.choice([1, 2, 3, 3, 3, 4, 5, 7]))
        s = int(rng.choice([1, 1, 1, 2, 2, 3]))
        p = int(rng.integers(0, 3))
        h = int(rng.integers(kh, 26))
        w = int(rng.integers(kw, 40))
        if rng.random() < 0.6:                 # plane pitches that are 16-byte multiples: the TMA-staged kernels
            w = max(kw, (w + 2 * p + 7) // 8 * 8 - 2 * p)
        if h + 2 * p < kh or w + 2 * p < kw:
            continue
        n = int(rng.integers(1, 5))
        c = int(rng.choice([1, 2, 3, 5, 8, 9, 16, 17, 24, 40]))
        co = int(rng.choice([1, 3, 8, 20, 64, 65, 130, 260]))
        ho = (h + 2 * p - kh) // s + 1
        wo = (w + 2 * p - kw) // s + 1
        if n * co * ho * wo * c * kh * kw > 60_000_000:      # keep the oracle in the seconds range
            continue
        layers.append(workloads.Layer(f"fuzz{len(layers)}_{n}x{c}x{h}x{w}_co{co}_k{kh}x{kw}_s{s}_p{p}", n, c, h, w, co,
                                      kh, kw, s, p, 9000 + len(layers), "normal01", "he_normal"))
    return layers


FUZZ = random_layers(20260725, 64)


@pytest.mark.parametrize("layer", FUZZ, ids=lambda l: l.name)
def test_random_layer_all_paths(layer):
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    for es, tdt in ((4, torch.float32), (2, torch.float16)):
        raw = x.to(tdt).view(torch.int32 if es == 4 else torch.int16)
        assert np.array_equal(gpu_transform(raw, dims), oracle.transform(raw.numpy(), dims)), (layer.name, es)
    yr32, ar32 = oracle.conv_direct(*oracle_inputs(x, f, "f32"), dims)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    check_conv(y, yr32, ar32, "f32", layer.name)
    xo, fo = oracle_inputs(x, f, "f16")
    yr16, ar16 = oracle.conv_direct(xo, fo, dims)
    for precision in ("f16", "f16-mat", "f16-shift", "f16-stem", "f16-gather"):
        y, _, _ = gpu_conv(x, f, dims, precision)
        check_conv(y, yr16, ar16, precision, layer.name)


@pytest.mark.parametrize("layer", FUZZ, ids=lambda l: l.name)
def test_random_layer_f32_tile_forms(layer, monkeypatch):
    """The fp32 kernel's forms that only large layers take by themselves, forced on the random layers:
    128-position tiles with the 16-position register tile (and with it the staged epilogue wherever Ho*Wo
    is no multiple of 4, and 96-channel tiles for Co = 130 and 260), then the same with the window operand
    gathered with k along the lanes, then 64-position tiles with k-blocks of 32."""
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    yr, ar = oracle.conv_direct(*oracle_inputs(x, f, "f32"), dims)
    for bm, tall, klanes, bk in (("128", "1", "0", None), ("128", "1", "1", None), ("64", "0", "0", "32")):
        monkeypatch.setenv("IM2WIN_F32_BM", bm)
        monkeypatch.setenv("IM2WIN_F32_TALL", tall)
        monkeypatch.setenv("IM2WIN_F32_KLANES", klanes)
        if bk:
            monkeypatch.setenv("IM2WIN_F32_BK", bk)
        y, _, _ = gpu_conv(x, f, dims, "f32")
        check_conv(y, yr, ar, "f32", f"{layer.name} bm={bm} tall={tall} klanes={klanes}")


@pytest.mark.parametrize("layer", FUZZ, ids=lambda l: l.name)
def test_random_layer_nhwc_paths(layer, monkeypatch):
    """The same layers through the channel-innermost (NHWC) form: the transform from both input layouts
    bit for bit, the convolution through the kernel the library picks and through each of its two
    kernels forced, and once with the fused epilogue (bias, ReLU, binary16 NHWC store)."""
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    raw = x.half().view(torch.int16)
    got = gpu_transform_nhwc(raw, dims, "nchw")
    want = oracle.transform_nhwc(raw.numpy(), dims, "nchw", got.shape[-1])
    assert np.array_equal(got, want), layer.name
    assert np.array_equal(gpu_transform_nhwc(raw, dims, "nhwc"), want), layer.name
    xo, fo = oracle_inputs(x, f, "f16")
    yr, ar = oracle.conv_direct(xo, fo, dims)
    for kernel in ("default", "shift", "overlap"):
        if kernel != "default":
            monkeypatch.setenv("IM2WIN_NHWC_KERNEL", kernel)
        check_conv(gpu_conv_nhwc(x, f, dims), yr, ar, "f16", f"{layer.name} {kernel}")
    monkeypatch.delenv("IM2WIN_NHWC_KERNEL")
    bias = torch.randn(layer.Co, generator=torch.Generator().manual_seed(layer.seed + 7)).numpy() * 0.5
    y_pre, a2 = oracle.epilogue(yr, ar, dims, bias=bias, relu=True, out16=False, nhwc=True)
    y = gpu_conv_nhwc(x, f, dims, bias=bias, relu=True, out16=True, y_nhwc=True)
    check_fused(y, y_pre, a2, True, f"{layer.name} fused")
