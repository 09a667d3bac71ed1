"""Parity of the CUDA path (through the C ABI) with the CPU oracle, element by element.

Transform: bit-exact.  Convolution: |gpu - oracle| <= 1e-5 * sum|x||w| (fp32) and
<= 2e-3 * sum|x||w| (fp16 inputs, oracle on binary16-rounded inputs), per output element.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_20725_b200 import binding, workloads
from paper_2608_20725_b200.workloads import Layer
from gpu_helpers import (assert_guards_intact, check_conv, gpu_conv, gpu_layer_keep_window, gpu_transform,
                         guarded, oracle_inputs)

pytestmark = pytest.mark.gpu


def L(name, N, C, H, W, Co, Kh, Kw, s, p, seed=0, xd="normal01", fd="he_normal"):
    return Layer(name, N, C, H, W, Co, Kh, Kw, s, p, seed, xd, fd)


# Small layers that still span several tiles (128 positions, 64/128/256 channels, 16/64-wide
# k-blocks) and leave ragged tails in every dimension.
SMALL = [
    workloads.LAYERS["cfg1"],
    L("tail_pos", 3, 5, 13, 11, 7, 3, 3, 1, 1, 11),            # P = 429: 3 full tiles + a ragged one
    L("k147", 2, 3, 37, 37, 64, 7, 7, 2, 3, 12),                # K = 147 (pads to 160 / 192)
    L("co_tail", 2, 16, 12, 12, 72, 3, 3, 1, 1, 13),            # Co = 72: two fp32 channel tiles, one masked
    L("co_300", 1, 8, 10, 10, 300, 3, 3, 1, 1, 14),             # Co = 300: 256 + 44 for the tensor-core tile
    L("rect", 2, 4, 9, 14, 10, 2, 5, 1, 2, 15),                 # Kh != Kw
    L("rect2", 2, 4, 14, 9, 10, 5, 2, 2, 0, 16),
    L("stride3", 2, 6, 17, 19, 12, 3, 3, 3, 1, 17),
    L("one_by_one", 3, 40, 7, 7, 33, 1, 1, 1, 0, 18),
    L("k11", 1, 6, 30, 30, 20, 11, 11, 1, 5, 19),
    L("k5s2", 2, 10, 21, 21, 24, 5, 5, 2, 2, 20),
    L("single_out", 1, 3, 3, 3, 2, 3, 3, 1, 0, 21),             # Ho = Wo = 1
    L("deep", 2, 130, 7, 7, 140, 3, 3, 1, 1, 22),               # K = 1170: many k-blocks, odd strips (54 B)
    L("wide_row", 1, 2, 4, 300, 5, 3, 3, 1, 1, 23),             # one output row longer than a tile
    L("uncovered_cols", 1, 3, 10, 12, 4, 3, 4, 3, 0, 24),       # (Wp - Kw) % s != 0: trailing columns never read
    L("pair_odd", 3, 16, 18, 22, 260, 3, 3, 1, 1, 25),          # Co > 256 and an odd number of position tiles (CTA pairs)
    L("pair_s2", 2, 24, 16, 14, 200, 3, 3, 2, 1, 26),           # CTA pairs with stride 2
    L("vec_w16", 2, 5, 11, 16, 6, 3, 3, 1, 1, 27),              # W a multiple of 8: vector-load transform, odd pad
    L("vec_w24_p2", 3, 3, 9, 24, 4, 5, 5, 1, 2, 28),            # ... even pad, Kh = 5
    L("vec_w32_k1", 2, 7, 6, 32, 9, 1, 1, 1, 0, 29),            # ... Kh = 1, no pad
    L("vec_w12", 2, 4, 10, 12, 5, 3, 3, 1, 1, 30),              # W = 12: 8-byte vectors for fp16, 16-byte for fp32
    L("vec_w6_s2", 2, 3, 9, 6, 4, 3, 3, 2, 1, 31),              # W = 6: no vectors (12- / 24-byte rows), stride 2
    L("vec_w16_k7", 2, 3, 20, 16, 4, 7, 7, 2, 3, 32),           # tall kernel with vector loads (fp16), stride 2
    L("vec_w24_k11", 1, 2, 26, 24, 3, 11, 11, 1, 5, 33),        # Kh = 11 with vector loads (fp16)
    L("cls2_s2", 2, 12, 12, 12, 20, 3, 3, 2, 1, 34),            # fp16 plane pitch 8 (mod 16): two channel classes, stride 2
    L("cls2_wide", 3, 10, 9, 10, 260, 3, 3, 1, 1, 35),          # ... with CTA pairs
    L("cls2_deep", 2, 40, 9, 10, 24, 3, 3, 1, 1, 36),           # ... several k-blocks per class (lane tables per class)
    L("cls2_odd", 2, 22, 9, 10, 24, 3, 3, 1, 1, 37),            # ... 11 channels per class: ragged last octet
    L("rag_s4", 2, 3, 39, 39, 20, 11, 11, 4, 0, 38),            # Wp % s = 3: cut-short last virtual column, one short k-block
    L("rag_s3", 3, 5, 20, 22, 12, 4, 4, 3, 0, 39),              # Wp % s = 1, K2 = 20: two MMA steps
    L("rag_s2_deep", 2, 20, 15, 15, 12, 5, 5, 2, 1, 40),        # Wp = 17 with stride 2, two k-blocks (the last one short)
    L("stem_rag4", 1, 3, 23, 131, 20, 11, 11, 4, 0, 41),        # one-k-block kernel: strip segments, stride 4, tensor ends off a 16-byte boundary
    L("stem_rag2", 2, 3, 21, 75, 24, 7, 7, 2, 0, 42),           # ... stride 2, odd strips
    L("stem_rag3", 2, 5, 14, 100, 12, 4, 4, 3, 0, 43),          # ... stride 3, K2 = 20
    L("stem_c8", 2, 8, 20, 40, 40, 5, 5, 1, 2, 44),             # ... K2 = 40, image segments
    L("stem_imgs", 6, 3, 8, 8, 16, 3, 3, 1, 1, 45),             # ... a tile that touches three images
    L("stem_wide", 2, 3, 12, 40, 300, 3, 3, 1, 1, 46),          # ... two channel tiles (filter streamed)
]


@pytest.mark.parametrize("layer", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("es", [4, 2])
@pytest.mark.parametrize("kernel", ["strips", "strips-scalar", "columns"])
def test_transform_bit_exact_small(layer, es, kernel, monkeypatch):
    """All transform kernels (the strip kernel the library picks, with vector loads where the
    row length allows and element-wise otherwise, and the column kernel it falls back to for
    very long strips) against the oracle, bit for bit."""
    if kernel == "columns":
        monkeypatch.setenv("IM2WIN_TRANSFORM_KERNEL", "columns")
    if kernel == "strips-scalar":
        monkeypatch.setenv("IM2WIN_TRANSFORM_SCALAR", "1")
    dims = layer.dims()
    x, _ = workloads.make_inputs(layer)
    xb = x if es == 4 else x.half()
    raw = xb.view(torch.int32 if es == 4 else torch.int16)
    got = gpu_transform(raw, dims)
    want = oracle.transform(raw.numpy(), dims)
    assert got.shape == want.shape and np.array_equal(got, want)


def test_transform_long_strips_use_the_column_kernel():
    """A strip longer than the staging limit (Kh*Wp*4 bytes > 96 KB) takes the fallback path."""
    layer = L("long", 1, 2, 5, 9000, 1, 3, 3, 1, 1, 33)
    dims = layer.dims()
    x, _ = workloads.make_inputs(layer)
    raw = x.view(torch.int32)
    assert np.array_equal(gpu_transform(raw, dims), oracle.transform(raw.numpy(), dims))


def test_transform_preserves_special_bit_patterns():
    layer = L("bits", 2, 3, 9, 10, 1, 3, 3, 2, 2, 30)
    dims = layer.dims()
    g = torch.Generator().manual_seed(31)
    n = 2 * 3 * 9 * 10
    raw32 = torch.randint(-2 ** 31, 2 ** 31 - 1, (n,), generator=g, dtype=torch.int64).to(torch.int32).reshape(2, 3, 9, 10)
    raw32.view(-1)[:4] = torch.tensor([0x7fc01234, -2 ** 31, -1, 0x7f800001], dtype=torch.int64).to(torch.int32)
    assert np.array_equal(gpu_transform(raw32, dims), oracle.transform(raw32.numpy(), dims))
    raw16 = torch.randint(-2 ** 15, 2 ** 15 - 1, (n,), generator=g, dtype=torch.int64).to(torch.int16).reshape(2, 3, 9, 10)
    raw16.view(-1)[:3] = torch.tensor([0x7e01, -2 ** 15, -1], dtype=torch.int64).to(torch.int16)
    assert np.array_equal(gpu_transform(raw16, dims), oracle.transform(raw16.numpy(), dims))


@pytest.mark.parametrize("layer", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("precision", ["f32", "f16", "f16-shift", "f16-mat", "f16-stem", "f16-gather"])
def test_conv_parity_small(layer, precision):
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, precision)
    xo, fo = oracle_inputs(x, f, precision)
    yr, ar = oracle.conv_direct(xo, fo, dims)
    check_conv(y, yr, ar, precision, layer.name)


@pytest.mark.parametrize("layer", [SMALL[1], SMALL[2], SMALL[4], SMALL[8], SMALL[10], SMALL[12]], ids=lambda l: l.name)
@pytest.mark.parametrize("precision", ["f32", "f16", "f16-shift", "f16-mat", "f16-stem", "f16-gather"])
def test_conv_exact_on_integer_inputs(layer, precision):
    """x in {-2..2}, filter in {-1,0,1}: every partial sum is a small integer, so any summation
    order gives the oracle's value exactly.  Separates indexing errors from rounding."""
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, precision)
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    assert np.array_equal(y.astype(np.float64), yr)


@pytest.mark.parametrize("layer", [SMALL[1], SMALL[2], L("wide_co", 3, 20, 11, 13, 150, 3, 3, 1, 1, 47),
                                   L("co96", 2, 12, 30, 29, 96, 5, 5, 2, 2, 48), L("co200", 1, 9, 14, 15, 200, 3, 3, 1, 1, 49)],
                         ids=lambda l: l.name)
@pytest.mark.parametrize("bm,bk", [("64", "16"), ("64", "32"), ("128", "16"), ("128", "tall"), ("64", "tall")])
def test_conv_f32_both_tile_heights(layer, bm, bk, monkeypatch):
    """The fp32 kernel's 64- and 128-position tiles (the library picks by grid size), on 64-, 96- and
    128-channel tiles (96 where that pads the output channels least: 96 and 150 here, not 200), and the
    64-position tiles with both k-blocks, all with the 8 x 8 register tile; then the 16 x 8 register tile
    (what 128-position tiles of 64 and 128 channels take by default) on 128 x 64, 128 x 128 and 64 x 128
    tiles: exact on integer-valued inputs, within tolerance on the seeded ones."""
    monkeypatch.setenv("IM2WIN_F32_BM", bm)
    if bk == "tall":
        monkeypatch.setenv("IM2WIN_F32_TALL", "1")
    else:
        monkeypatch.setenv("IM2WIN_F32_BK", bk)
        monkeypatch.setenv("IM2WIN_F32_TALL", "0")
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    assert np.array_equal(y.astype(np.float64), yr)
    x, f = workloads.make_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    yr, ar = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    check_conv(y, yr, ar, "f32", layer.name)


@pytest.mark.parametrize("layer", [SMALL[1], SMALL[2], SMALL[28], L("wide_co", 3, 20, 11, 13, 150, 3, 3, 1, 1, 47),
                                   L("co96_s4", 3, 3, 63, 67, 96, 11, 11, 4, 0, 50)], ids=lambda l: l.name)
def test_conv_f32_gather_with_k_along_lanes(layer, monkeypatch):
    """The fp32 kernel's second way of gathering the window operand (a warp's copy instruction covers
    eight consecutive k of four positions; the library takes it for windows 128 bytes or more apart),
    forced on 128-position tiles of 64, 96 and 128 channels, with ragged position and channel tails."""
    monkeypatch.setenv("IM2WIN_F32_BM", "128")
    monkeypatch.setenv("IM2WIN_F32_KLANES", "1")
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    assert np.array_equal(y.astype(np.float64), yr)
    x, f = workloads.make_inputs(layer)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    yr, ar = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    check_conv(y, yr, ar, "f32", layer.name)


def test_f16_inputs_are_the_oracles_rounding():
    """The cast that feeds the fp16 path (torch .half()) and the oracle's rounding agree bit for bit."""
    layer = workloads.LAYERS["cfg5k11"].with_batch(1)
    x, f = workloads.make_inputs(layer)
    for t in (x, f):
        bits, _ = oracle.round_to_f16(t.numpy())
        assert np.array_equal(bits, t.half().view(torch.int16).numpy().view(np.uint16))


def test_delta_filter_reproduces_input_on_gpu():
    C = 24
    x = torch.randn((2, C, 10, 12), generator=torch.Generator().manual_seed(40))
    f = torch.zeros((C, C, 3, 3))
    for c in range(C):
        f[c, c, 1, 1] = 1.0
    dims = dict(N=2, C=C, H=10, W=12, Co=C, Kh=3, Kw=3, stride=1, pad=1)
    y, _, _ = gpu_conv(x, f, dims, "f32")
    assert np.array_equal(y, x.numpy())
    y16, x16, _ = gpu_conv(x, f, dims, "f16")
    assert np.array_equal(y16, x16)


def test_layer_forward_host_matches_device_path():
    layer = L("host", 3, 6, 15, 13, 20, 3, 3, 2, 1, 50)
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    for precision, tdt, code in (("f32", torch.float32, binding.F32), ("f16", torch.float16, binding.F16)):
        y_dev, _, _ = gpu_conv(x, f, dims, precision)
        xh = x.to(tdt).pin_memory()
        fh = f.to(tdt).pin_memory()
        _, _, ho, wo = binding.im2win_workspace_size(dims, code)
        yh = torch.empty((layer.N, layer.Co, ho, wo), dtype=torch.float32).pin_memory()
        nbytes = binding.im2win_layer_workspace_size(dims, code)
        whole, ws = guarded(nbytes + 192, torch.uint8, 0x33)   # +192 keeps the view 256-byte aligned
        ws = ws[192:]
        assert ws.data_ptr() % 256 == 0
        binding.im2win_layer_forward_host(xh, fh, yh, ws, dims)
        torch.cuda.synchronize()
        assert_guards_intact(whole, nbytes + 192, 0x33)
        assert np.array_equal(yh.numpy(), y_dev)


@pytest.mark.parametrize("n", [9, 16])
def test_layer_forward_host_in_batch_chunks(n):
    """Layers above 8 MB go through the host path in batch chunks on auxiliary streams; the
    result must not depend on the chunking (ragged last chunk for N = 9), also when the call is
    repeated back to back on the same buffers."""
    layer = L("host_chunks", n, 32, 64, 64, 64, 3, 3, 1, 1, 51)
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    for precision, tdt, code in (("f32", torch.float32, binding.F32), ("f16", torch.float16, binding.F16)):
        y_dev, _, _ = gpu_conv(x, f, dims, precision)
        xh = x.to(tdt).pin_memory()
        fh = f.to(tdt).pin_memory()
        _, _, ho, wo = binding.im2win_workspace_size(dims, code)
        yh = torch.full((layer.N, layer.Co, ho, wo), float("nan"), dtype=torch.float32).pin_memory()
        nbytes = binding.im2win_layer_workspace_size(dims, code)
        whole, ws = guarded(nbytes + 192, torch.uint8, 0x33)
        ws = ws[192:]
        for _ in range(2):
            binding.im2win_layer_forward_host(xh, fh, yh, ws, dims)
        torch.cuda.synchronize()
        assert_guards_intact(whole, nbytes + 192, 0x33)
        assert np.array_equal(yh.numpy(), y_dev), precision


@pytest.mark.parametrize("layer", [SMALL[1], SMALL[4], SMALL[12], SMALL[15], SMALL[16]], ids=lambda l: l.name)
def test_pack_once_then_convolve_twice(layer):
    """im2win_pack_filter + im2win_conv_packed (twice, on different inputs) give what the one-call
    forms give, bit for bit, in both precisions."""
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    x2 = torch.flip(x, dims=[0, 3]).contiguous()
    for precision, tdt in (("f32", torch.float32), ("f16", torch.float16)):
        fd = f.to(tdt).cuda().contiguous()
        window, scratch, y = binding.alloc_layer_buffers(dims, tdt)
        binding.im2win_pack_filter(fd, scratch, dims)
        for xin in (x, x2):
            want, _, _ = gpu_conv(xin, f, dims, precision)
            binding.im2win_transform(xin.to(tdt).cuda().contiguous(), window, dims)
            y.fill_(float("nan"))
            binding.im2win_conv_packed(window, y, scratch, dims)
            binding.im2win_check_status(scratch)
            assert np.array_equal(y.cpu().numpy(), want), (layer.name, precision)


def test_repeated_calls_are_deterministic_and_do_not_depend_on_stale_scratch():
    layer = SMALL[3]
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    for precision in ("f32", "f16"):
        y1, _, _ = gpu_conv(x, f, dims, precision)
        y2, _, _ = gpu_conv(x, f, dims, precision)
        assert np.array_equal(y1, y2)


@pytest.mark.parametrize("pair", ["0", "1"])
def test_mat_kernel_with_and_without_cta_pairs(pair, monkeypatch):
    """The matrix-transpose fp16 kernel in its one-CTA and CTA-pair forms on a wide layer."""
    monkeypatch.setenv("IM2WIN_F16_PAIR", pair)
    for layer in (SMALL[15], SMALL[16], SMALL[4]):
        dims = layer.dims()
        x, f = workloads.make_small_integer_inputs(layer)
        y, _, _ = gpu_conv(x, f, dims, "f16-mat")
        yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        assert np.array_equal(y.astype(np.float64), yr), layer.name


@pytest.mark.parametrize("tall", ["0", "1"])
def test_shift_kernel_with_and_without_tall_tiles(tall, monkeypatch):
    """The gathering shifted-view kernel with 128- and 256-position tiles, on layers whose stride
    divides the strip width and on layers where it does not."""
    monkeypatch.setenv("IM2WIN_F16_TALL", tall)
    by_name = {l.name: l for l in SMALL}
    for name in ("k11", "k5s2", "k147", "rag_s4", "rag_s3", "rag_s2_deep", "wide_row"):
        layer = by_name[name]
        dims = layer.dims()
        x, f = workloads.make_small_integer_inputs(layer)
        y, _, _ = gpu_conv(x, f, dims, "f16-shift")
        yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        assert np.array_equal(y.astype(np.float64), yr), name


@pytest.mark.parametrize("generic", ["0", "1"])
@pytest.mark.parametrize("ctas", ["1", "2"])
def test_stem_kernel_variants(generic, ctas, monkeypatch):
    """The one-k-block fp16 kernel with its unrolled (3 channels, Kh in 3/5/7/11) and its table-driven
    re-layout, one and two CTAs per SM."""
    monkeypatch.setenv("IM2WIN_F16_STEM_GENERIC", generic)
    monkeypatch.setenv("IM2WIN_F16_STEM_CTAS", ctas)
    by_name = {l.name: l for l in SMALL}
    for name in ("cfg1", "stem_rag4", "stem_rag2", "stem_imgs", "stem_wide", "stem_c8"):
        layer = by_name[name]
        dims = layer.dims()
        x, f = workloads.make_small_integer_inputs(layer)
        y, _, _ = gpu_conv(x, f, dims, "f16-stem")
        yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        assert np.array_equal(y.astype(np.float64), yr), name


@pytest.mark.parametrize("bufs", ["1", "2"])
def test_stem_kernel_staged_epilogue(bufs, monkeypatch):
    """The opt-in epilogue of the one-k-block kernel that writes each output plane's run with aligned
    16-byte stores through a staging buffer (one or two buffers): runs that start on every 16-byte
    phase, tiles that straddle images (which store from the registers), several tiles per CTA."""
    monkeypatch.setenv("IM2WIN_F16_STEM_EPI", bufs)
    by_name = {l.name: l for l in SMALL}
    layers = [by_name[n] for n in ("cfg1", "stem_rag4", "stem_rag2", "stem_rag3", "stem_imgs", "stem_wide", "stem_c8")]
    layers += [workloads.TABLE1_LAYERS["cv3"].with_batch(4), workloads.TABLE1_LAYERS["cv7"].with_batch(3)]
    for layer in layers:
        dims = layer.dims()
        x, f = workloads.make_small_integer_inputs(layer)
        y, _, _ = gpu_conv(x, f, dims, "f16-stem")
        yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        assert np.array_equal(y.astype(np.float64), yr), layer.name


@pytest.mark.parametrize("name", ["cfg2", "cfg4a", "cfg5k3"])
def test_full_size_mat_kernel_sampled(name):
    """The matrix-transpose fp16 kernel forced at benchmark sizes, on sampled outputs."""
    layer = workloads.LAYERS[name]
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    total = layer.N * layer.Co * ho * wo
    rng = np.random.default_rng(layer.seed + 7)
    idx = np.concatenate([rng.integers(0, total, 4096), [0, total - 1, wo - 1, ho * wo - 1, total - ho * wo]])
    y, _, _ = gpu_conv(x, f, dims, "f16-mat")
    xo, fo = oracle_inputs(x, f, "f16-mat")
    yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
    check_conv(y.reshape(-1)[idx], yr, ar, "f16-mat", layer.name)
    one = dict(dims, N=1)
    yi, ai = oracle.conv_im2win(xo[-1:], fo, one)
    check_conv(y[-1:], yi, ai, "f16-mat", layer.name + " last image")


def _sample_indices(total, count, seed, extra=()):
    rng = np.random.default_rng(seed)
    return np.concatenate([rng.integers(0, total, count), np.asarray(list(extra), dtype=np.int64)])


def _whole_conv_check(y, xo, fo, dims, precision, name, images_per_pass):
    """Every output element of y against the oracle's im2win route, a few images at a time."""
    worst = 0.0
    for n0 in range(0, dims["N"], images_per_pass):
        n1 = min(dims["N"], n0 + images_per_pass)
        yr, ar = oracle.conv_im2win(xo[n0:n1], fo, dict(dims, N=n1 - n0))
        worst = max(worst, check_conv(y[n0:n1], yr, ar, precision, f"{name} images {n0}..{n1 - 1}"))
    return worst


@pytest.mark.parametrize("name", ["cfg5k7", "cfg5k11"])
def test_full_size_wide_kernels_sampled(name):
    """The two largest sweep layers at benchmark size (K = 12 544 and 30 976), in the launch
    configuration the benchmark times: 65 536 sampled outputs from Eq. 1, two whole images (the
    first and the last) through the im2win route, and the transform of every image bit for bit."""
    layer = workloads.LAYERS[name]
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    total = layer.N * layer.Co * ho * wo
    idx = _sample_indices(total, 65536, layer.seed + 11, [0, total - 1, wo - 1, ho * wo - 1, total - ho * wo])
    for precision in layer.precisions:
        tdt = torch.float32 if precision == "f32" else torch.float16
        raw = x.to(tdt).view(torch.int32 if precision == "f32" else torch.int16)
        got = gpu_transform(raw, dims)
        assert np.array_equal(got, oracle.transform(raw.numpy(), dims)), (name, precision)
        del got
        y, _, _ = gpu_conv(x, f, dims, precision)
        xo, fo = oracle_inputs(x, f, precision)
        yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
        check_conv(y.reshape(-1)[idx], yr, ar, precision, layer.name)
        for n in (0, layer.N - 1):
            yi, ai = oracle.conv_im2win(xo[n:n + 1], fo, dict(dims, N=1))
            check_conv(y[n:n + 1], yi, ai, precision, f"{layer.name} image {n}")
        del y


# ------------------------------------------------- the paper's Table 1 layers ----
TABLE1 = [workloads.TABLE1_LAYERS[k] for k in ("cv1", "cv2", "cv3", "cv5", "cv6", "cv7", "cv8", "cv9", "cv10",
                                                "cv11", "cv12")]


def _table1_check(layer, precisions, samples):
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    total = layer.N * layer.Co * ho * wo
    idx = _sample_indices(total, samples, layer.seed + 3, [0, total - 1, wo - 1, ho * wo - 1, total - ho * wo])
    images = (0, layer.N // 2, layer.N - 1)
    for precision in precisions:
        tdt = torch.float32 if precision == "f32" else torch.float16
        raw = x.to(tdt).view(torch.int32 if precision == "f32" else torch.int16)
        y, wins = gpu_layer_keep_window(x, f, dims, precision, images)
        for n in images:
            want = oracle.transform(raw[n:n + 1].numpy(), dict(dims, N=1))
            assert np.array_equal(wins[n], want), (layer.name, precision, n)
        del wins
        xo, fo = oracle_inputs(x, f, precision)
        yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
        check_conv(y.reshape(-1)[idx], yr, ar, precision, layer.name)
        for n in (layer.N // 2, layer.N - 1):
            yi, ai = oracle.conv_im2win(xo[n:n + 1], fo, dict(dims, N=1))
            check_conv(y[n:n + 1], yi, ai, precision, f"{layer.name} image {n}")
        del y, xo


@pytest.mark.parametrize("layer", TABLE1, ids=lambda l: l.name)
def test_table1_layers_at_batch_256(layer):
    """The paper's benchmark layers (Table 1: no padding, strides 1, 2 and 4, 3 to 512 channels) at
    the paper's batch of 256, as the benchmark launches them: transform bit for bit on the first,
    middle and last image, convolution on 16 384 sampled outputs (Eq. 1) and on two whole images."""
    _table1_check(layer, layer.precisions, 16384)


@pytest.mark.parametrize("precision", ["f32", "f16"])
def test_table1_cv4_at_batch_256(precision):
    """cv4 at batch 256: the one layer whose window tensor (2.8 G elements, 11.2 GB in fp32) passes
    2^31 elements, so image bases need 64-bit arithmetic.  65 536 sampled outputs (a quarter of them
    in images whose window offset exceeds 2^31 elements), the transform of the first, middle and last
    image and the convolution of the middle and last image whole."""
    layer = workloads.TABLE1_LAYERS["cv4"]
    dims = layer.dims()
    ho, wo = oracle.out_dims(dims)
    per_image = oracle.window_elems(dict(dims, N=1))
    assert per_image * (layer.N - 1) > 2 ** 31 and per_image * (layer.N // 2) < 2 ** 31
    _table1_check(layer, (precision,), 65536)


# ------------------------------------------------------------ full-size layers ----
FULL = [workloads.LAYERS[k] for k in ("cfg2", "cfg3", "cfg4a", "cfg4b", "cfg4c", "cfg5k1", "cfg5k3", "cfg5k5")]


@pytest.mark.parametrize("layer", FULL, ids=lambda l: l.name)
def test_full_size_whole_tensors(layer):
    """At the benchmark's sizes and launch configuration: the transform of every image bit for bit
    and EVERY output element of the convolution within tolerance (the oracle's im2win route over
    the whole batch), plus 4096 sampled outputs from Eq. 1 as a second route, in both precisions."""
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    total = layer.N * layer.Co * ho * wo
    idx = _sample_indices(total, 4096, layer.seed, [0, total - 1, wo - 1, ho * wo - 1, total - ho * wo])
    for precision in layer.precisions:
        tdt = torch.float32 if precision == "f32" else torch.float16
        raw = x.to(tdt).view(torch.int32 if precision == "f32" else torch.int16)
        got = gpu_transform(raw, dims)
        assert np.array_equal(got, oracle.transform(raw.numpy(), dims)), (layer.name, precision)
        del got
        y, _, _ = gpu_conv(x, f, dims, precision)
        xo, fo = oracle_inputs(x, f, precision)
        yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
        check_conv(y.reshape(-1)[idx], yr, ar, precision, layer.name)
        _whole_conv_check(y, xo, fo, dims, precision, layer.name, 16)
        del y
