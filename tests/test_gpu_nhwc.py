"""Parity of the channel-innermost (NHWC) form of the path with the CPU oracle: transform bit for
bit, convolution (tensor cores, TMA-fed) within the fp16 tolerance, every epilogue option, every
tile shape the library can be made to take, and the benchmark's deep layers whole."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_20725_b200 import binding, workloads
from paper_2608_20725_b200.workloads import Layer
from gpu_helpers import check_conv, check_fused, gpu_conv_nhwc, gpu_transform_nhwc, oracle_inputs

pytestmark = pytest.mark.gpu


def L(name, N, C, H, W, Co, Kh, Kw, s, p, seed=0, xd="normal01", fd="he_normal"):
    return Layer(name, N, C, H, W, Co, Kh, Kw, s, p, seed, xd, fd)


SMALL = [
    L("tail_pos", 3, 5, 13, 11, 7, 3, 3, 1, 1, 11),             # C = 5 -> 8 stored channels, ragged tiles
    L("c8", 2, 8, 12, 12, 72, 3, 3, 1, 1, 13),
    L("k_tail", 2, 24, 9, 10, 24, 3, 3, 1, 1, 36),              # K = 216: last k-block 24 wide
    L("co_300", 1, 8, 10, 10, 300, 3, 3, 1, 1, 14),             # Co = 300: two channel tiles, CTA pairs, one ragged
    L("rect", 2, 4, 9, 14, 10, 2, 5, 1, 2, 15),                 # Kh != Kw
    L("rect2", 2, 4, 14, 9, 10, 5, 2, 2, 0, 16),
    L("stride3", 2, 6, 17, 19, 12, 3, 3, 3, 1, 17),
    L("one_by_one", 3, 40, 7, 7, 33, 1, 1, 1, 0, 18),
    L("k11", 1, 6, 30, 30, 20, 11, 11, 1, 5, 19),
    L("k5s2", 2, 10, 21, 21, 24, 5, 5, 2, 2, 20),
    L("single_out", 1, 3, 3, 3, 2, 3, 3, 1, 0, 21),             # Ho = Wo = 1: 128 strips per tile
    L("deep", 2, 130, 7, 7, 140, 3, 3, 1, 1, 22),               # K = 1224: 20 k-blocks (K split eligible)
    L("wide_row", 1, 2, 4, 300, 5, 3, 3, 1, 1, 23),             # one output row longer than a tile: 3 tiles per strip
    L("uncovered_cols", 1, 3, 10, 12, 4, 3, 4, 3, 0, 24),
    L("pair_odd", 3, 16, 18, 22, 260, 3, 3, 1, 1, 25),          # odd number of position tiles with CTA pairs
    L("pair_s2", 2, 24, 16, 14, 200, 3, 3, 2, 1, 26),
    L("stem7", 2, 3, 37, 37, 64, 7, 7, 2, 3, 12),
    L("many_kb", 1, 64, 9, 9, 40, 5, 5, 1, 2, 27),              # 25 k-blocks: the stage ring wraps several times
    L("one_by_one_s2", 2, 24, 14, 14, 40, 1, 1, 2, 0, 28),      # kernel narrower than the stride: one column class of two is read
    L("one_by_one_big", 5, 72, 13, 13, 136, 1, 1, 1, 0, 29),    # 1x1 over several full position tiles
]


@pytest.mark.parametrize("layer", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("layout,variant", [("nchw", "default"), ("nchw", "rows"), ("nchw", "rows3"), ("nchw", "padded"),
                                            ("nhwc", "default"), ("nhwc", "chunks")])
def test_transform_nhwc_bit_exact(layer, layout, variant, monkeypatch):
    """From either input layout; from NCHW through the kernel the library picks (one block per strip
    for up to 8 channels, else blocks of input rows) and through the per-row kernel forced, with
    one and with three rows per block; from NHWC through the kernel the library picks (one block per
    strip when the channel count is a multiple of 8) and through the chunk-per-thread kernel forced."""
    if variant == "padded":               # the per-row kernel's padded shared-memory rows instead of swizzled ones
        monkeypatch.setenv("IM2WIN_NHWC_TRANSFORM", "rows")
        monkeypatch.setenv("IM2WIN_NHWC_TRANSFORM_SWZ", "0")
    elif variant == "chunks":
        monkeypatch.setenv("IM2WIN_NHWC_TRANSFORM", "chunks")
    elif variant != "default":
        monkeypatch.setenv("IM2WIN_NHWC_TRANSFORM", "rows")
    if variant == "rows3":
        monkeypatch.setenv("IM2WIN_NHWC_TRANSFORM_ROWS", "3")
    dims = layer.dims()
    x, _ = workloads.make_inputs(layer)
    raw = x.half().view(torch.int16)
    got = gpu_transform_nhwc(raw, dims, layout)
    cp = got.shape[-1]
    want = oracle.transform_nhwc(raw.numpy(), dims, "nchw", cp)
    assert cp == (layer.C + 7) // 8 * 8 and got.shape == want.shape
    assert np.array_equal(got, want)


def test_transform_nhwc_preserves_special_bit_patterns():
    layer = L("bits", 2, 11, 9, 10, 1, 3, 3, 2, 2, 30)
    dims = layer.dims()
    g = torch.Generator().manual_seed(31)
    raw = torch.randint(-2 ** 15, 2 ** 15 - 1, (2, 11, 9, 10), generator=g, dtype=torch.int64).to(torch.int16)
    raw.view(-1)[:3] = torch.tensor([0x7e01, -2 ** 15, -1], dtype=torch.int64).to(torch.int16)
    for layout in ("nchw", "nhwc"):
        assert np.array_equal(gpu_transform_nhwc(raw, dims, layout), oracle.transform_nhwc(raw.numpy(), dims, "nchw", 16))


def _reference(x, f, dims, bias=None, relu=False, out16=False, y_nhwc=False):
    xo, fo = oracle_inputs(x, f, "f16")
    y, a = oracle.conv_direct(xo, fo, dims)
    # the value before the store rounding, and the rounded one
    y_pre, a2 = oracle.epilogue(y, a, dims, bias=bias, relu=relu, out16=False, nhwc=y_nhwc)
    y_post, _ = oracle.epilogue(y, a, dims, bias=bias, relu=relu, out16=out16, nhwc=y_nhwc)
    return y_pre, y_post, a2


@pytest.mark.parametrize("layer", SMALL, ids=lambda l: l.name)
@pytest.mark.parametrize("layout,kernel", [("nchw", "overlap"), ("nhwc", "shift"), ("nchw", "default")])
def test_conv_nhwc_parity_small(layer, layout, kernel, monkeypatch):
    """Plain epilogue (fp32, NCHW out) from either input layout, through either kernel and the one
    the library picks."""
    if kernel != "default":
        monkeypatch.setenv("IM2WIN_NHWC_KERNEL", kernel)
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    y = gpu_conv_nhwc(x, f, dims, x_layout=layout)
    y_pre, _, a = _reference(x, f, dims)
    check_conv(y, y_pre, a, "f16", layer.name)


@pytest.mark.parametrize("layer", [SMALL[0], SMALL[2], SMALL[3], SMALL[4], SMALL[6], SMALL[7], SMALL[9], SMALL[11],
                                   SMALL[12], SMALL[14], SMALL[15], SMALL[18], SMALL[19]], ids=lambda l: l.name)
@pytest.mark.parametrize("kernel", ["overlap", "shift"])
@pytest.mark.parametrize("bn,pair,ksplit", [("64", "0", "1"), ("128", "0", "1"), ("128", "1", "1"), ("256", "0", "1"),
                                            ("256", "1", "1"), ("128", "0", "3"), ("256", "1", "2"), ("64", "0", "20")])
def test_conv_nhwc_exact_on_integer_inputs_every_tile_shape(layer, kernel, bn, pair, ksplit, monkeypatch):
    """Integer-valued inputs (order-independent sums) through both kernels (overlapping-row copies
    and shifted views; a layer the shifted-view kernel cannot take runs the other one), every tile
    width, with and without CTA pairs, with K split over several CTAs (partial sums added with
    red.global.add.f32)."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", kernel)
    monkeypatch.setenv("IM2WIN_NHWC_BN", bn)
    monkeypatch.setenv("IM2WIN_NHWC_PAIR", pair)
    monkeypatch.setenv("IM2WIN_NHWC_KSPLIT", ksplit)
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    for y_nhwc in (False, True):
        y = gpu_conv_nhwc(x, f, dims, y_nhwc=y_nhwc)
        assert np.array_equal(y, yr.transpose(0, 2, 3, 1) if y_nhwc else yr), (layer.name, y_nhwc)


@pytest.mark.parametrize("layer", [SMALL[1], SMALL[3], SMALL[6], SMALL[9], SMALL[11]], ids=lambda l: l.name)
@pytest.mark.parametrize("out16", [False, True])
@pytest.mark.parametrize("y_nhwc", [False, True])
@pytest.mark.parametrize("bias,relu", [(False, False), (True, False), (False, True), (True, True)])
def test_conv_nhwc_epilogue_options(layer, out16, y_nhwc, bias, relu, monkeypatch):
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "shift" if (bias != relu) else "overlap")
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    b = None
    if bias:
        b = torch.randn(layer.Co, generator=torch.Generator().manual_seed(layer.seed + 5)).numpy() * 0.5
    y = gpu_conv_nhwc(x, f, dims, bias=b, relu=relu, out16=out16, y_nhwc=y_nhwc, packed=bias and relu)
    y_pre, y_post, a = _reference(x, f, dims, b, relu, out16, y_nhwc)
    check_fused(y, y_pre, a, out16, f"{layer.name} out16={out16} nhwc={y_nhwc} bias={bias} relu={relu}")
    if relu:
        assert np.all(y >= 0)
    if out16:
        # the stored value is a binary16 number within one spacing of the oracle's own rounding
        assert np.array_equal(y, y.astype(np.float16).astype(np.float64))


@pytest.mark.parametrize("raster,stages,bn,ksplit", [("1", "7", "64", "1"), ("1", "2", "128", "2"), ("0", "2", "256", "1"),
                                                      ("1", "3", "64", "3")])
def test_conv_nhwc_overlap_item_order_and_ring_depth(raster, stages, bn, ksplit, monkeypatch):
    """The ablation switches of the overlapping-row kernel (work items in channel-tile-major order, a
    shallower operand ring) change when a tile is computed, never what: exact on integer-valued inputs on a
    layer with several position tiles, several channel tiles and a ragged last one."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "overlap")
    monkeypatch.setenv("IM2WIN_NHWC_RASTER", raster)
    monkeypatch.setenv("IM2WIN_NHWC_STAGES", stages)
    monkeypatch.setenv("IM2WIN_NHWC_BN", bn)
    monkeypatch.setenv("IM2WIN_NHWC_KSPLIT", ksplit)
    layer = L("order_depth", 5, 24, 19, 23, 150, 3, 3, 1, 1, 63)
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    assert np.array_equal(gpu_conv_nhwc(x, f, dims), yr)
    assert np.array_equal(gpu_conv_nhwc(x, f, dims, y_nhwc=True), yr.transpose(0, 2, 3, 1))


@pytest.mark.parametrize("layer", [L("many_items", 16, 16, 40, 40, 48, 3, 3, 1, 1, 60),
                                   L("many_items_s2", 12, 8, 61, 62, 20, 5, 5, 2, 2, 61)], ids=lambda l: l.name)
@pytest.mark.parametrize("dual", ["0", "1"])
def test_conv_nhwc_two_mma_issuers(layer, dual, monkeypatch):
    """More tile pairs than CTA pairs with a resident filter: every CTA works through several items,
    with one MMA-issuing warp and with two (even and odd items on halves of the activation ring).
    Exact on integer-valued inputs, within tolerance on the seeded ones."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "shift")
    monkeypatch.setenv("IM2WIN_NHWC_DUAL", dual)
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    yr, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    assert np.array_equal(gpu_conv_nhwc(x, f, dims), yr)
    x, f = workloads.make_inputs(layer)
    y_pre, _, a = _reference(x, f, dims)
    check_conv(gpu_conv_nhwc(x, f, dims), y_pre, a, "f16", layer.name)


_SHORT_LAST_ROUND = L("short_last_round", 13, 128, 24, 26, 300, 7, 7, 1, 3, 62)    # 14 k2-blocks x 7 kernel columns per item
_short_last_round_refs = {}


def _short_last_round_reference():
    """The oracle's results for the layer above, computed once for all variants of the test."""
    if not _short_last_round_refs:
        dims = _SHORT_LAST_ROUND.dims()
        xi, fi = workloads.make_small_integer_inputs(_SHORT_LAST_ROUND)
        yi, _ = oracle.conv_direct(xi.numpy(), fi.numpy(), dims)
        x, f = workloads.make_inputs(_SHORT_LAST_ROUND)
        y_pre, _, a = _reference(x, f, dims)
        _short_last_round_refs.update(xi=xi, fi=fi, yi=yi, x=x, f=f, y_pre=y_pre, a=a)
    return _short_last_round_refs


@pytest.mark.parametrize("tail", ["k", "n", "off"])
def test_conv_nhwc_short_last_round(tail, monkeypatch):
    """78 tile items on 74 CTA pairs with a streamed filter: the four tiles of the last round are handed
    out as K parts (part 0 stores and raises the tile's flag, the others wait for it and add with
    red.global.add.f32), as channel parts, or whole.  Exact on integer-valued inputs (three calls on
    the same scratch: the flags carry a per-launch value), within tolerance on the seeded ones; with a
    ReLU the K parts must not be taken (the result stays exact)."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "shift")
    if tail == "off":
        monkeypatch.setenv("IM2WIN_NHWC_TAIL", "0")
    if tail == "n":
        monkeypatch.setenv("IM2WIN_NHWC_TAIL_K", "0")
    dims = _SHORT_LAST_ROUND.dims()
    r = _short_last_round_reference()
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims), r["yi"])
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims, packed=True, repeat=3), r["yi"])
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims, relu=True), np.maximum(r["yi"], 0))
    check_conv(gpu_conv_nhwc(r["x"], r["f"], dims), r["y_pre"], r["a"], "f16", _SHORT_LAST_ROUND.name)


def test_conv_nhwc_flag_wait_is_bounded(monkeypatch):
    """The K parts of a short last round wait for part 0's flag.  With the poll limit lowered (word 1 of
    the status block) and the flag kept down (marker in word 2) those waits run out: the kernel returns,
    the status reads IM2WIN_ERR_TIMEOUT, nothing faults or hangs, and the next call on the same buffers
    (a fresh filter pack clears the block) is exact."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "shift")
    dims = _SHORT_LAST_ROUND.dims()
    r = _short_last_round_reference()
    xd, fd = r["xi"].half().cuda(), r["fi"].half().cuda()
    window, scratch, y = binding.alloc_nhwc_buffers(dims)
    binding.im2win_transform_nhwc(xd, binding.NCHW, window, dims)
    binding.im2win_pack_filter_nhwc(fd, scratch, dims)
    torch.cuda.synchronize()
    words = scratch[:256].view(torch.int32)
    words[1] = 4096                       # poll limit of every wait of the next kernel
    words[2] = 0x0d0a11ff                 # part 0 of every split tile keeps its flag down
    binding.im2win_conv_packed_nhwc(window, y, scratch, dims)
    with pytest.raises(binding.Im2winError) as err:
        binding.im2win_check_status(scratch)          # synchronises: the kernel did return
    assert err.value.code == 7
    binding.im2win_conv_f16_nhwc(window, fd, y, scratch, dims)
    binding.im2win_check_status(scratch)
    assert np.array_equal(y.cpu().double().numpy().reshape(r["yi"].shape), r["yi"])


@pytest.mark.parametrize("tail", ["runs", "halves", "off"])
def test_conv_nhwc_overlap_short_last_round(tail, monkeypatch):
    """The same layer through the overlapping-row kernel without a K split of every tile: 78 tile items on
    74 CTA pairs.  The four tiles of the last round are handed out as runs of their reduction (the CTA that
    starts a tile adds the other CTAs' partial sums from the scratch area once their flags are up, then
    applies bias / ReLU and stores), as half tiles, or whole.  Exact on integer-valued inputs, also with a
    bias and a ReLU (which the runs must pass through unchanged) and on three calls on the same scratch;
    within tolerance on the seeded inputs."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "overlap")
    monkeypatch.setenv("IM2WIN_NHWC_KSPLIT", "1")
    if tail == "off":
        monkeypatch.setenv("IM2WIN_NHWC_TAIL", "0")
    if tail == "halves":
        monkeypatch.setenv("IM2WIN_NHWC_STREAM", "0")
    dims = _SHORT_LAST_ROUND.dims()
    r = _short_last_round_reference()
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims), r["yi"])
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims, packed=True, repeat=3), r["yi"])
    b = (np.arange(_SHORT_LAST_ROUND.Co, dtype=np.float32) % 7) - 3.0
    want = np.maximum(r["yi"] + b[None, :, None, None], 0)
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims, bias=b, relu=True), want)
    assert np.array_equal(gpu_conv_nhwc(r["xi"], r["fi"], dims, bias=b, relu=True, y_nhwc=True),
                          want.transpose(0, 2, 3, 1))
    check_conv(gpu_conv_nhwc(r["x"], r["f"], dims), r["y_pre"], r["a"], "f16", _SHORT_LAST_ROUND.name)


def test_conv_nhwc_overlap_flag_wait_is_bounded(monkeypatch):
    """The CTA that starts a tile of a last round handed out as runs waits for the flags of the CTAs that
    hold the rest of its reduction.  With the poll limit lowered and the flags kept down those waits run
    out: the kernel returns, the status reads IM2WIN_ERR_TIMEOUT, and the next call is exact."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", "overlap")
    monkeypatch.setenv("IM2WIN_NHWC_KSPLIT", "1")
    dims = _SHORT_LAST_ROUND.dims()
    r = _short_last_round_reference()
    xd, fd = r["xi"].half().cuda(), r["fi"].half().cuda()
    window, scratch, y = binding.alloc_nhwc_buffers(dims)
    binding.im2win_transform_nhwc(xd, binding.NCHW, window, dims)
    binding.im2win_pack_filter_nhwc(fd, scratch, dims)
    torch.cuda.synchronize()
    words = scratch[:256].view(torch.int32)
    words[1] = 4096
    words[2] = 0x0d0a11ff
    binding.im2win_conv_packed_nhwc(window, y, scratch, dims)
    with pytest.raises(binding.Im2winError) as err:
        binding.im2win_check_status(scratch)
    assert err.value.code == 7
    binding.im2win_conv_f16_nhwc(window, fd, y, scratch, dims)
    binding.im2win_check_status(scratch)
    assert np.array_equal(y.cpu().double().numpy().reshape(r["yi"].shape), r["yi"])


def test_conv_nhwc_exact_with_integer_bias_relu_and_half_store():
    """Small integers all the way: bias, ReLU and the binary16 store must reproduce the oracle exactly."""
    layer = SMALL[2]
    dims = layer.dims()
    x, f = workloads.make_small_integer_inputs(layer)
    b = np.arange(layer.Co, dtype=np.float32) - 10.0
    y, a = oracle.conv_direct(x.numpy(), f.numpy(), dims)
    for y_nhwc in (False, True):
        want, _ = oracle.epilogue(y, a, dims, bias=b, relu=True, out16=True, nhwc=y_nhwc)
        got = gpu_conv_nhwc(x, f, dims, bias=b, relu=True, out16=True, y_nhwc=y_nhwc)
        assert np.abs(want).max() < 2048 and np.array_equal(got, want)


def test_nhwc_argument_errors_come_before_any_launch():
    lib = binding.lib()
    import ctypes
    s = binding.as_shape(SMALL[1].dims())
    e = binding.Epilogue(None, 2, 0, 0)
    assert lib.im2win_conv_f16_nhwc(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_void_p(1024), ctypes.byref(e),
                                    ctypes.c_void_p(2048), 1 << 30, ctypes.byref(s), None) == 1
    e = binding.Epilogue(None, 0, 5, 0)
    assert lib.im2win_conv_f16_nhwc(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_void_p(1024), ctypes.byref(e),
                                    ctypes.c_void_p(2048), 1 << 30, ctypes.byref(s), None) == 1
    assert lib.im2win_conv_f16_nhwc(None, ctypes.c_void_p(512), ctypes.c_void_p(1024), None,
                                    ctypes.c_void_p(2048), 1 << 30, ctypes.byref(s), None) == 2
    assert lib.im2win_conv_f16_nhwc(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_void_p(1028), None,
                                    ctypes.c_void_p(2048), 1 << 30, ctypes.byref(s), None) == 3
    assert lib.im2win_conv_f16_nhwc(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_void_p(1024), None,
                                    ctypes.c_void_p(2048), 16, ctypes.byref(s), None) == 4
    assert lib.im2win_transform_nhwc(ctypes.c_void_p(256), 7, ctypes.c_void_p(512), ctypes.byref(s), None) == 1


FULL = [workloads.LAYERS[k] for k in ("cfg2", "cfg3", "cfg4a", "cfg4b", "cfg4c", "cfg5k1", "cfg5k3", "cfg5k5")]


@pytest.mark.parametrize("layer", FULL, ids=lambda l: l.name)
def test_nhwc_full_size_whole_tensors(layer):
    """At the benchmark's sizes and launch configuration: the NHWC transform of every image bit for
    bit and EVERY output element of the convolution within tolerance, plus 4096 outputs from Eq. 1."""
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    raw = x.half().view(torch.int16)
    got = gpu_transform_nhwc(raw, dims, "nchw")
    assert np.array_equal(got, oracle.transform_nhwc(raw.numpy(), dims, "nchw", got.shape[-1]))
    del got
    y = gpu_conv_nhwc(x, f, dims)
    xo, fo = oracle_inputs(x, f, "f16")
    total = layer.N * layer.Co * ho * wo
    idx = np.concatenate([np.random.default_rng(layer.seed).integers(0, total, 4096), [0, total - 1]])
    yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
    check_conv(y.reshape(-1)[idx], yr, ar, "f16", layer.name)
    for n0 in range(0, layer.N, 16):
        n1 = min(layer.N, n0 + 16)
        yi, ai = oracle.conv_im2win(xo[n0:n1], fo, dict(dims, N=n1 - n0))
        check_conv(y[n0:n1], yi, ai, "f16", f"{layer.name} images {n0}..{n1 - 1}")


@pytest.mark.parametrize("name", ["cfg5k7", "cfg5k11"])
def test_nhwc_full_size_last_round_as_runs_with_fused_epilogue(name):
    """The two longest reductions at benchmark size with bias, ReLU and the binary16 store: 224 tiles on 74
    CTA pairs, the two tiles of the last round shared between CTAs as runs of the reduction (partial sums
    through the scratch area, the epilogue applied once by the CTA that starts the tile).  16 384 sampled
    outputs from Eq. 1 with the epilogue applied in binary64, and the first and last image whole through
    the oracle's im2win route and epilogue."""
    layer = workloads.LAYERS[name]
    dims = layer.dims()
    relu16 = binding.make_epilogue(None, True, torch.float16, binding.NCHW)
    assert binding.im2win_nhwc_kernel_name(dims, relu16) == "f16-nhwc-overlap+runs"
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    b = np.linspace(-0.5, 0.5, layer.Co).astype(np.float32)
    y = gpu_conv_nhwc(x, f, dims, bias=b, relu=True, out16=True)
    xo, fo = oracle_inputs(x, f, "f16")
    total = layer.N * layer.Co * ho * wo
    idx = np.concatenate([np.random.default_rng(layer.seed + 5).integers(0, total, 16384), [0, total - 1]])
    yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
    co = (idx // (ho * wo)) % layer.Co
    check_fused(y.reshape(-1)[idx], np.maximum(yr + b[co].astype(np.float64), 0.0), ar + np.abs(b[co]), True, name)
    for n in (0, layer.N - 1):
        d1 = dict(dims, N=1)
        yi, ai = oracle.conv_im2win(xo[n:n + 1], fo, d1)
        yi, ai = oracle.epilogue(yi, ai, d1, bias=b, relu=True, out16=False)
        check_fused(y[n:n + 1], yi, ai, True, f"{name} image {n}")


@pytest.mark.parametrize("name,kernel", [("cfg2", "overlap"), ("cfg4a", "shift"), ("cfg4b", "shift"), ("cfg4c", "shift"),
                                         ("cfg4c", "overlap"), ("cfg5k3", "overlap"), ("cfg5k3", "shift"), ("cfg5k5", "shift")])
def test_nhwc_full_size_forced_kernel_sampled(name, kernel, monkeypatch):
    """Both kernels at benchmark size wherever the library would pick the other one: 16 384 sampled
    outputs from Eq. 1 and two whole images."""
    monkeypatch.setenv("IM2WIN_NHWC_KERNEL", kernel)
    layer = workloads.LAYERS[name]
    dims = layer.dims()
    x, f = workloads.make_inputs(layer)
    ho, wo = oracle.out_dims(dims)
    y = gpu_conv_nhwc(x, f, dims)
    xo, fo = oracle_inputs(x, f, "f16")
    total = layer.N * layer.Co * ho * wo
    idx = np.concatenate([np.random.default_rng(layer.seed + 1).integers(0, total, 16384), [0, total - 1]])
    yr, ar = oracle.conv_direct_points(xo, fo, dims, idx)
    check_conv(y.reshape(-1)[idx], yr, ar, "f16", f"{name} {kernel}")
    for n in (0, layer.N - 1):
        yi, ai = oracle.conv_im2win(xo[n:n + 1], fo, dict(dims, N=1))
        check_conv(y[n:n + 1], yi, ai, "f16", f"{name} {kernel} image {n}")
