"""Pins of the oracle's second half: the epilogue options of Algorithm 1's last step (bias, ReLU,
binary16 store, NHWC store) and the channel-innermost (NHWC) im2win tensor of the paper's
tensor-core section.  No GPU needed.

The paper prints no values for either, so the pins are what the mathematics fixes: hand-computed
numbers, brute force against Eq. 1 (itself pinned in test_oracle_pins.py), constructions with
numpy slicing that share no code with the oracle, and an independent library routine.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle


def shp(N, C, H, W, Co, Kh, Kw, s, p):
    return dict(N=N, C=C, H=H, W=W, Co=Co, Kh=Kh, Kw=Kw, stride=s, pad=p)


# ------------------------------------------------- one-step binary64 -> binary16 rounding ----
def test_f64_to_f16_roundtrip_exhaustive():
    bits = np.arange(65536, dtype=np.uint16)
    vals = oracle.f16_bits_to_f64(bits)
    got, back = oracle.round_f64_to_f16(vals)
    nan = np.isnan(vals)
    assert np.array_equal(got[~nan], bits[~nan])
    assert np.array_equal(back[~nan], vals[~nan])
    assert np.all(np.isnan(back[nan]))


def test_f64_to_f16_midpoints_tie_to_even_and_neighbours_do_not():
    """Every midpoint between adjacent non-negative halves is exact in binary64: it must go to the
    neighbour with the even bit pattern; one binary64 ulp to either side must go to that side."""
    lo = np.arange(0, 0x7bff, dtype=np.uint16)                 # finite halves below the largest
    a = oracle.f16_bits_to_f64(lo)
    b = oracle.f16_bits_to_f64(lo + 1)
    mid = (a + b) / 2
    assert np.all((mid > a) & (mid < b))
    got, _ = oracle.round_f64_to_f16(mid)
    even = np.where(lo % 2 == 0, lo, lo + 1)
    assert np.array_equal(got, even)
    assert np.array_equal(oracle.round_f64_to_f16(np.nextafter(mid, np.inf))[0], lo + 1)
    assert np.array_equal(oracle.round_f64_to_f16(np.nextafter(mid, -np.inf))[0], lo)
    # the same on the negative side
    assert np.array_equal(oracle.round_f64_to_f16(-mid)[0], even | 0x8000)


def test_f64_to_f16_limits_and_specials():
    r = lambda v: int(oracle.round_f64_to_f16(np.array([v]))[0][0])
    assert r(65504.0) == 0x7bff and r(65519.999) == 0x7bff and r(65520.0) == 0x7c00 and r(1e300) == 0x7c00
    assert r(-65520.0) == 0xfc00
    assert r(2.0 ** -24) == 1 and r(2.0 ** -25) == 0 and r(np.nextafter(2.0 ** -25, 1.0)) == 1
    assert r(1e-320) == 0 and r(-1e-320) == 0x8000 and r(0.0) == 0 and r(-0.0) == 0x8000
    assert r(np.inf) == 0x7c00 and r(-np.inf) == 0xfc00
    assert np.isnan(oracle.round_f64_to_f16(np.array([np.nan]))[1][0])


def test_f64_to_f16_rounds_once_where_a_detour_through_binary32_rounds_twice():
    """1 + 2^-11 is a binary16 midpoint (ties to 1.0).  A binary64 value a hair above it must go up;
    rounding it to binary32 first lands exactly on the midpoint and then ties down: the one-step
    routine must not reproduce that."""
    v = 1.0 + 2.0 ** -11 + 2.0 ** -40
    one_step = oracle.round_f64_to_f16(np.array([v]))[1][0]
    assert one_step == 1.0 + 2.0 ** -10
    two_step = oracle.round_to_f16(np.array([np.float32(v)]))[1][0]
    assert float(two_step) == 1.0
    # on values that ARE binary32 numbers both routines agree bit for bit
    rng = np.random.default_rng(5)
    f = np.concatenate([rng.standard_normal(200000).astype(np.float32) * np.float32(s) for s in (1e-6, 1e-3, 1.0, 300.0, 7e4)])
    assert np.array_equal(oracle.round_f64_to_f16(f.astype(np.float64))[0], oracle.round_to_f16(f)[0])
    # and with numpy's own binary64 -> binary16 conversion
    d = rng.standard_normal(300000) * np.repeat([1e-7, 1e-2, 50.0], 100000)
    assert np.array_equal(oracle.round_f64_to_f16(d)[0], d.astype(np.float16).view(np.uint16))


# --------------------------------------------------------------------------- epilogue ----
def test_epilogue_worked_example_by_hand():
    """1x1x2x2 input, 2 output channels, 1x1 kernel: y = f*x by hand, then bias, ReLU, binary16."""
    sh = shp(1, 1, 2, 2, 2, 1, 1, 1, 0)
    x = np.array([[[[1.0, -2.0], [0.5, 3.0]]]], dtype=np.float32)
    f = np.array([[[[2.0]]], [[[-1.0]]]], dtype=np.float32)
    y, a = oracle.conv_direct(x, f, sh)
    assert np.array_equal(y, [[[[2.0, -4.0], [1.0, 6.0]], [[-1.0, 2.0], [-0.5, -3.0]]]])
    bias = np.array([0.25, 1.0], dtype=np.float32)
    yb, ab = oracle.epilogue(y, a, sh, bias=bias)
    assert np.array_equal(yb, [[[[2.25, -3.75], [1.25, 6.25]], [[0.0, 3.0], [0.5, -2.0]]]])
    assert np.array_equal(ab, a + np.array([0.25, 1.0]).reshape(1, 2, 1, 1))
    yr, _ = oracle.epilogue(y, a, sh, bias=bias, relu=True)
    assert np.array_equal(yr, [[[[2.25, 0.0], [1.25, 6.25]], [[0.0, 3.0], [0.5, 0.0]]]])
    # 2049 is not a binary16 number (spacing 2 above 2048): ties to even -> 2048
    y2 = np.full_like(y, 2049.0)
    y16, _ = oracle.epilogue(y2, a, sh, out16=True)
    assert np.all(y16 == 2048.0)
    y3 = np.full_like(y, 2051.0)
    assert np.all(oracle.epilogue(y3, a, sh, out16=True)[0] == 2052.0)
    # NHWC store is the transposition, nothing else
    yn, an = oracle.epilogue(y, a, sh, bias=bias, relu=True, nhwc=True)
    assert np.array_equal(yn, yr.transpose(0, 2, 3, 1)) and np.array_equal(an, ab.transpose(0, 2, 3, 1))
    # the inputs were not modified
    assert y[0, 0, 0, 1] == -4.0


def test_epilogue_bias_equals_an_extra_all_ones_channel():
    """Without padding, adding bias[co] is the convolution with one more input channel that is 1
    everywhere and whose filter has bias[co] at one tap and zeros elsewhere."""
    rng = np.random.default_rng(11)
    sh = shp(2, 3, 7, 8, 4, 3, 2, 2, 0)
    x = rng.standard_normal((2, 3, 7, 8)).astype(np.float32)
    f = rng.standard_normal((4, 3, 3, 2)).astype(np.float32)
    bias = rng.standard_normal(4).astype(np.float32)
    y, a = oracle.conv_direct(x, f, sh)
    yb, ab = oracle.epilogue(y, a, sh, bias=bias)
    x2 = np.concatenate([x, np.ones((2, 1, 7, 8), np.float32)], axis=1)
    f2 = np.concatenate([f, np.zeros((4, 1, 3, 2), np.float32)], axis=1)
    f2[:, 3, 1, 0] = bias
    y2, a2 = oracle.conv_direct(x2, f2, dict(sh, C=4))
    assert np.allclose(yb, y2, rtol=0, atol=1e-12 * np.abs(a2).max())
    assert np.allclose(ab, a2, rtol=0, atol=1e-12 * np.abs(a2).max())


def test_epilogue_relu_properties_and_library_cross_check():
    rng = np.random.default_rng(12)
    sh = shp(2, 4, 9, 9, 5, 3, 3, 1, 1)
    x = rng.standard_normal((2, 4, 9, 9)).astype(np.float32)
    f = rng.standard_normal((5, 4, 3, 3)).astype(np.float32)
    bias = rng.standard_normal(5).astype(np.float32)
    y, a = oracle.conv_direct(x, f, sh)
    yb, _ = oracle.epilogue(y, a, sh, bias=bias)
    yr, _ = oracle.epilogue(y, a, sh, bias=bias, relu=True)
    assert np.array_equal(yr, np.maximum(yb, 0.0))              # definition
    assert np.all(yr >= 0) and np.array_equal(yr[yb > 0], yb[yb > 0])
    assert (yb < 0).any() and (yb > 0).any()
    # order of the steps: bias BEFORE the ReLU (relu(y) + b differs wherever y < 0 < y + b or b < 0)
    wrong = np.maximum(y, 0.0) + bias.reshape(1, 5, 1, 1).astype(np.float64)
    assert not np.array_equal(wrong, yr)
    lib = torch.relu(torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(f).double(),
                                                torch.from_numpy(bias).double(), stride=1, padding=1)).numpy()
    assert np.allclose(yr, lib, rtol=0, atol=1e-12 * a.max())
    # binary16 store = the one-step rounding of the fp64 value, applied after bias and ReLU
    y16, _ = oracle.epilogue(y, a, sh, bias=bias, relu=True, out16=True)
    assert np.array_equal(y16, oracle.round_f64_to_f16(yr)[1])
    assert np.array_equal(y16, yr.astype(np.float16).astype(np.float64))


# ---------------------------------------------------- channel-innermost im2win tensor ----
NHWC_SHAPES = [shp(2, 3, 7, 6, 2, 3, 3, 1, 1), shp(1, 5, 9, 8, 2, 2, 4, 2, 0), shp(2, 4, 8, 11, 3, 4, 2, 3, 2),
               shp(1, 8, 5, 5, 2, 1, 1, 1, 0), shp(1, 3, 12, 12, 2, 7, 7, 2, 3)]


def _numpy_window_nhwc(x_nchw, sh, cp):
    """win[n][ho][k][u][c] = xpad[n][c][ho*s+u][k], by padding and slicing."""
    N, C, H, W, Kh, s, p = sh["N"], sh["C"], sh["H"], sh["W"], sh["Kh"], sh["stride"], sh["pad"]
    ho, _ = oracle.out_dims(sh)
    xp = np.pad(x_nchw, ((0, 0), (0, 0), (p, p), (p, p)))
    out = np.zeros((N, ho, W + 2 * p, Kh, cp), dtype=x_nchw.dtype)
    for m in range(ho):
        for u in range(Kh):
            out[:, m, :, u, :C] = xp[:, :, m * s + u, :].transpose(0, 2, 1)
    return out


@pytest.mark.parametrize("sh", NHWC_SHAPES, ids=lambda d: "x".join(str(v) for v in d.values()))
@pytest.mark.parametrize("layout", ["nchw", "nhwc"])
def test_transform_nhwc_matches_slicing_and_the_nchw_tensor(sh, layout):
    n = sh["N"] * sh["C"] * sh["H"] * sh["W"]
    x = (np.arange(n, dtype=np.int32) + 1).reshape(sh["N"], sh["C"], sh["H"], sh["W"])     # unique, non-zero
    xin = x if layout == "nchw" else np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    for cp in (sh["C"], (sh["C"] + 7) // 8 * 8):
        got = oracle.transform_nhwc(xin, sh, layout, cp)
        assert got.size == oracle.window_elems_nhwc(sh, cp)
        assert np.array_equal(got, _numpy_window_nhwc(x, sh, cp))
        assert np.all(got[..., sh["C"]:] == 0)
        # same elements as Eq. 2's tensor, channel moved innermost
        nchw = oracle.transform(x, sh)                                       # [N, C, Ho, Wp*Kh] with k*Kh+u
        ho = nchw.shape[2]
        want = nchw.reshape(sh["N"], sh["C"], ho, sh["W"] + 2 * sh["pad"], sh["Kh"]).transpose(0, 2, 3, 4, 1)
        assert np.array_equal(got[..., :sh["C"]], want)
    # 16-bit patterns travel verbatim as well
    x16 = (x % 65521).astype(np.uint16)
    xin16 = x16 if layout == "nchw" else np.ascontiguousarray(x16.transpose(0, 2, 3, 1))
    assert np.array_equal(oracle.transform_nhwc(xin16, sh, layout), _numpy_window_nhwc(x16, sh, sh["C"]))


def test_transform_nhwc_windows_are_contiguous_runs_in_v_u_c_order():
    sh = shp(1, 3, 6, 7, 1, 2, 3, 2, 1)
    rng = np.random.default_rng(3)
    x = rng.integers(1, 1000, (1, 3, 6, 7)).astype(np.int32)
    cp = 8
    win = oracle.transform_nhwc(x, sh, "nchw", cp)
    ho, wo = oracle.out_dims(sh)
    xp = np.pad(x, ((0, 0), (0, 0), (1, 1), (1, 1)))
    flat = win.reshape(1, ho, -1)
    for m, q in itertools.product(range(ho), range(wo)):
        start = q * sh["stride"] * sh["Kh"] * cp
        run = flat[0, m, start:start + sh["Kw"] * sh["Kh"] * cp].reshape(sh["Kw"], sh["Kh"], cp)
        for v, u, c in itertools.product(range(sh["Kw"]), range(sh["Kh"]), range(3)):
            assert run[v, u, c] == xp[0, c, m * sh["stride"] + u, q * sh["stride"] + v]


def test_nhwc_route_equals_direct_by_brute_force():
    """Every small shape (incl. Kh != Kw, strides, pads, channel padding, both input layouts): the
    NHWC im2win route gives Eq. 1's sums (same term set; integer data makes them exact)."""
    rng = np.random.default_rng(21)
    count = 0
    for N, C, H, W, Co, Kh, Kw, s, p in itertools.product((1, 2), (1, 3), (5, 6), (4, 7), (2,), (1, 2, 3), (1, 3), (1, 2), (0, 1, 2)):
        if H + 2 * p < Kh or W + 2 * p < Kw:
            continue
        sh = shp(N, C, H, W, Co, Kh, Kw, s, p)
        x = rng.integers(-3, 4, (N, C, H, W)).astype(np.float32)
        f = rng.integers(-2, 3, (Co, C, Kh, Kw)).astype(np.float32)
        y, a = oracle.conv_direct(x, f, sh)
        for layout, cp in (("nchw", C), ("nhwc", C + 5)):
            xin = x if layout == "nchw" else np.ascontiguousarray(x.transpose(0, 2, 3, 1))
            y2, a2 = oracle.conv_im2win_nhwc(xin, f, sh, layout, cp)
            assert np.array_equal(y, y2) and np.array_equal(a, a2), sh
        count += 1
    assert count > 250


def test_nhwc_route_on_real_values_and_image_ranges():
    rng = np.random.default_rng(22)
    sh = shp(3, 6, 10, 9, 4, 3, 3, 2, 1)
    x = rng.standard_normal((3, 6, 10, 9)).astype(np.float32)
    f = rng.standard_normal((4, 6, 3, 3)).astype(np.float32)
    y, a = oracle.conv_direct(x, f, sh)
    y2, a2 = oracle.conv_im2win_nhwc(x, f, sh, "nchw", 8)
    assert np.allclose(y, y2, rtol=0, atol=1e-12 * a.max()) and np.allclose(a, a2, rtol=0, atol=1e-12 * a.max())
    y3, _ = oracle.conv_im2win_nhwc(x, f, sh, "nchw", 8, 1, 3)
    assert np.array_equal(y3, y2[1:3])
    lib = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(f).double(), stride=2, padding=1).numpy()
    assert np.allclose(y2, lib, rtol=0, atol=1e-12 * a.max())
