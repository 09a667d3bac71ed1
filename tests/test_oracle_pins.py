"""Pins of the CPU oracle against what the paper and the mathematics fix.

Each test is chosen so that a plausible mistake in the oracle (a dropped term,
a flipped kernel, a transposed index, a wrong stride or padding offset) fails
at least one of them.  None of these tests needs a GPU.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from conftest import read_golden


def shp(N, C, H, W, Co, Kh, Kw, s, p):
    return dict(N=N, C=C, H=H, W=W, Co=Co, Kh=Kh, Kw=Kw, stride=s, pad=p)


# ----------------------------------------------------------------- sizes ----
def test_table1_output_sizes():
    """Table 1: twelve (input, filter, stride) -> output triples, incl. the floor case cv4."""
    rows = read_golden("table1_layers.txt")
    assert len(rows) == 12
    for name, ci, hi, wi, co, hf, wf, s, ho, wo in rows:
        got = oracle.out_dims(shp(256, int(ci), int(hi), int(wi), int(co), int(hf), int(wf), int(s), 0))
        assert got == (int(ho), int(wo)), name


def test_fig1_shapes_and_sizes():
    """Fig. 1: 1x3x3x3 input, 2x3x2x2 filter -> 1x2x2x2 output; 36 window vs 48 im2col elements."""
    (row,) = read_golden("fig1_shapes.txt")
    N, C, H, W, Co, Kh, Kw, s, p, ho, wo, nwin, ncol = map(int, row)
    sh = shp(N, C, H, W, Co, Kh, Kw, s, p)
    assert oracle.out_dims(sh) == (ho, wo)
    assert oracle.window_elems(sh) == nwin
    assert oracle.im2col_elems(sh) == ncol


def test_cv4_window_bytes_consistent_with_reported_memory():
    """The paper reports 11.7 GB for fp32 im2win on cv4; the window tensor is 11.2 GB of it."""
    (row,) = read_golden("cv4_memory.txt")
    *dims, reported = row
    sh = shp(*map(int, dims))
    win_bytes = oracle.window_elems(sh) * 4
    assert win_bytes == 256 * 64 * 109 * 7 * 224 * 4
    out_bytes = 256 * 64 * 109 * 109 * 4
    in_bytes = 256 * 64 * 224 * 224 * 4
    # window alone is below the reported total, window+output+input is not far above it
    assert win_bytes / 1e9 < float(reported) < (win_bytes + out_bytes + in_bytes) / 1e9 + 1.0


@pytest.mark.parametrize("s", [1, 2, 3])
def test_window_vs_im2col_size_relation(s):
    """The window tensor is smaller than im2col iff s < Kw and equal at s == Kw (no padding,
    (W - Kw) divisible by s); the saving is N*C*Ho*Kh*(Wo-1)*(Kw-s)."""
    Kw = 3
    W = Kw + 4 * s
    sh = shp(2, 3, 9, W, 4, 2, Kw, s, 0)
    ho, wo = oracle.out_dims(sh)
    diff = oracle.im2col_elems(sh) - oracle.window_elems(sh)
    assert diff == 2 * 3 * ho * 2 * (wo - 1) * (Kw - s)
    assert (diff > 0) == (s < Kw) and (diff == 0) == (s == Kw)


def test_invalid_shapes_rejected():
    with pytest.raises(ValueError):
        oracle.out_dims(shp(1, 1, 2, 2, 1, 3, 3, 1, 0))
    with pytest.raises(ValueError):
        oracle.out_dims(shp(1, 1, 4, 4, 1, 3, 3, 0, 0))


# ------------------------------------------------------------- transform ----
def _coded_input(N, C, H, W):
    """Every element holds its own flat index + 1 (exact in float32 below 2^24)."""
    return (np.arange(N * C * H * W, dtype=np.float32) + 1).reshape(N, C, H, W)


@pytest.mark.parametrize("dims", [
    (2, 3, 5, 6, 1, 3, 3, 1, 1), (1, 2, 7, 5, 1, 2, 3, 2, 0), (2, 1, 6, 6, 1, 3, 2, 3, 2),
    (1, 2, 9, 9, 1, 7, 7, 2, 3), (1, 1, 4, 5, 1, 1, 1, 1, 0), (1, 2, 8, 7, 1, 3, 5, 2, 1),
])
def test_transform_decodes_to_source_coordinates(dims):
    """With x = unique codes, every window-tensor entry names its source element.

    The expected coordinate is derived from the sliding-window picture, not from
    Eq. 2: entry j of strip (n, c, ho) is row (j mod Kh) and column (j div Kh) of
    the Kh-row band of the padded image that output row ho reads.
    """
    N, C, H, W, Co, Kh, Kw, s, p = dims
    sh = shp(*dims)
    x = _coded_input(N, C, H, W)
    win = oracle.transform(x, sh)
    ho_n, _ = oracle.out_dims(sh)
    Wp = W + 2 * p
    assert win.shape == (N, C, ho_n, Kh * Wp)
    xpad = np.zeros((N, C, H + 2 * p, Wp), dtype=np.float32)
    xpad[:, :, p:p + H, p:p + W] = x
    for n, c, ho in itertools.product(range(N), range(C), range(ho_n)):
        band = xpad[n, c, ho * s: ho * s + Kh, :]            # Kh x Wp
        assert np.array_equal(win[n, c, ho], band.T.reshape(-1)), (n, c, ho)


def test_transform_windows_are_contiguous_runs():
    """Each sliding window of Eq. 1 appears as one contiguous run of Kh*Kw entries,
    starting (wo*s)*Kh into the strip, in column-major (height-fastest) order."""
    dims = (1, 2, 8, 9, 1, 3, 4, 2, 1)
    N, C, H, W, Co, Kh, Kw, s, p = dims
    sh = shp(*dims)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    win = oracle.transform(x, sh)
    ho_n, wo_n = oracle.out_dims(sh)
    xpad = np.pad(x, ((0, 0), (0, 0), (p, p), (p, p)))
    for c, ho, wo in itertools.product(range(C), range(ho_n), range(wo_n)):
        patch = xpad[0, c, ho * s: ho * s + Kh, wo * s: wo * s + Kw]
        run = win[0, c, ho, wo * s * Kh: wo * s * Kh + Kh * Kw]
        assert np.array_equal(run, patch.T.reshape(-1))


def test_transform_multiplicity_and_zero_fill():
    """Input element (h, w) appears once per output row whose band covers row h; all other
    entries are +0 bit patterns."""
    dims = (1, 1, 7, 5, 1, 3, 3, 2, 1)
    N, C, H, W, Co, Kh, Kw, s, p = dims
    sh = shp(*dims)
    x = _coded_input(N, C, H, W)
    win = oracle.transform(x, sh)
    ho_n, _ = oracle.out_dims(sh)
    flat = win.reshape(-1)
    for h in range(H):
        mult = sum(1 for ho in range(ho_n) if ho * s <= h + p < ho * s + Kh)
        for w in range(W):
            assert np.count_nonzero(flat == x[0, 0, h, w]) == mult
    nonzero = sum(sum(1 for ho in range(ho_n) if ho * s <= h + p < ho * s + Kh) for h in range(H)) * W
    assert np.count_nonzero(flat.view(np.uint32)) == nonzero


def test_transform_identity_when_kh1_stride1_nopad():
    x = np.random.default_rng(2).standard_normal((2, 3, 4, 5)).astype(np.float32)
    win = oracle.transform(x, shp(2, 3, 4, 5, 1, 1, 3, 1, 0))
    assert np.array_equal(win.reshape(x.shape), x)


def test_transform_copies_bit_patterns_verbatim_16bit_and_32bit():
    """NaN payloads and -0.0 survive; the 16-bit path moves half bit patterns."""
    sh = shp(1, 1, 3, 3, 1, 2, 2, 1, 1)
    x32 = np.array([0x7fc01234, 0x80000000, 0xffffffff, 1, 2, 3, 4, 5, 6], dtype=np.uint32).reshape(1, 1, 3, 3)
    w32 = oracle.transform(x32, sh)
    x16 = np.array([0x7e01, 0x8000, 0xffff, 1, 2, 3, 4, 5, 6], dtype=np.uint16).reshape(1, 1, 3, 3)
    w16 = oracle.transform(x16, sh)
    assert w32.dtype == np.uint32 and w16.dtype == np.uint16
    # same permutation in both widths
    lut = {int(a): int(b) for a, b in zip(x32.reshape(-1), x16.reshape(-1))}
    lut[0] = 0
    assert [lut[int(v)] for v in w32.reshape(-1)] == [int(v) for v in w16.reshape(-1)]
    assert sorted(set(w32.reshape(-1).tolist())) == sorted(set(x32.reshape(-1).tolist()) | {0})


# ----------------------------------------------------------- convolution ----
def test_worked_example_by_hand():
    """x = [[1,2,3],[4,5,6],[7,8,9]], f = [[1,2],[3,4]], stride 1, no padding.
    By hand (cross-correlation): 1+4+12+20, 2+6+15+24, 4+10+21+32, 5+12+24+36."""
    x = np.arange(1, 10, dtype=np.float32).reshape(1, 1, 3, 3)
    f = np.array([[1, 2], [3, 4]], dtype=np.float32).reshape(1, 1, 2, 2)
    want = np.array([[37, 47], [67, 77]], dtype=np.float64).reshape(1, 1, 2, 2)
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, a = fn(x, f, shp(1, 1, 3, 3, 1, 2, 2, 1, 0))
        assert np.array_equal(y, want)
        assert np.array_equal(a, want)       # all terms positive => a == y


def test_worked_example_stride2_pad1_by_hand():
    """Same x, f = [[1,0],[0,-1]], stride 2, padding 1: windows of the 5x5 padded image at
    rows/cols {0,2}: y = [[0-1, 0-3],[0-7, 5-9]]... computed by hand below."""
    x = np.arange(1, 10, dtype=np.float32).reshape(1, 1, 3, 3)
    f = np.array([[1, 0], [0, -1]], dtype=np.float32).reshape(1, 1, 2, 2)
    # padded image P (5x5) has x at P[1:4,1:4]; y[m][n] = P[2m][2n] - P[2m+1][2n+1]
    # y[0][0] = 0 - 1, y[0][1] = 0 - 3, y[1][0] = 0 - 7, y[1][1] = 5 - 9
    want = np.array([[-1, -3], [-7, -4]], dtype=np.float64).reshape(1, 1, 2, 2)
    wanta = np.array([[1, 3], [7, 14]], dtype=np.float64).reshape(1, 1, 2, 2)
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, a = fn(x, f, shp(1, 1, 3, 3, 1, 2, 2, 2, 1))
        assert np.array_equal(y, want)
        assert np.array_equal(a, wanta)


TINY = [
    (N, C, H, W, Co, Kh, Kw, s, p)
    for N, C, Co in [(1, 1, 1), (2, 3, 2)]
    for H, W in [(4, 5), (7, 6)]
    for Kh, Kw in [(1, 1), (2, 3), (3, 2), (3, 3)]
    for s in (1, 2, 3)
    for p in (0, 1, 2)
]


def test_im2win_route_equals_direct_by_brute_force():
    """Eq. 3 over the window tensor has the same term set as Eq. 1: equal to fp64 noise on
    random data, exactly equal on integer data, over a grid of tiny shapes incl. Kh != Kw."""
    rng = np.random.default_rng(3)
    for dims in TINY:
        N, C, H, W, Co, Kh, Kw, s, p = dims
        sh = shp(*dims)
        x = rng.standard_normal((N, C, H, W)).astype(np.float32)
        f = rng.standard_normal((Co, C, Kh, Kw)).astype(np.float32)
        y1, a1 = oracle.conv_direct(x, f, sh)
        y2, a2 = oracle.conv_im2win(x, f, sh)
        assert np.all(np.abs(y1 - y2) <= 1e-13 * a1 + 1e-300), dims
        assert np.allclose(a1, a2, rtol=1e-13, atol=0), dims
        xi = rng.integers(-3, 4, (N, C, H, W)).astype(np.float32)
        fi = rng.integers(-3, 4, (Co, C, Kh, Kw)).astype(np.float32)
        yi1, _ = oracle.conv_direct(xi, fi, sh)
        yi2, _ = oracle.conv_im2win(xi, fi, sh)
        assert np.array_equal(yi1, yi2), dims


@pytest.mark.parametrize("dims", [
    (2, 3, 8, 9, 4, 3, 3, 1, 1), (1, 4, 11, 10, 3, 5, 3, 2, 2), (2, 2, 9, 9, 2, 7, 7, 2, 3),
    (1, 5, 6, 7, 6, 1, 1, 1, 0), (1, 3, 12, 12, 2, 2, 4, 3, 1),
])
def test_against_library_convolution(dims):
    """torch.nn.functional.conv2d in float64 on the CPU is an independent routine."""
    N, C, H, W, Co, Kh, Kw, s, p = dims
    sh = shp(*dims)
    g = torch.Generator().manual_seed(4)
    x = torch.randn((N, C, H, W), generator=g)
    f = torch.randn((Co, C, Kh, Kw), generator=g)
    ref = torch.nn.functional.conv2d(x.double(), f.double(), stride=s, padding=p).numpy()
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, a = fn(x.numpy(), f.numpy(), sh)
        assert y.shape == ref.shape
        assert np.all(np.abs(y - ref) <= 1e-13 * a)
    aref = torch.nn.functional.conv2d(x.double().abs(), f.double().abs(), stride=s, padding=p).numpy()
    assert np.allclose(a, aref, rtol=1e-13)


@pytest.mark.parametrize("K", [1, 3, 5])
def test_delta_filter_reproduces_input(K):
    C, H, W = 3, 6, 7
    x = np.random.default_rng(5).standard_normal((2, C, H, W)).astype(np.float32)
    f = np.zeros((C, C, K, K), dtype=np.float32)
    for c in range(C):
        f[c, c, K // 2, K // 2] = 1.0
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, _ = fn(x, f, shp(2, C, H, W, C, K, K, 1, K // 2))
        assert np.array_equal(y, x.astype(np.float64))


def test_off_centre_delta_shifts_the_image():
    """A delta at (u, v) = (0, 2) of a 3x3 filter with padding 1 reads x[h-1][w+1]:
    catches a swapped u/v or a wrong padding offset."""
    x = np.random.default_rng(6).standard_normal((1, 1, 5, 6)).astype(np.float32)
    f = np.zeros((1, 1, 3, 3), dtype=np.float32)
    f[0, 0, 0, 2] = 1.0
    want = np.zeros((1, 1, 5, 6))
    want[0, 0, 1:, :-1] = x[0, 0, :-1, 1:]
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, _ = fn(x, f, shp(1, 1, 5, 6, 1, 3, 3, 1, 1))
        assert np.array_equal(y, want)


def test_one_by_one_kernel_is_a_plain_gemm():
    N, C, H, W, Co = 2, 5, 4, 3, 6
    rng = np.random.default_rng(7)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    f = rng.standard_normal((Co, C, 1, 1)).astype(np.float32)
    want = np.einsum("oc,nchw->nohw", f[:, :, 0, 0].astype(np.float64), x.astype(np.float64))
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        y, a = fn(x, f, shp(N, C, H, W, Co, 1, 1, 1, 0))
        assert np.all(np.abs(y - want) <= 1e-13 * a)


def test_bilinearity():
    dims = (2, 3, 7, 8, 4, 3, 3, 2, 1)
    sh = shp(*dims)
    rng = np.random.default_rng(8)
    # values with few mantissa bits so that a*x1 + b*x2 is exact in float32
    x1 = rng.integers(-8, 9, (2, 3, 7, 8)).astype(np.float32) / 4
    x2 = rng.integers(-8, 9, (2, 3, 7, 8)).astype(np.float32) / 4
    f1 = rng.integers(-8, 9, (4, 3, 3, 3)).astype(np.float32) / 8
    f2 = rng.integers(-8, 9, (4, 3, 3, 3)).astype(np.float32) / 8
    a_, b_ = 2.0, -0.5
    for fn in (oracle.conv_direct, oracle.conv_im2win):
        lhs, _ = fn(a_ * x1 + b_ * x2, f1, sh)
        r1, _ = fn(x1, f1, sh)
        r2, _ = fn(x2, f1, sh)
        assert np.array_equal(lhs, a_ * r1 + b_ * r2)
        lhs, _ = fn(x1, a_ * f1 + b_ * f2, sh)
        r2, _ = fn(x1, f2, sh)
        assert np.array_equal(lhs, a_ * r1 + b_ * r2)


def test_direct_points_match_full_direct():
    dims = (2, 3, 9, 8, 4, 3, 3, 2, 1)
    sh = shp(*dims)
    rng = np.random.default_rng(9)
    x = rng.standard_normal((2, 3, 9, 8)).astype(np.float32)
    f = rng.standard_normal((4, 3, 3, 3)).astype(np.float32)
    y, a = oracle.conv_direct(x, f, sh)
    idx = rng.integers(0, y.size, 50)
    yp, ap = oracle.conv_direct_points(x, f, sh, idx)
    assert np.array_equal(yp, y.reshape(-1)[idx]) and np.array_equal(ap, a.reshape(-1)[idx])


def test_im2win_range_matches_full():
    dims = (4, 2, 6, 6, 3, 3, 3, 1, 1)
    sh = shp(*dims)
    rng = np.random.default_rng(10)
    x = rng.standard_normal((4, 2, 6, 6)).astype(np.float32)
    f = rng.standard_normal((3, 2, 3, 3)).astype(np.float32)
    y, a = oracle.conv_im2win(x, f, sh)
    ys, as_ = oracle.conv_im2win_range(x, f, sh, 1, 3)
    assert np.array_equal(ys, y[1:3]) and np.array_equal(as_, a[1:3])


# -------------------------------------------------------- binary16 rounding ----
def test_f16_roundtrip_exhaustive():
    """All 65 536 half patterns: widen -> round back is the identity (NaNs stay NaNs)."""
    bits = np.arange(65536, dtype=np.uint16)
    as_f32 = bits.view(np.float16).astype(np.float32)
    got, back = oracle.round_to_f16(as_f32)
    nan = np.isnan(as_f32)
    assert np.array_equal(got[~nan], bits[~nan])
    assert np.array_equal(back[~nan], as_f32[~nan])
    assert np.all(np.isnan(back[nan])) and np.all((got[nan] & 0x7c00) == 0x7c00) and np.all(got[nan] & 0x3ff)
    assert np.array_equal(oracle.f16_bits_to_f64(bits)[~nan], as_f32[~nan].astype(np.float64))


def test_f16_ties_to_even_and_limits():
    pos = np.arange(0, 0x7c00, dtype=np.uint16)                  # finite non-negative halves
    lo = pos[:-1].view(np.float16).astype(np.float64)
    hi = pos[1:].view(np.float16).astype(np.float64)
    mid = ((lo + hi) / 2).astype(np.float32)                     # exact in float32
    assert np.array_equal(mid.astype(np.float64), (lo + hi) / 2)
    got, _ = oracle.round_to_f16(mid)
    want = np.where(pos[:-1] % 2 == 0, pos[:-1], pos[1:])        # the even neighbour
    assert np.array_equal(got, want)
    # just above / below a midpoint goes to the nearer neighbour
    up, _ = oracle.round_to_f16(np.nextafter(mid, np.float32(np.inf)))
    dn, _ = oracle.round_to_f16(np.nextafter(mid, np.float32(-np.inf)))
    assert np.array_equal(up, pos[1:]) and np.array_equal(dn, pos[:-1])
    special = np.array([65519.996, 65520.0, 1e10, -1e10, 2.0 ** -25, 2.0 ** -25 * 1.0001, 2.0 ** -26, -0.0,
                        np.inf, -np.inf], dtype=np.float32)
    got, _ = oracle.round_to_f16(special)
    assert got.tolist() == [0x7bff, 0x7c00, 0x7c00, 0xfc00, 0x0000, 0x0001, 0x0000, 0x8000, 0x7c00, 0xfc00]


def test_f16_matches_library_conversion_on_random_values():
    rng = np.random.default_rng(11)
    v = np.concatenate([
        rng.standard_normal(200000).astype(np.float32),
        (rng.standard_normal(200000) * 0.008).astype(np.float32),          # reaches half subnormals
        (rng.standard_normal(100000) * 1e-5).astype(np.float32),
        rng.integers(0, 2 ** 32, 200000, dtype=np.uint64).astype(np.uint32).view(np.float32),
    ])
    v = v[~np.isnan(v)]
    got, back = oracle.round_to_f16(v)
    with np.errstate(over="ignore"):
        lib = v.astype(np.float16)
    assert np.array_equal(got, lib.view(np.uint16))
    assert np.array_equal(back, lib.astype(np.float32))
