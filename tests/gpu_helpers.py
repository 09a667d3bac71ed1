"""Helpers of the GPU parity tests: run the CUDA path through the C ABI with guard bands
around every output buffer, and compare with the CPU oracle."""
import os

import numpy as np
import torch

import oracle
from paper_2608_20725_b200 import binding

TOL_F32 = 1e-5     # |gpu - oracle| <= TOL * sum |x||w|   (fp32 path)
TOL_F16 = 2e-3     # same, fp16 inputs with fp32 accumulation, oracle on fp16-rounded inputs

GUARD = 64         # guard elements before and after each output buffer


def guarded(numel, dtype, fill):
    """A device buffer with GUARD canary elements on both sides; returns (whole, view)."""
    whole = torch.full((numel + 2 * GUARD,), fill, dtype=dtype, device="cuda")
    return whole, whole[GUARD:GUARD + numel]


def assert_guards_intact(whole, numel, fill):
    head = whole[:GUARD].cpu()
    tail = whole[GUARD + numel:].cpu()
    ref = torch.full((GUARD,), fill, dtype=whole.dtype)
    assert torch.equal(head.view(torch.uint8), ref.view(torch.uint8)), "write before the buffer"
    assert torch.equal(tail.view(torch.uint8), ref.view(torch.uint8)), "write past the buffer"


def gpu_transform(x_cpu: torch.Tensor, dims: dict) -> np.ndarray:
    """x (float32/float16/int32/int16 CPU tensor) -> window tensor as a numpy array of the same dtype."""
    code = binding.F32 if x_cpu.element_size() == 4 else binding.F16
    tdt = torch.float32 if code == binding.F32 else torch.float16
    wb, _, ho, _ = binding.im2win_workspace_size(dims, code)
    n = wb // x_cpu.element_size()
    whole, win = guarded(n, tdt, 7.0)
    xd = x_cpu.contiguous().view(tdt).cuda()
    binding.im2win_transform(xd, win, dims)
    torch.cuda.synchronize()
    assert_guards_intact(whole, n, 7.0)
    out = win.cpu().view(x_cpu.dtype).numpy()
    return out.reshape(dims["N"], dims["C"], ho, dims["Kh"] * (dims["W"] + 2 * dims["pad"]))


def gpu_conv(x_cpu: torch.Tensor, f_cpu: torch.Tensor, dims: dict, precision: str):
    """Transform + convolution on the GPU.  precision 'f32', 'f16' (the kernel the library picks),
    'f16-shift' (the gathering shifted-view kernel forced), 'f16-mat' (the matrix-transpose
    shifted-view kernel forced), 'f16-stem' (the one-k-block kernel where it can run) or 'f16-gather' (the general fp16 kernel forced); inputs are cast with torch's
    round-to-nearest-even conversion.  Returns (y float32 numpy, x_used, f_used as float32 numpy)."""
    if precision in ("f16-gather", "f16-shift", "f16-mat", "f16-stem"):
        os.environ["IM2WIN_F16_KERNEL"] = precision.split("-")[1]
        try:
            return gpu_conv(x_cpu, f_cpu, dims, "f16")
        finally:
            del os.environ["IM2WIN_F16_KERNEL"]
    tdt = torch.float32 if precision == "f32" else torch.float16
    code = binding.F32 if precision == "f32" else binding.F16
    xd = x_cpu.to(tdt).cuda().contiguous()
    fd = f_cpu.to(tdt).cuda().contiguous()
    wb, sb, ho, wo = binding.im2win_workspace_size(dims, code)
    nwin = wb // xd.element_size()
    nout = dims["N"] * dims["Co"] * ho * wo
    wwhole, win = guarded(nwin, tdt, 3.0)
    ywhole, y = guarded(nout, torch.float32, -123.0)
    swhole, scratch = guarded(sb, torch.uint8, 0x5a)
    assert scratch.data_ptr() % 16 == 0 and y.data_ptr() % 16 == 0 and win.data_ptr() % 16 == 0
    binding.im2win_transform(xd, win, dims)
    if precision == "f32":
        binding.im2win_conv_f32(win, fd, y, scratch, dims)
    else:
        binding.im2win_conv_f16(win, fd, y, scratch, dims)
    binding.im2win_check_status(scratch)
    assert_guards_intact(wwhole, nwin, 3.0)
    assert_guards_intact(ywhole, nout, -123.0)
    assert_guards_intact(swhole, sb, 0x5a)
    yh = y.cpu().numpy().reshape(dims["N"], dims["Co"], ho, wo)
    return yh, xd.float().cpu().numpy(), fd.float().cpu().numpy()


def gpu_layer_keep_window(x_cpu: torch.Tensor, f_cpu: torch.Tensor, dims: dict, precision: str, images):
    """Transform + convolution like gpu_conv, for layers whose window tensor is too large to copy to
    the host whole: returns (y float32 numpy, {n: window of image n as a raw-integer numpy array
    [1, C, Ho, Kh*Wp]} for n in `images`)."""
    tdt = torch.float32 if precision == "f32" else torch.float16
    idt = torch.int32 if precision == "f32" else torch.int16
    code = binding.F32 if precision == "f32" else binding.F16
    xd = x_cpu.to(tdt).cuda().contiguous()
    fd = f_cpu.to(tdt).cuda().contiguous()
    wb, sb, ho, wo = binding.im2win_workspace_size(dims, code)
    nwin = wb // xd.element_size()
    nout = dims["N"] * dims["Co"] * ho * wo
    wwhole, win = guarded(nwin, tdt, 3.0)
    ywhole, y = guarded(nout, torch.float32, -123.0)
    swhole, scratch = guarded(sb, torch.uint8, 0x5a)
    binding.im2win_transform(xd, win, dims)
    if precision == "f32":
        binding.im2win_conv_f32(win, fd, y, scratch, dims)
    else:
        binding.im2win_conv_f16(win, fd, y, scratch, dims)
    binding.im2win_check_status(scratch)
    assert_guards_intact(wwhole, nwin, 3.0)
    assert_guards_intact(ywhole, nout, -123.0)
    assert_guards_intact(swhole, sb, 0x5a)
    per = nwin // dims["N"]
    strip = dims["Kh"] * (dims["W"] + 2 * dims["pad"])
    wins = {n: win[n * per:(n + 1) * per].cpu().view(idt).numpy().reshape(1, dims["C"], ho, strip) for n in images}
    yh = y.cpu().numpy().reshape(dims["N"], dims["Co"], ho, wo)
    return yh, wins


def oracle_inputs(x_cpu: torch.Tensor, f_cpu: torch.Tensor, precision: str):
    """The values the oracle computes on: fp32 inputs as they are, or rounded to binary16 by the
    oracle's own routine for the fp16 path."""
    x = x_cpu.numpy().astype(np.float32)
    f = f_cpu.numpy().astype(np.float32)
    if precision.startswith("f16"):
        _, x = oracle.round_to_f16(x)
        _, f = oracle.round_to_f16(f)
    return x, f


def check_conv(y_gpu, y_ref, a_ref, precision, what=""):
    tol = TOL_F32 if precision == "f32" else TOL_F16
    err = np.abs(y_gpu.astype(np.float64) - y_ref)
    bound = tol * a_ref
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what} {precision}: {bad.sum()} of {bad.size} outputs out of tolerance; worst at {i}: "
                             f"gpu={y_gpu[i]!r} oracle={y_ref[i]!r} err={err[i]:.3e} bound={bound[i]:.3e}")
    zero = a_ref == 0
    assert np.all(y_gpu[zero] == 0), f"{what}: outputs with no non-zero term must be exactly 0"
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(a_ref > 0, err / a_ref, 0.0)
    return float(rel.max())


# ------------------------------------------------------- channel-innermost (NHWC) form ----
def gpu_transform_nhwc(x_nchw_bits: torch.Tensor, dims: dict, x_layout: str) -> np.ndarray:
    """x (int16 CPU tensor [N,C,H,W] of binary16 patterns) -> NHWC window tensor [N,Ho,Wp,Kh,Cp] (int16),
    feeding the library the input in `x_layout` ("nchw" or "nhwc")."""
    wb, _, ho, _, cp = binding.im2win_nhwc_workspace_size(dims)
    n = wb // 2
    whole, win = guarded(n, torch.float16, 7.0)
    xin = x_nchw_bits if x_layout == "nchw" else x_nchw_bits.permute(0, 2, 3, 1)
    xd = xin.contiguous().view(torch.float16).cuda()
    binding.im2win_transform_nhwc(xd, binding.NCHW if x_layout == "nchw" else binding.NHWC, win, dims)
    torch.cuda.synchronize()
    assert_guards_intact(whole, n, 7.0)
    return win.cpu().view(torch.int16).numpy().reshape(dims["N"], ho, dims["W"] + 2 * dims["pad"], dims["Kh"], cp)


def gpu_conv_nhwc(x_cpu: torch.Tensor, f_cpu: torch.Tensor, dims: dict, x_layout="nchw", bias=None, relu=False,
                  out16=False, y_nhwc=False, packed=False, repeat=1):
    """NHWC transform + convolution through the C ABI with guard bands.  Returns y as a float64 numpy
    array in the requested layout ([N,Co,Ho,Wo] or [N,Ho,Wo,Co])."""
    xh = x_cpu.half()
    xin = xh if x_layout == "nchw" else xh.permute(0, 2, 3, 1)
    xd = xin.contiguous().cuda()
    fd = f_cpu.half().cuda().contiguous()
    wb, sb, ho, wo, _ = binding.im2win_nhwc_workspace_size(dims)
    nout = dims["N"] * dims["Co"] * ho * wo
    odt = torch.float16 if out16 else torch.float32
    wwhole, win = guarded(wb // 2, torch.float16, 3.0)
    ywhole, y = guarded(nout, odt, -123.0)
    swhole, scratch = guarded(sb, torch.uint8, 0x5a)
    bd = None if bias is None else torch.as_tensor(bias, dtype=torch.float32).cuda().contiguous()
    epi = binding.make_epilogue(bd, relu, odt, binding.NHWC if y_nhwc else binding.NCHW)
    binding.im2win_transform_nhwc(xd, binding.NCHW if x_layout == "nchw" else binding.NHWC, win, dims)
    if packed:
        binding.im2win_pack_filter_nhwc(fd, scratch, dims)
        for _ in range(repeat):                      # the same packed filter and scratch, call after call
            binding.im2win_conv_packed_nhwc(win, y, scratch, dims, epi)
    else:
        binding.im2win_conv_f16_nhwc(win, fd, y, scratch, dims, epi)
    binding.im2win_check_status(scratch)
    assert_guards_intact(wwhole, wb // 2, 3.0)
    assert_guards_intact(ywhole, nout, -123.0)
    assert_guards_intact(swhole, sb, 0x5a)
    shape = (dims["N"], ho, wo, dims["Co"]) if y_nhwc else (dims["N"], dims["Co"], ho, wo)
    return y.cpu().double().numpy().reshape(shape)


def half_ulp_spacing(v: np.ndarray) -> np.ndarray:
    """Spacing of binary16 numbers at |v| (2^-24 in the subnormal range)."""
    with np.errstate(over="ignore"):
        h = np.minimum(np.abs(v), 65504.0).astype(np.float16)
    return np.spacing(h).astype(np.float64)


def check_fused(y_gpu, y_ref, a_ref, out16, what=""):
    """|gpu - oracle| <= 2e-3 * (sum|x||w| + |bias|) (+ one binary16 spacing at |y| when the store is
    binary16), y_ref being the oracle's value BEFORE the store rounding; exact zeros where nothing
    contributes."""
    err = np.abs(y_gpu - y_ref)
    bound = TOL_F16 * a_ref + (half_ulp_spacing(y_ref) if out16 else 0.0)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outputs out of tolerance; worst at {i}: "
                             f"gpu={y_gpu[i]!r} oracle={y_ref[i]!r} err={err[i]:.3e} bound={bound[i]:.3e}")
    assert np.all(y_gpu[a_ref == 0] == 0), f"{what}: outputs with no non-zero term must be exactly 0"
