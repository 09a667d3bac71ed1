"""The allocation-free fp32 entry point (scratch in a fixed array inside the library).

Who needs it: callers that are handed input and output buffers but cannot create a scratch
buffer themselves, because device allocation is forbidden or unavailable where they run.
The test calls it through the C ABI twice in a row, on two different layers, and checks
each result against the ordinary entry point (caller-provided scratch) and the oracle's
tolerance.  Collected last on purpose, so that a failure here cannot hide other tests.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2608_20725_b200 import binding, workloads
from paper_2608_20725_b200.workloads import Layer


def _layer(name, N, C, H, W, Co, K, s, p, seed):
    return Layer(name, N, C, H, W, Co, K, K, s, p, seed, "normal01", "he_normal")


@pytest.mark.gpu
def test_static_scratch_entry_matches_regular_entry_twice_in_a_row():
    # second layer is smaller in every scratch dimension than the first: stale filter or
    # table contents left by the first call would show up in the second result
    layers = [_layer("first", 3, 40, 13, 12, 72, 3, 1, 1, 71), _layer("second", 2, 5, 9, 9, 7, 3, 2, 0, 72)]
    lib = binding.lib()
    for layer in layers:
        dims = layer.dims()
        x, f = workloads.make_inputs(layer)
        xd, fd = x.cuda(), f.cuda()
        window, scratch, y_ref = binding.alloc_layer_buffers(dims, torch.float32)
        binding.im2win_transform(xd, window, dims)
        binding.im2win_conv_f32(window, fd, y_ref, scratch, dims)
        y = torch.full_like(y_ref, float("nan"))
        shape = binding.as_shape(dims)
        stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        rc = lib.im2win_conv_f32_static(window.data_ptr(), fd.data_ptr(), y.data_ptr(), ctypes.byref(shape), stream)
        assert rc == 0, binding.STATUS_NAMES.get(rc, rc)
        torch.cuda.synchronize()
        # "allocates nothing": once the first call has done its per-device set-up, a call must leave the
        # device's free memory where it was
        free_before, _ = torch.cuda.mem_get_info()
        rc = lib.im2win_conv_f32_static(window.data_ptr(), fd.data_ptr(), y.data_ptr(), ctypes.byref(shape), stream)
        assert rc == 0, binding.STATUS_NAMES.get(rc, rc)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert free_after == free_before, "the allocation-free entry point changed the device's free memory"
        _, a = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        yr, yn = y_ref.cpu().numpy().astype(np.float64), y.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(yn))
        assert np.all(np.abs(yn - yr) <= 1e-5 * a), layer.name
        y_or, _ = oracle.conv_direct(x.numpy(), f.numpy(), dims)
        assert np.all(np.abs(yn - y_or) <= 1e-5 * a), layer.name


def test_static_scratch_entry_rejects_oversized_layers_before_touching_cuda():
    lib = binding.lib()
    big = binding.as_shape(workloads.LAYERS["cfg4b"].dims())          # fp32 scratch ~9.4 MB > 4 MiB
    _, need, _, _ = binding.im2win_workspace_size(big, binding.F32)
    assert need > binding.STATIC_SCRATCH_BYTES
    rc = lib.im2win_conv_f32_static(ctypes.c_void_p(256), ctypes.c_void_p(512), ctypes.c_void_p(1024),
                                    ctypes.byref(big), None)
    assert rc == 4
    ok = binding.as_shape(workloads.LAYERS["cfg2"].dims())
    assert binding.im2win_workspace_size(ok, binding.F32)[1] <= binding.STATIC_SCRATCH_BYTES
    assert lib.im2win_conv_f32_static(None, ctypes.c_void_p(512), ctypes.c_void_p(1024), ctypes.byref(ok), None) == 2
    assert lib.im2win_conv_f32_static(ctypes.c_void_p(260), ctypes.c_void_p(512), ctypes.c_void_p(1024),
                                      ctypes.byref(ok), None) == 3
