"""The bounded device-side waits and the status word (IM2WIN_ERR_TIMEOUT).

Nothing here faults, traps or hangs the GPU: a wait that cannot complete gives up after a poll
limit, raises the status word and the kernel returns normally (its tensor memory freed), which
is what the tests check.  The limit is lowered through word 1 of the status block and one
barrier arrival of the one-k-block fp16 kernel is left out through the marker in word 2 (both
testing aids read by the kernels; the filter pack clears the block, so the words are written
between im2win_pack_filter and im2win_conv_packed).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_20725_b200 import binding, workloads
from paper_2608_20725_b200.workloads import Layer
from gpu_helpers import check_conv, oracle_inputs

pytestmark = pytest.mark.gpu

DROP_ARRIVE = 0x0d0a11fe      # marker of word 2 (csrc/ptx_sm100.cuh)

TINY = Layer("tiny_stem", 1, 3, 8, 8, 16, 3, 3, 1, 1, 71, "normal01", "he_normal")   # one tile, one CTA


def _status_words(scratch):
    return scratch[:256].view(torch.int32)


def test_check_status_maps_a_raised_status_word_to_timeout():
    """The host side alone: a non-zero word 0 reads as IM2WIN_ERR_TIMEOUT; the next filter pack
    clears it and a convolution on the same scratch then reports success."""
    dims = TINY.dims()
    x, f = workloads.make_inputs(TINY)
    window, scratch, y = binding.alloc_layer_buffers(dims, torch.float16)
    scratch.zero_()
    binding.im2win_check_status(scratch)
    _status_words(scratch)[0] = 1
    with pytest.raises(binding.Im2winError) as err:
        binding.im2win_check_status(scratch)
    assert err.value.code == 7
    binding.im2win_transform(x.half().cuda(), window, dims)
    binding.im2win_conv_f16(window, f.half().cuda(), y, scratch, dims)
    binding.im2win_check_status(scratch)


def test_a_wait_that_cannot_complete_gives_up_and_the_kernel_returns():
    dims = TINY.dims()
    x, f = workloads.make_inputs(TINY)
    xd, fd = x.half().cuda(), f.half().cuda()
    window, scratch, y = binding.alloc_layer_buffers(dims, torch.float16)
    binding.im2win_transform(xd, window, dims)
    binding.im2win_pack_filter(fd, scratch, dims)
    torch.cuda.synchronize()
    words = _status_words(scratch)
    words[1] = 4096               # poll limit of every wait of the next kernel
    words[2] = DROP_ARRIVE        # the copy warp leaves out its first arrival
    y.fill_(float("nan"))
    binding.im2win_conv_packed(window, y, scratch, dims)
    with pytest.raises(binding.Im2winError) as err:
        binding.im2win_check_status(scratch)          # synchronises: the kernel did return
    assert err.value.code == 7
    assert int(words[0].item()) == 1
    # the context is usable and the tensor memory was given back: the same layer, from the start
    for _ in range(2):
        binding.im2win_conv_f16(window, fd, y, scratch, dims)
        binding.im2win_check_status(scratch)
        xo, fo = oracle_inputs(x, f, "f16")
        yr, ar = oracle.conv_direct(xo, fo, dims)
        check_conv(y.cpu().numpy(), yr, ar, "f16", "after a timed-out call")
    # and a layer that needs all 512 tensor-memory columns of an SM
    wide = Layer("after_timeout_wide", 2, 16, 14, 14, 160, 3, 3, 1, 1, 72, "normal01", "he_normal")
    x2, f2 = workloads.make_inputs(wide)
    w2, s2, y2 = binding.alloc_layer_buffers(wide.dims(), torch.float16)
    binding.im2win_transform(x2.half().cuda(), w2, wide.dims())
    binding.im2win_conv_f16(w2, f2.half().cuda(), y2, s2, wide.dims())
    binding.im2win_check_status(s2)
    xo, fo = oracle_inputs(x2, f2, "f16")
    yr, ar = oracle.conv_direct(xo, fo, wide.dims())
    check_conv(y2.cpu().numpy(), yr, ar, "f16", wide.name)
