"""Host-side checks of the C ABI: the library builds, loads, exports every declared symbol,
reports closed-form sizes and rejects bad arguments before launching anything.  No GPU needed."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2608_20725_b200 import binding, workloads
from conftest import ROOT


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "im2win.h")).read()
    # strip comments, then collect function declarators
    code = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(im2win_[a-z0-9_]+)\s*\(", code))
    assert declared, "no declarations found"
    lib = binding.lib()
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in im2win.h but not exported"
    assert declared == set(binding.EXPORTS)


def test_status_strings():
    lib = binding.lib()
    seen = set()
    for code in range(8):
        s = lib.im2win_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert lib.im2win_status_string(99).decode() == "unknown status"


@pytest.mark.parametrize("layer", list(workloads.LAYERS.values()) + list(workloads.TABLE1_LAYERS.values()),
                         ids=lambda l: l.name)
def test_window_bytes_equal_closed_form(layer):
    """window_bytes is exactly N*C*Ho*Kh*(W+2p)*esize -- compared with the oracle's count --
    and never larger than im2col's N*C*Kh*Kw*Ho*Wo elements when stride < Kw."""
    for code, es in ((binding.F32, 4), (binding.F16, 2)):
        wb, sb, ho, wo = binding.im2win_workspace_size(layer, code)
        assert (ho, wo) == oracle.out_dims(layer.dims())
        assert wb == oracle.window_elems(layer.dims()) * es
        assert sb >= 256 + layer.Co * layer.C * layer.Kh * layer.Kw * es
        if layer.stride < layer.Kw and layer.pad == 0:
            assert wb <= oracle.im2col_elems(layer.dims()) * es


def test_layer_workspace_covers_all_buffers():
    layer = workloads.LAYERS["cfg4a"]
    for code, es in ((binding.F32, 4), (binding.F16, 2)):
        wb, sb, ho, wo = binding.im2win_workspace_size(layer, code)
        total = binding.im2win_layer_workspace_size(layer, code)
        need = (layer.N * layer.C * layer.H * layer.W * es + layer.Co * layer.C * layer.Kh * layer.Kw * es
                + wb + sb + layer.N * layer.Co * ho * wo * 4)
        assert need <= total <= need + 5 * 256


BAD_SHAPES = [
    dict(N=0, C=1, H=4, W=4, Co=1, Kh=3, Kw=3, stride=1, pad=0),
    dict(N=1, C=1, H=4, W=4, Co=1, Kh=3, Kw=3, stride=0, pad=0),
    dict(N=1, C=1, H=4, W=4, Co=1, Kh=3, Kw=3, stride=1, pad=-1),
    dict(N=1, C=1, H=2, W=4, Co=1, Kh=3, Kw=3, stride=1, pad=0),     # Ho < 1
    dict(N=1, C=1, H=4, W=2, Co=1, Kh=3, Kw=3, stride=1, pad=0),     # Wo < 1
    dict(N=1, C=-3, H=4, W=4, Co=1, Kh=3, Kw=3, stride=1, pad=0),
]


@pytest.mark.parametrize("bad", BAD_SHAPES)
def test_invalid_shapes_rejected(bad):
    with pytest.raises(binding.Im2winError) as e:
        binding.im2win_workspace_size(bad, binding.F32)
    assert e.value.code == 1


def test_unsupported_and_bad_dtype():
    huge = dict(N=1, C=4096, H=4096, W=4096, Co=1, Kh=3, Kw=3, stride=1, pad=0)   # per-image window >= 2^31 elements
    with pytest.raises(binding.Im2winError) as e:
        binding.im2win_workspace_size(huge, binding.F32)
    assert e.value.code == 5
    ok = dict(N=1, C=1, H=4, W=4, Co=1, Kh=3, Kw=3, stride=1, pad=0)
    with pytest.raises(binding.Im2winError) as e:
        binding.im2win_workspace_size(ok, 7)
    assert e.value.code == 1


def test_null_and_misaligned_pointers_rejected_before_launch():
    """These return before any CUDA call, so they are safe without a device."""
    lib = binding.lib()
    s = binding.make_shape(1, 1, 4, 4, 1, 3, 3, 1, 0)
    sp = ctypes.byref(s)
    assert lib.im2win_transform(None, ctypes.c_void_p(256), sp, 0, None) == 2
    assert lib.im2win_transform(ctypes.c_void_p(256), ctypes.c_void_p(256), None, 0, None) == 2
    assert lib.im2win_transform(ctypes.c_void_p(256), ctypes.c_void_p(264), sp, 0, None) == 3
    assert lib.im2win_transform(ctypes.c_void_p(256), ctypes.c_void_p(512), sp, 5, None) == 1
    assert lib.im2win_conv_f32(ctypes.c_void_p(256), None, ctypes.c_void_p(512), ctypes.c_void_p(768), 1 << 20, sp, None) == 2
    assert lib.im2win_conv_f32(ctypes.c_void_p(256), ctypes.c_void_p(1024), ctypes.c_void_p(520), ctypes.c_void_p(768),
                               1 << 20, sp, None) == 3
    assert lib.im2win_conv_f16(ctypes.c_void_p(256), ctypes.c_void_p(1024), ctypes.c_void_p(512), ctypes.c_void_p(768),
                               16, sp, None) == 4
    assert lib.im2win_check_status(None, None) == 2
    vp = ctypes.c_void_p
    assert lib.im2win_pack_filter(None, vp(768), 1 << 20, sp, 0, None) == 2
    assert lib.im2win_pack_filter(vp(1024), vp(776), 1 << 20, sp, 0, None) == 3
    assert lib.im2win_pack_filter(vp(1024), vp(768), 16, sp, 1, None) == 4
    assert lib.im2win_pack_filter(vp(1024), vp(768), 1 << 20, sp, 7, None) == 1
    assert lib.im2win_conv_packed(None, vp(512), vp(768), 1 << 20, sp, 0, None) == 2
    assert lib.im2win_conv_packed(vp(256), vp(520), vp(768), 1 << 20, sp, 1, None) == 3
    assert lib.im2win_conv_packed(vp(256), vp(512), vp(768), 16, sp, 0, None) == 4
    assert lib.im2win_layer_forward_host(ctypes.c_void_p(256), ctypes.c_void_p(256), ctypes.c_void_p(256),
                                         ctypes.c_void_p(128), 1 << 30, sp, 0, None) == 3
    assert lib.im2win_layer_forward_host(ctypes.c_void_p(256), ctypes.c_void_p(256), ctypes.c_void_p(256),
                                         ctypes.c_void_p(256), 16, sp, 0, None) == 4


def test_nhwc_kernel_name_query():
    """Host-only: which NHWC kernel a layer takes (reports and tests use it).  Wide-kernel stride-1
    layers take the shifted views, stride 2 with a 3-wide kernel the overlapping rows; the longest
    reductions split every tile's K or, with any epilogue, share the tiles of a short last round by
    runs of the reduction; short reductions (3x3) do neither."""
    import torch
    name = binding.im2win_nhwc_kernel_name
    assert name(workloads.LAYERS["cfg2"].dims()) == "f16-nhwc-shift"
    assert name(workloads.LAYERS["cfg5k5"].dims()) == "f16-nhwc-shift"
    assert name(workloads.LAYERS["cfg4c"].dims()) == "f16-nhwc-overlap"
    relu16 = binding.make_epilogue(None, True, torch.float16, binding.NCHW)
    assert name(workloads.LAYERS["cfg5k11"].dims()) == "f16-nhwc-overlap+ksplit"
    assert name(workloads.LAYERS["cfg5k7"].dims()) == "f16-nhwc-overlap+runs"
    assert name(workloads.LAYERS["cfg5k11"].dims(), relu16) == "f16-nhwc-overlap+runs"
    assert name(workloads.LAYERS["cfg5k7"].dims(), relu16) == "f16-nhwc-overlap+runs"
    assert name(workloads.LAYERS["cfg4a"].dims(), relu16) == "f16-nhwc-overlap"
    huge = dict(workloads.LAYERS["cfg2"].dims(), C=40000)       # beyond the NHWC transform's staging
    assert name(huge) == "none"
