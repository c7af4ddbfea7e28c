"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, validates descriptors and infers integer shapes exactly like the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

from paper_1901_00858_b200 import binding as hgc
from paper_1901_00858_b200 import build as hgc_build
from paper_1901_00858_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    hgc_build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hgc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hgc_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_symbols()
    assert "hgc_conv_forward" in names and "hgc_conv_desc_create" in names and len(names) >= 14
    L = ctypes.CDLL(hgc.LIB_PATH)
    for nm in names:
        assert hasattr(L, nm), f"{nm} is declared in hgc.h but not exported"


def test_status_strings():
    for code in range(7):
        assert hgc.status_string(code)
    assert hgc.status_string(0) == "ok"
    assert "unknown" in hgc.status_string(12345)


@pytest.mark.parametrize("bad", [
    dict(n=0), dict(c=0), dict(h=0), dict(w=0), dict(k=0), dict(r=0), dict(s=0), dict(group=0),
    dict(stride_h=0), dict(stride_w=0), dict(dil_h=0), dict(dil_w=0), dict(pad_h=-1), dict(pad_w=-1),
    dict(c=6, group=4), dict(k=6, group=4, c=8), dict(h=2, r=3), dict(w=4, s=3, dil_w=2),
])
def test_invalid_descriptors_are_rejected(bad):
    base = dict(n=1, c=4, h=8, w=8, k=4, r=3, s=3)
    base.update(bad)
    with pytest.raises(hgc.HgcError) as e:
        hgc.ConvDesc(**base)
    assert e.value.status == hgc.HGC_INVALID_ARG


def test_null_arguments():
    L = hgc.lib()
    assert L.hgc_conv_desc_create(None, None) == hgc.HGC_INVALID_ARG
    h = ctypes.c_void_p(123)
    assert L.hgc_conv_desc_create(ctypes.byref(h), None) == hgc.HGC_INVALID_ARG
    assert not h.value
    assert L.hgc_conv_desc_destroy(None) == hgc.HGC_OK
    d = hgc.ConvDesc(1, 3, 8, 8, 4, 3, 3)
    assert L.hgc_conv_forward(d.handle, None, None, None, None, 0, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_forward(None, 16, 16, None, 16, 0, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_forward(d.handle, 32, 48, None, 66, 0, None) == hgc.HGC_BAD_ALIGNMENT
    assert L.hgc_conv_forward(d.handle, 32, 48, 6, 64, 0, None) == hgc.HGC_BAD_ALIGNMENT
    assert L.hgc_conv_output_dims(None, None, None, None, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_set_workspace(d.handle, 128, 10) == hgc.HGC_BAD_ALIGNMENT
    assert L.hgc_conv_set_workspace(d.handle, None, 10) == hgc.HGC_INVALID_ARG
    assert L.hgc_layout_nchw_to_nhwc(16, 32, 1, 3, 4, 4, 4, None) == hgc.HGC_INVALID_ARG  # c_pad % 8
    assert L.hgc_layout_nchw_to_nhwc(16, 32, 1, 9, 4, 4, 8, None) == hgc.HGC_INVALID_ARG  # c_pad < c
    assert L.hgc_weights_repack(16, 32, 6, 3, 3, 3, 4, 8, None) == hgc.HGC_INVALID_ARG    # k % group


def test_output_dims_of_the_workloads(oracle):
    for wl in workloads.all_workloads():
        for l in wl.layers:
            d = hgc.ConvDesc(wl.batch, l.c, l.h, l.h, l.k, l.r, l.r, l.pad, l.pad, l.stride, l.stride,
                             l.dil, l.dil, l.group)
            assert d.output_dims() == (wl.batch, l.k, l.out, l.out), (wl.name, l.name)
            d.close()


@settings(max_examples=300, deadline=None)
@given(st.integers(1, 200), st.integers(1, 200), st.integers(1, 9), st.integers(1, 9), st.integers(0, 5),
       st.integers(0, 5), st.integers(1, 5), st.integers(1, 5), st.integers(1, 3), st.integers(1, 3))
def test_shape_inference_matches_oracle_exactly(oracle, h, w, r, s, ph, pw, sh, sw, dh, dw):
    P, Q = oracle.out_dim(h, r, ph, sh, dh), oracle.out_dim(w, s, pw, sw, dw)
    args = dict(n=2, c=4, h=h, w=w, k=6, r=r, s=s, pad_h=ph, pad_w=pw, stride_h=sh, stride_w=sw,
                dil_h=dh, dil_w=dw, group=2)
    if P < 1 or Q < 1:
        with pytest.raises(hgc.HgcError) as e:
            hgc.ConvDesc(**args)
        assert e.value.status == hgc.HGC_INVALID_ARG
    else:
        d = hgc.ConvDesc(**args)
        assert d.output_dims() == (2, 6, P, Q)
        d.close()


def test_planner_paths():
    dw = hgc.ConvDesc(2, 32, 14, 14, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32)
    assert dw.path() == hgc.HGC_PATH_DEPTHWISE
    forced = hgc.ConvDesc(2, 32, 14, 14, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32, hgc.HGC_FLAG_FORCE_DIRECT)
    assert forced.path() == hgc.HGC_PATH_DIRECT
    dil = hgc.ConvDesc(2, 32, 14, 14, 32, 3, 3, 2, 2, 1, 1, 2, 2, 32)
    assert dil.path() == hgc.HGC_PATH_DIRECT      # dilated depthwise: generic kernel
    mult = hgc.ConvDesc(2, 32, 14, 14, 64, 3, 3, 1, 1, 1, 1, 1, 1, 32)
    assert mult.path() == hgc.HGC_PATH_DIRECT     # channel multiplier 2: generic kernel


def test_plan_info_reports_tiling_and_activation_source():
    """The planner runs on the host: its choices can be checked without a GPU."""
    keys = {"path", "kb", "halo", "tn", "th", "pitch", "ncols", "tiles", "stages", "taps", "x_source", "k_slices",
            "grid", "shared_tiles", "pair", "fused_layout", "row_pairs", "replicas", "y_store"}
    cases = [
        # (n, c, h, w, k, r, s, pad, stride), x_source
        ((16, 256, 56, 56, 256, 3, 3, 1, 1), 0),   # NHWC copy of x
        ((64, 64, 56, 56, 256, 1, 1, 0, 1), 1),    # 1x1 on a plane of a multiple of 8 pixels: x itself
        ((64, 1024, 14, 14, 256, 1, 1, 0, 1), 0),  # 196 pixels: rows of x are not 16-byte aligned
        ((16, 3, 224, 224, 64, 3, 3, 1, 1), 2),    # stride-1 stem: overlapping windows
        ((32, 3, 224, 224, 32, 3, 3, 1, 2), 3),    # strided stem: expanded copy
    ]
    for (n, c, h, w, k, r, s, pad, stride), source in cases:
        d = hgc.ConvDesc(n, c, h, w, k, r, s, pad, pad, stride, stride, 1, 1, 1)
        assert d.path() == hgc.HGC_PATH_IGEMM
        info = d.plan_info()
        assert set(info) == keys
        assert info["x_source"] == source, info
        assert info["kb"] in (16, 32, 64) and 16 <= info["ncols"] <= 256 and info["ncols"] % 16 == 0
        assert info["tn"] >= 1 and info["th"] >= 1 and info["stages"] >= 2 and info["tiles"] >= 1
        assert info["k_slices"] == 1
        # an accumulator tile never holds more than 256 columns
        assert info["tn"] * info["th"] * info["pitch"] - (info["pitch"] - d.output_dims()[3]) <= 256
        d.close()
    fc = hgc.ConvDesc.inner_product(64, 4096, 4096)
    info = fc.plan_info()   # few tiles: several CTAs share the reduction of a tile, one way or the other
    assert (info["k_slices"] in (2, 4, 8) or info["shared_tiles"] == 1) and info["tn"] == 64, info
    fc.close()
    dw = hgc.ConvDesc(2, 32, 14, 14, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32)
    assert dw.plan_info()["kb"] == 0   # not the tensor-core path: zeros


def test_launch_counter_readable():
    assert hgc.kernel_launch_count() >= 0


def test_batchnorm_entry_points_validate_their_arguments():
    """No launch: every call below must be refused on the host."""
    import ctypes
    L = hgc.lib()
    ok_ptr = ctypes.c_void_p(0x10000)           # never dereferenced: the calls fail before any launch
    f = ctypes.c_void_p(0x20000)
    assert hgc.batchnorm_workspace_bytes(16, 64, 224 * 224) == 2 * 64 * 16 * 25 * 4   # 25 groups of <= 2048 per plane
    assert hgc.batchnorm_workspace_bytes(2, 3, 2048) == 2 * 3 * 2 * 1 * 4
    assert hgc.batchnorm_workspace_bytes(0, 3, 10) == 0
    bad = [
        (None, ok_ptr, 1, 1, 10, 0.0, 0, 0, f, f, ok_ptr, hgc.HGC_INVALID_ARG),      # x NULL
        (ok_ptr, ok_ptr, 0, 1, 10, 0.0, 0, 0, f, f, ok_ptr, hgc.HGC_INVALID_ARG),    # n < 1
        (ok_ptr, ok_ptr, 1, 1, 0, 0.0, 0, 0, f, f, ok_ptr, hgc.HGC_INVALID_ARG),     # hw < 1
        (ok_ptr, ok_ptr, 1, 1, 10, -1.0, 0, 0, f, f, ok_ptr, hgc.HGC_INVALID_ARG),   # eps < 0
        (ok_ptr, ok_ptr, 1, 1, 10, 0.0, 9, 0, f, f, ok_ptr, hgc.HGC_INVALID_ARG),    # shift out of range
        (ok_ptr, ok_ptr, 1, 1, 10, 0.0, 0, 0, None, f, ok_ptr, hgc.HGC_INVALID_ARG),  # mean NULL
        (ok_ptr, ok_ptr, 1, 70000, 10, 0.0, 0, 0, f, f, ok_ptr, hgc.HGC_UNSUPPORTED),  # too many channels
        (ctypes.c_void_p(0x10002), ok_ptr, 1, 1, 10, 0.0, 0, 0, f, f, ok_ptr, hgc.HGC_BAD_ALIGNMENT),
        (ok_ptr, ok_ptr, 1, 1, 10, 0.0, 0, 0, f, f, None, hgc.HGC_NO_WORKSPACE),     # statistics need scratch
    ]
    for *args, want in bad:
        assert L.hgc_batchnorm_forward(*args, None) == want, args
    assert L.hgc_bn_fold(None, None, f, f, None, None, 0.0, 4, 9, ok_ptr, ok_ptr, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_bn_fold(ok_ptr, None, f, f, None, None, 0.0, 0, 9, ok_ptr, ok_ptr, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_bn_fold(ok_ptr, None, f, f, None, None, -1.0, 4, 9, ok_ptr, ok_ptr, None) == hgc.HGC_INVALID_ARG


def test_static_entry_point_refuses_layouts_it_does_not_have():
    """hgc_conv_forward_static takes NCHW tensors on the tensor-core path only: a layout flag or the
    direct-path flag is refused before anything is queued (no GPU needed: the pointers are never
    dereferenced), where silently ignoring it would hand back a tensor in the wrong layout."""
    L = hgc.lib()
    ptr = ctypes.c_void_p(0x10000)
    for flags in (hgc.HGC_FLAG_X_NHWC, hgc.HGC_FLAG_Y_NHWC, hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC,
                  hgc.HGC_FLAG_FORCE_DIRECT):
        p = hgc.hgc_conv_params(1, 32, 8, 8, 32, 3, 3, 1, 1, 1, 1, 1, 1, 1, flags)
        assert L.hgc_conv_forward_static(ctypes.byref(p), ptr, ptr, None, ptr, 0, None) == hgc.HGC_UNSUPPORTED
    p = hgc.hgc_conv_params(1, 32, 8, 8, 32, 3, 3, 1, 1, 1, 1, 1, 1, 1, 0)
    assert L.hgc_conv_forward_static(ctypes.byref(p), None, ptr, None, ptr, 0, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_forward_static(ctypes.byref(p), ctypes.c_void_p(0x10002), ptr, None, ptr, 0, None) == hgc.HGC_BAD_ALIGNMENT
    bad = hgc.hgc_conv_params(1, 32, 8, 8, 32, 3, 3, 1, 1, 0, 1, 1, 1, 1, 0)     # stride 0
    assert L.hgc_conv_forward_static(ctypes.byref(bad), ptr, ptr, None, ptr, 0, None) == hgc.HGC_INVALID_ARG


def test_scheduling_flags_change_the_plan_not_the_layer():
    """HGC_FLAG_CTA_PAIRS is opt-in; shared tiles are the planner's choice (this layer: 3.03 waves of
    long tiles), forced by HGC_FLAG_SHARED_TILES and forbidden by HGC_FLAG_WHOLE_TILES; the plan
    reports them, and none changes the output shape or the path."""
    args = (16, 256, 56, 56, 256, 3, 3, 1, 1, 1, 1, 1, 1, 1)
    auto = hgc.ConvDesc(*args)
    assert auto.plan_info()["pair"] == 0 and auto.plan_info()["shared_tiles"] == 1
    base = hgc.ConvDesc(*args, flags=hgc.HGC_FLAG_WHOLE_TILES)
    assert base.plan_info()["pair"] == 0 and base.plan_info()["shared_tiles"] == 0
    assert hgc.ConvDesc(*args, flags=hgc.HGC_FLAG_WHOLE_TILES | hgc.HGC_FLAG_SHARED_TILES).plan_info()["shared_tiles"] == 0
    # layers whose tiles are short, or fewer than 2.5 per CTA, keep whole tiles unless asked
    small = (16, 512, 28, 28, 512, 3, 3, 1, 1, 1, 1, 1, 1, 1)
    assert hgc.ConvDesc(*small).plan_info()["shared_tiles"] == 0
    assert hgc.ConvDesc(*small, flags=hgc.HGC_FLAG_SHARED_TILES).plan_info()["shared_tiles"] == 1
    pairs = hgc.ConvDesc(*args, flags=hgc.HGC_FLAG_CTA_PAIRS)
    info = pairs.plan_info()
    assert info["pair"] == 1 and info["ncols"] % 16 == 0 and info["ncols"] <= 256 and info["grid"] <= 74
    shared = hgc.ConvDesc(*args, flags=hgc.HGC_FLAG_SHARED_TILES)
    assert shared.plan_info()["shared_tiles"] == 1 and shared.plan_info()["grid"] == 148
    assert shared.workspace_bytes() > base.workspace_bytes()          # hand-over slots
    for d in (pairs, shared):
        assert d.output_dims() == base.output_dims() and d.path() == base.path()
    # a layer with 128 output channels has nothing to pair
    assert hgc.ConvDesc(16, 128, 112, 112, 128, 3, 3, 1, 1, flags=hgc.HGC_FLAG_CTA_PAIRS).plan_info()["pair"] == 0


def test_gather_flag_replaces_the_layout_pass_on_small_planes():
    """1x1 layers on 14x14 planes (8-byte plane starts) take the NHWC copy of x unless
    HGC_FLAG_GATHER_X asks the kernel's own warps to fetch x: then no copy is planned."""
    args = (64, 1024, 14, 14, 256, 1, 1, 0, 0, 1, 1, 1, 1, 1)
    plain = hgc.ConvDesc(*args)
    gather = hgc.ConvDesc(*args, flags=hgc.HGC_FLAG_GATHER_X)
    assert plain.plan_info()["x_source"] == 0 and gather.plan_info()["x_source"] == 4
    assert gather.plan_info()["th"] == 14 and gather.plan_info()["tn"] == 1          # a tile is one plane
    assert gather.workspace_bytes() + 2 * 64 * 1024 * 14 * 14 <= plain.workspace_bytes()
    assert gather.output_dims() == plain.output_dims() and gather.path() == plain.path()
    # planes the copy engine can address, odd planes and ragged channel blocks are not gathered
    for other in ((2, 64, 16, 16, 64), (2, 64, 7, 7, 64), (2, 96, 14, 14, 64), (2, 64, 20, 20, 64)):
        d = hgc.ConvDesc(*other, 1, 1, flags=hgc.HGC_FLAG_GATHER_X)
        assert d.plan_info()["x_source"] != 4, other


def test_plan_reports_how_the_output_is_written():
    """[18] of the plan: staged tiles through a tensor map (rows of whole 16-byte vectors), whole
    planes of a 1x1 layer as bulk copies (14x14, 7x7: 32-channel blocks contiguous in y), else plain stores."""
    assert hgc.ConvDesc(16, 64, 56, 56, 64, 3, 3, 1, 1).plan_info()["y_store"] == 1
    assert hgc.ConvDesc(64, 256, 14, 14, 1024, 1, 1, 0, 0).plan_info()["y_store"] == 2
    assert hgc.ConvDesc(64, 256, 14, 14, 256, 3, 3, 1, 1).plan_info()["y_store"] == 0      # junk columns between rows
    assert hgc.ConvDesc(64, 512, 7, 7, 2048, 1, 1, 0, 0).plan_info()["y_store"] == 2       # four images per tile
    assert hgc.ConvDesc(64, 256, 14, 14, 1000, 1, 1, 0, 0).plan_info()["y_store"] == 0     # K % 32 != 0
    assert hgc.ConvDesc(2, 256, 14, 14, 1024, 1, 1, 0, 0).plan_info()["y_store"] == 0      # few images: tiles of a few rows
    assert hgc.ConvDesc(64, 256, 14, 14, 1024, 1, 1, 0, 0, flags=hgc.HGC_FLAG_Y_NHWC).plan_info()["y_store"] == 1


def test_64_channel_layers_fill_the_mma():
    """Layers of 64 output channels leave half of the 128-row MMA idle.  Wide stride-1 layers with
    several kernel rows run as row pairs (odd output rows in the upper lanes: tiles of two rows, one
    more kernel row); epilogue-bound ones with a short reduction hold their weight rows twice."""
    rp = hgc.ConvDesc(16, 64, 224, 224, 64, 3, 3, 1, 1).plan_info()
    assert rp["row_pairs"] == 1 and rp["th"] == 1 and rp["tiles"] == 16 * 112 and rp["replicas"] == 1
    # not: odd output height, narrow planes, strides, channels-last output, other channel counts
    for args, kw in [((16, 64, 223, 224, 64, 3, 3, 1, 1), {}), ((64, 64, 56, 56, 64, 3, 3, 1, 1), {}),
                     ((16, 64, 224, 224, 64, 3, 3, 1, 1, 2, 2), {}), ((16, 64, 224, 224, 128, 3, 3, 1, 1), {}),
                     ((16, 64, 224, 224, 64, 3, 3, 1, 1), {"flags": hgc.HGC_FLAG_Y_NHWC}),
                     ((16, 64, 224, 224, 64, 1, 1, 0, 0), {})]:
        assert hgc.ConvDesc(*args, **kw).plan_info()["row_pairs"] == 0, args
    assert hgc.ConvDesc(16, 3, 224, 224, 64, 3, 3, 1, 1).plan_info()["replicas"] == 2     # stem: 6 MMAs per tile
    assert hgc.ConvDesc(32, 32, 112, 112, 64, 1, 1, 0, 0).plan_info()["replicas"] == 2    # 1x1, 32 channels in
    assert hgc.ConvDesc(64, 256, 56, 56, 64, 1, 1, 0, 0).plan_info()["replicas"] == 1     # long reduction
    assert hgc.ConvDesc(16, 64, 112, 112, 128, 3, 3, 1, 1).plan_info()["replicas"] == 1


def test_block_descriptor_validation():
    """hgc_dwpw_desc_create: argument checks and planning run on the host."""
    L = hgc.lib()
    h = ctypes.c_void_p()
    ok = hgc.hgc_dwpw_params(32, 512, 14, 14, 512, 1, hgc.HGC_FLAG_Y_NHWC)
    assert L.hgc_dwpw_desc_create(ctypes.byref(h), ctypes.byref(ok)) == hgc.HGC_OK
    n, k, p, q = (ctypes.c_int32() for _ in range(4))
    assert L.hgc_conv_output_dims(h, ctypes.byref(n), ctypes.byref(k), ctypes.byref(p), ctypes.byref(q)) == hgc.HGC_OK
    assert (n.value, k.value, p.value, q.value) == (32, 512, 14, 14)
    ptr = ctypes.c_void_p(0x10000)
    # a block descriptor is not a layer descriptor, and needs its workspace
    assert L.hgc_conv_forward(h, ptr, ptr, None, ptr, 0, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_set_weights(h, ptr, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_dwpw_forward(h, ptr, ptr, None, ptr, None, ptr, 1, 1, None) == hgc.HGC_NO_WORKSPACE
    assert L.hgc_dwpw_forward(h, None, ptr, None, ptr, None, ptr, 1, 1, None) == hgc.HGC_INVALID_ARG
    assert L.hgc_conv_desc_destroy(h) == hgc.HGC_OK
    s2 = hgc.hgc_dwpw_params(2, 64, 15, 17, 128, 2, 0)           # stride 2 on an odd plane: 8 x 9 outputs
    assert L.hgc_dwpw_desc_create(ctypes.byref(h), ctypes.byref(s2)) == hgc.HGC_OK
    assert L.hgc_conv_output_dims(h, ctypes.byref(n), ctypes.byref(k), ctypes.byref(p), ctypes.byref(q)) == hgc.HGC_OK
    assert (p.value, q.value) == (8, 9)
    assert L.hgc_conv_desc_destroy(h) == hgc.HGC_OK
    for bad, want in [(hgc.hgc_dwpw_params(1, 32, 8, 8, 32, 3, 0), hgc.HGC_INVALID_ARG),      # stride 3
                      (hgc.hgc_dwpw_params(1, 32, 8, 8, 32, 1, hgc.HGC_FLAG_X_NHWC), hgc.HGC_INVALID_ARG),  # other flags
                      (hgc.hgc_dwpw_params(0, 32, 8, 8, 32, 1, 0), hgc.HGC_INVALID_ARG),
                      (hgc.hgc_dwpw_params(1, 12, 8, 8, 32, 1, 0), hgc.HGC_UNSUPPORTED)]:     # 12 channels
        assert L.hgc_dwpw_desc_create(ctypes.byref(h), ctypes.byref(bad)) == want
    layer = hgc.ConvDesc(1, 32, 8, 8, 32, 3, 3, 1, 1)
    assert L.hgc_dwpw_forward(layer.handle, ptr, ptr, None, ptr, None, ptr, 1, 1, None) == hgc.HGC_INVALID_ARG
