"""GPU parity of the tensor-core path, one case per way it can feed and drain the MMA: where the
activation tiles come from (NHWC copy, x itself for 1x1 layers, overlapping windows or an
expanded copy for few-channel stems), which epilogue writes y (TMA store, copy), tile shapes with
several images, ragged last tiles and partially filled channel tiles.  Every case is compared
with the CPU oracle element by element; outputs are NaN-filled before the call."""
import zlib

import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import check_close, params_dict, run_layer

pytestmark = pytest.mark.gpu

X_NHWC_COPY, X_DIRECT, X_WINDOWS, X_PATCHES = 0, 1, 2, 3


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


CASES = [
    # (id, params, expected activation source or None)
    ("1x1 direct 56x56 k256", params_dict(2, 64, 56, 56, 256, 1, 1), X_DIRECT),
    ("1x1 direct 28x28 k200 (tile rows in whole 8-pixel steps)", params_dict(3, 128, 28, 28, 200, 1, 1), X_DIRECT),
    ("1x1 direct 8x8 single tile", params_dict(1, 64, 8, 8, 128, 1, 1), X_DIRECT),
    ("1x1 direct c40 (channel tail in the block)", params_dict(2, 40, 16, 24, 48, 1, 1), X_DIRECT),
    ("1x1 14x14 (copy epilogue, 4-byte words)", params_dict(5, 256, 14, 14, 136, 1, 1), X_NHWC_COPY),
    ("1x1 7x7 several images per tile", params_dict(9, 512, 7, 7, 130, 1, 1), X_NHWC_COPY),
    ("1x1 stride 2", params_dict(2, 64, 28, 28, 96, 1, 1, 0, 0, 2, 2), X_NHWC_COPY),
    ("1x1 grouped", params_dict(2, 64, 12, 12, 64, 1, 1, 0, 0, 1, 1, 1, 1, 4), X_NHWC_COPY),
    ("3x3 224 wide rows k64", params_dict(1, 64, 20, 224, 64, 3, 3, 1, 1), X_NHWC_COPY),
    ("3x3 c256 32-channel stages", params_dict(2, 256, 24, 24, 160, 3, 3, 1, 1), X_NHWC_COPY),
    ("3x3 13x13 odd plane (copy epilogue with junk columns)", params_dict(3, 96, 13, 13, 72, 3, 3, 1, 1), X_NHWC_COPY),
    ("3x3 7x7 several images per tile", params_dict(7, 64, 7, 7, 40, 3, 3, 1, 1), X_NHWC_COPY),
    ("3x3 stride 2", params_dict(2, 96, 15, 15, 200, 3, 3, 1, 1, 2, 2), X_NHWC_COPY),
    ("5x5 grouped pad 2", params_dict(1, 96, 27, 27, 256, 5, 5, 2, 2, 1, 1, 1, 1, 2), X_NHWC_COPY),
    ("3x3 dilation 2", params_dict(2, 24, 20, 18, 30, 3, 3, 2, 2, 1, 1, 2, 2), X_NHWC_COPY),
    ("3x1 and unpadded rows", params_dict(2, 40, 10, 40, 16, 3, 1, 1, 0), X_NHWC_COPY),
    ("1x1 5x5 c4096 k96: reduction split over several CTAs, ragged channel tile", params_dict(3, 4096, 5, 5, 96, 1, 1), X_NHWC_COPY),
    ("1x1 7x7 c2048 k200: reduction split, one-row tiles", params_dict(2, 2048, 7, 7, 200, 1, 1), X_NHWC_COPY),
    ("1x1 3x5 c4096 k64: reduction split, several images per tile", params_dict(4, 4096, 3, 5, 64, 1, 1), X_NHWC_COPY),
    ("stem 3x3 c3 stride 1 (windows)", params_dict(2, 3, 32, 40, 16, 3, 3, 1, 1), X_WINDOWS),
    ("stem 7x7 c3 stride 2 (windows)", params_dict(2, 3, 64, 64, 64, 7, 7, 3, 3, 2, 2), X_WINDOWS),
    ("stem 11x11 c3 stride 4 (windows)", params_dict(1, 3, 67, 67, 96, 11, 11, 0, 0, 4, 4), X_WINDOWS),
    ("stem 7x7 c3 stride 2, 224 wide (dense rows of 4-channel pixels, two rows per tile)",
     params_dict(2, 3, 20, 224, 64, 7, 7, 3, 3, 2, 2), X_WINDOWS),
    ("stem 5x5 c4 stride 2 (dense rows of 4-channel pixels)", params_dict(2, 4, 37, 45, 40, 5, 5, 2, 2, 2, 2), X_WINDOWS),
    ("stem 7x7 c3 stride 1 along H, 2 along W", params_dict(2, 3, 30, 50, 24, 7, 7, 3, 3, 1, 2), X_WINDOWS),
    ("stem 7x7 c1 stride 1 along H, 2 along W (49 values under the kernel: patches)",
     params_dict(2, 1, 30, 50, 24, 7, 7, 3, 3, 1, 2), X_PATCHES),
    ("stem 9x9 c3 stride 2 (64-element windows)", params_dict(1, 3, 41, 41, 32, 9, 9, 4, 4, 2, 2), X_WINDOWS),
    ("stem 5x5 c5 stride 2 (8-channel pixels: one request per window)", params_dict(2, 5, 33, 33, 16, 5, 5, 2, 2, 2, 2), X_WINDOWS),
    ("stem 5x5 c3 stride 1 (dense rows, shared kernel rows)", params_dict(2, 3, 30, 70, 48, 5, 5, 2, 2), X_WINDOWS),
    ("stem 3x3 c8 stride 1, 250 wide (dense rows at the column limit)", params_dict(1, 8, 9, 250, 16, 3, 3, 1, 1), X_WINDOWS),
    ("stem 3x3 c3 stride 1, 256 wide (rows too wide for the dense form)", params_dict(1, 3, 6, 256, 16, 3, 3, 1, 1), X_WINDOWS),
    ("stem 3x3 c3 stride 2 (patches)", params_dict(2, 3, 64, 48, 32, 3, 3, 1, 1, 2, 2), X_PATCHES),
    ("stem 3x3 c1 stride 2 (patches)", params_dict(3, 1, 33, 31, 24, 3, 3, 1, 1, 2, 2), X_PATCHES),
    ("stem 3x3 c4 stride 2, 44 wide (patches from aligned words)", params_dict(2, 4, 30, 44, 16, 3, 3, 1, 1, 2, 2), X_PATCHES),
    ("stem 3x3 c1 stride 2 x 1, 70 wide, pad 2 x 1 (patches from aligned words)", params_dict(3, 1, 21, 70, 24, 3, 3, 2, 1, 1, 2), X_PATCHES),
    ("stem 3x3 c4 stride 2 dilated (patches)", params_dict(2, 4, 30, 30, 20, 3, 3, 2, 2, 2, 2, 2, 2), X_PATCHES),
    ("stem 5x5 c2 stride 3 (patches, generic expansion)", params_dict(2, 2, 29, 35, 20, 5, 5, 2, 2, 3, 3), X_PATCHES),
    ("stem 1x1 c8 stride 2 (patches)", params_dict(2, 8, 18, 18, 16, 1, 1, 0, 0, 2, 2), X_PATCHES),
    # 64 output channels: odd output rows in the upper accumulator lanes (row pairs) ...
    ("row pairs 3x3 c16 112 wide", params_dict(2, 16, 10, 112, 64, 3, 3, 1, 1), X_NHWC_COPY),
    ("row pairs 3x3 c64 224 wide, two images", params_dict(2, 64, 6, 224, 64, 3, 3, 1, 1), X_NHWC_COPY),
    ("row pairs 2x3 c32 120 wide, pad 1", params_dict(3, 32, 9, 120, 64, 2, 3, 1, 1), X_NHWC_COPY),
    ("row pairs 5x1 c24 unpadded columns, pad 2 rows", params_dict(1, 24, 8, 136, 64, 5, 1, 2, 0), X_NHWC_COPY),
    ("row pairs 3x3 c40 without padding (channel tail)", params_dict(2, 40, 12, 130, 64, 3, 3, 0, 0), X_NHWC_COPY),
    ("row pairs 4x3 c64 248 wide (250 columns)", params_dict(1, 64, 7, 248, 64, 4, 3, 1, 1), X_NHWC_COPY),
    # ... or, for epilogue-bound layers, the weight rows twice (replicas that take other pixels)
    ("replicas 1x1 c32 112x112 k64", params_dict(2, 32, 112, 112, 64, 1, 1), X_DIRECT),
    ("replicas 1x1 c64 56x56 k64", params_dict(8, 64, 56, 56, 64, 1, 1), X_DIRECT),
    ("replicas stem 3x3 c3 224 wide k64 (32-pixel units)", params_dict(2, 3, 12, 224, 64, 3, 3, 1, 1), X_WINDOWS),
    ("replicas 1x1 c32 27x72 k64 (64-pixel units, ragged tiles)", params_dict(8, 32, 27, 72, 64, 1, 1), X_DIRECT),
    ("replicas stem 3x3 c3 200 wide k64 (64-pixel units, ragged)", params_dict(2, 3, 20, 200, 64, 3, 3, 1, 1), X_WINDOWS),
]


@pytest.mark.parametrize("name,a,source", CASES, ids=[c[0] for c in CASES])
def test_igemm_mode(hgc, oracle, name, a, source):
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    P = oracle.ConvParams(**a)
    d = hgc.ConvDesc(**a)
    assert d.path() == hgc.HGC_PATH_IGEMM, name
    if source is not None:
        assert d.plan_info()["x_source"] == source, (name, d.plan_info())
    if name.startswith("row pairs"):
        assert d.plan_info()["row_pairs"] == 1, d.plan_info()
    if name.startswith("replicas"):
        assert d.plan_info()["replicas"] == 2, d.plan_info()
    if "reduction split" in name:
        # several CTAs per tile: reduction slices with a second pass, or CTAs that hand their
        # accumulators over inside the one launch
        assert d.plan_info()["k_slices"] > 1 or d.plan_info()["shared_tiles"] == 1, d.plan_info()
    d.close()
    for relu, bias, registered in ((True, b, True), (False, None, False)):
        ref = oracle.conv_fast(P, x, w, bias, relu)
        got, path = run_layer(hgc, a, x, w, bias, relu, register_weights=registered)
        assert path == hgc.HGC_PATH_IGEMM
        check_close(got, ref, what=f"{name} relu={relu}")


SCHED_CASES = [
    # (id, params, flags by name, what the plan must report)
    ("pairs 3x3 c128 k256 24x24 (TMA-store epilogue)", params_dict(3, 128, 24, 24, 256, 3, 3, 1, 1), ("pairs",), {"pair": 1}),
    ("pairs 3x3 c96 k384 13x13 (copy epilogue, second CTA of the last channel pair idle)",
     params_dict(3, 96, 13, 13, 384, 3, 3, 1, 1), ("pairs",), {"pair": 1}),
    ("pairs 3x3 c64 k520 7x7 (several images per sub-tile, odd number of sub-tiles, ragged channels)",
     params_dict(7, 64, 7, 7, 520, 3, 3, 1, 1), ("pairs",), {"pair": 1}),
    ("pairs 3x3 stride 2 c96 k256 (one tap per stage)", params_dict(2, 96, 15, 15, 256, 3, 3, 1, 1, 2, 2), ("pairs",), {"pair": 1}),
    ("pairs 1x1 14x14 c256 k1024", params_dict(4, 256, 14, 14, 1024, 1, 1), ("pairs",), {"pair": 1}),
    ("pairs grouped 3x3 g2 c128 k512", params_dict(2, 128, 12, 12, 512, 3, 3, 1, 1, 1, 1, 1, 1, 2), ("pairs",), {"pair": 1}),
    ("pairs k128: not eligible, single CTAs", params_dict(2, 64, 16, 16, 128, 3, 3, 1, 1), ("pairs",), {"pair": 0}),
    ("shared 3x3 c256 k256 56x56 n2 (tiles over 148 CTAs: ranges end inside tiles)",
     params_dict(2, 256, 56, 56, 256, 3, 3, 1, 1), ("shared",), {"shared_tiles": 1}),
    ("shared 3x3 c512 k512 14x14 n3 (a tile over several CTAs)", params_dict(3, 512, 14, 14, 512, 3, 3, 1, 1), ("shared",),
     {"shared_tiles": 1}),
    ("shared 1x1 5x5 c4096 k96 (inner-product shape, many CTAs per tile)", params_dict(3, 4096, 5, 5, 96, 1, 1), ("shared",),
     {"shared_tiles": 1}),
    ("shared 1x1 direct 28x28 c512 k384", params_dict(3, 512, 28, 28, 384, 1, 1), ("shared",), {"shared_tiles": 1}),
    ("pairs + shared 3x3 c256 k256 28x28 n5", params_dict(5, 256, 28, 28, 256, 3, 3, 1, 1), ("pairs", "shared"),
     {"pair": 1, "shared_tiles": 1}),
    ("pairs + shared 3x3 c512 k512 14x14 n3", params_dict(3, 512, 14, 14, 512, 3, 3, 1, 1), ("pairs", "shared"),
     {"pair": 1, "shared_tiles": 1}),
    ("fused layout 3x3 c64 k64 56x56 n5 (64-channel units)", params_dict(5, 64, 56, 56, 64, 3, 3, 1, 1), ("fused",),
     {"fused_layout": 1}),
    ("fused layout 3x3 c40 k72 24x40 n3 (32-channel units, ragged channel and pixel units)",
     params_dict(3, 40, 24, 40, 72, 3, 3, 1, 1), ("fused",), {"fused_layout": 1}),
    ("fused layout 3x3 stride 2 c128 k96 34x32 n2", params_dict(2, 128, 34, 32, 96, 3, 3, 1, 1, 2, 2), ("fused",),
     {"fused_layout": 1}),
    ("fused layout 5x5 grouped c96 k64 24x24 n2", params_dict(2, 96, 24, 24, 64, 5, 5, 2, 2, 1, 1, 1, 1, 2), ("fused",),
     {"fused_layout": 1}),
    ("fused layout: 13x13 plane keeps the separate pass", params_dict(2, 96, 13, 13, 72, 3, 3, 1, 1), ("fused",),
     {"fused_layout": 0}),
    # 1x1 layers on planes that start on 8-byte boundaries: x gathered by the kernel's own warps
    ("gather 1x1 14x14 c256 k256 n3 (several stages in flight, two channel tiles)", params_dict(3, 256, 14, 14, 256, 1, 1),
     ("gather",), {"x_source": 4}),
    ("gather 1x1 14x14 c1024 k72 n2 (ring laps, ragged channel tile)", params_dict(2, 1024, 14, 14, 72, 1, 1), ("gather",),
     {"x_source": 4}),
    ("gather 1x1 10x10 c192 k130 n5", params_dict(5, 192, 10, 10, 130, 1, 1), ("gather",), {"x_source": 4}),
    ("gather 1x1 2x2 c64 k16 n2 (one piece per channel)", params_dict(2, 64, 2, 2, 16, 1, 1), ("gather",), {"x_source": 4}),
    ("gather 1x1 12x21 c64 k64 n2 (252 pixels: all 256 accumulator columns)", params_dict(2, 64, 12, 21, 64, 1, 1), ("gather",),
     {"x_source": 4}),
    ("gather: 16-byte planes go through the copy engine", params_dict(2, 64, 16, 15, 64, 1, 1), ("gather",), {"x_source": 1}),
    ("gather: 7x7 planes keep the layout pass", params_dict(2, 64, 7, 7, 64, 1, 1), ("gather",), {"x_source": 0}),
    ("gather: c96 keeps the layout pass", params_dict(2, 96, 14, 14, 64, 1, 1), ("gather",), {"x_source": 0}),
]


@pytest.mark.parametrize("name,a,flag_names,want", SCHED_CASES, ids=[c[0] for c in SCHED_CASES])
def test_scheduling_flags(hgc, oracle, name, a, flag_names, want):
    """CTA pairs (cta_group::2), tiles shared by several CTAs, the layout pass inside the
    tensor-core kernel and x gathered by the kernel's own warps are opt-in schedules of the same layer: the plan must report them where
    asked for, and the results must match the oracle."""
    flags = ((hgc.HGC_FLAG_CTA_PAIRS if "pairs" in flag_names else 0) | (hgc.HGC_FLAG_SHARED_TILES if "shared" in flag_names else 0)
             | (hgc.HGC_FLAG_FUSED_LAYOUT if "fused" in flag_names else 0) | (hgc.HGC_FLAG_GATHER_X if "gather" in flag_names else 0))
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    P = oracle.ConvParams(**a)
    d = hgc.ConvDesc(flags=flags, **a)
    assert d.path() == hgc.HGC_PATH_IGEMM, name
    info = d.plan_info()
    d.close()
    for key, value in want.items():
        assert info[key] == value, (name, info)
    for relu, bias in ((True, b), (False, None)):
        ref = oracle.conv_fast(P, x, w, bias, relu)
        first = None
        for rep in range(2):   # twice: the second launch finds the first one's hand-over flags lowered again
            got, _ = run_layer(hgc, a, x, w, bias, relu, flags=flags, register_weights=True)
            check_close(got, ref, what=f"{name} relu={relu} rep={rep}")
            if first is None:
                first = got
            else:
                assert np.array_equal(first.view(np.uint16), got.view(np.uint16)), "the schedule must be deterministic"


PLANE_CASES = [
    # (name, layer, flags, plan keys): tiles of whole output planes of 1x1 layers leave as one bulk copy per 32-channel block
    ("14x14 c64 k256 n40", params_dict(40, 64, 14, 14, 256, 1, 1), 0, {"y_store": 2, "th": 14, "tn": 1}),
    ("10x10 c128 k160 n48 (ragged last group of columns)", params_dict(48, 128, 10, 10, 160, 1, 1), 0, {"y_store": 2, "tn": 1}),
    ("2x2 c64 k32 n70 (several images per tile, last tile short)", params_dict(70, 64, 2, 2, 32, 1, 1), 0, {"y_store": 2}),
    ("6x6 c64 k64 n120 stride 2 from 12x12", params_dict(120, 64, 12, 12, 64, 1, 1, 0, 0, 2, 2), 0, {"y_store": 2, "th": 6}),
    ("6x6 c64 k96 n200 (two images per tile)", params_dict(200, 64, 6, 6, 96, 1, 1), 0, {"y_store": 2, "tn": 2}),
    ("14x14 c256 k256 n20, x gathered by the kernel's warps", params_dict(20, 256, 14, 14, 256, 1, 1), "gather", {"y_store": 2, "x_source": 4}),
    ("3x3 stride 2, 12x12 -> 6x6, c64 k64 n40 (taps do not share a tile: columns are pixels)",
     params_dict(40, 64, 12, 12, 64, 3, 3, 1, 1, 2, 2), 0, {"y_store": 2, "halo": 0}),
    ("3x3 stride 2, 14x14 -> 7x7, c64 k64 n150 (two images per tile)", params_dict(150, 64, 14, 14, 64, 3, 3, 1, 1, 2, 2), 0,
     {"y_store": 2, "tn": 2}),
    ("k72: channel blocks are not whole, copy epilogue", params_dict(40, 64, 14, 14, 72, 1, 1), 0, {"y_store": 0}),
    ("7x7 c512 k256 n64 (98-byte planes: 2-byte staging stores, one image per tile)", params_dict(64, 512, 7, 7, 256, 1, 1), 0,
     {"y_store": 2, "tn": 1}),
    ("7x7 c64 k2048 n33 (four images per tile, the last tile short)", params_dict(33, 64, 7, 7, 2048, 1, 1), 0, {"y_store": 2, "tn": 4}),
    ("3x3 planes c64 k32 n130", params_dict(130, 64, 3, 3, 32, 1, 1), 0, {"y_store": 2}),
    ("1x2 planes c64 k64 n300 (eight images per tile)", params_dict(300, 64, 1, 2, 64, 1, 1), 0, {"y_store": 2, "tn": 8}),
    ("7x7 c64 k64 n64: tiles of four rows, copy epilogue", params_dict(64, 64, 7, 7, 64, 1, 1), 0, {"y_store": 0}),
    ("3x3 on 14x14: junk columns between rows, copy epilogue", params_dict(64, 64, 14, 14, 64, 3, 3, 1, 1), 0, {"y_store": 0}),
]


@pytest.mark.parametrize("name,a,flags,want", PLANE_CASES, ids=[c[0] for c in PLANE_CASES])
def test_whole_plane_epilogue(hgc, oracle, name, a, flags, want):
    """Whole-tensor comparison of the layers whose tiles are written as bulk copies, and of their
    neighbours that must keep the copy epilogue; the output buffer is NaN-filled with guard bands."""
    fl = hgc.HGC_FLAG_GATHER_X if flags == "gather" else flags
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    d = hgc.ConvDesc(flags=fl, **a)
    info = d.plan_info()
    d.close()
    for key, value in want.items():
        assert info[key] == value, (name, info)
    for relu, bias in ((True, b), (False, None)):
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, bias, relu)
        got, _ = run_layer(hgc, a, x, w, bias, relu, flags=fl)
        check_close(got, ref, what=f"{name} relu={relu}")


def test_scheduling_flags_channels_last(hgc, oracle):
    """The same schedules with channels-last activations on both sides."""
    from gpu_util import to_dev, to_host
    import torch
    a = params_dict(3, 128, 20, 20, 256, 3, 3, 1, 1)
    rng = np.random.default_rng(99)
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], 3, 3, 1)
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
    for extra in (hgc.HGC_FLAG_CTA_PAIRS, hgc.HGC_FLAG_SHARED_TILES, hgc.HGC_FLAG_CTA_PAIRS | hgc.HGC_FLAG_SHARED_TILES):
        d = hgc.ConvDesc(flags=hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC | extra, **a)
        d.ensure_workspace()
        xd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1)))
        wd, bd = to_dev(w), to_dev(b)
        y = torch.full((3, 20, 20, 256), float("nan"), dtype=torch.float16, device="cuda")
        d.set_weights(wd)
        hgc.conv_forward(d, xd, wd, bd, y, True)
        torch.cuda.synchronize()
        assert d.last_device_status() == hgc.HGC_OK
        check_close(to_host(y).transpose(0, 3, 1, 2), ref, what=f"channels-last flags {extra}")
        d.close()


def test_same_descriptor_new_tensors(hgc, oracle):
    """A descriptor keeps tensor maps over x and y between calls: new pointers must re-encode them."""
    import torch
    from gpu_util import to_dev, to_host
    a = params_dict(2, 64, 16, 16, 128, 1, 1)
    rng = np.random.default_rng(5)
    d = hgc.ConvDesc(**a)
    d.ensure_workspace()
    P = oracle.ConvParams(**a)
    for rep in range(3):
        x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], 1, 1, 1)
        xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
        y = torch.full((2, 128, 16, 16), float("nan"), dtype=torch.float16, device="cuda")
        hgc.conv_forward(d, xd, wd, bd, y, True)
        torch.cuda.synchronize()
        check_close(to_host(y), oracle.conv_fast(P, x, w, b, True), what=f"rep {rep}")
    d.close()


def test_launch_overlap_gives_the_same_results(hgc, oracle):
    """With programmatic dependent launch on, a chain of dependent kernels (layout pass ->
    tensor-core kernel, twice on the same descriptor and workspace, then a depthwise layer) must
    still see every predecessor's writes."""
    import torch
    from gpu_util import to_dev, to_host
    a = params_dict(2, 96, 20, 20, 72, 3, 3, 1, 1)
    rng = np.random.default_rng(77)
    P = oracle.ConvParams(**a)
    d = hgc.ConvDesc(**a)
    d.ensure_workspace()
    dw_a = params_dict(2, 72, 20, 20, 72, 3, 3, 1, 1, 1, 1, 1, 1, 72)
    dw = hgc.ConvDesc(**dw_a)
    hgc.set_launch_overlap(True)
    try:
        for rep in range(3):
            x, w, b = workloads.random_layer_tensors(rng, 2, 96, 20, 20, 72, 3, 3, 1)
            _, w2, b2 = workloads.random_layer_tensors(rng, 2, 72, 20, 20, 72, 3, 3, 72)
            xd, wd, bd, w2d, b2d = to_dev(x), to_dev(w), to_dev(b), to_dev(w2), to_dev(b2)
            y = torch.full((2, 72, 20, 20), float("nan"), dtype=torch.float16, device="cuda")
            z = torch.full((2, 72, 20, 20), float("nan"), dtype=torch.float16, device="cuda")
            hgc.conv_forward(d, xd, wd, bd, y, True)
            hgc.conv_forward(dw, y, w2d, b2d, z, False)     # reads what the kernel before wrote
            torch.cuda.synchronize()
            ref_y = oracle.conv_fast(P, x, w, b, True)
            check_close(to_host(y), ref_y, what=f"overlap rep {rep} conv")
            ref_z = oracle.conv_fast(oracle.ConvParams(**dw_a), to_host(y), w2, b2, False)
            check_close(to_host(z), ref_z, what=f"overlap rep {rep} depthwise")
    finally:
        hgc.set_launch_overlap(False)
    d.close()
    dw.close()


NHWC_CASES = [
    # (id, params, x channels-last, y channels-last)
    ("3x3 c64 k128 both channels-last", params_dict(2, 64, 20, 24, 128, 3, 3, 1, 1), True, True),
    ("3x3 c256 k72 odd plane both", params_dict(3, 256, 13, 13, 72, 3, 3, 1, 1), True, True),
    ("1x1 c128 k200 28x28 both", params_dict(2, 128, 28, 28, 200, 1, 1), True, True),
    ("1x1 c512 7x7 several images per tile both", params_dict(9, 512, 7, 7, 130, 1, 1), True, True),
    ("3x3 stride 2 c96 both", params_dict(2, 96, 15, 15, 200, 3, 3, 1, 1, 2, 2), True, True),
    ("grouped 5x5 both", params_dict(1, 96, 27, 27, 256, 5, 5, 2, 2, 1, 1, 1, 1, 2), True, True),
    ("stem c3: NCHW in, channels-last out", params_dict(2, 3, 32, 40, 16, 3, 3, 1, 1), False, True),
    ("last layer: channels-last in, NCHW out", params_dict(2, 64, 16, 16, 40, 3, 3, 1, 1), True, False),
    ("wide rows 224 channels-last out", params_dict(1, 64, 6, 224, 64, 3, 3, 1, 1), True, True),
    ("rows of 100: a full and a ragged store per row", params_dict(2, 32, 5, 100, 48, 3, 3, 1, 1), True, True),
    ("k = 100: channel runs not 16-byte aligned, plain stores", params_dict(2, 64, 14, 14, 100, 3, 3, 1, 1), True, True),
    ("4 groups of 24 output channels", params_dict(2, 64, 12, 12, 96, 3, 3, 1, 1, 1, 1, 1, 1, 4), True, True),
    ("1x1 c64 k256 56x56: wide epilogue", params_dict(2, 64, 56, 56, 256, 1, 1), True, True),
    ("7x7 planes: nine rows per store, several images per tile", params_dict(9, 512, 7, 7, 128, 1, 1), True, True),
    ("14x14 planes k256: four rows per store", params_dict(3, 256, 14, 14, 256, 3, 3, 1, 1), True, True),
    ("28x28 planes k64: two rows per store, ragged last tile", params_dict(2, 128, 28, 28, 64, 3, 3, 1, 1), True, True),
    ("15x15 odd rows k96: junk pixel slots between rows", params_dict(2, 64, 15, 15, 96, 3, 3, 1, 1), True, True),
    ("stem c3 k64 windows, channels-last out", params_dict(2, 3, 24, 40, 64, 3, 3, 1, 1), False, True),
    ("stem 7x7 stride 2 c3 k64 patches, channels-last out", params_dict(2, 3, 38, 38, 64, 7, 7, 3, 3, 2, 2), False, True),
    ("grouped: 2 groups of 64 output channels", params_dict(2, 64, 12, 20, 128, 3, 3, 1, 1, 1, 1, 1, 1, 2), True, True),
    ("7x7 c2048 k128: channels-last in, few tiles (split reduction), NCHW out", params_dict(2, 2048, 7, 7, 128, 3, 3, 1, 1), True, False),
    ("7x7 c2048 k128: both channels-last (no split)", params_dict(2, 2048, 7, 7, 128, 3, 3, 1, 1), True, True),
    ("dilated 3x3 c64 k64 channels-last", params_dict(2, 64, 20, 20, 64, 3, 3, 2, 2, 1, 1, 2, 2), True, True),
]


@pytest.mark.parametrize("name,a,xl,yl", NHWC_CASES, ids=[c[0] for c in NHWC_CASES])
def test_channels_last_flags(hgc, oracle, name, a, xl, yl):
    import torch
    from gpu_util import to_dev, to_host
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)          # NCHW
    flags = (hgc.HGC_FLAG_X_NHWC if xl else 0) | (hgc.HGC_FLAG_Y_NHWC if yl else 0)
    d = hgc.ConvDesc(flags=flags, **a)
    assert d.path() == hgc.HGC_PATH_IGEMM
    n, k, p, q = d.output_dims()
    d.ensure_workspace()
    xin = np.ascontiguousarray(x.transpose(0, 2, 3, 1)) if xl else x
    xd, wd, bd = to_dev(xin), to_dev(w), to_dev(b)
    yshape = (n, p, q, k) if yl else (n, k, p, q)
    y = torch.full(yshape, float("nan"), dtype=torch.float16, device="cuda")
    hgc.conv_forward(d, xd, wd, bd, y, True)
    torch.cuda.synchronize()
    assert d.last_device_status() == hgc.HGC_OK
    got = to_host(y)
    if yl:
        got = np.ascontiguousarray(got.transpose(0, 3, 1, 2))
    check_close(got, ref, what=name)
    d.close()


DW_NHWC_CASES = [
    ("112x112 c32", params_dict(2, 32, 112, 112, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32)),
    ("56x56 c128 stride 2", params_dict(2, 128, 56, 56, 128, 3, 3, 1, 1, 2, 2, 1, 1, 128)),
    ("14x14 c512", params_dict(3, 512, 14, 14, 512, 3, 3, 1, 1, 1, 1, 1, 1, 512)),
    ("7x7 c1024", params_dict(2, 1024, 7, 7, 1024, 3, 3, 1, 1, 1, 1, 1, 1, 1024)),
    ("odd plane 13x9 c24, ragged strips", params_dict(2, 24, 13, 9, 24, 3, 3, 1, 1, 1, 1, 1, 1, 24)),
    ("15x15 stride 2 c40", params_dict(1, 40, 15, 15, 40, 3, 3, 1, 1, 2, 2, 1, 1, 40)),
    ("no padding 10x12 c16", params_dict(2, 16, 10, 12, 16, 3, 3, 0, 0, 1, 1, 1, 1, 16)),
    ("c64 odd plane 37x21 (TMA-fed, ragged tiles)", params_dict(2, 64, 37, 21, 64, 3, 3, 1, 1, 1, 1, 1, 1, 64)),
    ("c96 no padding 20x50 (TMA-fed, three 32-channel blocks)", params_dict(3, 96, 20, 50, 96, 3, 3, 0, 0, 1, 1, 1, 1, 96)),
    ("c128 padding 2, 33x40 (TMA-fed)", params_dict(1, 128, 33, 40, 128, 3, 3, 2, 2, 1, 1, 1, 1, 128)),
    ("c32 56x56 many tiles per block (TMA-fed)", params_dict(8, 32, 56, 56, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32)),
    ("padding 2, stride 2, 9x11 c8", params_dict(2, 8, 9, 11, 8, 3, 3, 2, 2, 2, 2, 1, 1, 8)),
]


@pytest.mark.parametrize("name,a", DW_NHWC_CASES, ids=[c[0] for c in DW_NHWC_CASES])
def test_depthwise_channels_last(hgc, oracle, name, a):
    import torch
    from gpu_util import to_dev, to_host
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], 3, 3, a["group"])
    d = hgc.ConvDesc(flags=hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC, **a)
    assert d.path() == hgc.HGC_PATH_DEPTHWISE
    n, k, p, q = d.output_dims()
    xd, wd, bd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1))), to_dev(w), to_dev(b)
    for relu, bias, bias_d in ((True, b, bd), (False, None, None)):
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, bias, relu)
        y = torch.full((n, p, q, k), float("nan"), dtype=torch.float16, device="cuda")
        hgc.conv_forward(d, xd, wd, bias_d, y, relu)
        torch.cuda.synchronize()
        check_close(np.ascontiguousarray(to_host(y).transpose(0, 3, 1, 2)), ref, what=f"{name} relu={relu}")
    assert d.last_device_status() == hgc.HGC_OK
    d.close()


def test_channels_last_flags_are_refused_where_they_cannot_apply(hgc):
    with pytest.raises(hgc.HgcError):     # a depthwise layer takes the flags only together
        hgc.ConvDesc(2, 32, 14, 14, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32, flags=hgc.HGC_FLAG_Y_NHWC)
    with pytest.raises(hgc.HgcError):     # and only with whole 16-byte vectors of channels
        hgc.ConvDesc(2, 12, 14, 14, 12, 3, 3, 1, 1, 1, 1, 1, 1, 12,
                     flags=hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC)
    with pytest.raises(hgc.HgcError):     # 3 input channels are not a whole number of 16-byte vectors
        hgc.ConvDesc(2, 3, 14, 14, 32, 3, 3, 1, 1, flags=hgc.HGC_FLAG_X_NHWC)


def test_channels_last_chain_with_registered_weights(hgc, oracle):
    """Four layers that hand their activations on channels-last: NCHW enters the first layer and
    leaves the last, nothing is converted in between (y of one layer is x of the next).  Weights
    are registered once per layer.  Compared with the same chain through the oracle, every
    intermediate rounded to fp16 exactly where the layers do."""
    import torch
    from gpu_util import to_dev, to_host
    rng = np.random.default_rng(77)
    n = 2
    chain = [  # (params, flags)
        (params_dict(n, 3, 30, 36, 32, 3, 3, 1, 1), hgc.HGC_FLAG_Y_NHWC),
        (params_dict(n, 32, 30, 36, 64, 3, 3, 1, 1), hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC),
        (params_dict(n, 64, 30, 36, 64, 1, 1), hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC),
        (params_dict(n, 64, 30, 36, 40, 3, 3, 1, 1, 2, 2), hgc.HGC_FLAG_X_NHWC),
    ]
    x0 = rng.uniform(0.0, 1.0, (n, 3, 30, 36)).astype(np.float16)
    ref = x0
    cur = to_dev(x0)
    keep = []
    for a, fl in chain:
        _, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
        ref = oracle.conv_fast(oracle.ConvParams(**a), ref, w, b, True)
        d = hgc.ConvDesc(flags=fl, **a)
        assert d.path() == hgc.HGC_PATH_IGEMM
        d.ensure_workspace()
        wd, bd = to_dev(w), to_dev(b)
        d.set_weights(wd)
        nn, k, p, q = d.output_dims()
        shape = (nn, p, q, k) if fl & hgc.HGC_FLAG_Y_NHWC else (nn, k, p, q)
        y = torch.full(shape, float("nan"), dtype=torch.float16, device="cuda")
        hgc.conv_forward(d, cur, wd, bd, y, True)
        keep.append((d, wd, bd, cur))
        cur = y
    torch.cuda.synchronize()
    for d, *_ in keep:
        assert d.last_device_status() == hgc.HGC_OK
    check_close(to_host(cur), ref, what="channels-last chain")
    for d, *_ in keep:
        d.close()
