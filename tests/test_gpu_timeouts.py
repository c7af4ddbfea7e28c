"""Failure detection without a fault: every device-side wait of the TMA-fed kernels is bounded.
The tests shorten the bound to a few milliseconds and make one copy never arrive (the first CTA
announces it and does not issue it), then check what a caller sees: the launch ends by itself,
the status reads HGC_DEVICE_TIMEOUT once, forwards are skipped until it has been read, and the
next forward on the same descriptor is correct again.  Nothing here traps, faults or waits
without bound."""
import time

import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import check_close, params_dict, to_dev, to_host

pytestmark = pytest.mark.gpu
LIMIT_NS = 2_000_000     # 2 ms per wait


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _forward(hgc, d, xd, wd, bd, shape, relu=True):
    import torch
    y = torch.full(shape, float("nan"), dtype=torch.float16, device="cuda")
    hgc.conv_forward(d, xd, wd, bd, y, relu)
    torch.cuda.synchronize()
    return y


@pytest.mark.parametrize("name,a,flags_name,drop", [
    ("one tile on one CTA, second ring stage", params_dict(1, 32, 8, 8, 32, 3, 3, 1, 1), "", 1),
    ("several CTAs, first stage of the first CTA", params_dict(4, 64, 16, 16, 256, 3, 3, 1, 1), "", 0),
    ("CTA pairs: the first CTA's copies of a stage", params_dict(2, 64, 12, 12, 256, 3, 3, 1, 1), "pairs", 2),
    ("tiles shared between CTAs: a part that is never handed over", params_dict(2, 256, 24, 24, 256, 3, 3, 1, 1), "shared", 0),
    ("layout pass inside the kernel", params_dict(2, 64, 24, 24, 64, 3, 3, 1, 1), "fused", 1),
    ("whole-plane epilogue (the warps of a lane quarter meet on a bounded barrier)", params_dict(40, 64, 14, 14, 256, 1, 1), "", 0),
    ("x gathered by the kernel's own warps: the weight copy of a later stage", params_dict(20, 256, 14, 14, 256, 1, 1), "gather", 1),
])
def test_tensor_core_wait_runs_out_and_the_descriptor_recovers(hgc, oracle, name, a, flags_name, drop):
    import torch
    flags = {"": 0, "pairs": hgc.HGC_FLAG_CTA_PAIRS, "shared": hgc.HGC_FLAG_SHARED_TILES,
             "fused": hgc.HGC_FLAG_FUSED_LAYOUT, "gather": hgc.HGC_FLAG_GATHER_X}[flags_name]
    rng = np.random.default_rng(3)
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
    d = hgc.ConvDesc(flags=flags, **a)
    assert d.path() == hgc.HGC_PATH_IGEMM
    d.ensure_workspace()
    shape = d.output_dims()
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    d.set_weights(wd)
    check_close(to_host(_forward(hgc, d, xd, wd, bd, shape)), ref, what=name + " (before)")
    assert d.last_device_status() == hgc.HGC_OK
    try:
        hgc.debug_set_wait_limit_ns(LIMIT_NS)
        hgc.debug_drop_copies(drop)
        t0 = time.time()
        _forward(hgc, d, xd, wd, bd, shape)
        assert time.time() - t0 < 2.0, "the launch must end within a few wait limits"
        hgc.debug_drop_copies(-1)
        # the word is still raised: this forward is skipped and leaves y as it was
        y_skipped = _forward(hgc, d, xd, wd, bd, shape)
        assert bool(torch.isnan(y_skipped).all())
        assert d.last_device_status() == hgc.HGC_DEVICE_TIMEOUT
        assert d.last_device_status() == hgc.HGC_OK          # reading it cleared it
    finally:
        hgc.debug_drop_copies(-1)
        hgc.debug_set_wait_limit_ns(0)
    for rep in range(2):
        check_close(to_host(_forward(hgc, d, xd, wd, bd, shape)), ref, what=f"{name} (after, {rep})")
    assert d.last_device_status() == hgc.HGC_OK
    d.close()


def test_depthwise_copy_never_arrives(hgc, oracle):
    """The TMA-fed channels-last depthwise kernel: same form."""
    import torch
    a = params_dict(2, 64, 20, 20, 64, 3, 3, 1, 1, 1, 1, 1, 1, 64)
    rng = np.random.default_rng(4)
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], 3, 3, 64)
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
    d = hgc.ConvDesc(flags=hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC, **a)
    assert d.path() == hgc.HGC_PATH_DEPTHWISE
    n, k, p, q = d.output_dims()
    xd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1)))
    wd, bd = to_dev(w), to_dev(b)

    def run():
        return to_host(_forward(hgc, d, xd, wd, bd, (n, p, q, k))).transpose(0, 3, 1, 2)

    check_close(run(), ref, what="depthwise channels-last (before)")
    assert d.last_device_status() == hgc.HGC_OK
    try:
        hgc.debug_set_wait_limit_ns(LIMIT_NS)
        hgc.debug_drop_copies(0)
        t0 = time.time()
        run()
        assert time.time() - t0 < 2.0
        assert d.last_device_status() == hgc.HGC_DEVICE_TIMEOUT
        assert d.last_device_status() == hgc.HGC_OK
    finally:
        hgc.debug_drop_copies(-1)
        hgc.debug_set_wait_limit_ns(0)
    check_close(run(), ref, what="depthwise channels-last (after)")
    assert d.last_device_status() == hgc.HGC_OK
    d.close()
