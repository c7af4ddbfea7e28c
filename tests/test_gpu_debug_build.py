"""The checked build (libhgc_debug.so, -DHGC_DEBUG): every global access that a kernel addresses by
hand is tested against the tensors of the call.  The same layers as elsewhere must give the same
results with no access outside them; and with the registered ranges cut short (test hook) the
accesses at the end of the tensors must be reported and skipped, while nothing faults.
Runs in a child process: a process loads one build of the library."""
import os
import subprocess
import sys
import textwrap

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = textwrap.dedent(r'''
    import sys, zlib
    import numpy as np
    sys.path.insert(0, ROOT); sys.path.insert(0, ROOT + "/tests")
    import torch
    import oracle
    oracle.build()
    from paper_1901_00858_b200 import binding as hgc, workloads
    from gpu_util import check_close, params_dict, run_layer, to_dev, to_host
    hgc.use_checked_build()
    assert hgc.debug_checked_build()

    NHWC = hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC
    cases = [
        # tensor-core path: TMA-store, copy and channels-last epilogues, stems, shared and paired tiles
        ("3x3 56x56", params_dict(2, 64, 56, 56, 128, 3, 3, 1, 1), 0),
        ("3x3 14x14 copy epilogue, words with junk columns", params_dict(3, 128, 14, 14, 136, 3, 3, 1, 1), 0),
        ("3x3 13x13 copy epilogue, 2-byte stores", params_dict(3, 96, 13, 13, 72, 3, 3, 1, 1), 0),
        ("1x1 in place", params_dict(2, 64, 56, 56, 256, 1, 1), 0),
        ("1x1 7x7", params_dict(9, 512, 7, 7, 130, 1, 1), 0),
        ("row pairs", params_dict(2, 16, 10, 112, 64, 3, 3, 1, 1), 0),
        ("replicated rows", params_dict(2, 32, 112, 112, 64, 1, 1), 0),
        ("stem windows", params_dict(2, 3, 32, 40, 16, 3, 3, 1, 1), 0),
        ("stem patches", params_dict(2, 3, 64, 48, 32, 3, 3, 1, 1, 2, 2), 0),
        ("split reduction", params_dict(3, 4096, 5, 5, 96, 1, 1), 0),
        ("shared tiles", params_dict(2, 256, 24, 24, 256, 3, 3, 1, 1), hgc.HGC_FLAG_SHARED_TILES),
        ("pairs", params_dict(2, 64, 12, 12, 256, 3, 3, 1, 1), hgc.HGC_FLAG_CTA_PAIRS),
        ("layout pass inside the kernel", params_dict(2, 64, 24, 24, 64, 3, 3, 1, 1), hgc.HGC_FLAG_FUSED_LAYOUT),
        ("grouped", params_dict(1, 96, 27, 27, 256, 5, 5, 2, 2, 1, 1, 1, 1, 2), 0),
        ("x gathered by the kernel's warps", params_dict(3, 128, 14, 14, 72, 1, 1), hgc.HGC_FLAG_GATHER_X),
        ("whole planes as bulk copies", params_dict(40, 64, 14, 14, 96, 1, 1), 0),
        ("whole planes as bulk copies, several images per tile", params_dict(33, 64, 7, 7, 256, 1, 1), 0),
        # depthwise kernels (rows of whole vectors, column words, small rows, general), direct kernel
        ("depthwise 112x112", params_dict(2, 32, 112, 112, 32, 3, 3, 1, 1, 1, 1, 1, 1, 32), 0),
        ("depthwise 56x56 stride 2", params_dict(2, 64, 56, 56, 64, 3, 3, 1, 1, 2, 2, 1, 1, 64), 0),
        ("depthwise 28x28", params_dict(2, 64, 28, 28, 64, 3, 3, 1, 1, 1, 1, 1, 1, 64), 0),
        ("depthwise 14x14 stride 2", params_dict(2, 64, 14, 14, 64, 3, 3, 1, 1, 2, 2, 1, 1, 64), 0),
        ("depthwise 7x7", params_dict(3, 40, 7, 7, 40, 3, 3, 1, 1, 1, 1, 1, 1, 40), 0),
        ("depthwise 37x29", params_dict(2, 24, 37, 29, 24, 3, 3, 1, 1, 1, 1, 1, 1, 24), 0),
        ("direct (odd groups)", params_dict(2, 15, 9, 11, 10, 3, 2, 1, 0, 1, 1, 1, 1, 5), 0),
        ("direct (forced)", params_dict(2, 32, 12, 12, 48, 3, 3, 1, 1), hgc.HGC_FLAG_FORCE_DIRECT),
    ]
    for name, a, flags in cases:
        rng = np.random.default_rng(zlib.crc32(name.encode()))
        x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
        got, path = run_layer(hgc, a, x, w, b, True, flags=flags)
        check_close(got, ref, what=name)
        v = hgc.debug_violations()
        assert v["count"] == 0, (name, v)
    print("clean:", len(cases), "layers")

    # channels-last layers (plain 2-byte stores where the channel count is odd-ish, depthwise both forms)
    for name, a in [("nhwc k40", params_dict(2, 64, 9, 11, 40, 3, 3, 1, 1)),
                    ("nhwc depthwise", params_dict(2, 64, 20, 20, 64, 3, 3, 1, 1, 1, 1, 1, 1, 64)),
                    ("nhwc depthwise stride 2", params_dict(2, 24, 15, 15, 24, 3, 3, 1, 1, 2, 2, 1, 1, 24))]:
        rng = np.random.default_rng(zlib.crc32(name.encode()))
        x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
        d = hgc.ConvDesc(flags=NHWC, **a)
        d.ensure_workspace()
        n, k, p, q = d.output_dims()
        xd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1)))
        y = torch.full((n, p, q, k), float("nan"), dtype=torch.float16, device="cuda")
        hgc.conv_forward(d, xd, to_dev(w), to_dev(b), y, True)
        torch.cuda.synchronize()
        check_close(to_host(y).transpose(0, 3, 1, 2), ref, what=name)
        v = hgc.debug_violations()
        assert v["count"] == 0, (name, v)
        d.close()
    print("clean: channels-last")

    # the test hook: ranges 64 bytes short.  The kernels are the same, so their last accesses now
    # lie outside: they must be reported and skipped (the end of y keeps its NaN), nothing faults.
    name, a = "3x3 14x14 copy epilogue", params_dict(3, 128, 14, 14, 136, 3, 3, 1, 1)
    rng = np.random.default_rng(5)
    x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
    d = hgc.ConvDesc(**a)
    d.ensure_workspace()
    y = torch.full(d.output_dims(), float("nan"), dtype=torch.float16, device="cuda")
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    hgc.debug_shrink_ranges(64)
    try:
        hgc.conv_forward(d, xd, wd, bd, y, True)
        torch.cuda.synchronize()
    finally:
        hgc.debug_shrink_ranges(0)
    v = hgc.debug_violations()
    assert v["count"] > 0 and v["line"] > 0 and v["bytes"] > 0, v
    got = to_host(y).ravel()
    assert np.isnan(got[-32:].astype(np.float32)).all(), "the skipped stores must not have happened"
    assert d.last_device_status() == hgc.HGC_OK
    # and the descriptor is as good as before
    y.fill_(float("nan"))
    hgc.conv_forward(d, xd, wd, bd, y, True)
    torch.cuda.synchronize()
    check_close(to_host(y), ref, what=name + " (after)")
    assert hgc.debug_violations()["count"] == 0
    d.close()
    print("hook: reported", v["count"], "accesses, first at source line", v["line"])
    print("CHECKED BUILD OK")
''')


def test_checked_build_runs_the_layers_without_an_access_outside_their_tensors():
    lib = os.path.join(ROOT, "paper_1901_00858_b200", "libhgc_debug.so")
    assert os.path.exists(lib), "build it with `python -m paper_1901_00858_b200.build`"
    r = subprocess.run([sys.executable, "-c", "ROOT = %r\n" % ROOT + CHILD], capture_output=True, text=True, timeout=900)
    sys.stdout.write(r.stdout[-3000:])
    sys.stderr.write(r.stderr[-3000:])
    assert r.returncode == 0 and "CHECKED BUILD OK" in r.stdout
