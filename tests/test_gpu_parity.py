"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded float16 inputs.  Tolerance: |gpu - ref| <= 2e-3 + 1e-2*|ref|."""
import json
import os

import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import (attach_guarded_workspace, check_close, check_guards, guarded_output, layer_args, max_ulp_error,
                      params_dict, run_layer, sample_coords, to_dev, to_host)

pytestmark = pytest.mark.gpu
F16 = np.float16
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
# Beyond the tolerance, a correct kernel differs from the fp64 oracle only where its fp32 sum falls
# on the other side of a binary16 rounding boundary: by one unit in the last place, on a fraction
# of the outputs that grows with the reduction length (measured: 0.03 % at 27 terms, 0.3 % at
# 1152, 0.5 % at 2304, about 1 % at 4608).  A dropped tap, a wrong padding column, binary16
# accumulation or a double rounding moves many outputs by many units, so both numbers are asserted.
MIN_BIT_IDENTICAL = 0.985
MAX_ULP = 1


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _hand_examples():
    with open(os.path.join(GOLDEN, "hand_examples.json")) as f:
        return json.load(f)["examples"]


@pytest.mark.parametrize("flags", [0, 1], ids=["planned", "forced-direct"])
@pytest.mark.parametrize("ex", _hand_examples(), ids=lambda e: e["id"])
def test_hand_examples_on_gpu(hgc, oracle, ex, flags):
    from test_oracle_pins import _example_tensors
    P = oracle.ConvParams(**ex["params"])
    x, w, b = _example_tensors(ex, P)
    args = params_dict(**ex["params"])
    y, _ = run_layer(hgc, args, x, w, b, ex["relu"], flags=flags)
    assert list(y.shape) == ex["out_shape"]
    if "expected_bits" in ex:   # fp32 holds this sum exactly: the GPU must round like the oracle
        assert [format(v, "04x") for v in y.view(np.uint16).ravel()] == ex["expected_bits"]
    else:                        # small exact integers/halves: exact on the GPU as well
        assert y.ravel().astype(np.float64).tolist() == [float(v) for v in ex["expected"]]


def _random_descriptor(rng):
    g = int(rng.choice([1, 1, 2, 3, 4, -1]))
    cg, kg = int(rng.integers(1, 41)), int(rng.integers(1, 41))
    if g == -1:   # depthwise, sometimes with a channel multiplier
        g, cg, kg = int(rng.integers(1, 70)), 1, int(rng.choice([1, 1, 1, 2]))
    h, w = int(rng.integers(1, 41)), int(rng.integers(1, 41))
    r, s = int(rng.integers(1, 8)), int(rng.integers(1, 8))
    if rng.random() < 0.4:
        r = s = 3
    ph, pw = int(rng.integers(0, 5)), int(rng.integers(0, 5))
    sh, sw = int(rng.integers(1, 6)), int(rng.integers(1, 6))
    if rng.random() < 0.5:
        sh = sw = int(rng.integers(1, 3))
    dh, dw = int(rng.integers(1, 4)), int(rng.integers(1, 4))
    if rng.random() < 0.5:
        dh = dw = 1
    n = int(rng.integers(1, 4))
    return params_dict(n, g * cg, h, w, g * kg, r, s, ph, pw, sh, sw, dh, dw, g)


@pytest.mark.parametrize("flags", [0, 1], ids=["planned", "forced-direct"])
def test_random_descriptors(hgc, oracle, flags):
    rng = np.random.default_rng(20240 + flags)
    done = 0
    paths = set()
    while done < 160:
        a = _random_descriptor(rng)
        if oracle.out_dim(a["h"], a["r"], a["pad_h"], a["stride_h"], a["dil_h"]) < 1 or \
           oracle.out_dim(a["w"], a["s"], a["pad_w"], a["stride_w"], a["dil_w"]) < 1:
            with pytest.raises(hgc.HgcError) as e:
                hgc.ConvDesc(**a)
            assert e.value.status == hgc.HGC_INVALID_ARG
            continue
        x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"],
                                                 a["group"])
        relu = bool(rng.integers(0, 2))
        bias = b if rng.integers(0, 2) else None
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, bias, relu)
        got, path = run_layer(hgc, a, x, w, bias, relu, flags=flags)
        paths.add(path)
        assert got.shape == ref.shape
        check_close(got, ref, what=str(a))
        done += 1
    if flags:
        assert paths == {hgc.HGC_PATH_DIRECT}


@pytest.mark.parametrize("plane", [7, 13, 14, 27, 28, 33, 56, 57, 112, 113, 150])
@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_planes(hgc, oracle, plane, stride):
    """3x3 depthwise at the MobileNet plane sizes and at odd, ragged ones; several images and a
    channel count that leaves a ragged last CTA."""
    rng = np.random.default_rng(plane * 10 + stride)
    n, c = 3, 37
    if plane >= 112:
        n, c = 2, 5
    for pad in (1, 0):
        a = params_dict(n, c, plane, plane + (plane % 5), c, 3, 3, pad, pad, stride, stride, 1, 1, c)
        x, w, b = workloads.random_layer_tensors(rng, n, c, a["h"], a["w"], c, 3, 3, c)
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
        got, path = run_layer(hgc, a, x, w, b, True)
        assert path == hgc.HGC_PATH_DEPTHWISE
        check_close(got, ref, what=f"dw plane {plane} stride {stride} pad {pad}")
        got2, _ = run_layer(hgc, a, x, w, None, False)
        check_close(got2, oracle.conv_fast(oracle.ConvParams(**a), x, w, None, False), what="dw no bias")


@pytest.mark.parametrize("plane", [14, 28])
@pytest.mark.parametrize("stride", [1, 2])
def test_depthwise_square_small_planes(hgc, oracle, plane, stride):
    """The 28x28 and 14x14 planes of MobileNet (one column word per lane, several planes per
    warp): a plane count that leaves the last warp partly filled, with and without bias/ReLU."""
    rng = np.random.default_rng(500 + plane + stride)
    n, c = 3, 37
    a = params_dict(n, c, plane, plane, c, 3, 3, 1, 1, stride, stride, 1, 1, c)
    x, w, b = workloads.random_layer_tensors(rng, n, c, plane, plane, c, 3, 3, c)
    for relu, bias in ((True, b), (False, None), (False, b)):
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, bias, relu)
        got, path = run_layer(hgc, a, x, w, bias, relu)
        assert path == hgc.HGC_PATH_DEPTHWISE
        check_close(got, ref, what=f"dw square {plane} stride {stride} relu={relu}")


@pytest.mark.parametrize("h,w,stride", [(56, 56, 1), (112, 112, 1), (24, 40, 1), (9, 8, 1), (56, 56, 2), (112, 112, 2),
                                        (40, 24, 2), (16, 8, 2), (30, 72, 2)])
def test_depthwise_row_vector_shapes(hgc, oracle, h, w, stride):
    """Planes whose rows are whole 16-byte vectors take the shuffle-based kernel: cover warp
    boundaries inside rows, half-full last vectors (Q % 8 == 4) and ragged last strips."""
    rng = np.random.default_rng(h * 7 + w + stride)
    n, c = 2, 19
    a = params_dict(n, c, h, w, c, 3, 3, 1, 1, stride, stride, 1, 1, c)
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, c, 3, 3, c)
    for relu, bias in ((True, b), (False, None)):
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, wt, bias, relu)
        got, path = run_layer(hgc, a, x, wt, bias, relu)
        assert path == hgc.HGC_PATH_DEPTHWISE
        check_close(got, ref, what=f"dw rowvec {h}x{w} s{stride}")


@pytest.mark.parametrize("cfg,batch", [(0, 1), (1, 1), (2, 1), (3, 1)])
def test_configs_whole_tensor(hgc, oracle, cfg, batch):
    """Configs small enough for the oracle to compute every output."""
    wl = workloads.workload(cfg, batch)
    for li, l in enumerate(wl.layers):
        x, w, b = workloads.make_tensors(cfg, batch, li, l)
        a = layer_args(batch, l)
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, l.relu)
        assert float(np.abs(ref.astype(np.float64)).max()) < 65504
        got, _ = run_layer(hgc, a, x, w, b, l.relu, register_weights=True)
        err, same = check_close(got, ref, what=f"{wl.name}/{l.name}")
        ulp = max_ulp_error(got, ref)
        print(f"{wl.name}/{l.name}: bit-identical {same:.5f}, max error {ulp} ulp, {err:.2e} abs")
        assert same >= MIN_BIT_IDENTICAL and ulp <= MAX_ULP, (wl.name, l.name, same, ulp)


def _unique_layers(wl):
    seen, out = set(), []
    for li, l in enumerate(wl.layers):
        key = (l.c, l.h, l.k, l.r, l.stride, l.pad, l.group, l.relu)
        if key not in seen:
            seen.add(key)
            out.append((li, l))
    return out


def _whole_tensor_layer(hgc, oracle, a, x, w, b, relu, flags, what):
    """One full-size layer in the configuration the bench times (planner's path, registered
    weights, guarded output and workspace): EVERY output element against the oracle."""
    import torch
    d = hgc.ConvDesc(flags=flags, **a)
    n, k, p, q = d.output_dims()
    ws_whole = attach_guarded_workspace(d)
    x_cl, y_cl = bool(flags & hgc.HGC_FLAG_X_NHWC), bool(flags & hgc.HGC_FLAG_Y_NHWC)
    xd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1)) if x_cl else x)
    wd, bd = to_dev(w), to_dev(b)
    y_whole, y = guarded_output((n, p, q, k) if y_cl else (n, k, p, q))
    d.set_weights(wd)
    hgc.conv_forward(d, xd, wd, bd, y, relu)
    torch.cuda.synchronize()
    assert d.last_device_status() == hgc.HGC_OK
    check_guards(y_whole, what + " (y)")
    if ws_whole is not None:
        check_guards(ws_whole, what + " (workspace)")
    got = to_host(y)
    if y_cl:
        got = np.ascontiguousarray(got.transpose(0, 3, 1, 2))
    info = d.plan_info()
    d.close()
    del xd, wd, bd, y, y_whole, ws_whole
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, relu)
    assert float(np.abs(ref.astype(np.float32)).max()) < 65504
    err, same = check_close(got, ref, what=what)
    ulp = max_ulp_error(got, ref)
    print(f"{what}: {got.size} outputs, bit-identical {same:.5f}, max error {ulp} ulp, {err:.2e} abs")
    assert same >= MIN_BIT_IDENTICAL and ulp <= MAX_ULP, (what, same, ulp, info)


@pytest.mark.parametrize("cfg,batch", [(2, 16), (3, 32), (4, 64)])
def test_configs_full_size_whole_tensor(hgc, oracle, cfg, batch):
    """The three throughput configurations at full size, in the launch configuration the bench
    times: every unique layer, every output element against the oracle (the tile plans for
    several images per tile, multi-wave schedules and wide epilogues only occur here)."""
    wl = workloads.workload(cfg, batch)
    for li, l in _unique_layers(wl):
        x, w, b = workloads.make_tensors(cfg, batch, li, l)
        _whole_tensor_layer(hgc, oracle, layer_args(batch, l), x, w, b, l.relu, 0, f"{wl.name}/{l.name}")


@pytest.mark.parametrize("cfg,batch", [(2, 16), (3, 32), (4, 64)])
def test_configs_full_size_channels_last_whole_tensor(hgc, oracle, cfg, batch):
    """The bench's channels-last leg at full size: every layer that takes the flags reads
    x[N][H][W][C] and writes y[N][P][Q][K]; every output element against the oracle."""
    wl = workloads.workload(cfg, batch)
    for li, l in _unique_layers(wl):
        a = layer_args(batch, l)
        flags = None
        for fl in (hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC, hgc.HGC_FLAG_Y_NHWC):
            try:
                hgc.ConvDesc(flags=fl, **a).close()
                flags = fl
                break
            except hgc.HgcError:
                pass
        if flags is None:
            continue
        x, w, b = workloads.make_tensors(cfg, batch, li, l)
        _whole_tensor_layer(hgc, oracle, a, x, w, b, l.relu, flags, f"{wl.name}/{l.name} channels-last")


@pytest.mark.parametrize("kind", ["tensor cores", "channels-last", "depthwise", "depthwise channels-last",
                                  "1x1 reading x in place"])
def test_tensors_of_more_than_2_31_elements(hgc, oracle, kind):
    """Maximum sizes: 700 (1400) images of 224x224, x and y of 2.25 G elements (4.5 GB) each, so every
    flat index beyond the first 2^31 elements needs 64-bit arithmetic.  Inputs are generated on the
    device; the oracle evaluates sampled outputs including the last ones."""
    import torch
    n, c, k, r, pad, group = 700, 64, 64, 3, 1, 1
    if kind.startswith("depthwise"):
        group = 64
    if kind.startswith("1x1"):
        n, c, k, r, pad = 1400, 32, 32, 1, 0
    cl = "channels-last" in kind
    a = params_dict(n, c, 224, 224, k, r, r, pad, pad, 1, 1, 1, 1, group)
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    x = torch.empty((n, c, 224, 224), dtype=torch.float16, device="cuda").uniform_(0, 1, generator=g)
    w = (torch.randn((k, c // group, r, r), device="cuda", generator=g) * float(np.sqrt(2.0 / (c // group * r * r)))).to(torch.float16)
    b = torch.empty(k, dtype=torch.float16, device="cuda").uniform_(-0.1, 0.1, generator=g)
    assert x.numel() > 2 ** 31
    d = hgc.ConvDesc(flags=(hgc.HGC_FLAG_X_NHWC | hgc.HGC_FLAG_Y_NHWC) if cl else 0, **a)
    assert d.path() == (hgc.HGC_PATH_DEPTHWISE if group > 1 else hgc.HGC_PATH_IGEMM)
    d.ensure_workspace()
    nn, kk, p, q = d.output_dims()
    y = torch.full((nn, p, q, kk) if cl else (nn, kk, p, q), float("nan"), dtype=torch.float16, device="cuda")
    xin = x.permute(0, 2, 3, 1).contiguous() if cl else x
    hgc.conv_forward(d, xin, w, b, y, True)
    torch.cuda.synchronize()
    del xin
    assert d.last_device_status() == hgc.HGC_OK
    assert bool(torch.isfinite(y).all())
    rng = np.random.default_rng(5)
    pts = np.stack([rng.integers(0, nn, 4000), rng.integers(0, kk, 4000), rng.integers(0, p, 4000),
                    rng.integers(0, q, 4000)], 1).astype(np.int64)
    pts[:6] = [[nn - 1, kk - 1, p - 1, q - 1], [nn - 1, 0, 0, 0], [0, kk - 1, p - 1, 0], [nn - 1, kk - 1, 0, q - 1],
               [nn // 2 + 1, kk // 2, p // 2, q // 2], [0, 0, 0, 0]]
    ref = oracle.conv_points(oracle.ConvParams(**a), x.cpu().numpy(), w.cpu().numpy(), b.cpu().numpy(), True, pts)
    ct = torch.from_numpy(pts).cuda()
    got = y[ct[:, 0], ct[:, 2], ct[:, 3], ct[:, 1]] if cl else y[ct[:, 0], ct[:, 1], ct[:, 2], ct[:, 3]]
    check_close(to_host(got), ref, what=f"2^31 elements, {kind}")
    d.close()
    del x, y
    torch.cuda.empty_cache()


def test_forward_host_matches_device_forward(hgc, oracle):
    import torch
    rng = np.random.default_rng(4)
    a = params_dict(2, 6, 17, 19, 10, 3, 3, 1, 1, 2, 1, 1, 1, 2)
    x, w, b = workloads.random_layer_tensors(rng, 2, 6, 17, 19, 10, 3, 3, 2)
    ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
    d = hgc.ConvDesc(**a)
    d.ensure_workspace(host=True)
    xh = torch.from_numpy(x.view(np.int16)).pin_memory()
    wh = torch.from_numpy(w.view(np.int16)).pin_memory()
    bh = torch.from_numpy(b.view(np.int16)).pin_memory()
    yh = torch.empty(ref.shape, dtype=torch.int16).pin_memory()
    hgc.conv_forward_host(d, xh, wh, bh, yh, True)
    torch.cuda.synchronize()
    got = yh.numpy().view(F16)
    check_close(got, ref, what="forward_host")
    d.set_workspace(None)
    with pytest.raises(hgc.HgcError) as e:
        hgc.conv_forward_host(d, xh, wh, bh, yh, True)
    assert e.value.status == hgc.HGC_NO_WORKSPACE
