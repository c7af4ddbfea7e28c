"""GPU parity of the depthwise + pointwise block that runs as one kernel (hgc_dwpw_*): the oracle
is the composition the paper's engine would compute layer by layer, conv_fast(depthwise) rounded to
binary16, then conv_fast(pointwise), both in fp64 inside.  Every output element is compared."""
import zlib

import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import (attach_guarded_workspace, check_close, check_guards, guarded_output, max_ulp_error, params_dict,
                      to_dev, to_host)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _block_tensors(rng, n, c, h, w, k):
    x = rng.uniform(0.0, 1.0, (n, c, h, w)).astype(np.float16)
    w_dw = rng.normal(0.0, np.sqrt(2.0 / 9.0), (c, 1, 3, 3)).astype(np.float16)
    b_dw = rng.uniform(-0.1, 0.1, (c,)).astype(np.float16)
    w_pw = rng.normal(0.0, np.sqrt(2.0 / c), (k, c, 1, 1)).astype(np.float16)
    b_pw = rng.uniform(-0.1, 0.1, (k,)).astype(np.float16)
    return x, w_dw, b_dw, w_pw, b_pw


def _oracle_block(oracle, n, c, h, w, k, stride, x, w_dw, b_dw, w_pw, b_pw, relu_dw, relu_pw):
    dw = oracle.ConvParams(**params_dict(n, c, h, w, c, 3, 3, 1, 1, stride, stride, 1, 1, c))
    mid = oracle.conv_fast(dw, x, w_dw, b_dw, relu_dw)          # binary16, as the layer would store it
    p, q = mid.shape[2], mid.shape[3]
    pw = oracle.ConvParams(**params_dict(n, c, p, q, k, 1, 1))
    return oracle.conv_fast(pw, mid, w_pw, b_pw, relu_pw)


def _run_block(hgc, n, c, h, w, k, stride, x, w_dw, b_dw, w_pw, b_pw, relu_dw, relu_pw, y_nhwc, register):
    import torch
    d = hgc.DwPwDesc(n, c, h, w, k, stride, hgc.HGC_FLAG_Y_NHWC if y_nhwc else 0)
    nn, kk, p, q = d.output_dims()
    assert (nn, kk) == (n, k)
    ws_whole = attach_guarded_workspace(d)
    xd = to_dev(np.ascontiguousarray(x.transpose(0, 2, 3, 1)))
    wd, bd, wp, bp = to_dev(w_dw), to_dev(b_dw), to_dev(w_pw), to_dev(b_pw)
    y_whole, y = guarded_output((n, p, q, k) if y_nhwc else (n, k, p, q))
    if register:
        d.set_weights(wd, wp)
    hgc.dwpw_forward(d, xd, wd, bd, wp, bp, y, relu_dw, relu_pw)
    torch.cuda.synchronize()
    assert d.last_device_status() == hgc.HGC_OK
    check_guards(y_whole, "block y")
    check_guards(ws_whole, "block workspace")
    got = to_host(y)
    d.close()
    return np.ascontiguousarray(got.transpose(0, 3, 1, 2)) if y_nhwc else got


SMALL = [
    # (id, n, c, h, w, k, stride, y channels-last, relu_dw, relu_pw, bias)
    ("c32 k64 12x12", 2, 32, 12, 12, 64, 1, True, True, True, True),
    ("c64 k128 stride 2 odd plane 15x17, NCHW out", 3, 64, 15, 17, 128, 2, False, True, True, True),
    ("c24 k40: ragged channel block and channel tile, no ReLU, no bias", 2, 24, 9, 11, 40, 1, False, False, False, False),
    ("c136 k200: three channel blocks with a tail, NHWC plain stores", 2, 136, 10, 10, 200, 1, True, True, False, True),
    ("c512 k512 7x7 several images per tile", 9, 512, 7, 7, 512, 1, True, True, True, True),
    ("c256 k96 stride 2 on 28x28", 2, 256, 28, 28, 96, 2, True, True, True, True),
    ("c32 k64 one row", 1, 32, 1, 40, 64, 1, False, True, True, True),
]


@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_block_small_cases(hgc, oracle, case):
    name, n, c, h, w, k, stride, y_nhwc, relu_dw, relu_pw, bias = case
    rng = np.random.default_rng(zlib.crc32(name.encode()))
    x, w_dw, b_dw, w_pw, b_pw = _block_tensors(rng, n, c, h, w, k)
    if not bias:
        b_dw = b_pw = None
    ref = _oracle_block(oracle, n, c, h, w, k, stride, x, w_dw, b_dw, w_pw, b_pw, relu_dw, relu_pw)
    for register in (True, False):
        got = _run_block(hgc, n, c, h, w, k, stride, x, w_dw, b_dw, w_pw, b_pw, relu_dw, relu_pw, y_nhwc, register)
        check_close(got, ref, what=f"{name} registered={register}")


def test_block_mobilenet_blocks_full_size(hgc, oracle):
    """All 13 depthwise-separable blocks of the MobileNet-v1 workload at batch 32, every output
    element; the unfused channels-last layers give the same bits up to the intermediate's ties."""
    wl = workloads.workload(3, 32)
    layers = wl.expanded()
    seen = set()
    rng = np.random.default_rng(31)
    for i in range(1, len(layers), 2):
        dw, pw = layers[i], layers[i + 1]
        assert dw.group == dw.c and pw.r == 1
        key = (dw.c, dw.h, dw.stride, pw.k)
        if key in seen:
            continue
        seen.add(key)
        x, w_dw, b_dw, w_pw, b_pw = _block_tensors(rng, 32, dw.c, dw.h, dw.h, pw.k)
        ref = _oracle_block(oracle, 32, dw.c, dw.h, dw.h, pw.k, dw.stride, x, w_dw, b_dw, w_pw, b_pw, True, True)
        got = _run_block(hgc, 32, dw.c, dw.h, dw.h, pw.k, dw.stride, x, w_dw, b_dw, w_pw, b_pw, True, True, True, True)
        err, same = check_close(got, ref, what=f"block {dw.name}+{pw.name}")
        print(f"block {dw.name}+{pw.name}: {got.size} outputs, bit-identical {same:.5f}, max error "
              f"{max_ulp_error(got, ref)} ulp, {err:.2e} abs")
        assert same >= 0.98


def test_block_descriptor_is_not_a_layer_descriptor(hgc):
    import torch
    d = hgc.DwPwDesc(1, 32, 8, 8, 32)
    t = torch.zeros(64, dtype=torch.float16, device="cuda")
    with pytest.raises(hgc.HgcError) as e:
        hgc.conv_forward(d, t, t, None, t, True)
    assert e.value.status == hgc.HGC_INVALID_ARG
    with pytest.raises(hgc.HgcError) as e:          # no workspace attached yet
        hgc.dwpw_forward(d, t, t, None, t, None, t, True, True)
    assert e.value.status == hgc.HGC_NO_WORKSPACE
    d.close()
    with pytest.raises(hgc.HgcError) as e:
        hgc.DwPwDesc(1, 12, 8, 8, 32)               # 12 channels: not whole 8-channel chunks
    assert e.value.status == hgc.HGC_UNSUPPORTED
    with pytest.raises(hgc.HgcError) as e:
        hgc.DwPwDesc(1, 32, 8, 8, 32, stride=3)
    assert e.value.status == hgc.HGC_INVALID_ARG
