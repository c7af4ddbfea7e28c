"""The data-movement kernels are permutations: exact equality of bit patterns with the
numpy definitions."""
import numpy as np
import pytest

from gpu_util import to_dev, to_host

pytestmark = pytest.mark.gpu
F16 = np.float16


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


@pytest.mark.parametrize("n,c,h,w,c_pad", [
    (1, 3, 32, 32, 8), (2, 3, 227, 227, 8), (3, 64, 56, 56, 64), (2, 96, 27, 27, 96), (2, 48, 27, 27, 64),
    (5, 100, 7, 7, 104), (3, 130, 14, 14, 136), (1, 1, 1, 1, 8), (2, 7, 13, 5, 16), (1, 256, 28, 28, 256),
    (2, 65, 9, 8, 72),
])
def test_layout_round_trip_exact(hgc, oracle, n, c, h, w, c_pad):
    import torch
    rng = np.random.default_rng(n * 1000 + c)
    x = rng.uniform(-4, 4, (n, c, h, w)).astype(F16)
    want = oracle.nchw_to_nhwc(x, c_pad)
    xd = to_dev(x)
    out = torch.full((n, h, w, c_pad), float("nan"), dtype=torch.float16, device="cuda")
    hgc.layout_nchw_to_nhwc(xd, out, n, c, h, w, c_pad)
    torch.cuda.synchronize()
    got = to_host(out)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    back = torch.full((n, c, h, w), float("nan"), dtype=torch.float16, device="cuda")
    hgc.layout_nhwc_to_nchw(out, back, n, c, h, w, c_pad)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(back).view(np.uint16), x.view(np.uint16))
    assert np.array_equal(to_host(back).view(np.uint16), oracle.nhwc_to_nchw(want, c).view(np.uint16))


@pytest.mark.parametrize("k,cg,r,s,group,c_pad", [
    (16, 3, 3, 3, 1, 8), (256, 48, 5, 5, 2, 64), (96, 3, 11, 11, 1, 8), (12, 5, 1, 1, 3, 8),
    (64, 64, 3, 3, 1, 64), (10, 17, 2, 3, 2, 24),
])
def test_weights_repack_exact(hgc, oracle, k, cg, r, s, group, c_pad):
    import torch
    rng = np.random.default_rng(k + cg)
    w = rng.normal(0, 1, (k, cg, r, s)).astype(F16)
    want = oracle.repack_weights(w, group, c_pad)
    out = torch.full(want.shape, float("nan"), dtype=torch.float16, device="cuda")
    hgc.weights_repack(to_dev(w), out, k, cg, r, s, group, c_pad)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(out).view(np.uint16), want.view(np.uint16))
