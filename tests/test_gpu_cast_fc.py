"""GPU parity of the two layers next to the convolution path: the converter's FP32 -> FP16 cast
(bit-exact against the oracle, overflow count included) and the inner-product layer (within the
convolution's tolerance), both through the C ABI."""
import numpy as np
import pytest

from gpu_util import check_close, to_dev, to_host

pytestmark = pytest.mark.gpu
F16 = np.float16


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _cast_inputs(rng, count):
    kinds = rng.integers(0, 6, size=count)
    v = np.empty(count, dtype=np.float64)
    v[kinds == 0] = rng.normal(0, 1, np.count_nonzero(kinds == 0))
    v[kinds == 1] = rng.normal(0, 400, np.count_nonzero(kinds == 1))
    v[kinds == 2] = rng.uniform(-70000, 70000, np.count_nonzero(kinds == 2))      # around the overflow edge
    v[kinds == 3] = rng.uniform(-1e-4, 1e-4, np.count_nonzero(kinds == 3))        # fp16 subnormals
    v[kinds == 4] = rng.uniform(-1e-7, 1e-7, np.count_nonzero(kinds == 4))        # underflow to zero
    m = kinds == 5                                                                # exact ties
    v[m] = (1024 + rng.integers(0, 1023, np.count_nonzero(m)) + 0.5) * 2.0 ** rng.integers(-24, 5, np.count_nonzero(m))
    src = v.astype(np.float32)
    special = np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65520.0, -65520.0, 65519.996, 1e38, -1e38, np.nan],
                       dtype=np.float32)
    src[:special.size] = special[:min(special.size, count)]
    return src


@pytest.mark.parametrize("count", [1, 7, 8, 9, 1000, 8 * 256 * 3 + 5, 1 << 20, (1 << 22) + 3])
def test_cast_is_bit_exact(hgc, oracle, count):
    import torch
    rng = np.random.default_rng(count)
    src = _cast_inputs(rng, count)
    want, want_over = oracle.cast_f32_to_f16(src)
    s = torch.from_numpy(src).cuda()
    d = torch.full((count,), float("nan"), dtype=torch.float16, device="cuda")
    over = torch.zeros(1, dtype=torch.int64, device="cuda")
    hgc.cast_f32_to_f16(s, d, overflow_count=over)
    torch.cuda.synchronize()
    got = to_host(d)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got.view(np.uint16)[~nan], want.view(np.uint16)[~nan])
    assert int(over.item()) == want_over
    # without a counter
    d2 = torch.empty_like(d)
    hgc.cast_f32_to_f16(s, d2)
    torch.cuda.synchronize()
    assert np.array_equal(to_host(d2).view(np.uint16)[~nan], want.view(np.uint16)[~nan])


def test_cast_rejects_bad_arguments(hgc):
    import torch
    s = torch.zeros(64, dtype=torch.float32, device="cuda")
    d = torch.zeros(64, dtype=torch.float16, device="cuda")
    with pytest.raises(hgc.HgcError):
        hgc.cast_f32_to_f16(s[1:], d, count=8)       # src not 16-byte aligned
    with pytest.raises(hgc.HgcError):
        hgc.cast_f32_to_f16(s, d, count=-1)
    hgc.cast_f32_to_f16(s, d, count=0)               # no-op


@pytest.mark.parametrize("n,c,k", [(3, 100, 10), (64, 512, 1000), (256, 1024, 256), (1, 4096, 130), (17, 9, 33)])
def test_inner_product(hgc, oracle, n, c, k):
    import torch
    rng = np.random.default_rng(n * 1000 + c + k)
    x = rng.uniform(-1, 1, size=(n, c)).astype(F16)
    w = rng.normal(0, np.sqrt(2.0 / c), size=(k, c)).astype(F16)
    b = rng.uniform(-0.1, 0.1, size=(k,)).astype(F16)
    d = hgc.ConvDesc.inner_product(n, c, k)
    assert d.output_dims() == (n, k, 1, 1)
    d.ensure_workspace()
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    for relu, bias, bias_d in ((True, b, bd), (False, None, None)):
        y = torch.full((n, k), float("nan"), dtype=torch.float16, device="cuda")
        hgc.conv_forward(d, xd, wd, bias_d, y, relu)
        torch.cuda.synchronize()
        assert d.last_device_status() == hgc.HGC_OK
        check_close(to_host(y), oracle.inner_product(x, w, bias, relu), what=f"fc {n}x{c}->{k} relu={relu}")
    d.close()


def test_inner_product_keeps_a_wide_sum(hgc, oracle):
    """4096 ones: FP16 accumulation would stall at 2048 (the overflow/precision problem of
    Section 3.1); the FP32 accumulator gives 4096 exactly."""
    import torch
    d = hgc.ConvDesc.inner_product(2, 4096, 16)
    d.ensure_workspace()
    x = torch.ones((2, 4096), dtype=torch.float16, device="cuda")
    w = torch.ones((16, 4096), dtype=torch.float16, device="cuda")
    y = torch.zeros((2, 16), dtype=torch.float16, device="cuda")
    hgc.conv_forward(d, x, w, None, y, False)
    torch.cuda.synchronize()
    assert torch.all(y == 4096).item()
    d.close()


def test_cast_of_more_than_2_31_values(hgc, oracle):
    """2^31 + 12345 values (8.6 GB in, 4.3 GB out): a sample of a million positions, the last ones
    included, must carry exactly the oracle's bits (the tail after the last group of 8 too)."""
    import torch
    count = 2 ** 31 + 12345
    g = torch.Generator(device="cuda")
    g.manual_seed(9)
    src = torch.empty(count, dtype=torch.float32, device="cuda").normal_(0, 300.0, generator=g)
    src[-1] = 70000.0          # a finite value that overflows, at the very end
    dst = torch.zeros(count, dtype=torch.float16, device="cuda")
    over = torch.zeros(1, dtype=torch.int64, device="cuda")
    hgc.cast_f32_to_f16(src, dst, overflow_count=over)
    torch.cuda.synchronize()
    idx = torch.randint(0, count, (1 << 20,), device="cuda", generator=g)
    idx[:5] = torch.tensor([count - 1, count - 2, count - 9, 2 ** 31, 0], device="cuda")
    sample = src[idx].cpu().numpy()
    ref, _ = oracle.cast_f32_to_f16(sample)
    got = dst[idx].cpu().numpy()
    assert np.array_equal(got.view(np.uint16), ref.view(np.uint16))
    assert int(over.item()) >= 1
    assert bool(torch.isinf(dst[-1]))
    del src, dst
    torch.cuda.empty_cache()
