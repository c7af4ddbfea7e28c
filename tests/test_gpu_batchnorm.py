"""GPU parity of the batch-norm layer (grouped mean, shift before squaring) and of the folding of
stored statistics into a convolution, against the CPU oracle, through the C ABI."""
import numpy as np
import pytest

from gpu_util import check_close, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def make_x(rng, shape, kind):
    n, c = shape[0], shape[1]
    if kind == "image":          # pixel values 0..255 (the section's overflow example)
        return rng.integers(0, 256, size=shape).astype(np.float16)
    if kind == "small":          # data with small values (the section's case for shifting by 32)
        return (rng.normal(0, 1, size=shape) * 2.0 ** -9).astype(np.float16)
    scale = rng.uniform(0.1, 8.0, size=(1, c, 1, 1))
    offset = rng.normal(0, 4.0, size=(1, c, 1, 1))
    return (rng.normal(0, 1, size=shape) * scale + offset).astype(np.float16)


def run_bn(hgc, x, eps, shift_log2=0, stored=None):
    import torch
    n, c = x.shape[0], x.shape[1]
    hw = int(np.prod(x.shape[2:]))
    xd = to_dev(x)
    y = torch.full(x.shape, float("nan"), dtype=torch.float16, device="cuda")
    if stored is None:
        mean = torch.full((c,), float("nan"), dtype=torch.float32, device="cuda")
        var = torch.full((c,), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.empty(hgc.batchnorm_workspace_bytes(n, c, hw), dtype=torch.uint8, device="cuda")
        hgc.batchnorm_forward(xd, y, eps, mean, var, ws, shift_log2=shift_log2)
    else:
        mean = torch.from_numpy(stored[0].astype(np.float32)).cuda()
        var = torch.from_numpy(stored[1].astype(np.float32)).cuda()
        hgc.batchnorm_forward(xd, y, eps, mean, var, None, use_stored=True)
    torch.cuda.synchronize()
    return to_host(y), mean.cpu().numpy(), var.cpu().numpy()


SHAPES = [
    ("tiny odd plane", (2, 5, 7, 6), "mixed"),
    ("56x56: a full group and a ragged one per plane", (4, 64, 56, 56), "mixed"),
    ("50x50: planes not 16-byte aligned", (3, 16, 50, 50), "mixed"),
    ("112x112: seven groups per plane", (16, 8, 112, 112), "image"),
    ("7x7 planes, many channels", (9, 130, 7, 7), "mixed"),
    ("one image, one channel", (1, 1, 33, 65), "small"),
    ("image-valued 224x224", (2, 3, 224, 224), "image"),
]


@pytest.mark.parametrize("name,shape,kind", SHAPES, ids=[s[0] for s in SHAPES])
def test_batchnorm_matches_oracle(hgc, oracle, name, shape, kind):
    rng = np.random.default_rng(int(np.prod(shape)) + len(name))
    x = make_x(rng, shape, kind)
    eps = 0.0 if kind == "small" else 1e-5
    ref, rmean, rvar = oracle.batchnorm(x, eps)
    got, mean, var = run_bn(hgc, x, eps)
    # statistics: FP32 sums of up to 2048 values, then of the group values
    assert np.all(np.abs(mean - rmean) <= 1e-5 * np.abs(rmean) + 1e-6 * np.sqrt(rvar) + 1e-12), name
    assert np.all(np.abs(var - rvar) <= 2e-5 * rvar), name
    check_close(got, ref, what=name)


def test_shift_before_squaring_does_not_change_the_result(hgc, oracle):
    """Multiplying by 1/32 or 32 before the square and shifting back is exact in FP32."""
    rng = np.random.default_rng(5)
    x = make_x(rng, (3, 12, 40, 40), "image")
    base, m0, v0 = run_bn(hgc, x, 1e-5, 0)
    for s in (-5, 5):
        got, m, v = run_bn(hgc, x, 1e-5, s)
        assert np.array_equal(got.view(np.uint16), base.view(np.uint16))
        assert np.array_equal(m, m0) and np.array_equal(v, v0)
    # small data shifted up by 32: same statement
    xs = make_x(rng, (2, 4, 24, 24), "small")
    a, _, va = run_bn(hgc, xs, 0.0, 0)
    b, _, vb = run_bn(hgc, xs, 0.0, 5)
    assert np.array_equal(a.view(np.uint16), b.view(np.uint16)) and np.array_equal(va, vb)
    check_close(a, oracle.batchnorm(xs, 0.0)[0], what="small data")


def test_batchnorm_is_deterministic(hgc):
    rng = np.random.default_rng(6)
    x = make_x(rng, (8, 32, 28, 28), "mixed")
    a = run_bn(hgc, x, 1e-5)
    b = run_bn(hgc, x, 1e-5)
    assert np.array_equal(a[0].view(np.uint16), b[0].view(np.uint16))
    assert np.array_equal(a[1], b[1]) and np.array_equal(a[2], b[2])


def test_batchnorm_with_stored_statistics(hgc, oracle):
    rng = np.random.default_rng(7)
    x = make_x(rng, (3, 20, 17, 19), "mixed")
    mean = rng.normal(0, 2, 20).astype(np.float32).astype(np.float64)
    var = rng.uniform(0.25, 9, 20).astype(np.float32).astype(np.float64)
    ref, _, _ = oracle.batchnorm(x, 1e-3, mean, var)
    got, m, v = run_bn(hgc, x, 1e-3, stored=(mean, var))
    assert np.array_equal(m.astype(np.float64), mean) and np.array_equal(v.astype(np.float64), var)   # untouched
    check_close(got, ref, what="stored statistics")


def test_fold_matches_oracle_and_the_folded_convolution_normalises(hgc, oracle):
    import torch
    from paper_1901_00858_b200 import workloads
    rng = np.random.default_rng(8)
    n, c, h, w_, k = 2, 64, 14, 14, 96
    x, w, b = workloads.random_layer_tensors(rng, n, c, h, w_, k, 3, 3, 1)
    mean = rng.normal(0, 0.5, k).astype(np.float32)
    var = rng.uniform(0.25, 4, k).astype(np.float32)
    gamma = rng.uniform(0.5, 2, k).astype(np.float32)
    beta = rng.normal(0, 1, k).astype(np.float32)
    eps = 1e-5
    wr, br = oracle.bn_fold(w, b, mean, var, eps, gamma, beta)
    wd, bd = to_dev(w), to_dev(b)
    wo, bo = torch.empty_like(wd), torch.empty_like(bd)
    hgc.bn_fold(wd, bd, torch.from_numpy(mean).cuda(), torch.from_numpy(var).cuda(), eps, wo, bo,
                gamma=torch.from_numpy(gamma).cuda(), beta=torch.from_numpy(beta).cuda())
    torch.cuda.synchronize()
    gw, gb = to_host(wo), to_host(bo)
    # FP32 factor against the oracle's FP64 one: at most one FP16 ulp apart, nearly always equal
    for got, ref in ((gw, wr), (gb, br)):
        g64, r64 = got.astype(np.float64), ref.astype(np.float64)
        assert np.all(np.abs(g64 - r64) <= np.abs(r64) * 2.0 ** -10 + 2.0 ** -24)
        assert np.mean(got.view(np.uint16) == ref.view(np.uint16)) > 0.99
    # without bias, gamma, beta
    wo2, bo2 = torch.empty_like(wd), torch.empty_like(bd)
    hgc.bn_fold(wd, None, torch.from_numpy(mean).cuda(), torch.from_numpy(var).cuda(), eps, wo2, bo2)
    torch.cuda.synchronize()
    wr2, br2 = oracle.bn_fold(w, None, mean, var, eps)
    assert np.mean(to_host(wo2).view(np.uint16) == wr2.view(np.uint16)) > 0.99
    assert np.all(np.abs(to_host(bo2).astype(np.float64) - br2.astype(np.float64)) <= np.abs(br2.astype(np.float64)) * 2.0 ** -10 + 2.0 ** -24)
    # the folded layer on the GPU = conv -> stored-statistics batch norm -> scale/shift (+ ReLU) in FP64
    d = hgc.ConvDesc(n, c, h, w_, k, 3, 3, 1, 1)
    d.ensure_workspace()
    y = torch.full((n, k, h, w_), float("nan"), dtype=torch.float16, device="cuda")
    hgc.conv_forward(d, to_dev(x), wo, bo, y, True)
    torch.cuda.synchronize()
    xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (1, 1), (1, 1)))
    conv = np.zeros((n, k, h, w_))
    for r in range(3):
        for s in range(3):
            conv += np.einsum("nchw,kc->nkhw", xp[:, :, r:r + h, s:s + w_], w.astype(np.float64)[:, :, r, s])
    conv += b.astype(np.float64).reshape(1, k, 1, 1)
    a = gamma.astype(np.float64) / np.sqrt(var.astype(np.float64) + eps)
    want = np.maximum((conv - mean.reshape(1, k, 1, 1)) * a.reshape(1, k, 1, 1) + beta.reshape(1, k, 1, 1), 0.0)
    got = to_host(y).astype(np.float64)
    # the folded weights carry one extra FP16 rounding each: a slightly wider band than a plain layer
    assert np.all(np.abs(got - want) <= 4e-3 + 1e-2 * np.abs(want))
    d.close()


def test_batchnorm_on_more_than_2_31_elements(hgc, oracle):
    """700 x 64 x 224 x 224 (2.25 G elements).  Every plane holds every value 0..255 equally
    often, so the statistics have the closed form the oracle is pinned to (mean 255/2, variance
    (256^2 - 1)/12) and every output is one of 256 values, which the oracle computes from those
    statistics."""
    import torch
    n, c, h, w = 700, 64, 224, 224
    hw = h * w
    assert hw % 256 == 0 and n * c * hw > 2 ** 31
    plane = (torch.arange(hw, device="cuda") % 256).to(torch.float16)
    x = plane.expand(n, c, hw).contiguous().view(n, c, h, w)
    y = torch.empty_like(x)
    mean = torch.empty(c, dtype=torch.float32, device="cuda")
    var = torch.empty(c, dtype=torch.float32, device="cuda")
    ws = torch.empty(hgc.batchnorm_workspace_bytes(n, c, hw), dtype=torch.uint8, device="cuda")
    hgc.batchnorm_forward(x, y, 1e-5, mean, var, ws, shift_log2=-5)
    torch.cuda.synchronize()
    m, v = mean.cpu().numpy().astype(np.float64), var.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(m - 127.5) <= 127.5e-5) and np.all(np.abs(v - (256.0 ** 2 - 1) / 12) <= 2e-5 * 5461.25)
    # the 256 possible outputs, from the oracle with the closed-form statistics
    vals = np.arange(256, dtype=np.float64).reshape(1, 1, 16, 16).astype(np.float16)
    table, _, _ = oracle.batchnorm(vals, 1e-5, np.array([127.5]), np.array([(256.0 ** 2 - 1) / 12]))
    table = torch.from_numpy(table.reshape(256).view(np.int16)).cuda().view(torch.float16).float()
    # sampled outputs, including the very last ones
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    idx = torch.randint(0, n * c * hw, (200000,), device="cuda", generator=g)
    idx[:4] = torch.tensor([n * c * hw - 1, n * c * hw - 2, 2 ** 31 + 5, 0], device="cuda")
    got = y.view(-1)[idx].float()
    ref = table[(idx % hw) % 256]
    err = (got - ref).abs()
    assert bool((err <= 2e-3 + 1e-2 * ref.abs()).all()), float(err.max())
    del x, y
    torch.cuda.empty_cache()
