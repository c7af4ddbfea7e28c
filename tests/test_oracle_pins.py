"""Pins for the CPU oracle: hand-worked examples, closed forms, library restatements and
invariants.  None of these calls the CUDA path; a dropped term, a wrong sign or index, a
transposed operand or a narrow accumulator in the oracle fails at least one of them."""
import json
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st
from scipy.signal import correlate2d

from paper_1901_00858_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
F16 = np.float16


def _bits_list(hexes):
    return np.array([int(h, 16) for h in hexes], dtype=np.uint16).view(F16)


def _example_tensors(ex, P):
    n, c, h, w = P.n, P.c, P.h, P.w
    wshape = (P.k, P.c // P.group, P.r, P.s)
    if "x_bits" in ex:
        x = _bits_list(ex["x_bits"]).reshape(n, c, h, w)
        wt = _bits_list(ex["w_bits"]).reshape(wshape)
        b = _bits_list(ex["bias_bits"]) if ex.get("bias_bits") else None
    elif "x_fill" in ex:
        x = np.full((n, c, h, w), ex["x_fill"], dtype=F16)
        wt = np.full(wshape, ex["w_fill"], dtype=F16)
        b = None if ex.get("bias") is None else np.array(ex["bias"], dtype=F16)
    else:
        x = np.array(ex["x"], dtype=F16).reshape(n, c, h, w)
        wt = np.array(ex["w"], dtype=F16).reshape(wshape)
        b = None if ex.get("bias") is None else np.array(ex["bias"], dtype=F16)
    return x, wt, b


def load_hand_examples():
    with open(os.path.join(GOLDEN, "hand_examples.json")) as f:
        return json.load(f)["examples"]


@pytest.mark.parametrize("ex", load_hand_examples(), ids=lambda e: e["id"])
@pytest.mark.parametrize("impl", ["conv_naive", "conv_fast", "conv_points"])
def test_hand_examples(oracle, ex, impl):
    P = oracle.ConvParams(**ex["params"])
    x, wt, b = _example_tensors(ex, P)
    if impl == "conv_points":
        shape = ex["out_shape"]
        coords = np.stack(np.meshgrid(*[np.arange(d) for d in shape], indexing="ij"), -1).reshape(-1, 4)
        y = oracle.conv_points(P, x, wt, b, ex["relu"], coords).reshape(shape)
    else:
        y = getattr(oracle, impl)(P, x, wt, b, ex["relu"])
    assert list(y.shape) == ex["out_shape"]
    if "expected_bits" in ex:
        assert [format(v, "04x") for v in y.view(np.uint16).ravel()] == ex["expected_bits"]
    else:
        assert y.ravel().astype(np.float64).tolist() == [float(v) for v in ex["expected"]]


def test_out_dim_golden(oracle):
    with open(os.path.join(GOLDEN, "out_dims.json")) as f:
        cases = json.load(f)["cases"]
    for size, k, pad, stride, dil, want in cases:
        assert oracle.out_dim(size, k, pad, stride, dil) == want, (size, k, pad, stride, dil)


@settings(max_examples=300, deadline=None)
@given(st.integers(1, 300), st.integers(1, 11), st.integers(0, 6), st.integers(1, 6), st.integers(1, 4))
def test_out_dim_counts_valid_window_positions(oracle, size, k, pad, stride, dil):
    """Brute force: count start positions t = -pad, -pad+stride, ... whose dilated window
    [t, t + dil*(k-1)] ends inside the padded line."""
    extent = dil * (k - 1) + 1
    count = 0
    t = -pad
    while t + extent <= size + pad:
        count += 1
        t += stride
    got = oracle.out_dim(size, k, pad, stride, dil)
    assert (got if got > 0 else 0) == count


def test_workload_planes_agree_with_formula(oracle):
    for wl in workloads.all_workloads():
        for l in wl.layers:
            assert oracle.out_dim(l.h, l.r, l.pad, l.stride, l.dil) == l.out, (wl.name, l.name)


# ---- binary16 conversion ---------------------------------------------------------------

def test_half_to_double_all_patterns(oracle):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = bits.view(F16).astype(np.float64)
    got = np.array([oracle.half_bits_to_double(int(b)) for b in bits])
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], want[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def test_double_to_half_roundtrip_midpoints_and_ties(oracle):
    bits = np.arange(0x7c01, dtype=np.uint32).astype(np.uint16)   # +0 .. +inf
    vals = bits.view(F16).astype(np.float64)
    d2h = oracle.double_to_half_bits
    for sgn, sbit in ((1.0, 0), (-1.0, 0x8000)):
        for i in range(0, len(bits) - 1, 7):           # every 7th pattern: 4500 cases per sign
            lo, hi = vals[i], vals[i + 1]
            assert d2h(sgn * lo) == (int(bits[i]) | sbit)
            if np.isinf(hi):
                mid = 65520.0
            else:
                mid = (lo + hi) / 2                       # exact in fp64
            even = int(bits[i]) if (bits[i] & 1) == 0 else int(bits[i + 1])
            assert d2h(sgn * mid) == (even | sbit), (i, mid)
            assert d2h(sgn * np.nextafter(mid, 0.0)) == (int(bits[i]) | sbit)
            assert d2h(sgn * np.nextafter(mid, np.inf)) == (int(bits[i + 1]) | sbit)
    assert d2h(65504.0) == 0x7bff and d2h(65519.99) == 0x7bff and d2h(65520.0) == 0x7c00
    assert d2h(1e300) == 0x7c00 and d2h(-1e300) == 0xfc00
    assert d2h(2.0 ** -25) == 0x0000            # tie between 0 and the smallest subnormal -> even
    assert d2h(np.nextafter(2.0 ** -25, 1.0)) == 0x0001
    assert d2h(-0.0) == 0x8000


def test_double_to_half_matches_numpy_on_random_doubles(oracle):
    rng = np.random.default_rng(7)
    v = np.concatenate([rng.normal(0, 1, 4000), rng.normal(0, 1e-6, 2000), rng.normal(0, 3e4, 2000)])
    want = v.astype(F16).view(np.uint16)
    got = np.array([oracle.double_to_half_bits(float(t)) for t in v], dtype=np.uint16)
    assert np.array_equal(got, want)


# ---- invariants and restatements ---------------------------------------------------------

def _dyadic(rng, shape, lo=-8, hi=8, scale=0.25):
    """Small dyadic rationals: every product and partial sum below is exact in fp64 and the
    results are exact in binary16, so equalities are bit-for-bit whatever the summation order."""
    return (rng.integers(lo, hi + 1, size=shape) * scale).astype(F16)


def test_1x1_conv_is_matmul(oracle):
    rng = np.random.default_rng(1)
    n, c, h, w, k = 2, 37, 5, 6, 19
    x = _dyadic(rng, (n, c, h, w), -4, 4, 0.5)
    wt = _dyadic(rng, (k, c, 1, 1), -4, 4, 0.5)
    b = _dyadic(rng, (k,))
    P = oracle.ConvParams(n, c, h, w, k, 1, 1)
    y = oracle.conv_fast(P, x, wt, b, relu=False)
    W = wt.reshape(k, c).astype(np.float64)
    want = np.empty((n, k, h, w))
    for i in range(n):
        want[i] = (W @ x[i].reshape(c, h * w).astype(np.float64) + b.astype(np.float64)[:, None]).reshape(k, h, w)
    assert np.abs(want).max() < 2048  # integers/halves below 2048 are exact in binary16
    assert np.array_equal(y.astype(np.float64), want)
    assert np.array_equal(oracle.conv_naive(P, x, wt, b, relu=False), y)


@pytest.mark.parametrize("r,dil", [(1, 1), (3, 1), (3, 2), (5, 1), (5, 3), (7, 2)])
def test_centred_delta_kernel_reproduces_input(oracle, r, dil):
    rng = np.random.default_rng(r * 10 + dil)
    n, c, h, w = 2, 3, 9, 11
    x = rng.uniform(-1, 1, (n, c, h, w)).astype(F16)
    wt = np.zeros((c, c, r, r), dtype=F16)
    for ch in range(c):
        wt[ch, ch, r // 2, r // 2] = 1
    pad = (r - 1) // 2 * dil
    P = oracle.ConvParams(n, c, h, w, c, r, r, pad, pad, 1, 1, dil, dil)
    for fn in (oracle.conv_naive, oracle.conv_fast):
        y = fn(P, x, wt)
        assert np.array_equal(y.view(np.uint16), x.view(np.uint16))


@pytest.mark.parametrize("r0,s0,pad,dil", [(0, 0, 1, 1), (2, 1, 1, 1), (0, 2, 0, 1), (2, 2, 2, 2), (1, 0, 3, 2)])
def test_shifted_delta_shifts_input(oracle, r0, s0, pad, dil):
    rng = np.random.default_rng(5)
    h, w, r = 8, 9, 3
    x = rng.uniform(-1, 1, (1, 1, h, w)).astype(F16)
    wt = np.zeros((1, 1, r, r), dtype=F16)
    wt[0, 0, r0, s0] = 1
    P = oracle.ConvParams(1, 1, h, w, 1, r, r, pad, pad, 1, 1, dil, dil)
    y = oracle.conv_fast(P, x, wt)
    dy, dx = r0 * dil - pad, s0 * dil - pad     # y[p,q] = X[p+dy, q+dx]
    want = np.zeros(y.shape, dtype=F16)
    for p in range(y.shape[2]):
        for q in range(y.shape[3]):
            i, j = p + dy, q + dx
            if 0 <= i < h and 0 <= j < w:
                want[0, 0, p, q] = x[0, 0, i, j]
    assert np.array_equal(y, want)
    assert np.array_equal(oracle.conv_naive(P, x, wt), want)


def test_linearity_in_x(oracle):
    rng = np.random.default_rng(2)
    n, c, h, w, k, r = 1, 4, 7, 8, 5, 3
    x1 = _dyadic(rng, (n, c, h, w), -4, 4, 0.5)
    x2 = _dyadic(rng, (n, c, h, w), -4, 4, 0.5)
    wt = _dyadic(rng, (k, c, r, r), -2, 2, 0.5)
    P = oracle.ConvParams(n, c, h, w, k, r, r, 1, 1, 2, 1, 1, 1)
    a = 2.0
    lhs = oracle.conv_fast(P, (a * x1.astype(np.float64) + x2.astype(np.float64)).astype(F16), wt)
    rhs = a * oracle.conv_fast(P, x1, wt).astype(np.float64) + oracle.conv_fast(P, x2, wt).astype(np.float64)
    assert np.array_equal(lhs.astype(np.float64), rhs)


@pytest.mark.parametrize("group", [2, 3, 6])
def test_groups_are_independent_convs_on_channel_slices(oracle, group):
    rng = np.random.default_rng(group)
    n, c, h, w, k, r = 2, 6, 6, 7, 12, 3
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, k, r, r, group)
    P = oracle.ConvParams(n, c, h, w, k, r, r, 1, 1, 1, 1, 1, 1, group)
    y = oracle.conv_fast(P, x, wt, b, relu=True)
    cg, kg = c // group, k // group
    for gi in range(group):
        Pg = oracle.ConvParams(n, cg, h, w, kg, r, r, 1, 1)
        yg = oracle.conv_fast(Pg, x[:, gi * cg:(gi + 1) * cg], wt[gi * kg:(gi + 1) * kg], b[gi * kg:(gi + 1) * kg], relu=True)
        assert np.array_equal(y[:, gi * kg:(gi + 1) * kg].view(np.uint16), yg.view(np.uint16))


@pytest.mark.parametrize("stride", [2, 3])
def test_stride_is_subsampling_of_stride_1(oracle, stride):
    rng = np.random.default_rng(stride)
    n, c, h, w, k, r = 1, 3, 11, 13, 4, 3
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, k, r, r, 1)
    y1 = oracle.conv_fast(oracle.ConvParams(n, c, h, w, k, r, r, 1, 1), x, wt, b)
    ys = oracle.conv_fast(oracle.ConvParams(n, c, h, w, k, r, r, 1, 1, stride, stride), x, wt, b)
    assert np.array_equal(ys.view(np.uint16), y1[:, :, ::stride, ::stride].view(np.uint16))


@pytest.mark.parametrize("dil", [2, 3])
def test_dilation_is_dense_conv_with_zero_stuffed_kernel(oracle, dil):
    rng = np.random.default_rng(dil)
    n, c, h, w, k, r = 1, 2, 12, 10, 3, 3
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, k, r, r, 1)
    ext = dil * (r - 1) + 1
    stuffed = np.zeros((k, c, ext, ext), dtype=F16)
    stuffed[:, :, ::dil, ::dil] = wt
    yd = oracle.conv_fast(oracle.ConvParams(n, c, h, w, k, r, r, 2, 2, 1, 1, dil, dil), x, wt, b)
    y1 = oracle.conv_fast(oracle.ConvParams(n, c, h, w, k, ext, ext, 2, 2), x, stuffed, b)
    assert np.array_equal(yd.view(np.uint16), y1.view(np.uint16))


@pytest.mark.parametrize("pad,stride", [(0, 1), (2, 1), (1, 2)])
def test_against_scipy_correlate2d(oracle, pad, stride):
    """Independent library restatement: per (k, c) plane correlation in float64, summed."""
    rng = np.random.default_rng(11 + pad)
    n, c, h, w, k, r, s = 2, 3, 9, 8, 4, 3, 2
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, k, r, s, 1)
    P = oracle.ConvParams(n, c, h, w, k, r, s, pad, pad, stride, stride)
    y = oracle.conv_fast(P, x, wt, b, relu=True)
    xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    want = np.empty(y.shape, dtype=F16)
    for i in range(n):
        for ko in range(k):
            acc = sum(correlate2d(xp[i, ci], wt[ko, ci].astype(np.float64), mode="valid") for ci in range(c))
            acc = acc[::stride, ::stride] + float(b[ko])
            want[i, ko] = np.maximum(acc, 0).astype(F16)
    # fp64 sums in another order: allow one binary16 step on rare ties, nothing more
    diff = np.abs(y.astype(np.float64) - want.astype(np.float64))
    assert np.all(diff <= np.spacing(np.abs(want).astype(F16)).astype(np.float64))
    assert np.mean(y.view(np.uint16) == want.view(np.uint16)) > 0.999


def test_pad_larger_than_kernel_gives_bias_border(oracle):
    x = np.ones((1, 1, 2, 2), dtype=F16)
    wt = np.ones((1, 1, 1, 1), dtype=F16)
    b = np.array([0.25], dtype=F16)
    y = oracle.conv_fast(oracle.ConvParams(1, 1, 2, 2, 1, 1, 1, 2, 3), x, wt, b)
    assert y.shape == (1, 1, 6, 8)
    want = np.full((6, 8), 0.25)
    want[2:4, 3:5] = 1.25
    assert np.array_equal(y[0, 0].astype(np.float64), want)


def test_invalid_parameters_are_rejected(oracle):
    x = np.zeros((1, 4, 4, 4), dtype=F16)
    with pytest.raises(ValueError):
        oracle.conv_fast(oracle.ConvParams(1, 4, 4, 4, 6, 3, 3, group=4), x, np.zeros((6, 1, 3, 3), dtype=F16))
    with pytest.raises(ValueError):
        oracle.conv_fast(oracle.ConvParams(1, 4, 4, 4, 4, 5, 5), x, np.zeros((4, 4, 5, 5), dtype=F16))


_desc = st.tuples(
    st.integers(1, 2), st.sampled_from([1, 2, 3, 4, 0]), st.integers(1, 6), st.integers(1, 6),
    st.integers(1, 12), st.integers(1, 12), st.integers(1, 5), st.integers(1, 5),
    st.integers(0, 3), st.integers(0, 3), st.integers(1, 4), st.integers(1, 4),
    st.integers(1, 3), st.integers(1, 3), st.booleans(), st.booleans(), st.integers(0, 2 ** 31))


@settings(max_examples=150, deadline=None)
@given(_desc)
def test_fast_is_bit_identical_to_naive(oracle, d):
    n, g, cg, kg, h, w, r, s, ph, pw, sh, sw, dh, dw, relu, has_bias, seed = d
    if g == 0:          # depthwise
        g, cg = cg * 3, 1
    c, k = g * cg, g * kg
    if oracle.out_dim(h, r, ph, sh, dh) < 1 or oracle.out_dim(w, s, pw, sw, dw) < 1:
        return
    rng = np.random.default_rng(seed)
    x, wt, b = workloads.random_layer_tensors(rng, n, c, h, w, k, r, s, g)
    P = oracle.ConvParams(n, c, h, w, k, r, s, ph, pw, sh, sw, dh, dw, g)
    bias = b if has_bias else None
    y0 = oracle.conv_naive(P, x, wt, bias, relu)
    y1 = oracle.conv_fast(P, x, wt, bias, relu)
    assert np.array_equal(y0.view(np.uint16), y1.view(np.uint16))
    coords = np.stack(np.meshgrid(*[np.arange(t) for t in y0.shape], indexing="ij"), -1).reshape(-1, 4)
    y2 = oracle.conv_points(P, x, wt, bias, relu, coords)
    assert np.array_equal(y2.view(np.uint16), y0.view(np.uint16).ravel())


def test_layout_definitions_round_trip(oracle):
    rng = np.random.default_rng(3)
    x = rng.uniform(-1, 1, (2, 5, 3, 4)).astype(F16)
    xp = oracle.nchw_to_nhwc(x, 8)
    assert xp.shape == (2, 3, 4, 8) and np.all(xp[..., 5:] == 0)
    assert xp[1, 2, 3, 4] == x[1, 4, 2, 3]
    assert np.array_equal(oracle.nhwc_to_nchw(xp, 5), x)
    wt = rng.uniform(-1, 1, (6, 2, 3, 3)).astype(F16)
    wp = oracle.repack_weights(wt, 3, 8)
    assert wp.shape == (3, 2, 3, 3, 8)
    assert wp[2, 1, 0, 2, 1] == wt[5, 1, 0, 2] and np.all(wp[..., 2:] == 0)


# ---- the converter's cast and the inner-product layer (oracle functions added for the next rows) ----

def test_cast_matches_numpy_on_every_class_of_value(oracle):
    """ref_cast_f32_to_f16 against numpy's float32 -> float16 conversion (an independent
    implementation of IEEE round-to-nearest-even): normals, subnormals, ties, overflow, signed
    zeros, infinities; NaN stays NaN."""
    rng = np.random.default_rng(11)
    parts = [
        rng.normal(0, 1, 20000), rng.normal(0, 300, 20000), rng.uniform(-70000, 70000, 20000),
        rng.uniform(-1e-4, 1e-4, 20000), rng.uniform(-1e-7, 1e-7, 20000),   # fp16 subnormals and below
        np.array([0.0, -0.0, np.inf, -np.inf, 65504.0, 65519.996, 65520.0, -65520.0, 65536.0, 1e30, -1e30,
                  2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0000001, 3 * 2.0 ** -25, 2.0 ** -14, 2.0 ** -14 - 2.0 ** -25]),
        # exact ties between neighbouring fp16 values in several binades: (m + 0.5) * 2^(e-10)
        np.array([(1024 + m + 0.5) * 2.0 ** (e - 10) for e in (-14, -3, 0, 7, 15) for m in (0, 1, 2, 511, 1022)]),
    ]
    src = np.concatenate(parts).astype(np.float32)
    got, n_over = oracle.cast_f32_to_f16(src)
    with np.errstate(over="ignore"):
        want = src.astype(np.float16)
    assert np.array_equal(got.view(np.uint16), want.view(np.uint16))
    finite_in = np.isfinite(src)
    assert n_over == int(np.count_nonzero(finite_in & np.isinf(want)))
    assert n_over > 0
    nan_out, n2 = oracle.cast_f32_to_f16(np.array([np.nan, -np.nan, 1.0], dtype=np.float32))
    assert np.isnan(nan_out[0]) and np.isnan(nan_out[1]) and nan_out[2] == 1.0 and n2 == 0


def test_cast_is_the_identity_on_values_that_are_already_fp16(oracle):
    bits = np.arange(0, 0x10000, dtype=np.uint32).astype(np.uint16)
    h = bits.view(np.float16)
    keep = ~np.isnan(h)
    got, n_over = oracle.cast_f32_to_f16(h[keep].astype(np.float32))
    assert np.array_equal(got.view(np.uint16), bits[keep]) and n_over == 0


def test_inner_product_matches_float64_matmul(oracle):
    """y = x W^T + b in float64 (numpy matmul), rounded once: the oracle's loop must agree
    bit for bit wherever the float64 sums agree, i.e. within one fp16 ulp everywhere and
    exactly on small integer-valued data where no rounding happens at all."""
    rng = np.random.default_rng(3)
    x = rng.integers(-4, 5, size=(7, 33)).astype(F16)
    w = rng.integers(-3, 4, size=(11, 33)).astype(F16)
    b = rng.integers(-5, 6, size=(11,)).astype(F16)
    want = (x.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64))
    for relu in (False, True):
        ref = np.maximum(want, 0) if relu else want
        got = oracle.inner_product(x, w, b, relu)
        assert np.array_equal(got.astype(np.float64), ref)     # integers < 2048: exact in fp16
    xr = rng.uniform(-1, 1, size=(5, 400)).astype(F16)
    wr = rng.normal(0, 0.07, size=(9, 400)).astype(F16)
    got = oracle.inner_product(xr, wr, None, False).astype(np.float64)
    want = xr.astype(np.float64) @ wr.astype(np.float64).T
    assert np.all(np.abs(got - want) <= np.abs(want) * 2.0 ** -11 + 2.0 ** -25)   # half an ulp of fp16


def test_inner_product_is_a_1x1_convolution_on_a_1x1_plane(oracle):
    rng = np.random.default_rng(4)
    x = rng.uniform(-1, 1, size=(6, 50)).astype(F16)
    w = rng.normal(0, 0.2, size=(13, 50)).astype(F16)
    b = rng.uniform(-0.1, 0.1, size=(13,)).astype(F16)
    P = oracle.ConvParams(6, 50, 1, 1, 13, 1, 1, 0, 0, 1, 1, 1, 1, 1)
    conv = oracle.conv_naive(P, x.reshape(6, 50, 1, 1), w.reshape(13, 50, 1, 1), b, True)
    fc = oracle.inner_product(x, w, b, True)
    assert np.array_equal(conv.reshape(6, 13).view(np.uint16), fc.view(np.uint16))


def test_wide_accumulation_in_the_inner_product(oracle):
    """4096 ones times ones: a sum carried in FP16 stalls at 2048; the layer must give 4096."""
    x = np.ones((1, 4096), dtype=F16)
    w = np.ones((2, 4096), dtype=F16)
    assert np.array_equal(oracle.inner_product(x, w, None, False), np.full((1, 2), 4096, dtype=F16))


# ---- batch norm (Section 3.1) ------------------------------------------------------------------

def test_batchnorm_hand_examples(oracle):
    """{1,2,3,4}: mean 5/2, variance 5/4, outputs -+3/sqrt(5) and -+1/sqrt(5).  Two images of one
    pixel {0, 2}: mean 1, variance 1, outputs -1 and 1 (the statistics run over images too)."""
    y, m, v = oracle.batchnorm(np.array([[[[1, 2], [3, 4]]]], dtype=F16), 0.0)
    assert m[0] == 2.5 and v[0] == 1.25
    want = np.array([-3, -1, 1, 3], dtype=np.float64) / np.sqrt(5.0)
    assert np.array_equal(y.ravel(), want.astype(F16))
    y, m, v = oracle.batchnorm(np.array([[[[0]]], [[[2]]]], dtype=F16), 0.0)
    assert (m[0], v[0]) == (1.0, 1.0) and y.ravel().tolist() == [-1.0, 1.0]
    # eps enters under the root: {0, 2} with eps = 3 gives -+1/2
    y, _, _ = oracle.batchnorm(np.array([[[[0]]], [[[2]]]], dtype=F16), 3.0)
    assert y.ravel().tolist() == [-0.5, 0.5]


def test_batchnorm_matches_float64_numpy_per_channel(oracle):
    rng = np.random.default_rng(11)
    x = (rng.normal(0, 1, size=(3, 5, 7, 6)) * np.array([1, 4, 0.25, 10, 1]).reshape(1, 5, 1, 1)
         + np.array([0, 3, -1, 20, 0.5]).reshape(1, 5, 1, 1)).astype(F16)
    eps = 1e-5
    y, m, v = oracle.batchnorm(x, eps)
    xd = x.astype(np.float64)
    mean = xd.mean(axis=(0, 2, 3))
    var = xd.var(axis=(0, 2, 3))          # biased, like the layer
    assert np.allclose(m, mean, rtol=1e-13, atol=1e-15) and np.allclose(v, var, rtol=1e-12, atol=0)
    want = (xd - mean.reshape(1, 5, 1, 1)) / np.sqrt(var.reshape(1, 5, 1, 1) + eps)
    # both are fp64 before the one rounding; different summation orders can flip a rare tie
    err = np.abs(y.astype(np.float64) - want)
    assert np.all(err <= np.abs(want) * 2.0 ** -11 + 2.0 ** -25)
    assert np.mean(y.view(np.uint16) == want.astype(F16).view(np.uint16)) > 0.999


def test_batchnorm_output_has_zero_mean_and_unit_variance(oracle):
    rng = np.random.default_rng(12)
    x = rng.uniform(0, 255, size=(4, 3, 16, 16)).astype(F16)
    y, _, _ = oracle.batchnorm(x, 0.0)
    yd = y.astype(np.float64)
    assert np.all(np.abs(yd.mean(axis=(0, 2, 3))) < 2e-4)
    assert np.all(np.abs(yd.var(axis=(0, 2, 3)) - 1.0) < 2e-3)


def test_batchnorm_ignores_exact_shifts_and_positive_scales(oracle):
    """x + 16 and 4 * x are exact in fp16 for multiples of 1/64 in [0, 8): the normalised output
    has the same bits (eps = 0)."""
    rng = np.random.default_rng(13)
    x = (rng.integers(0, 512, size=(2, 4, 9, 5)) / 64.0).astype(F16)
    base, _, _ = oracle.batchnorm(x, 0.0)
    shifted, ms, _ = oracle.batchnorm((x.astype(np.float64) + 16.0).astype(F16), 0.0)
    scaled, _, vs = oracle.batchnorm((x.astype(np.float64) * 4.0).astype(F16), 0.0)
    assert np.array_equal(base.view(np.uint16), shifted.view(np.uint16))
    assert np.array_equal(base.view(np.uint16), scaled.view(np.uint16))
    # a negative scale mirrors the output
    neg, _, _ = oracle.batchnorm((-x.astype(np.float64)).astype(F16), 0.0)
    assert np.array_equal((-base).view(np.uint16), neg.view(np.uint16))


def test_batchnorm_image_valued_data_does_not_overflow(oracle):
    """The case the section names: pixel values 0..255, many of them.  Every value 0..255 equally
    often: mean 255/2, variance (256^2 - 1)/12.  (A sum, or a square, carried in FP16 would have
    left the finite range after a few hundred values.)"""
    x = np.tile(np.arange(256, dtype=np.float64), 64).reshape(4, 1, 64, 64).astype(F16)
    y, m, v = oracle.batchnorm(x, 0.0)
    assert m[0] == 127.5 and v[0] == (256.0 ** 2 - 1.0) / 12.0
    assert np.all(np.isfinite(y.astype(np.float64)))
    assert y.ravel()[0] == F16(-127.5 / np.sqrt(v[0])) and y.ravel()[255] == F16(127.5 / np.sqrt(v[0]))


def test_batchnorm_with_stored_statistics(oracle):
    rng = np.random.default_rng(14)
    x = rng.normal(2, 3, size=(2, 6, 5, 5)).astype(F16)
    y0, m, v = oracle.batchnorm(x, 1e-3)
    y1, m1, v1 = oracle.batchnorm(x, 1e-3, m, v)          # its own statistics handed back in
    assert np.array_equal(y0.view(np.uint16), y1.view(np.uint16)) and np.array_equal(m, m1) and np.array_equal(v, v1)
    mean = rng.normal(0, 1, 6)
    var = rng.uniform(0.5, 2, 6)
    y2, _, _ = oracle.batchnorm(x, 1e-3, mean, var)
    want = (x.astype(np.float64) - mean.reshape(1, 6, 1, 1)) / np.sqrt(var.reshape(1, 6, 1, 1) + 1e-3)
    assert np.array_equal(y2.view(np.uint16), want.astype(F16).view(np.uint16))


def test_bn_fold_restates_the_formula_and_commutes_with_a_1x1_convolution(oracle):
    rng = np.random.default_rng(15)
    k, c = 7, 24
    w = rng.normal(0, 0.2, size=(k, c, 1, 1)).astype(F16)
    b = rng.uniform(-0.5, 0.5, size=k).astype(F16)
    mean, var = rng.normal(0, 1, k), rng.uniform(0.25, 4, k)
    gamma, beta = rng.uniform(0.5, 2, k), rng.normal(0, 1, k)
    eps = 1e-5
    wf, bf = oracle.bn_fold(w, b, mean, var, eps, gamma, beta)
    a = gamma / np.sqrt(var + eps)
    assert np.array_equal(wf.view(np.uint16), (w.astype(np.float64) * a.reshape(k, 1, 1, 1)).astype(F16).view(np.uint16))
    assert np.array_equal(bf.view(np.uint16), ((b.astype(np.float64) - mean) * a + beta).astype(F16).view(np.uint16))
    # defaults: gamma = 1, beta = 0, no bias
    wf1, bf1 = oracle.bn_fold(w, None, mean, var, eps)
    a1 = 1.0 / np.sqrt(var + eps)
    assert np.array_equal(wf1.view(np.uint16), (w.astype(np.float64) * a1.reshape(k, 1, 1, 1)).astype(F16).view(np.uint16))
    assert np.array_equal(bf1.view(np.uint16), (-mean * a1).astype(F16).view(np.uint16))
    # the folded layer computes what conv -> batch norm (stored statistics) -> scale/shift computes
    x = rng.uniform(-1, 1, size=(3, c, 4, 4)).astype(F16)
    P = oracle.ConvParams(3, c, 4, 4, k, 1, 1, 0, 0, 1, 1, 1, 1, 1)
    folded = oracle.conv_naive(P, x, wf, bf, False).astype(np.float64)
    conv = np.einsum("nchw,kc->nkhw", x.astype(np.float64), w.astype(np.float64).reshape(k, c)) + \
        b.astype(np.float64).reshape(1, k, 1, 1)
    want = (conv - mean.reshape(1, k, 1, 1)) * a.reshape(1, k, 1, 1) + beta.reshape(1, k, 1, 1)
    assert np.all(np.abs(folded - want) <= 2e-3 + 1e-2 * np.abs(want))
