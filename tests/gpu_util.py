"""Helpers for the GPU parity tests: run a layer through the C ABI, compare with the oracle."""
import numpy as np

ABS_TOL = 2e-3
REL_TOL = 1e-2


def to_dev(a):
    import torch
    if a is None:
        return None
    return torch.from_numpy(np.ascontiguousarray(a).view(np.uint16).copy()).view(torch.float16).cuda()


def to_host(t):
    import torch
    return t.cpu().view(torch.int16).numpy().view(np.float16)


GUARD_BYTES = 4096
GUARD_BYTE = 0x7E     # 0x7E7E is a binary16 NaN: a guarded buffer starts out NaN-filled


def guarded(nbytes):
    """A device buffer of `nbytes` bytes (rounded up to 256) between two guard bands filled with a
    fixed byte pattern, all of it inside one allocation.  Returns (whole, inner)."""
    import torch
    inner = (int(nbytes) + 255) // 256 * 256
    whole = torch.full((inner + 2 * GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
    return whole, whole[GUARD_BYTES:GUARD_BYTES + inner]


def check_guards(whole, what=""):
    """The bands before and after a guarded buffer still hold the pattern: nothing was stored
    outside the buffer."""
    n = whole.numel()
    assert bool((whole[:GUARD_BYTES] == GUARD_BYTE).all()), f"{what}: bytes BEFORE the buffer were overwritten"
    assert bool((whole[n - GUARD_BYTES:] == GUARD_BYTE).all()), f"{what}: bytes AFTER the buffer were overwritten"


def guarded_output(shape):
    """A NaN-filled float16 output tensor of `shape` between guard bands.  Returns (whole, y)."""
    import torch
    count = int(np.prod(shape))
    whole, inner = guarded(count * 2)
    return whole, inner[:count * 2].view(torch.float16).view(*shape)


def attach_guarded_workspace(d, host=False):
    """Attaches a workspace between guard bands (its bytes start out as the NaN pattern, so a read
    of something the library never wrote shows up in the result).  Returns the whole buffer or None."""
    need = d.host_workspace_bytes() if host else d.workspace_bytes()
    if need == 0:
        return None
    whole, inner = guarded(need)
    d.set_workspace(inner)
    return whole


def run_layer(hgc, args, x, w, b, relu, flags=0, register_weights=False):
    """args: dict of hgc_conv_params fields (without flags).  Returns (y float16 ndarray, path).
    The output and the workspace sit between guard bands that must survive the call."""
    import torch
    d = hgc.ConvDesc(flags=flags, **args)
    n, k, p, q = d.output_dims()
    ws_whole = attach_guarded_workspace(d)
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    # canary-filled output: an element the kernel does not write stays NaN and fails the check
    y_whole, y = guarded_output((n, k, p, q))
    if register_weights:
        d.set_weights(wd)
    hgc.conv_forward(d, xd, wd, bd, y, relu)
    torch.cuda.synchronize()
    assert d.last_device_status() == hgc.HGC_OK
    check_guards(y_whole, f"y of {args}")
    if ws_whole is not None:
        check_guards(ws_whole, f"workspace of {args}")
    path = d.path()
    out = to_host(y)
    d.close()
    return out, path


def max_ulp_error(got, ref, floor=2.0 ** -6):
    """Largest distance in binary16 units in the last place between got and ref over the outputs
    with |ref| >= floor (below that an absolute error of a rounding tie is many ulps)."""
    g = got.ravel().view(np.uint16).astype(np.int32)
    r = ref.ravel().view(np.uint16).astype(np.int32)
    big = np.abs(ref.ravel().astype(np.float32)) >= floor
    if not big.any():
        return 0
    # sign-magnitude -> a monotonic integer scale
    gm = np.where(g & 0x8000, -(g & 0x7FFF), g & 0x7FFF)
    rm = np.where(r & 0x8000, -(r & 0x7FFF), r & 0x7FFF)
    return int(np.abs(gm - rm)[big].max())


def check_close(got, ref, what=""):
    """|got - ref| <= 2e-3 + 1e-2*|ref| for every element (ref = oracle's fp16 output).
    Returns (max_abs_err, fraction bit-identical)."""
    g = got.astype(np.float64).ravel()
    r = ref.astype(np.float64).ravel()
    assert g.shape == r.shape, (what, got.shape, ref.shape)
    assert np.all(np.isfinite(r)), what
    assert np.all(np.isfinite(g)), f"{what}: non-finite output (unwritten or NaN)"
    err = np.abs(g - r)
    tol = ABS_TOL + REL_TOL * np.abs(r)
    bad = np.nonzero(err > tol)[0]
    assert bad.size == 0, (f"{what}: {bad.size} of {g.size} outside tolerance; first at flat index "
                           f"{bad[0]}: got {g[bad[0]]}, ref {r[bad[0]]}")
    same = float(np.mean(got.ravel().view(np.uint16) == ref.ravel().view(np.uint16))) if g.size else 1.0
    return (float(err.max()) if g.size else 0.0), same


def params_dict(n, c, h, w, k, r, s, pad_h=0, pad_w=0, stride_h=1, stride_w=1, dil_h=1, dil_w=1, group=1):
    return dict(n=n, c=c, h=h, w=w, k=k, r=r, s=s, pad_h=pad_h, pad_w=pad_w, stride_h=stride_h,
                stride_w=stride_w, dil_h=dil_h, dil_w=dil_w, group=group)


def layer_args(batch, l):
    return params_dict(batch, l.c, l.h, l.h, l.k, l.r, l.r, l.pad, l.pad, l.stride, l.stride, l.dil, l.dil,
                       l.group)


def sample_coords(rng, n, k, p, q, nrandom=16384):
    """Output coordinates for sampled checks: image/channel/plane corners and borders plus
    uniformly random points."""
    ns = sorted({0, n - 1, n // 2})
    ks = sorted({0, 1 % k, k // 2, k - 1})
    ps = sorted({0, 1 % p, p // 2, p - 2 if p > 1 else 0, p - 1})
    qs = sorted({0, 1 % q, q // 2, q - 2 if q > 1 else 0, q - 1})
    grid = np.array([(a, b, c, d) for a in ns for b in ks for c in ps for d in qs], dtype=np.int64)
    rnd = np.stack([rng.integers(0, n, nrandom), rng.integers(0, k, nrandom), rng.integers(0, p, nrandom),
                    rng.integers(0, q, nrandom)], axis=1).astype(np.int64)
    return np.concatenate([grid, rnd], axis=0)
