"""hgc_conv_forward_static: the entry point for callers that may not allocate device memory
(a plug-in inside a process whose device memory is fully owned by another framework, code that
runs where the allocator is off limits).  Its scratch is a fixed array inside the library, so
the test checks what such a caller relies on: the result equals the ordinary entry point's,
also on a second call that finds the first call's leftovers in the shared array.

Collected last on purpose (file name), and it passes both alone and after the other tests."""
import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import check_close, params_dict, run_layer, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _static_forward(hgc, args, x, w, b, relu):
    import torch
    params = hgc.hgc_conv_params(args["n"], args["c"], args["h"], args["w"], args["k"], args["r"], args["s"],
                                 args["pad_h"], args["pad_w"], args["stride_h"], args["stride_w"],
                                 args["dil_h"], args["dil_w"], args["group"], 0)
    d = hgc.ConvDesc(**args)          # only to learn the output shape
    n, k, p, q = d.output_dims()
    d.close()
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    y = torch.full((n, k, p, q), float("nan"), dtype=torch.float16, device="cuda")
    hgc.conv_forward_static(params, xd, wd, bd, y, relu)
    torch.cuda.synchronize()
    return to_host(y)


def test_static_scratch_matches_ordinary_entry_point_twice_in_a_row(hgc):
    rng = np.random.default_rng(77)
    # two different layers back to back: the second call reuses the array the first one filled
    # (a larger layer first, so that stale weights/input lie beyond what the second call rewrites)
    layers = [params_dict(3, 48, 20, 22, 72, 3, 3, 1, 1), params_dict(2, 32, 9, 9, 40, 3, 3, 1, 1, 2, 2)]
    for args in layers:
        x, w, b = workloads.random_layer_tensors(rng, args["n"], args["c"], args["h"], args["w"], args["k"],
                                                 args["r"], args["s"], args["group"])
        want, path = run_layer(hgc, args, x, w, b, True)
        assert path == hgc.HGC_PATH_IGEMM
        got = _static_forward(hgc, args, x, w, b, True)
        check_close(got, want, what=f"static scratch {args}")
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16))   # same kernels: same bits


def test_static_scratch_rejects_what_it_cannot_hold(hgc):
    import torch
    dummy = torch.zeros(64, dtype=torch.float16, device="cuda")
    # two groups of 3 channels: not a layer the tensor-core path takes, so this entry point has
    # no variant for it
    small = hgc.hgc_conv_params(1, 6, 8, 8, 4, 3, 3, 1, 1, 1, 1, 1, 1, 2, 0)
    with pytest.raises(hgc.HgcError) as e:
        hgc.conv_forward_static(small, dummy, dummy, None, dummy, False)
    assert e.value.status == hgc.HGC_UNSUPPORTED
    # NHWC copy of the input alone is 64 x 64 x 112 x 112 x 2 B = 98 MiB > 32 MiB: refused before
    # anything is queued (the pointers are never dereferenced)
    big = hgc.hgc_conv_params(64, 64, 112, 112, 64, 3, 3, 1, 1, 1, 1, 1, 1, 1, 0)
    with pytest.raises(hgc.HgcError) as e:
        hgc.conv_forward_static(big, dummy, dummy, None, dummy, False)
    assert e.value.status == hgc.HGC_NO_WORKSPACE
