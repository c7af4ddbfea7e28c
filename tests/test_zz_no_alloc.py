"""hgc_conv_forward_static: the entry point for callers that may not allocate device memory
(a plug-in inside a process whose device memory is fully owned by another framework, code that
runs where the allocator is off limits).  Its scratch is a fixed array inside the library, so
the tests check what such a caller relies on: the result is the layer the oracle computes and
equals the ordinary entry point's, also on calls that find an earlier, larger call's leftovers
in the shared array, in every way the tensor-core path lays its scratch out; and the call does
not change the amount of free device memory.

Collected last on purpose (file name), and it passes both alone and after the other tests."""
import numpy as np
import pytest

from paper_1901_00858_b200 import workloads
from gpu_util import check_close, guarded_output, check_guards, params_dict, run_layer, to_dev, to_host

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def hgc():
    import torch
    assert torch.cuda.is_available()
    from paper_1901_00858_b200 import binding
    binding.lib()
    return binding


def _params(hgc, args, flags=0):
    return hgc.hgc_conv_params(args["n"], args["c"], args["h"], args["w"], args["k"], args["r"], args["s"],
                               args["pad_h"], args["pad_w"], args["stride_h"], args["stride_w"],
                               args["dil_h"], args["dil_w"], args["group"], flags)


def _static_forward(hgc, args, x, w, b, relu, free_must_not_change=False):
    import torch
    d = hgc.ConvDesc(**args)          # only to learn the output shape
    n, k, p, q = d.output_dims()
    d.close()
    xd, wd, bd = to_dev(x), to_dev(w), to_dev(b)
    y_whole, y = guarded_output((n, k, p, q))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    hgc.conv_forward_static(_params(hgc, args), xd, wd, bd, y, relu)
    torch.cuda.synchronize()
    free_after = torch.cuda.mem_get_info()[0]
    if free_must_not_change:
        assert free_after == free_before, "the call changed the amount of free device memory"
    check_guards(y_whole, f"static y {args}")
    return to_host(y)


# a larger layer first, so that stale weights, input copies and partial sums lie where the
# later, smaller calls put theirs (and beyond)
BIG = params_dict(3, 48, 40, 44, 72, 3, 3, 1, 1)
MODES = [
    ("NHWC copy, 3x3", params_dict(2, 32, 9, 9, 40, 3, 3, 1, 1, 2, 2)),
    ("stem 3->16 3x3 stride 1 (bordered copy, dense rows)", params_dict(2, 3, 20, 24, 16, 3, 3, 1, 1)),
    ("stem 3->16 3x3 stride 2 (expanded copy)", params_dict(2, 3, 21, 25, 16, 3, 3, 1, 1, 2, 2)),
    ("stem 7x7 stride 2 (windows of 4-channel pixels)", params_dict(1, 3, 30, 34, 24, 7, 7, 3, 3, 2, 2)),
    ("1x1 64->64 on 8x8 (x read in place)", params_dict(2, 64, 8, 8, 64, 1, 1)),
    ("inner product 4096->130 (split reduction: partial sums in the array)", params_dict(4, 4096, 1, 1, 130, 1, 1)),
    ("1x1 5x5 c4096 k96 (split reduction on a small plane)", params_dict(3, 4096, 5, 5, 96, 1, 1)),
    ("grouped 5x5", params_dict(1, 96, 13, 13, 64, 5, 5, 2, 2, 1, 1, 1, 1, 2)),
]


@pytest.mark.parametrize("name,args", MODES, ids=[m[0] for m in MODES])
def test_static_scratch_after_a_larger_call(hgc, oracle, name, args):
    rng = np.random.default_rng(77)
    for a in (BIG, args, args):          # the mode under test runs twice in a row after the large layer
        x, w, b = workloads.random_layer_tensors(rng, a["n"], a["c"], a["h"], a["w"], a["k"], a["r"], a["s"], a["group"])
        ref = oracle.conv_fast(oracle.ConvParams(**a), x, w, b, True)
        want, path = run_layer(hgc, a, x, w, b, True)
        assert path == hgc.HGC_PATH_IGEMM
        got = _static_forward(hgc, a, x, w, b, True, free_must_not_change=a is not BIG)
        check_close(got, ref, what=f"static scratch vs oracle: {name} {a}")
        assert np.array_equal(got.view(np.uint16), want.view(np.uint16)), name   # same kernels, same plan: same bits


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
    # channels-last tensors and the direct path are not what this entry point does: refused, not ignored
    ok = params_dict(1, 32, 8, 8, 32, 3, 3, 1, 1)
    for flags in (hgc.HGC_FLAG_X_NHWC, hgc.HGC_FLAG_Y_NHWC, hgc.HGC_FLAG_FORCE_DIRECT):
        with pytest.raises(hgc.HgcError) as e:
            hgc.conv_forward_static(_params(hgc, ok, flags), dummy, dummy, None, dummy, False)
        assert e.value.status == hgc.HGC_UNSUPPORTED
