"""A bounded device-side wait that runs out, watched from the host, without faulting anything.

Every wait of the tensor-core kernels on a copy or MMA barrier gives up after a cycle limit,
records a code in the device status word and lets the kernel run to its normal end.  The product
library's limit is about a second and nothing ever makes a wait run out, so this file loads the
test-hooks build of the same sources (``-DLORDBA_TEST_HOOKS``: the limit is about a millisecond
and ``lordba_test_skip_item`` makes the producer leave out the copy request of one pipeline item;
nothing is in flight for that item, so nothing can land late).  Checked: the call itself succeeds,
``lordba_device_status`` reports LORDBA_ETIMEOUT once and is clean afterwards, y holds either its
old values or the oracle's result and nothing else, and a following normal call is correct (for the
tcgen05 kernel this also shows that its tensor memory was freed).
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_2605_24058_b200 import build, lordba, workloads
from gpu_util import DeviceProj, assert_close, oracle_forward, torch_to_f64

pytestmark = pytest.mark.gpu

ETIMEOUT = 5


@pytest.fixture(scope="module")
def hooks():
    lib = lordba.bind(build.build_library(test_hooks=True))
    lib.lordba_test_skip_item.restype = ctypes.c_int
    lib.lordba_test_skip_item.argtypes = [ctypes.c_int]
    yield lib
    lib.lordba_test_skip_item(-1)
    lib.lordba_set_variant(lordba.VARIANT_AUTO)


def _forward(lib, d, T):
    p = d.proj()
    s = int(torch.cuda.current_stream().cuda_stream)
    return lib.lordba_adapter_forward_ex(ctypes.byref(p), T, lordba.BF16, s)


def _status(lib):
    code = ctypes.c_int(0)
    rc = lib.lordba_device_status(ctypes.byref(code), int(torch.cuda.current_stream().cuda_stream))
    return rc, int(code.value)


@pytest.mark.parametrize("kernel,skip", [("mma", 0), ("mma", 3), ("tc", 1)])
def test_a_wait_that_runs_out_is_reported_and_nothing_wrong_is_written(oracle, hooks, kernel, skip):
    # 150 token tiles of 16 (more than one wave: eight consumer warps, x items of 512 columns, so
    # d_in = 1024 is items 0 and 1 and the three y items of 512 columns are items 2, 3 and 4)
    T, d_in, d_out, r = 2400, 1024, 1536, 32
    p = workloads.make_projection(d_in, d_out, r, T, "bf16", seed=900)
    d = DeviceProj(p)
    y0 = d.y.clone()
    hooks.lordba_set_variant(lordba.VARIANT_MMA if kernel == "mma" else lordba.VARIANT_TC)
    assert _status(hooks) == (0, 0)

    hooks.lordba_test_skip_item(skip)
    assert _forward(hooks, d, T) == 0                     # the launch itself is fine
    rc, code = _status(hooks)                             # synchronises the stream
    assert rc == ETIMEOUT and code in (1, 2, 3, 4)
    assert _status(hooks) == (0, 0)                       # reading the word cleared it
    want = oracle_forward(oracle, p)
    got = torch_to_f64(d.y)
    if kernel == "mma" and skip == 3:
        # the second y item never arrived: its 512 columns keep their values, the rest is done
        assert torch.equal(d.y[:, 512:1024], y0[:, 512:1024])
        keep = np.ones(d_out, bool)
        keep[512:1024] = False
        assert_close(got[:, keep], want[:, keep], "bf16", "columns of the items that did arrive", scale_from=want)
    else:
        # an x item (chunk) never arrived: the first product is incomplete and nothing is written
        assert torch.equal(d.y, y0)

    # the same call without the hook, on the same library, is correct
    hooks.lordba_test_skip_item(-1)
    assert _forward(hooks, d, T) == 0
    assert _status(hooks) == (0, 0)
    if kernel == "mma" and skip == 3:
        assert_close(torch_to_f64(d.y[:, 512:1024]), want[:, 512:1024], "bf16", "after the timeout", scale_from=want)
    else:
        assert_close(torch_to_f64(d.y), want, "bf16", "after the timeout")


def test_a_wait_that_runs_out_in_a_cluster_stops_the_whole_cluster(oracle, hooks):
    """Eight token rows of a down projection: the CTAs of the tile share the first product as
    clusters.  With one CTA's first copy request left out, that CTA sends its partial sums to
    nobody, every CTA of every cluster gives up its wait for them, the status word reports it and
    y is untouched; the same call afterwards is correct."""
    T, d_in, d_out, r = 8, 11008, 4096, 16
    p = workloads.make_projection(d_in, d_out, r, T, "bf16", seed=901)
    d = DeviceProj(p)
    y0 = d.y.clone()
    hooks.lordba_set_variant(lordba.VARIANT_MMA)
    assert _status(hooks) == (0, 0)
    hooks.lordba_test_skip_item(0)
    assert _forward(hooks, d, T) == 0
    rc, code = _status(hooks)
    assert rc == ETIMEOUT and code in (1, 2, 3, 4)
    assert _status(hooks) == (0, 0)
    assert torch.equal(d.y, y0)
    hooks.lordba_test_skip_item(-1)
    assert _forward(hooks, d, T) == 0
    assert _status(hooks) == (0, 0)
    assert_close(torch_to_f64(d.y), oracle_forward(oracle, p), "bf16", "after the timeout in a cluster")


def test_product_library_has_no_hooks():
    assert not hasattr(lordba.load(), "lordba_test_skip_item")
