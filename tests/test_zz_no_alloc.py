"""The allocation-free host entry point, lordba_adapter_forward_host_static, against
lordba_adapter_forward_host and against the oracle.

Some callers hold their activations in host memory and cannot ask for device memory at the time
of the call (an allocation may stall the device, or the surrounding framework owns all of it).
For them the library stages x and y in a fixed buffer that ships inside its own image.  This file
checks, through the C ABI, that the result is bit for bit that of the workspace-taking entry point
(both run the same kernel on the same bytes), twice in a row on the shared buffer (the second call
is smaller, so that leftovers of the first would show), that it matches the oracle, that a call on
a stream of the caller's works, and that a call too large for the buffer is refused without
touching anything.

Collected last on purpose: a run that stops at the first failure has then already run every
other test.
"""
import numpy as np
import pytest
import torch

from paper_2605_24058_b200 import lordba, workloads
from gpu_util import DeviceProj, assert_close, np_to_torch, oracle_forward

pytestmark = pytest.mark.gpu


def _both_entries(p, stream=None):
    """Run one projection through both host entry points; return (static result, workspace result)."""
    d = DeviceProj(p)
    xh = np_to_torch(p.x, p.dtype, "cpu").pin_memory()
    y_static = np_to_torch(p.y, p.dtype, "cpu").pin_memory()
    y_ws = np_to_torch(p.y, p.dtype, "cpu").pin_memory()
    torch.cuda.synchronize()
    lordba.adapter_forward_host_static(xh, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, y_static, p.r,
                                       stream=stream)
    torch.cuda.synchronize()
    code = lordba.BF16 if p.dtype == "bf16" else lordba.F32
    ws = torch.empty(lordba.host_workspace_bytes(p.T, p.d_in, p.d_out, code), dtype=torch.uint8,
                     device="cuda:0")
    lordba.adapter_forward_host(xh, d.packed_A, d.packed_B, d.s_in, d.s_r, d.s_out, y_ws, p.r, ws, stream=stream)
    torch.cuda.synchronize()
    assert lordba.device_status() == 0
    return y_static, y_ws


def test_static_scratch_entry_matches_workspace_entry_twice_in_a_row(oracle):
    lordba.set_variant(lordba.VARIANT_AUTO)
    first = workloads.make_projection(1024, 1536, 16, 300, "bf16", seed=41)
    second = workloads.make_projection(512, 384, 8, 77, "f32", seed=42, scales="tiny")
    for p in (first, second):
        y_static, y_ws = _both_entries(p)
        want = oracle_forward(oracle, p)
        assert not np.array_equal(want, p.y_f64()), "the adapter term must have changed y"
        # same kernel, same bytes: the two entries agree bit for bit
        assert torch.equal(y_static, y_ws), "static scratch entry differs from the workspace entry (%s)" % p.dtype
        assert_close(y_static.to(torch.float64).numpy(), want, p.dtype, "static scratch entry vs oracle, %s" % p.dtype)


def test_static_scratch_entry_on_a_stream_of_the_caller(oracle):
    p = workloads.make_projection(768, 1024, 16, 200, "bf16", seed=44)
    stream = torch.cuda.Stream()
    y_static, y_ws = _both_entries(p, stream=stream)
    assert torch.equal(y_static, y_ws)
    assert_close(y_static.to(torch.float64).numpy(), oracle_forward(oracle, p), "bf16", "static scratch entry, side stream")


def test_static_scratch_entry_refuses_what_does_not_fit():
    p = workloads.make_projection(64, 64, 8, 4, "bf16", seed=43)
    d = DeviceProj(p)
    T = lordba.STATIC_SCRATCH_BYTES // (2 * (4096 + 4096)) + 1          # one row too many
    assert lordba.host_workspace_bytes(T, 4096, 4096, lordba.BF16) > lordba.STATIC_SCRATCH_BYTES
    n0 = lordba.launch_count()
    rc = lordba.load().lordba_adapter_forward_host_static(
        1, d.packed_A.data_ptr(), d.packed_B.data_ptr(), d.s_in.data_ptr(), d.s_r.data_ptr(),
        d.s_out.data_ptr(), 1, T, 4096, 4096, 16, lordba.BF16, None)
    assert rc == 6 and lordba.launch_count() == n0
    assert "scratch" in lordba.status_string(6)
