"""The allocation-free forward entry point (collected last on purpose).

hag_aggregate_fwd_static serves hosts that own all device memory themselves or
cannot afford the device-wide stall of a cudaMalloc, so it keeps the rows of the
aggregation nodes in an array inside the library image.  It must give exactly
what hag_aggregate_fwd gives with a caller-supplied workspace: on a first call,
on a second call that finds the previous call's rows still in the array, and
whether or not other tests used the library before in this process."""
import ctypes

import numpy as np
import pytest

import paper_1906_03707_b200 as hb
from paper_1906_03707_b200 import synth
from paper_1906_03707_b200.build import build as build_library

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

STATIC_SCRATCH_BYTES = 16 << 20


def _c_call(lib, h, reduce, dtype, x, out):
    stream = torch.cuda.current_stream().cuda_stream
    return lib.hag_aggregate_fwd_static(h._h, reduce, dtype, x.shape[1], x.data_ptr(), out.data_ptr(), stream)


def test_static_scratch_forward_equals_workspace_forward_twice_in_a_row():
    build_library()
    lib = hb.load_library()
    assert torch.cuda.is_available()
    w = synth.workload(2, scale=0.1)
    g = w.graph
    h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity).to_device(0)
    assert h.info()["num_agg"] > 0 and h.info()["num_levels"] > 1
    assert h.workspace_bytes(w.d) <= STATIC_SCRATCH_BYTES
    # two different inputs, one after the other: the second call meets the first call's rows in the array
    for call, (seed, reduce, name) in enumerate([(21, 0, "sum"), (22, 1, "mean")]):
        x = torch.from_numpy(synth.features(seed, g.n, w.d, "normal")).cuda()
        want = h.aggregate_fwd(x, name)
        got = torch.full_like(x, float("nan"))
        assert _c_call(lib, h, reduce, 0, x, got) == 0, f"call {call}"
        torch.cuda.synchronize()
        # same kernels, same order of additions: the tolerance of the parity tests (1e-5 * sum|terms| + 1e-6)
        # is met with zero difference
        assert torch.equal(got, want), f"call {call}"
    # bf16 storage goes through the same array
    xb = torch.from_numpy(synth.features(23, g.n, 64, "normal", "bf16")).cuda().to(torch.bfloat16)
    gotb = torch.empty_like(xb)
    assert _c_call(lib, h, 0, 1, xb, gotb) == 0
    torch.cuda.synchronize()
    assert torch.equal(gotb, h.aggregate_fwd(xb, "sum"))
    # the Python wrapper is the same call
    x = torch.from_numpy(synth.features(24, g.n, w.d, "normal")).cuda()
    out = torch.empty_like(x)
    assert torch.equal(h.aggregate_fwd_static(x, out, "mean"), h.aggregate_fwd(x, "mean"))


def test_static_scratch_rejects_what_does_not_fit_and_bad_arguments():
    build_library()
    lib = hb.load_library()
    w = synth.workload(2, scale=0.1)
    g = w.graph
    h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity).to_device(0)
    k = h.workspace_bytes(4) // 16                                  # scratch rows: aggregation nodes + long-row partials
    assert k >= h.info()["num_agg"] > 0
    d_big = 4 * (STATIC_SCRATCH_BYTES // (4 * k) // 4 + 1)          # smallest multiple of 4 that no longer fits
    assert k * d_big * 4 > STATIC_SCRATCH_BYTES
    x = torch.zeros((g.n, d_big), device="cuda")
    out = torch.full_like(x, 7.0)
    assert _c_call(lib, h, 0, 0, x, out) == 12                     # HAG_ERR_TOO_LARGE, nothing launched
    torch.cuda.synchronize()
    assert bool((out == 7.0).all())
    assert "scratch" in hb.status_str(12)
    d_fit = d_big - 4
    if d_fit > 0:
        xs = torch.from_numpy(synth.features(25, g.n, d_fit, "uniform")).cuda()
        os_ = torch.empty_like(xs)
        assert _c_call(lib, h, 0, 0, xs, os_) == 0
        torch.cuda.synchronize()
        assert torch.equal(os_, h.aggregate_fwd(xs, "sum"))
    small = torch.zeros((g.n, 16), device="cuda")
    assert lib.hag_aggregate_fwd_static(None, 0, 0, 16, small.data_ptr(), small.data_ptr(), None) == 1
    assert lib.hag_aggregate_fwd_static(h._h, 0, 0, 16, small.data_ptr(), small.data_ptr(), None) == 2   # out aliases x
    assert lib.hag_aggregate_fwd_static(h._h, 0, 3, 16, small.data_ptr(), out.data_ptr(), None) == 7     # dtype
    host_only = hb.Hag.build(g.row_ptr, g.col_idx, 10)
    assert lib.hag_aggregate_fwd_static(host_only._h, 0, 0, 16, small.data_ptr(), out.data_ptr(), None) == 11
