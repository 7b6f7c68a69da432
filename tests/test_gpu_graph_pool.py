"""GPU parity of the graph read-out (the mean-pooling layer of Section 5.1) against
the fp64 oracle, element by element, through the C ABI.

Tolerances as for the aggregation: fp32 |gpu - oracle| <= 1e-5 * Sigma|terms| + 1e-6;
bf16 the minimum of 1e-2 * Sigma|terms| + 1e-6 and the fp32 bound plus one bf16
output rounding.  The backward pass is a scaled copy: one rounding for the factor,
one for the product (and one to bf16).
"""
import ctypes

import numpy as np
import pytest

import paper_1906_03707_b200 as hb
from oracle import oracle as O
from paper_1906_03707_b200 import synth
from paper_1906_03707_b200.build import build as build_library

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _library():
    build_library()
    hb.load_library()
    assert torch.cuda.is_available(), "the parity tests need a CUDA device"


def _dev(a, dtype):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def _host(t):
    return t.float().cpu().numpy().astype(np.float64)


def _bound(scale, want, dtype):
    if dtype == "f32":
        return 1e-5 * scale + 1e-6
    return np.minimum(1e-2 * scale + 1e-6, 1e-5 * scale + 1e-6 + 2.0 ** -8 * np.abs(want))


def _segments(seed, m, max_len, lead=0, empty_every=0):
    rng = np.random.default_rng(seed)
    lens = rng.integers(1, max_len + 1, size=m)
    if empty_every:
        lens[::empty_every] = 0
    return (lead + np.concatenate([[0], np.cumsum(lens)])).astype(np.int32)


def _check(seg_ptr, n_rows, d, dtype, reduce, seed, dist="normal"):
    x = synth.features(seed, n_rows, d, dist, dtype)
    g = synth.features(seed + 1000, seg_ptr.shape[0] - 1, d, dist, dtype)
    sp = torch.from_numpy(seg_ptr).cuda()
    want, t = O.graph_pool_forward(seg_ptr, x.astype(np.float64), reduce)
    got = _host(hb.graph_pool_fwd(sp, _dev(x, dtype), reduce))
    err = np.abs(got - want)
    assert (err <= _bound(t, want, dtype)).all(), f"forward {reduce} {dtype}: worst {err.max():.3e}"
    wantg, tg = O.graph_pool_backward(seg_ptr, g.astype(np.float64), n_rows, reduce)
    out = torch.full((n_rows, d), float("nan"), device="cuda", dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
    gotg = _host(hb.graph_pool_bwd(sp, _dev(g, dtype), n_rows, reduce, out=out))
    errg = np.abs(gotg - wantg)
    assert (errg <= _bound(tg, wantg, dtype)).all(), f"backward {reduce} {dtype}: worst {errg.max():.3e}"
    return got, gotg


@pytest.mark.parametrize("reduce", ["mean", "sum"])
@pytest.mark.parametrize("dtype,d", [("f32", 64), ("f32", 4), ("f32", 20), ("f32", 132), ("f32", 256), ("bf16", 256), ("bf16", 8), ("bf16", 72)])
def test_ragged_batches(reduce, dtype, d):
    """Graphs of 1..150 nodes (several inner groups and a ragged tail), empty graphs,
    rows before the first and after the last graph, widths that fill a lane group
    partly, exactly, and more than once."""
    seg_ptr = _segments(11, 700, 150, lead=3, empty_every=9)
    _check(seg_ptr, int(seg_ptr[-1]) + 5, d, dtype, reduce, seed=21)


def test_batch_of_equal_graphs_like_the_classification_workload():
    """5 000 graphs of 100 nodes, 64 features (the block-diagonal workload shape)."""
    seg_ptr = (np.arange(5001, dtype=np.int64) * 100).astype(np.int32)
    _check(seg_ptr, 500000, 64, "f32", "mean", seed=3, dist="uniform")


def test_integer_features_are_exact_and_runs_repeat():
    seg_ptr = _segments(5, 300, 90)
    n = int(seg_ptr[-1])
    x = synth.features(8, n, 32, "int", "f32")
    sp = torch.from_numpy(seg_ptr).cuda()
    want, _ = O.graph_pool_forward(seg_ptr, x.astype(np.float64), "sum")
    a = hb.graph_pool_fwd(sp, _dev(x, "f32"), "sum")
    b = hb.graph_pool_fwd(sp, _dev(x, "f32"), "sum")
    assert np.array_equal(_host(a), want)
    assert torch.equal(a, b)


def test_one_long_graph_and_single_rows():
    seg_ptr = np.array([0, 1, 2, 5003, 5004], dtype=np.int32)
    _check(seg_ptr, 5004, 64, "f32", "mean", seed=4)


def test_no_graphs_and_argument_errors():
    lib = hb.load_library()
    sp = torch.zeros(1, dtype=torch.int32, device="cuda")
    x = torch.ones((6, 8), device="cuda")
    out = hb.graph_pool_fwd(sp, x, "mean")
    assert out.shape == (0, 8)
    gx = hb.graph_pool_bwd(sp, out, 6, "mean")
    assert not gx.any()                                             # rows that belong to no graph are cleared
    o = torch.empty((1, 8), device="cuda")
    vp = ctypes.c_void_p
    assert lib.hag_graph_pool_fwd(None, 1, 1, 0, 8, vp(x.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_NULL
    assert lib.hag_graph_pool_fwd(vp(sp.data_ptr()), -1, 1, 0, 8, vp(x.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_ARG
    assert lib.hag_graph_pool_fwd(vp(sp.data_ptr()), 0, 2, 0, 8, vp(x.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_ARG   # GCN mode
    assert lib.hag_graph_pool_fwd(vp(sp.data_ptr()), 0, 1, 7, 8, vp(x.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_DTYPE
    assert lib.hag_graph_pool_fwd(vp(sp.data_ptr()), 0, 1, 0, 6, vp(x.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_ALIGN
    assert lib.hag_graph_pool_fwd(vp(sp.data_ptr()), 0, 1, 0, 8, vp(x.data_ptr() + 4), vp(o.data_ptr()), None) == hb.HAG_ERR_ALIGN
    assert lib.hag_graph_pool_bwd(vp(sp.data_ptr()), 0, -1, 1, 0, 8, vp(o.data_ptr()), vp(x.data_ptr()), None) == hb.HAG_ERR_ARG
    torch.cuda.synchronize()
