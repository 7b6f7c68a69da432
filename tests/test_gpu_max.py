"""GPU parity of the element-wise max aggregation (GraphSAGE-P row of Table 1) against
the fp64 oracle, through the C ABI.

Forward: max does no arithmetic, so the result must equal the oracle's bit for bit,
for fp32 and for bf16 storage, over the HAG and over the plain graph; so must the
maxima the aggregation nodes hold.  Backward: sums of selected gradient components
in fp32, |gpu - oracle| <= 1e-5 * Sigma|terms| + 1e-6 (bf16: as for the sum
aggregation); with integer-valued gradients the sums are exact and must match bit
for bit, ties included.
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


def _check(g, capacity, d, dtype, seed, z=None, gr=None, exact_grad=False):
    h = hb.Hag.build(g.row_ptr, g.col_idx, capacity).to_device(0)
    z = synth.features(seed, g.n, d, "normal", dtype) if z is None else z
    gr = synth.features(seed + 1000, g.n, d, "normal", dtype) if gr is None else gr
    z64, g64 = z.astype(np.float64), gr.astype(np.float64)
    want = O.direct_max_forward(g.row_ptr, g.col_idx, z64)
    wantg, tg = O.direct_max_backward(g.row_ptr, g.col_idx, z64, g64)
    zd, gd = _dev(z, dtype), _dev(gr, dtype)
    for use_hag in (True, False):
        name = "hag" if use_hag else "csr"
        out, ws = h.max_fwd(zd, use_hag=use_hag)
        assert np.array_equal(_host(out), want), f"{name} max forward {dtype}"
        if use_hag and h.info()["num_agg"] > 0:
            arr = h.arrays()
            ahat = ws[: arr["num_agg"] * d].reshape(arr["num_agg"], d).cpu().numpy().astype(np.float64)
            full = np.concatenate([z64, ahat])
            j = np.random.default_rng(seed).integers(0, arr["num_agg"], size=64)
            agg_in = np.asarray(arr["agg_in"]).reshape(-1, 2)
            assert np.array_equal(ahat[j], np.maximum(full[agg_in[j, 0]], full[agg_in[j, 1]])), "aggregation-node maxima"
        gz = _host(h.max_bwd(zd, out, ws, gd, use_hag=use_hag))
        if exact_grad:
            assert np.array_equal(gz, wantg), f"{name} max backward {dtype} (integer gradients)"
        else:
            err = np.abs(gz - wantg)
            assert (err <= _bound(tg, wantg, dtype)).all(), f"{name} max backward {dtype}: worst {err.max():.3e}"
    h.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("index,scale", [(1, 1.0), (2, 0.1), (4, 0.01), (6, 0.05)])
def test_workload_shapes(index, scale, dtype):
    w = synth.workload(index, scale=scale)
    _check(w.graph, w.capacity, w.d if dtype == "f32" else max(w.d, 8), dtype, seed=index)


@pytest.mark.parametrize("dtype,d", [("f32", 4), ("f32", 20), ("f32", 64), ("f32", 132), ("f32", 256), ("bf16", 8), ("bf16", 72), ("bf16", 256)])
def test_widths(dtype, d):
    g = synth.workload(2, scale=0.04).graph
    _check(g, g.n // 4, d, dtype, seed=d)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_ties_and_integer_gradients_are_exact(dtype):
    """Features from {-1, 0, 1} tie almost everywhere; every maximiser receives the gradient, and integer
    gradients make the sums exact."""
    g = synth.workload(2, scale=0.06).graph
    z = synth.features(3, g.n, 32, "int", dtype)
    z = np.clip(z, -1, 1).astype(z.dtype)
    gr = synth.features(4, g.n, 32, "int", dtype)
    _check(g, g.n // 4, 32, dtype, seed=5, z=z, gr=gr, exact_grad=True)


@pytest.mark.parametrize("seed", range(8))
def test_random_graphs_with_empty_rows(seed):
    rng = np.random.default_rng(seed)
    g = synth.random_digraph(seed=seed, n=int(rng.integers(40, 400)), p=float(rng.uniform(0.01, 0.2)),
                             undirected=bool(seed % 2), self_loops=bool(seed % 3 == 0))
    _check(g, g.n // 2, 16, "f32", seed=seed)


def test_capacity_zero_and_long_rows():
    g = synth.workload(3, scale=0.02).graph           # hub rows of several hundred entries
    _check(g, 0, 32, "f32", seed=9)
    _check(g, g.n // 4, 32, "f32", seed=9)


def test_argument_errors():
    w = synth.workload(1)
    h = hb.Hag.build(w.graph.row_ptr, w.graph.col_idx, w.capacity).to_device(0)
    lib = hb.load_library()
    vp = ctypes.c_void_p
    z = torch.zeros((w.graph.n, 16), device="cuda")
    o = torch.zeros_like(z)
    ws = h.max_workspace(16, z.device)
    ws2 = h.max_workspace(16, z.device)
    hp = h._h
    assert lib.hag_max_fwd(None, 0, 16, vp(z.data_ptr()), vp(o.data_ptr()), vp(ws.data_ptr()), None) == hb.HAG_ERR_NULL
    assert lib.hag_max_fwd(hp, 0, 16, vp(z.data_ptr()), None, vp(ws.data_ptr()), None) == hb.HAG_ERR_NULL
    assert lib.hag_max_fwd(hp, 0, 16, vp(z.data_ptr()), vp(o.data_ptr()), None, None) == hb.HAG_ERR_WORKSPACE
    assert lib.hag_max_fwd(hp, 0, 16, vp(z.data_ptr()), vp(z.data_ptr()), vp(ws.data_ptr()), None) == hb.HAG_ERR_ARG
    assert lib.hag_max_fwd(hp, 3, 16, vp(z.data_ptr()), vp(o.data_ptr()), vp(ws.data_ptr()), None) == hb.HAG_ERR_DTYPE
    assert lib.hag_max_fwd(hp, 0, 6, vp(z.data_ptr()), vp(o.data_ptr()), vp(ws.data_ptr()), None) == hb.HAG_ERR_ALIGN
    assert lib.hag_max_fwd(hp, 0, 0, vp(z.data_ptr()), vp(o.data_ptr()), vp(ws.data_ptr()), None) == hb.HAG_ERR_ARG
    g = torch.zeros_like(z)
    gz = torch.zeros_like(z)
    args = (vp(z.data_ptr()), vp(o.data_ptr()), vp(ws.data_ptr()), vp(g.data_ptr()), vp(gz.data_ptr()))
    assert lib.hag_max_bwd(hp, 0, 16, *args, vp(ws.data_ptr()), None) == hb.HAG_ERR_ARG          # one buffer for both roles
    assert lib.hag_max_bwd(hp, 0, 16, *args, None, None) == hb.HAG_ERR_WORKSPACE
    assert lib.hag_max_bwd(hp, 0, 16, *args, vp(ws2.data_ptr()), None) == hb.HAG_OK
    assert lib.csr_max_bwd(hp, 0, 16, vp(z.data_ptr()), vp(o.data_ptr()), vp(g.data_ptr()), vp(z.data_ptr()), None) == hb.HAG_ERR_ARG
    host_only = hb.Hag.build(w.graph.row_ptr, w.graph.col_idx, w.capacity)
    assert lib.csr_max_fwd(host_only._h, 0, 16, vp(z.data_ptr()), vp(o.data_ptr()), None) == hb.HAG_ERR_NOT_ON_DEVICE
    torch.cuda.synchronize()


@pytest.mark.parametrize("dtype,d,ties", [("f32", 16, False), ("f32", 32, True), ("f32", 40, False), ("f32", 64, False),
                                           ("bf16", 32, False), ("bf16", 64, True), ("bf16", 128, False)])
def test_several_rows_per_warp_kernels(dtype, d, ties):
    """Launches of 4096 x (groups per warp) rows or more take a row per group of lanes, in the list's by-length order;
    rows of more than 128 entries among them are walked by the whole warp afterwards: the 70 000-row clique-union graph
    (rows up to several hundred entries), every group width, dead lanes (d = 40), ties with integer gradients."""
    w = synth.workload(6, scale=0.7)
    g = w.graph
    assert g.n >= 8 * 4096 and int(np.diff(g.row_ptr).max()) > 128
    if ties:
        z = np.clip(synth.features(3, g.n, d, "int", dtype), -1, 1).astype(np.float32)
        gr = synth.features(4, g.n, d, "int", dtype)
        # fp32 holds every integer sum exactly; a bf16 result is rounded, so that case keeps the tolerance
        _check(g, w.capacity, d, dtype, seed=6, z=z, gr=gr, exact_grad=(dtype == "f32"))
    else:
        _check(g, w.capacity, d, dtype, seed=d)


@pytest.mark.parametrize("index", [2, 4])
def test_full_size_workloads(index):
    """The 50 000-node clustered workload and the batch of 5 000 small graphs at full size, fp32, D = 64:
    every element of the forward result and of the gradient against the oracle."""
    w = synth.workload(index)
    _check(w.graph, w.capacity, w.d, "f32", seed=w.seed)


@pytest.mark.parametrize("index", [3, 5, 6])
def test_full_size_workloads_sampled_rows(index):
    """The two largest shapes (fp32 D = 128; bf16 D = 256) and the clique-union graph at full size, in the
    storage type of the workload: the oracle evaluates sampled rows one by one (forward rows, and gradient
    rows with the maxima of their out-neighbours), hub rows and empty-ish rows included."""
    w = synth.workload(index)
    g = w.graph
    h = hb.Hag.build(g.row_ptr, g.col_idx, w.capacity).to_device(0)
    z = synth.features(w.seed, g.n, w.d, "normal", w.dtype)
    gr = synth.upstream_grad(w.seed, g.n, w.d, "normal", w.dtype)
    rng = np.random.default_rng(index)
    deg = np.diff(g.row_ptr)
    out_deg = np.bincount(g.col_idx, minlength=g.n)
    rows = np.unique(np.concatenate([rng.choice(g.n, 1200, replace=False), np.argsort(deg)[-20:], np.argsort(deg)[:20],
                                     np.argsort(out_deg)[-20:], [0, g.n - 1]]))
    z64, g64 = z.astype(np.float64), gr.astype(np.float64)
    want = O.direct_max_forward(g.row_ptr, g.col_idx, z64, rows=rows)
    wantg, tg = O.direct_max_backward(g.row_ptr, g.col_idx, z64, g64, rows=rows)
    zd, gd = _dev(z, w.dtype), _dev(gr, w.dtype)
    for use_hag in (True, False):
        out, ws = h.max_fwd(zd, use_hag=use_hag)
        assert np.array_equal(_host(out)[rows], want), f"max forward use_hag={use_hag}"
        gz = _host(h.max_bwd(zd, out, ws, gd, use_hag=use_hag))[rows]
        err = np.abs(gz - wantg)
        assert (err <= _bound(tg, wantg, w.dtype)).all(), f"max backward use_hag={use_hag}: worst {err.max():.3e}"
    h.close()
