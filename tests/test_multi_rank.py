"""The N > 1 path on CPU: two gloo ranks shard a block-diagonal batch by graph, each builds
the HAG of its own graphs with the library (host code) and evaluates it with the
oracle; then they split the feature columns of one graph, each with the whole structure
from the library; the pieces must tile the unsharded results, and the timing reduction
must be the max over ranks."""
import os
import socket

import numpy as np
import pytest

import paper_1906_03707_b200 as hb
from oracle import oracle as O
from paper_1906_03707_b200 import sharding, synth
from paper_1906_03707_b200.build import build as build_library

torch = pytest.importorskip("torch")


def test_shard_range_tiles_the_units():
    for n_units in (0, 1, 7, 50, 5000):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(n_units, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n_units
            for (f0, c0), (f1, _) in zip(spans, spans[1:]):
                assert f0 + c0 == f1
            counts = [c for _, c in spans]
            assert max(counts) - min(counts) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def test_block_diagonal_shard_rejects_crossing_edges():
    g = synth.config4_graph(seed=5, n_graphs=4, graph_size=10)
    sharding.shard_block_diagonal(g, 10, 0, 2)
    bad = synth.csr_from_rows([[15]] + [[] for _ in range(19)])
    with pytest.raises(ValueError):
        sharding.shard_block_diagonal(bad, 10, 0, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, tmpdir):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        g = synth.config4_graph(seed=21, n_graphs=9, graph_size=40)
        mine = sharding.shard_block_diagonal(g, 40, rank, world)
        first = mine.meta["first_node"]
        h = hb.Hag.build(mine.row_ptr, mine.col_idx, mine.n // 4)
        arr = h.arrays()
        ref = O.canonical_hag(mine.row_ptr, O.greedy_pairmap(mine.row_ptr, mine.col_idx, mine.n // 4))
        assert np.array_equal(arr["agg_in"], ref.agg_in) and np.array_equal(arr["res_idx"], ref.res_idx)
        x = synth.features(3, g.n, 8, "uniform").astype(np.float64)
        out = O.hag_forward(ref, x[first:first + mine.n], "sum")
        gx = O.hag_backward(ref, x[first:first + mine.n], "sum")
        np.save(os.path.join(tmpdir, f"out{rank}.npy"), out)
        np.save(os.path.join(tmpdir, f"gx{rank}.npy"), gx)
        # second split: the feature columns of ONE graph; every rank holds the whole structure (built by the library,
        # evaluated over the library's own arrays) and a 16-byte-aligned slice of the columns: no exchange
        g2 = synth.config2_graph(seed=23, n=1200, n_comm=12)
        d2 = 24
        c0, cn = sharding.shard_columns(d2, rank, world, 4)
        h2 = hb.Hag.build(g2.row_ptr, g2.col_idx, g2.n // 4)
        a2 = h2.arrays()
        lay = O.CanonicalHag(g2.n, a2["num_agg"], a2["num_levels"], a2["level_ptr"], a2["agg_in"], a2["res_ptr"], a2["res_idx"],
                             a2["t_ptr"], a2["t_idx"], a2["in_degree"], None)
        x2 = synth.features(4, g2.n, d2, "normal").astype(np.float64)
        mine2 = np.ascontiguousarray(x2[:, c0:c0 + cn])
        np.save(os.path.join(tmpdir, f"cols_out{rank}.npy"), O.hag_forward(lay, mine2, "mean"))
        np.save(os.path.join(tmpdir, f"cols_gx{rank}.npy"), O.hag_backward(lay, mine2, "mean"))
        # timing reduction: slowest rank decides, units add up
        ms = sharding.max_over_ranks(10.0 + 5.0 * rank)
        units = sharding.sum_over_ranks(float(mine.n))
        thr = sharding.job_throughput(float(mine.n), 10.0 + 5.0 * rank)
        assert ms == 10.0 + 5.0 * (world - 1)
        assert units == float(g.n)
        assert abs(thr - g.n / (ms * 1e-3)) < 1e-6
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_tile_the_batch(tmp_path):
    import torch.multiprocessing as mp
    build_library()
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    g = synth.config4_graph(seed=21, n_graphs=9, graph_size=40)
    x = synth.features(3, g.n, 8, "uniform").astype(np.float64)
    want, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "sum")
    want_b, _ = O.direct_backward(g.row_ptr, g.col_idx, x, "sum")
    got = np.concatenate([np.load(tmp_path / f"out{r}.npy") for r in range(world)])
    got_b = np.concatenate([np.load(tmp_path / f"gx{r}.npy") for r in range(world)])
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(got_b, want_b, rtol=0, atol=1e-12)
    # the column split: side by side the ranks' slices are the whole result
    g2 = synth.config2_graph(seed=23, n=1200, n_comm=12)
    x2 = synth.features(4, g2.n, 24, "normal").astype(np.float64)
    want2, _ = O.direct_forward(g2.row_ptr, g2.col_idx, x2, "mean")
    want2_b, _ = O.direct_backward(g2.row_ptr, g2.col_idx, x2, "mean")
    got2 = np.concatenate([np.load(tmp_path / f"cols_out{r}.npy") for r in range(world)], axis=1)
    got2_b = np.concatenate([np.load(tmp_path / f"cols_gx{r}.npy") for r in range(world)], axis=1)
    assert got2.shape == want2.shape
    np.testing.assert_allclose(got2, want2, rtol=0, atol=1e-11)
    np.testing.assert_allclose(got2_b, want2_b, rtol=0, atol=1e-11)


def test_column_slices_tile_the_features_and_need_no_exchange():
    for d, eb, world in ((64, 4, 2), (64, 4, 3), (20, 4, 8), (256, 2, 8), (8, 2, 4)):
        parts = [sharding.shard_columns(d, r, world, eb) for r in range(world)]
        assert parts[0][0] == 0 and sum(c for _, c in parts) == d
        for (f0, c0), (f1, _) in zip(parts, parts[1:]):
            assert f1 == f0 + c0
        assert all((c * eb) % 16 == 0 and (f * eb) % 16 == 0 for f, c in parts)
    with pytest.raises(ValueError):
        sharding.shard_columns(6, 0, 2, 4)
    # every rank aggregates its own columns over the whole graph; side by side they are the full result
    g = synth.config1_graph()
    x = synth.features(5, g.n, 24, "normal").astype(np.float64)
    want, _ = O.direct_forward(g.row_ptr, g.col_idx, x, "mean")
    got = []
    for r in range(3):
        f, c = sharding.shard_columns(24, r, 3, 4)
        got.append(O.direct_forward(g.row_ptr, g.col_idx, np.ascontiguousarray(x[:, f:f + c]), "mean")[0])
    np.testing.assert_array_equal(np.concatenate(got, axis=1), want)
