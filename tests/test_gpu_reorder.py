"""taurus_reorder (Alg. 1, Sect. 3.8) against the oracle."""
import numpy as np
import pytest

import oracle
import taurus_gen as tg

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,V,scramble", [("large", 60_000, True), ("mid", 30_011, False), ("tiny", 10_000, True)])
def test_reorder_matches_the_oracle(name, V, scramble):
    import paper_2607_17374_b200 as tb
    w = tg.WORKLOADS[name] if V == tg.WORKLOADS[name].V else tg.scaled(tg.WORKLOADS[name], V, chunk=1024)
    g = tg.make_graph(w)
    init = np.random.default_rng(0).permutation(g.V).astype(np.int32) if scramble else None
    rank, pos, J, span = tb.reorder(g.V, g.E, g.row_ptr, g.col_idx, init, 5)
    o_rank, hist, o_pos = oracle.reorder(g.V, g.row_ptr, g.col_idx, init, 5)
    # positions: same arithmetic up to the summation order
    np.testing.assert_allclose(pos, o_pos, rtol=1e-11, atol=1e-9)
    # the order is a permutation, and sorts the oracle's positions (where positions nearly tie, either order is valid)
    assert np.array_equal(np.sort(rank), np.arange(g.V))
    by_rank = np.empty(g.V, np.int64); by_rank[rank] = np.arange(g.V)
    gaps = np.diff(o_pos[by_rank])
    assert gaps.min() >= -1e-9 * max(1.0, np.abs(o_pos).max())
    agree = float((rank == o_rank).mean())
    print("%s: ranks identical for %.4f of the vertices; span %d -> %d; J %.4g -> %.4g" % (w.name, agree, span[0], span[-1], J[0], J[-1]))
    assert agree > 0.999
    for it in range(6):
        assert abs(span[it] - hist[it][1]) <= 2e-4 * hist[it][1]      # equal unless near-ties were ordered differently
        assert abs(J[it] - hist[it][0]) <= 1e-6 * hist[it][0]
    if agree == 1.0:
        assert [int(x) for x in span] == [h[1] for h in hist]
    if scramble:
        assert span[-1] < span[0]


def test_reorder_rejects_bad_input():
    import paper_2607_17374_b200 as tb
    w = tg.WORKLOADS["tiny"]
    g = tg.make_graph(w)
    bad = g.col_idx.copy(); bad[5] = g.V + 3
    with pytest.raises(tb.TaurusError) as ei:
        tb.reorder(g.V, g.E, g.row_ptr, bad, None, 1)
    assert ei.value.code == tb.ERROR_CODES["INVALID_ARG"]


def test_relabel_csr_and_permute_rows_match_the_oracle():
    import torch
    import oracle
    import paper_2607_17374_b200 as tb
    w = tg.scaled(tg.WORKLOADS["large"], 50_000, chunk=2048)
    g = tg.make_graph(w)
    rng = np.random.default_rng(3)
    rank = rng.permutation(g.V).astype(np.int32)
    want = oracle.relabel_csr(g.V, g.row_ptr, g.col_idx, rank)
    got = tb.relabel_csr(g.V, g.E, g.row_ptr, g.col_idx, rank)                       # host pointers
    for a, b in zip(got, want):
        assert np.array_equal(a, b)
    dev = torch.device("cuda:0")
    got_dev = tb.relabel_csr(g.V, g.E, torch.from_numpy(g.row_ptr).to(dev), torch.from_numpy(g.col_idx).to(dev),
                             torch.from_numpy(rank).to(dev))                         # device pointers
    for a, b in zip(got_dev, want):
        assert np.array_equal(a, b)
    # rows: out[rank[v]] = in[v], padded pitches
    x = rng.normal(size=(g.V, 37)).astype(np.float32)
    xin = torch.zeros((g.V, 40), device=dev); xin[:, :37] = torch.from_numpy(x).to(dev)
    xout = torch.full((g.V, 48), -5.0, device=dev)
    tb.permute_rows(g.V, 37, xin, 40, torch.from_numpy(rank).to(dev), xout, 48)
    ref = np.empty_like(x); ref[rank] = x
    o = xout.cpu().numpy()
    assert np.array_equal(o[:, :37], ref) and (o[:, 37:] == -5.0).all()
    # errors: not a permutation, destination out of range, host matrices
    bad = rank.copy(); bad[5] = bad[6]
    with pytest.raises(tb.TaurusError) as ei:
        tb.relabel_csr(g.V, g.E, g.row_ptr, g.col_idx, bad)
    assert ei.value.code == tb.ERROR_CODES["INVALID_ARG"]
    badcol = g.col_idx.copy(); badcol[17] = g.V
    with pytest.raises(tb.TaurusError) as ei:
        tb.relabel_csr(g.V, g.E, g.row_ptr, badcol, rank)
    assert ei.value.code == tb.ERROR_CODES["INVALID_ARG"]
    with pytest.raises(tb.TaurusError) as ei:
        tb.permute_rows(g.V, 37, x, 37, rank, np.empty_like(x), 37)
    assert ei.value.code == tb.ERROR_CODES["INVALID_ARG"]


def test_reordered_graph_runs_through_the_hot_path():
    """taurus_reorder -> taurus_relabel_csr -> taurus_permute_rows -> one layer: the outputs are the original graph's
    outputs under the renaming (and fewer evictions on a scrambled banded graph)."""
    import torch
    from dataclasses import replace
    import oracle
    import paper_2607_17374_b200 as tb
    from gpu_harness import row_error, run_library
    w = replace(tg.scaled(tg.WORKLOADS["large"], 40_000, chunk=1024), dims=(64, 32), fanout=(0,), hub_count=0)
    g = tg.make_graph(w)
    scramble = np.random.default_rng(1).permutation(g.V).astype(np.int32)
    p1, c1, d1 = tb.relabel_csr(g.V, g.E, g.row_ptr, g.col_idx, scramble)            # a badly labelled version of the graph
    rank, _, J, span = tb.reorder(g.V, g.E, p1, c1, None, 5)
    assert span[-1] < span[0]
    p2, c2, d2 = tb.relabel_csr(g.V, g.E, p1, c1, rank)
    model = tg.make_model(w, bias_scale=0.3)
    x = tg.features(w.seed, 0, 0, g.V, 64)
    x1 = np.empty_like(x); x1[scramble] = x
    dev = torch.device("cuda:0")
    x2d = torch.empty((g.V, 64), device=dev)
    tb.permute_rows(g.V, 64, torch.from_numpy(x1).to(dev), 64, torch.from_numpy(rank).to(dev), x2d, 64)
    x2 = x2d.cpu().numpy()
    outs, evictions = [], []
    for (pp, cc, dd, xx) in [(p1, c1, d1, x1), (p2, c2, d2, x2)]:
        gg = tg.Graph(g.V, g.E, pp, cc, dd)
        ww = replace(w, pool_slots=int(g.V * 0.75))
        lib = run_library(ww, gg, model, xx)
        outs.append(lib["outs"][0]); evictions.append(lib["stats"][0]["evictions"])
    inl = oracle.build_in_lists(g.V, p1, c1)
    ms = oracle.message_sets(inl, 0, w.seed, 0)
    ref1 = oracle.layer_forward(ms, w.mode, np.diff(inl.ptr), np.diff(p1), x1.astype(np.float64), model.W_neigh[0], model.W_self[0],
                                model.bias[0], model.act[0])
    assert row_error(outs[0], ref1)[0] <= 1e-4
    assert row_error(outs[1][rank], ref1)[0] <= 1e-4          # the reordered run gives the same rows under the renaming
    print("evictions scrambled %d -> reordered %d" % tuple(evictions))
    assert evictions[1] < evictions[0]


def test_reorder_and_relabel_on_edgeless_and_single_vertex_graphs():
    import oracle
    import paper_2607_17374_b200 as tb
    for V in (1, 5):
        row_ptr = np.zeros(V + 1, np.int64)
        col = np.zeros(1, np.int32)[:0]
        start = np.arange(V, dtype=np.int32)[::-1].copy()
        rank, pos, J, span = tb.reorder(V, 0, row_ptr, col, start, 3)
        want_rank, _, _ = oracle.reorder(V, row_ptr, col, start, 3)
        assert np.array_equal(rank, want_rank) and (span == 0).all() and np.allclose(J, 0.0)
        p, c, d = tb.relabel_csr(V, 0, row_ptr, col, rank)
        assert np.array_equal(p, row_ptr) and c.size == 0 and (d == 0).all()
