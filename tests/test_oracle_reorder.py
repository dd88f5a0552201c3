"""Pins for the oracle's topology-aware reordering (Alg. 1 and the span analysis of Sect. 3.8): the update rules
are the stationary points of J, a worked three-vertex example, closed forms of the span, and the claimed effect."""
import numpy as np

import oracle
import taurus_gen as tg
from helpers import csr_from_edges, random_multigraph


def test_worked_example_on_a_three_vertex_path():
    """0 -> 1 -> 2 with r = (0, 1, 2); d = in-degree + 1 = (1, 2, 2).  By hand:
    mu = (0, 1/2, 3/2);  r' = ((0 + 1/4) / (1 + 1/2), (1/4 + 3/4) / (1/2 + 1/2), (3/4) / (1/2)) = (1/6, 1, 3/2)."""
    row_ptr, col = csr_from_edges(3, [(0, 1), (1, 2)])
    mu, r = oracle.reorder_step(3, row_ptr, col, np.array([0.0, 1.0, 2.0]))
    np.testing.assert_allclose(mu, [0.0, 0.5, 1.5], rtol=1e-15)
    np.testing.assert_allclose(r, [1.0 / 6.0, 1.0, 1.5], rtol=1e-15)
    # J by hand: v0: 0; v1: ((1 - .5)^2 + (0 - .5)^2) / 2 = .25; v2: ((2 - 1.5)^2 + (1 - 1.5)^2) / 2 = .25
    assert abs(oracle.dispersion_J(3, row_ptr, col, np.array([0.0, 1.0, 2.0]), mu) - 0.5) < 1e-15


def test_update_rules_are_the_minimisers_of_J():
    V, E = 60, 400
    row_ptr, col = random_multigraph(V, E, 21)
    rng = np.random.default_rng(21)
    r = rng.standard_normal(V) * 10
    mu, r_new = oracle.reorder_step(V, row_ptr, col, r)
    J0 = oracle.dispersion_J(V, row_ptr, col, r, mu)
    for _ in range(20):      # mu* minimises J(r, .): any perturbation raises it
        assert oracle.dispersion_J(V, row_ptr, col, r, mu + rng.standard_normal(V) * 0.1) > J0
    J1 = oracle.dispersion_J(V, row_ptr, col, r_new, mu)
    assert J1 <= J0
    for _ in range(20):      # r* minimises J(., mu)
        assert oracle.dispersion_J(V, row_ptr, col, r_new + rng.standard_normal(V) * 0.1, mu) > J1
    h = 1e-6                 # and the gradients vanish there
    for v in (0, 7, 33):
        e = np.zeros(V); e[v] = h
        g_mu = (oracle.dispersion_J(V, row_ptr, col, r, mu + e) - oracle.dispersion_J(V, row_ptr, col, r, mu - e)) / (2 * h)
        g_r = (oracle.dispersion_J(V, row_ptr, col, r_new + e, mu) - oracle.dispersion_J(V, row_ptr, col, r_new - e, mu)) / (2 * h)
        assert abs(g_mu) < 1e-6 and abs(g_r) < 1e-6


def test_span_closed_forms():
    V = 12
    ring_ptr, ring_col = csr_from_edges(V, [(u, (u + 1) % V) for u in range(V)])
    ident = np.arange(V)
    # every vertex v > 0 has in-neighbour v - 1: span 1; vertex 0 has in-neighbour V - 1: span V - 1
    assert oracle.total_span(V, ring_ptr, ring_col, ident) == (V - 1) + (V - 1)
    star_ptr, star_col = csr_from_edges(V, [(u, 0) for u in range(1, V)])
    assert oracle.total_span(V, star_ptr, star_col, ident) == V - 1          # only the centre has a span
    assert oracle.total_span(V, star_ptr, star_col, ident[::-1].copy()) == V - 1
    empty_ptr, empty_col = csr_from_edges(V, [])
    assert oracle.total_span(V, empty_ptr, empty_col, ident) == 0           # only self messages: L(v) = 0


def test_span_is_bounded_by_twice_v_times_bandwidth():
    """C(pi) <= 2 |V| B with B the largest edge length under pi (Sect. 3.8)."""
    V, rng = 400, np.random.default_rng(3)
    edges = [(u, min(V - 1, max(0, u + int(o)))) for u in range(V) for o in rng.integers(-9, 10, 4)]
    row_ptr, col = csr_from_edges(V, edges)
    src = np.repeat(np.arange(V), np.diff(row_ptr))
    B = int(np.abs(src - col).max())
    assert oracle.total_span(V, row_ptr, col, np.arange(V)) <= 2 * V * B


def test_ranks_break_ties_by_vertex_id():
    assert oracle.ranks_of(np.array([2.0, 1.0, 2.0, 0.5, 1.0])).tolist() == [3, 1, 4, 0, 2]


def test_five_iterations_reduce_the_span_of_a_scrambled_banded_graph():
    """The effect Sect. 3.8 / 4.4 claims: the reordering shortens the total span (and the dispersion J tracks it)."""
    w = tg.scaled(tg.WORKLOADS["large"], 30_000, chunk=1024)
    g = tg.make_graph(w)
    scrambled = np.random.default_rng(0).permutation(g.V)
    rank, hist, _ = oracle.reorder(g.V, g.row_ptr, g.col_idx, scrambled, 5)
    assert sorted(rank.tolist()) == list(range(g.V))
    assert hist[-1][1] < 0.85 * hist[0][1] and hist[-1][0] < hist[0][0]
    assert hist[1][1] < hist[0][1]


def test_relabelling_is_an_isomorphism():
    """Relabelled graph: same edges under the renaming, inverse relabelling restores the original, and a GNN layer
    on the relabelled graph with permuted features gives the permuted outputs (message passing does not depend on
    the names of the vertices)."""
    rng = np.random.default_rng(21)
    V, E = 300, 2500
    src = np.sort(rng.integers(0, V, E))
    col = rng.integers(0, V, E).astype(np.int32)
    row_ptr = np.zeros(V + 1, np.int64)
    np.cumsum(np.bincount(src, minlength=V), out=row_ptr[1:])
    rank = rng.permutation(V).astype(np.int32)
    p2, c2, d2 = oracle.relabel_csr(V, row_ptr, col, rank)
    # the same multiset of edges under the renaming
    old_edges = sorted(zip(rank[src].tolist(), rank[col].tolist()))
    src2 = np.repeat(np.arange(V), np.diff(p2))
    assert sorted(zip(src2.tolist(), c2.tolist())) == old_edges
    assert np.array_equal(d2, np.bincount(rank[col], minlength=V))
    # the inverse renaming restores the original arrays exactly (edge order inside a row is kept)
    inv = np.empty(V, np.int32); inv[rank] = np.arange(V, dtype=np.int32)
    p3, c3, _ = oracle.relabel_csr(V, p2, c2, inv)
    assert np.array_equal(p3, row_ptr) and np.array_equal(c3, col)
    ident = np.arange(V, dtype=np.int32)
    p4, c4, _ = oracle.relabel_csr(V, row_ptr, col, ident)
    assert np.array_equal(p4, row_ptr) and np.array_equal(c4, col)
    # one exact SAGE layer: out'[rank[v]] == out[v]
    h = rng.normal(size=(V, 6)); Wn = rng.normal(size=(6, 4)); Ws = rng.normal(size=(6, 4)); b = rng.normal(size=4)
    def layer(rp, cc, x):
        inl = oracle.build_in_lists(V, rp, cc)
        ms = oracle.message_sets(inl, 0, 1, 0)
        return oracle.layer_forward(ms, oracle.SAGE_MEAN, np.diff(inl.ptr), np.diff(rp), x, Wn, Ws, b, 1)
    out = layer(row_ptr, col, h)
    h2 = np.empty_like(h); h2[rank] = h
    out2 = layer(p2, c2, h2)
    assert np.allclose(out2[rank], out, rtol=1e-12, atol=1e-12)
