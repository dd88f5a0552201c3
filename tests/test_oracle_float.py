"""Pins for the float side of the oracle: everything here is fixed by the paper's
definitions (Eq. 1-2, the SAGEConv split, the normalised message) and by plain
linear algebra, not by the oracle's own code."""
import numpy as np
import pytest

import oracle
from helpers import csr_from_edges, dense_adjacency, random_multigraph


def _weights(rng, d_in, d_out):
    return rng.standard_normal((d_in, d_out)), rng.standard_normal((d_in, d_out)), rng.standard_normal(d_out)


def _layer(V, row_ptr, col, mode, h, Wn, Ws, b, act, fanout=0, seed=1, layer=0):
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, fanout, seed, layer)
    return oracle.layer_forward(ms, mode, np.diff(inl.ptr), np.diff(row_ptr), h, Wn, Ws, b, act)


@pytest.mark.parametrize("V,E,seed", [(7, 20, 0), (64, 400, 1), (200, 900, 2)])
@pytest.mark.parametrize("act", [0, 1])
def test_sage_mean_equals_dense_products(V, E, seed, act):
    """act(D_in^-1 A H W_neigh + H W_self + b) with A[v,u] = edge multiplicity (Eq. 1-2, mean aggregate)."""
    rng = np.random.default_rng(seed)
    row_ptr, col = random_multigraph(V, E, seed)
    A = dense_adjacency(V, row_ptr, col)
    din = A.sum(1)
    H = rng.standard_normal((V, 5))
    Wn, Ws, b = _weights(rng, 5, 3)
    z = (A @ H @ Wn) / np.maximum(din, 1.0)[:, None] + H @ Ws + b
    ref = np.maximum(z, 0) if act else z
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, Wn, Ws, b, act)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("V,E,seed", [(9, 30, 3), (128, 700, 4)])
def test_gcn_sym_equals_dense_products(V, E, seed):
    """D_in^-1/2 (A + I) D_out^-1/2 H W + b with degrees counting the implicit self message."""
    rng = np.random.default_rng(seed)
    row_ptr, col = random_multigraph(V, E, seed)
    A = dense_adjacency(V, row_ptr, col)
    din = A.sum(1) + 1.0
    dout = A.sum(0) + 1.0
    H = rng.standard_normal((V, 4))
    Wn, _, b = _weights(rng, 4, 6)
    ref = np.diag(din ** -0.5) @ (A + np.eye(V)) @ np.diag(dout ** -0.5) @ H @ Wn + b
    got = _layer(V, row_ptr, col, oracle.GCN_SYM, H, Wn, None, b, 0)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


@pytest.mark.parametrize("V,E,seed", [(9, 30, 13), (128, 700, 14)])
def test_gin_sum_equals_dense_products(V, E, seed):
    """act((A + (1 + eps) I) H W + b): sum aggregator, one shared weight ("GCN/GIN-style aggregation", Sect. 3.9)."""
    rng = np.random.default_rng(seed)
    row_ptr, col = random_multigraph(V, E, seed)
    A = dense_adjacency(V, row_ptr, col)
    H = rng.standard_normal((V, 4))
    Wn, _, b = _weights(rng, 4, 6)
    eps = 0.25
    ref = np.maximum((A + (1 + eps) * np.eye(V)) @ H @ Wn + b, 0)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, 0, 1, 0)
    got = oracle.layer_forward(ms, oracle.GIN_SUM, np.diff(inl.ptr), np.diff(row_ptr), H, Wn, None, b, 1, gin_eps=eps)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_directed_ring_is_a_shifted_copy():
    V = 11
    row_ptr, col = csr_from_edges(V, [(u, (u + 1) % V) for u in range(V)])
    H = np.arange(V * 3, dtype=np.float64).reshape(V, 3)
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, np.eye(3), np.zeros((3, 3)), np.zeros(3), 0)
    np.testing.assert_array_equal(got, np.roll(H, 1, axis=0))


def test_star_hub_is_mean_of_leaves_and_leaves_get_hub_row():
    V = 9  # vertex 0 is the centre, edges both ways
    edges = [(0, v) for v in range(1, V)] + [(v, 0) for v in range(1, V)]
    row_ptr, col = csr_from_edges(V, edges)
    rng = np.random.default_rng(5)
    H = rng.standard_normal((V, 4))
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, np.eye(4), np.zeros((4, 4)), np.zeros(4), 0)
    np.testing.assert_allclose(got[0], H[1:].mean(0), rtol=1e-13)
    for v in range(1, V):
        np.testing.assert_allclose(got[v], H[0], rtol=1e-13)


def test_complete_graph_constant_features():
    V = 6
    row_ptr, col = csr_from_edges(V, [(u, v) for u in range(V) for v in range(V) if u != v])
    H = np.full((V, 3), 2.5)
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, np.eye(3), np.zeros((3, 3)), np.zeros(3), 0)
    np.testing.assert_allclose(got, H, rtol=1e-14)


def test_vertex_without_in_edges_gets_only_self_term():
    V = 4
    row_ptr, col = csr_from_edges(V, [(0, 1), (0, 2), (1, 2)])  # vertices 0 and 3 have din = 0
    rng = np.random.default_rng(6)
    H = rng.standard_normal((V, 3))
    Wn, Ws, b = _weights(rng, 3, 2)
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, Wn, Ws, b, 1)
    for v in (0, 3):
        np.testing.assert_allclose(got[v], np.maximum(H[v] @ Ws + b, 0), rtol=1e-13)


def test_constant_features_return_the_constant():
    V, E = 300, 2000
    row_ptr, col = random_multigraph(V, E, 7)
    din = np.bincount(col, minlength=V)
    H = np.full((V, 4), -1.75)
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, np.eye(4), np.zeros((4, 4)), np.zeros(4), 0)
    np.testing.assert_allclose(got[din > 0], -1.75, rtol=1e-13)
    np.testing.assert_array_equal(got[din == 0], 0.0)


@pytest.mark.parametrize("mode", [oracle.SAGE_MEAN, oracle.GCN_SYM])
@pytest.mark.parametrize("fanout", [0, 3])
def test_linearity_in_the_features(mode, fanout):
    V, E = 150, 1500
    row_ptr, col = random_multigraph(V, E, 8)
    rng = np.random.default_rng(8)
    X, Y = rng.standard_normal((V, 6)), rng.standard_normal((V, 6))
    Wn, Ws, _ = _weights(rng, 6, 5)
    zero = np.zeros(5)
    f = lambda Z: _layer(V, row_ptr, col, mode, Z, Wn, Ws, zero, 0, fanout=fanout)
    a, b = 0.7, -2.3
    np.testing.assert_allclose(f(a * X + b * Y), a * f(X) + b * f(Y), rtol=0, atol=1e-12)


def test_split_weights_equal_concatenated_weight():
    """W [h_agg || h_v] = W_agg h_agg + W_self h_v (SAGEConv paragraph, Sect. 3.9)."""
    V, E = 80, 600
    row_ptr, col = random_multigraph(V, E, 9)
    rng = np.random.default_rng(9)
    H = rng.standard_normal((V, 5))
    Wn, Ws, b = _weights(rng, 5, 4)
    A = dense_adjacency(V, row_ptr, col)
    h_agg = (A @ H) / np.maximum(A.sum(1), 1.0)[:, None]
    W_cat = np.vstack([Wn, Ws])                      # (2d) x d'
    ref = np.maximum(np.hstack([h_agg, H]) @ W_cat + b, 0)
    got = _layer(V, row_ptr, col, oracle.SAGE_MEAN, H, Wn, Ws, b, 1)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_sampled_mean_equals_dense_product_over_sampled_edges():
    """Under sampling the mean runs over M(v) only: brute force with the sampled adjacency."""
    V, E, fanout = 60, 900, 4
    row_ptr, col = random_multigraph(V, E, 10)
    rng = np.random.default_rng(10)
    H = rng.standard_normal((V, 3))
    Wn, Ws, b = _weights(rng, 3, 3)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, fanout, 42, 1)
    A = np.zeros((V, V))
    src_of_edge = np.repeat(np.arange(V), np.diff(row_ptr))
    for e in np.flatnonzero(ms.prop):
        A[col[e], src_of_edge[e]] += 1
    assert (A.sum(1) == np.minimum(np.bincount(col, minlength=V), fanout)).all()
    ref = (A @ H @ Wn) / np.maximum(A.sum(1), 1)[:, None] + H @ Ws + b
    got = oracle.layer_forward(ms, oracle.SAGE_MEAN, np.diff(inl.ptr), np.diff(row_ptr), H, Wn, Ws, b, 0)
    np.testing.assert_allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_two_layers_chain_through_the_oracles_own_output():
    V, E = 50, 300
    row_ptr, col = random_multigraph(V, E, 11)
    rng = np.random.default_rng(11)
    X = rng.standard_normal((V, 4))
    W1n, W1s, b1 = _weights(rng, 4, 6)
    W2n, W2s, b2 = _weights(rng, 6, 2)
    A = dense_adjacency(V, row_ptr, col)
    Dinv = 1.0 / np.maximum(A.sum(1), 1.0)[:, None]
    h1 = np.maximum(Dinv * (A @ X @ W1n) + X @ W1s + b1, 0)
    h2 = Dinv * (A @ h1 @ W2n) + h1 @ W2s + b2
    outs = oracle.forward(V, row_ptr, col, X, oracle.SAGE_MEAN, [W1n, W2n], [W1s, W2s], [b1, b2], [1, 0], [0, 0], 1)
    np.testing.assert_allclose(outs[0], h1, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(outs[1], h2, rtol=1e-11, atol=1e-11)


def test_in_lists_are_sorted_by_source_with_duplicates_in_csr_order():
    V, E = 40, 500
    row_ptr, col = random_multigraph(V, E, 12)
    inl = oracle.build_in_lists(V, row_ptr, col)
    src_of_edge = np.repeat(np.arange(V), np.diff(row_ptr))
    for v in range(V):
        s = inl.src[inl.ptr[v]:inl.ptr[v + 1]]
        e = inl.eid[inl.ptr[v]:inl.ptr[v + 1]]
        assert (np.diff(e) > 0).all()               # CSR order == (source, position) order
        assert (col[e] == v).all() and (src_of_edge[e] == s).all()
    assert (np.diff(inl.ptr) == np.bincount(col, minlength=V)).all()


@pytest.mark.parametrize("mode", [oracle.SAGE_MEAN, oracle.GCN_SYM, oracle.GIN_SUM])
@pytest.mark.parametrize("fanout", [0, 3])
def test_subset_evaluation_equals_the_full_layer_on_those_rows(mode, fanout):
    """The destination-subset path (in-lists by a CSR scan) against the whole-graph path restricted to the same rows."""
    from helpers import random_multigraph
    V, E, F, H = 300, 2500, 12, 7
    row_ptr, col = random_multigraph(V, E, 5)
    rng = np.random.default_rng(2)
    h = rng.standard_normal((V, F))
    Wn, Ws, b = rng.standard_normal((F, H)), rng.standard_normal((F, H)), rng.standard_normal(H)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, fanout, 9, 1)
    din, dout = np.diff(inl.ptr), np.diff(row_ptr)
    full = oracle.layer_forward(ms, mode, din, dout, h, Wn, Ws, b, 1, gin_eps=0.25)
    dsts = np.unique(rng.integers(0, V, 40)).astype(np.int64)
    ptr, src, eid = oracle.subset_in_lists(V, row_ptr, col, dsts)
    for i, v in enumerate(dsts):                      # the scan finds exactly the in-list of the whole-graph builder
        assert (src[ptr[i]:ptr[i + 1]] == inl.src[inl.ptr[v]:inl.ptr[v + 1]]).all()
        assert (eid[ptr[i]:ptr[i + 1]] == inl.eid[inl.ptr[v]:inl.ptr[v + 1]]).all()
    kp, ks, ke = oracle.subset_message_sets(ptr, src, eid, dsts, fanout, 9, 1)
    for i, v in enumerate(dsts):
        assert sorted(ke[kp[i]:kp[i + 1]].tolist()) == sorted(ms.eid[ms.ptr[v]:ms.ptr[v + 1]].tolist())
    need = np.unique(np.concatenate([ks, dsts]))
    sub = oracle.subset_forward(mode, dsts, kp, ks, din[dsts], dout[dsts], need, dout[need], h[need], Wn, Ws, b, 1, gin_eps=0.25)
    assert np.abs(sub - full[dsts]).max() <= 1e-12
