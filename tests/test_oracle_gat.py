"""Pins of the oracle's GATConv layer against hand-worked values, a dense masked softmax and special cases."""
import os

import numpy as np
import pytest

import oracle
from oracle import gat

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "gat_example.txt")


def csr_from_edges(V, edges):
    edges = sorted(edges, key=lambda e: e[0])
    row_ptr = np.zeros(V + 1, np.int64)
    for u, _ in edges:
        row_ptr[u + 1] += 1
    row_ptr = np.cumsum(row_ptr)
    col = np.array([v for _, v in edges], np.int32)
    return row_ptr, col


def random_multigraph(V, E, seed):
    rng = np.random.default_rng(seed)
    edges = [(int(u), int(v)) for u, v in zip(rng.integers(0, V, E), rng.integers(0, V, E))]
    edges += edges[:E // 5]                     # repeated edges
    return csr_from_edges(V, edges)


def test_hand_worked_examples():
    cases = {}
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        c = cases.setdefault(t[0], {})
        if len(t) == 2:
            c["V"] = int(t[1])
        elif t[1] == "edges":
            x = [int(v) for v in t[2:]]
            c["edges"] = list(zip(x[0::2], x[1::2]))
        elif t[1] == "h":
            c["h"] = [float(v) for v in t[2:]]
        elif t[1] == "a_src":
            c.update(a_src=float(t[2]), a_dst=float(t[4]), slope=float(t[6]))
        elif t[1] == "out":
            c["out"] = [float(v) for v in t[2:]]
    assert set(cases) == {"A", "B"}
    for c in cases.values():
        row_ptr, col = csr_from_edges(c["V"], c["edges"])
        inl = oracle.build_in_lists(c["V"], row_ptr, col)
        ms = oracle.message_sets(inl, 0, 1, 0)
        out = gat.gat_layer_forward(ms, np.array(c["h"])[:, None], np.eye(1), [c["a_src"]], [c["a_dst"]], [0.0], 0, c["slope"])
        assert np.allclose(out[:, 0], c["out"], atol=2e-7, rtol=0)


@pytest.mark.parametrize("seed,act,slope", [(1, 0, 0.2), (2, 1, 0.2), (3, 0, 0.01)])
def test_dense_masked_softmax(seed, act, slope):
    V, d, dp = 40, 7, 5
    row_ptr, col = random_multigraph(V, 150, seed)
    rng = np.random.default_rng(seed)
    h = rng.normal(size=(V, d)); W = rng.normal(size=(d, dp)); b = rng.normal(size=dp)
    a_s, a_d = rng.normal(size=dp), rng.normal(size=dp)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, 0, 1, 0)
    got = gat.gat_layer_forward(ms, h, W, a_s, a_d, b, act, slope)
    # dense: A[v, u] = multiplicity of u -> v, plus the identity for the self message
    A = np.eye(V)
    for u in range(V):
        for k in range(row_ptr[u], row_ptr[u + 1]):
            A[col[k], u] += 1
    hp = h @ W
    S = (hp @ a_d)[:, None] + (hp @ a_s)[None, :]
    S = np.where(S > 0, S, slope * S)
    Wt = A * np.exp(S)
    alpha = Wt / Wt.sum(axis=1, keepdims=True)
    ref = alpha @ hp + b
    if act:
        ref = np.maximum(ref, 0)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_zero_attention_vector_is_a_plain_mean():
    V, d, dp = 200, 6, 4
    row_ptr, col = random_multigraph(V, 900, 7)
    rng = np.random.default_rng(7)
    h = rng.normal(size=(V, d)); W = rng.normal(size=(d, dp)); b = rng.normal(size=dp)
    inl = oracle.build_in_lists(V, row_ptr, col)
    for fanout in (0, 3):
        ms = oracle.message_sets(inl, fanout, 11, 0)
        got = gat.gat_layer_forward(ms, h, W, np.zeros(dp), np.zeros(dp), b, 0)
        hp = h @ W
        agg = oracle.aggregate(ms, np.arange(V), None, hp)          # the C aggregator: sum over M(v)
        ref = (agg + hp) / (ms.m[:, None] + 1.0) + b
        assert np.allclose(got, ref, rtol=1e-12, atol=1e-12)


def test_identity_slope_makes_the_destination_term_cancel():
    V, d = 60, 5
    row_ptr, col = random_multigraph(V, 300, 4)
    rng = np.random.default_rng(4)
    h = rng.normal(size=(V, d)); W = rng.normal(size=(d, d)); a_s = rng.normal(size=d)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, 0, 1, 0)
    o1 = gat.gat_layer_forward(ms, h, W, a_s, rng.normal(size=d), np.zeros(d), 0, slope=1.0)
    o2 = gat.gat_layer_forward(ms, h, W, a_s, np.zeros(d), np.zeros(d), 0, slope=1.0)
    assert np.allclose(o1, o2, rtol=1e-10, atol=1e-12)
    o3 = gat.gat_layer_forward(ms, h, W, a_s, rng.normal(size=d), np.zeros(d), 0, slope=0.2)
    assert not np.allclose(o1, o3, rtol=1e-3, atol=1e-6)            # with a real LeakyReLU it does not


def test_vertex_without_in_edges_and_large_fanout():
    V, d = 30, 4
    row_ptr, col = csr_from_edges(V, [(u, (u * 7 + 1) % (V - 1) + 1) for u in range(V)] * 2)   # vertex 0 has no in-edge
    rng = np.random.default_rng(2)
    h = rng.normal(size=(V, d)); W = rng.normal(size=(d, d)); b = rng.normal(size=d)
    a_s, a_d = rng.normal(size=d), rng.normal(size=d)
    inl = oracle.build_in_lists(V, row_ptr, col)
    exact = oracle.message_sets(inl, 0, 1, 0)
    assert exact.m[0] == 0
    out = gat.gat_layer_forward(exact, h, W, a_s, a_d, b, 1)
    assert np.allclose(out[0], np.maximum(h[0] @ W + b, 0))
    big = oracle.message_sets(inl, 64, 1, 0)
    assert np.array_equal(gat.gat_layer_forward(big, h, W, a_s, a_d, b, 1), out)


def test_several_heads_are_the_single_head_layer_per_column_block():
    """gat_layer_forward_heads against its definition written out: each head is the one-head layer on its own columns of
    W, a_src, a_dst and b; with one head it is the one-head layer itself."""
    from oracle import gat
    from helpers import random_multigraph
    V, E, F, H, heads = 60, 300, 5, 12, 3
    row_ptr, col = random_multigraph(V, E, 4)
    ms = oracle.message_sets(oracle.build_in_lists(V, row_ptr, col), 0, 1, 0)
    rng = np.random.default_rng(8)
    h, W = rng.standard_normal((V, F)), rng.standard_normal((F, H))
    a_s, a_d, b = rng.standard_normal(H), rng.standard_normal(H), rng.standard_normal(H)
    out = gat.gat_layer_forward_heads(ms, h, W, a_s, a_d, b, 1, heads, 0.2)
    d = H // heads
    for i in range(heads):
        blk = slice(i * d, (i + 1) * d)
        one = gat.gat_layer_forward(ms, h, W[:, blk], a_s[blk], a_d[blk], b[blk], 1, 0.2)
        assert np.array_equal(out[:, blk], one)
    assert np.array_equal(gat.gat_layer_forward_heads(ms, h, W, a_s, a_d, b, 0, 1, 0.2), gat.gat_layer_forward(ms, h, W, a_s, a_d, b, 0, 0.2))
    # heads differ: with different attention vectors two heads weight the same neighbours differently
    same_w = np.concatenate([W[:, :d], W[:, :d]], axis=1)
    two = gat.gat_layer_forward_heads(ms, h, same_w, np.concatenate([a_s[:d], 3 * a_s[:d]]), np.concatenate([a_d[:d], -a_d[:d]]),
                                      np.zeros(2 * d), 0, 2, 0.2)
    assert np.abs(two[:, :d] - two[:, d:]).max() > 1e-3
