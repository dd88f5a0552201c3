"""Statistics and determinism of the seeded input generator."""
import numpy as np

import taurus_gen as tg


def test_tiny_graph_shape_and_determinism():
    w = tg.WORKLOADS["tiny"]
    g1, g2 = tg.make_graph(w), tg.make_graph(w)
    assert g1.V == 10_000 and abs(g1.E - 100_000) <= 100
    assert (g1.row_ptr == g2.row_ptr).all() and (g1.col_idx == g2.col_idx).all()
    assert np.diff(g1.row_ptr).min() >= 1
    assert (g1.in_degree == np.bincount(g1.col_idx, minlength=g1.V)).all()
    assert g1.col_idx.min() >= 0 and g1.col_idx.max() < g1.V


def test_symmetric_graph_has_every_reverse_edge():
    w = tg.scaled(tg.WORKLOADS["mid"], 5_000, chunk=512)
    g = tg.make_graph(w)
    src = np.repeat(np.arange(g.V), np.diff(g.row_ptr))
    fwd = np.sort(src.astype(np.int64) * g.V + g.col_idx)
    rev = np.sort(g.col_idx.astype(np.int64) * g.V + src)
    assert (fwd == rev).all()
    assert (g.in_degree == np.diff(g.row_ptr)).all()
    assert abs(g.E - w.E) <= 0.002 * w.E


def test_hub_and_local_structure_of_a_scaled_large_graph():
    w = tg.scaled(tg.WORKLOADS["large"], 200_000, chunk=4096)
    g = tg.make_graph(w)
    assert abs(g.E - w.E) <= 0.002 * w.E
    top = np.sort(g.in_degree)[::-1]
    assert 0.5 * w.top_in < top[0] < 2.0 * w.top_in
    src = np.repeat(np.arange(g.V), np.diff(g.row_ptr))
    d = np.abs(src - g.col_idx.astype(np.int64))
    d = np.minimum(d, g.V - d)
    near = (d < 8 * 4 * w.chunk).mean()     # local edges sit within a few chunk widths
    assert near > 0.45


def test_features_are_standard_normal_and_row_addressable():
    x = tg.features(1, 0, 0, 4000, 100)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1) < 0.01
    y = tg.features(1, 0, 1000, 1010, 100)
    assert (x[1000:1010] == y).all()
    z = tg.features(1, 1, 1000, 1010, 100)
    assert not (z == y).all()
    padded = tg.features(1, 0, 1000, 1010, 100, ld=104)
    assert (padded[:, :100] == y).all() and (padded[:, 100:] == 0).all()


def test_weights_are_xavier_uniform():
    W = tg.weights(1, 0, 0, 100, 256)
    a = (6 / 356) ** 0.5
    assert W.min() >= -a and W.max() <= a and abs(W.std() - a / 3 ** 0.5) < 0.01 * a
    assert not (W == tg.weights(1, 0, 1, 100, 256)).all()
