"""CPU oracle for a GATConv layer (GATConv paragraph of Sect. 3.9).  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

The definition, pull-based and in fp64, one destination at a time:

    h'_u    = h_u W                                             transformed features (the first pass)
    e_uv    = LeakyReLU(a_src . h'_u + a_dst . h'_v)            a = [a_src || a_dst]
    alpha_uv = softmax over u in N(v) of e_uv                   neighbourhood-wise
    out_v   = act(sum_{u in N(v)} alpha_uv h'_u + b)

N(v) is the propagated in-multiset M(v) (all in-edges, or the sampled ones; a multi-edge counts once per
copy) together with v itself: every vertex aggregates a self message (Sect. 3.8), so a vertex without
in-edges keeps act(h'_v + b).  gat_layer_forward is one attention head; gat_layer_forward_heads applies the same
procedure per head (Sect. 3.9 treats several heads as independent repetitions) to column blocks of W, a_src, a_dst and b and
concatenates the heads' outputs.

Pins (tests/test_oracle_gat.py): two hand-worked examples (tests/golden/gat_example.txt), a dense masked
softmax on tiny multigraphs, uniform attention when a = 0 (a plain mean, checked against the C aggregator),
independence of a_dst when the slope is 1, vertices without in-edges, fanout >= max in-degree = exact.
Nothing here is parity unpinned.
"""
from __future__ import annotations

from typing import Optional

import numpy as np


def gat_layer_forward(ms, h: np.ndarray, W: np.ndarray, a_src: np.ndarray, a_dst: np.ndarray, bias: np.ndarray, act: int,
                      slope: float = 0.2, dst: Optional[np.ndarray] = None, magnitude: bool = False):
    """out_v for v in dst (default: all).  ms is the layer's MessageSets (ptr, src).

    magnitude=True returns (out, mag): mag_v = sum_u alpha_uv (|h_u| |W|) + |b|, the same weighted sum with every
    product of the transform replaced by its absolute value (the scale against which a rounding error of the sum is
    measured); `out` is unchanged by the flag."""
    hp = np.asarray(h, dtype=np.float64) @ np.asarray(W, dtype=np.float64)
    hp_abs = np.abs(np.asarray(h, dtype=np.float64)) @ np.abs(np.asarray(W, dtype=np.float64)) if magnitude else None
    s = hp @ np.asarray(a_src, dtype=np.float64)
    t = hp @ np.asarray(a_dst, dtype=np.float64)
    b = np.asarray(bias, dtype=np.float64)
    V = ms.m.size
    if dst is None:
        dst = np.arange(V, dtype=np.int64)
    out = np.empty((len(dst), hp.shape[1]), np.float64)
    mag = np.empty_like(out) if magnitude else None
    for i, v in enumerate(dst):
        v = int(v)
        nb = np.concatenate([ms.src[ms.ptr[v]:ms.ptr[v + 1]].astype(np.int64), [v]])
        e = s[nb] + t[v]
        e = np.where(e > 0, e, slope * e)
        w = np.exp(e - e.max())
        alpha = w / w.sum()
        z = alpha @ hp[nb] + b
        out[i] = np.maximum(z, 0.0) if act else z
        if magnitude:
            mag[i] = alpha @ hp_abs[nb] + np.abs(b)
    return (out, mag) if magnitude else out


def gat_layer_forward_heads(ms, h: np.ndarray, W: np.ndarray, a_src: np.ndarray, a_dst: np.ndarray, bias: np.ndarray, act: int,
                            heads: int, slope: float = 0.2, dst: Optional[np.ndarray] = None, magnitude: bool = False):
    """Several heads: head i owns columns [i * d, (i + 1) * d) of W, a_src, a_dst and bias (d = columns / heads) and is
    one call of gat_layer_forward; the outputs are concatenated in head order."""
    W = np.asarray(W)
    d = W.shape[1] // heads
    assert d * heads == W.shape[1]
    outs = [gat_layer_forward(ms, h, W[:, i * d:(i + 1) * d], np.asarray(a_src)[i * d:(i + 1) * d], np.asarray(a_dst)[i * d:(i + 1) * d],
                              np.asarray(bias)[i * d:(i + 1) * d], act, slope, dst, magnitude) for i in range(heads)]
    if magnitude:
        return np.concatenate([o[0] for o in outs], axis=1), np.concatenate([o[1] for o in outs], axis=1)
    return np.concatenate(outs, axis=1)
