"""The forward-error gate of the GPU parity tests, checked on the CPU: the magnitude row it divides by is the layer's
own expression over absolute values (so it bounds the value and equals it on non-negative data), and a result with a
dropped, doubled or misplaced message fails the gate by orders of magnitude while fp32 rounding passes it."""
from dataclasses import replace

import numpy as np
import pytest

import taurus_gen as tg
from gpu_harness import forward_error, layer_on_input, run_oracle


def _case(mode, heads=1):
    w = replace(tg.scaled(tg.WORKLOADS["mid"], 600, chunk=128, name="gate"), mode=mode, dims=(12, 8 * heads, 8 * heads),
                fanout=(0, 0), pool_slots=600, hub_count=0, gat_heads=heads)
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.2)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    return w, g, model, x0, run_oracle(w, g, model, x0)


@pytest.mark.parametrize("mode,heads", [(tg.SAGE_MEAN, 1), (tg.GCN_SYM, 1), (tg.GIN_SUM, 1), (tg.GAT, 1), (tg.GAT, 2)])
def test_magnitude_row_bounds_the_value_and_equals_it_on_nonnegative_data(mode, heads):
    w, g, model, x0, orc = _case(mode, heads)
    no_act = replace(model, act=[0] * w.L)
    ref, mag = layer_on_input(w, no_act, orc, 0, x0)
    assert mag.shape == ref.shape and (mag >= 0).all()
    assert (np.abs(ref) <= mag * (1 + 1e-12) + 1e-300).all()
    # the chained oracle output of layer 0 is what layer_on_input evaluates on x0
    ref_act, _ = layer_on_input(w, model, orc, 0, x0)
    assert np.array_equal(ref_act, orc["outs"][0])
    if mode != tg.GAT:      # attention weights depend on the signs of the inputs; the linear modes do not
        pos = replace(no_act, W_neigh=[np.abs(x) for x in model.W_neigh], W_self=[np.abs(x) for x in model.W_self],
                      bias=[np.abs(x) for x in model.bias])
        ref_p, mag_p = layer_on_input(w, pos, orc, 0, np.abs(x0))
        assert np.allclose(ref_p, mag_p, rtol=1e-12, atol=0)


@pytest.mark.parametrize("mode", [tg.SAGE_MEAN, tg.GCN_SYM, tg.GIN_SUM])
def test_gate_passes_rounding_and_fails_a_dropped_message(mode):
    w, g, model, x0, orc = _case(mode)
    ref, mag = layer_on_input(w, model, orc, 0, x0)
    assert forward_error(ref.astype(np.float32), ref, mag) < 1e-6          # fp32 rounding of the result
    # drop one message: remove one edge of the graph and evaluate the same layer
    u = int(np.argmax(np.diff(g.row_ptr)))
    e = int(g.row_ptr[u])
    v = int(g.col_idx[e])
    row_ptr = g.row_ptr.copy(); row_ptr[u + 1:] -= 1
    col = np.delete(g.col_idx, e)
    g2 = replace(g, E=g.E - 1, row_ptr=row_ptr, col_idx=col)
    orc2 = run_oracle(w, g2, model, x0)
    bad = orc2["outs"][0].copy()
    # the degrees of the damaged graph differ too; put back everything but the row that lost its message
    keep = np.ones(g.V, bool); keep[v] = False
    bad[keep] = ref[keep]
    assert forward_error(bad, ref, mag) > 1e-3
