"""GATConv in three passes on the GPU (GATConv paragraph of Sect. 3.9) against the fp64 pull-based oracle."""
from dataclasses import replace

import numpy as np
import pytest

import taurus_gen as tg
from gpu_harness import check_accounting, forward_error, layer_on_input, row_error, run_library, run_oracle

pytestmark = pytest.mark.gpu

TOL = 1e-4


def _check(w, **kw):
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.3)
    # attention vectors of order one, so that the scores spread over several units and the softmax is far from uniform
    model.att_src = [(a * 4).astype(np.float32) for a in model.att_src]
    model.att_dst = [(a * 4).astype(np.float32) for a in model.att_dst]
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0, **kw)
    orc = run_oracle(w, g, model, x0)
    for l in range(w.L):
        row, elem_max, elem = row_error(lib["outs"][l], orc["outs"][l])
        print("GAT layer %d: row-wise %.3e element-wise max %.3e over 1e-4: %d of %d" % (l, row, elem_max, int((elem > TOL).sum()), elem.size))
        assert row <= TOL, (l, row)
        assert orc["sims"][l].rc == 0
        check_accounting(lib["stats"][l], lib["chunk_log"][l], lib["reload_count"][l], orc["sims"][l], lib["completed"][l])
    return lib, orc


def test_gat_exact_with_eviction_and_hubs():
    w = tg.scaled(tg.WORKLOADS["large"], 40_000, chunk=1024)
    w = replace(w, mode=tg.GAT, dims=(96, 128, 32), fanout=(0, 0), pool_slots=20_000, hub_count=40)
    lib, _ = _check(w)
    assert lib["stats"][0]["evictions"] > 0 and lib["stats"][0]["hub_messages"] > 0


def test_gat_sampled_and_ragged_widths():
    w = tg.scaled(tg.WORKLOADS["large"], 30_000, chunk=2048)
    w = replace(w, mode=tg.GAT, dims=(70, 50, 7), fanout=(6, 3), pool_slots=30_000, hub_count=0)   # widths not multiples of 4: repacked
    _check(w)


def test_gat_csr_order_kernels_and_host_rows():
    w = tg.scaled(tg.WORKLOADS["large"], 30_000, chunk=2048)
    w = replace(w, mode=tg.GAT, dims=(64, 64, 16), fanout=(0, 5), pool_slots=18_000, hub_count=30)
    _check(w, flags=4)                       # no grouped order: CSR-order scatter
    _check(w, host_features=True)            # features and transformed rows staged from pinned host memory


def test_gat_dense_output_mode_simt_projection():
    w = tg.scaled(tg.WORKLOADS["mid"], 20_011, chunk=4096)
    w = replace(w, mode=tg.GAT, dims=(100, 256, 47), fanout=(0, 0))
    _check(w, dense_output=True)
    _check(w, flags=2)                       # FFMA projection


@pytest.mark.parametrize("flags", [0, 4])      # grouped scatter; CSR-order scatter
def test_gat_destination_with_thousands_of_in_edges(flags):
    """The softmax normaliser of a destination with thousands of in-edges sums positive terms that differ by many orders
    of magnitude; added one by one in fp32 the small ones are lost (2e-4 of the sum at 8 000 in-edges, every output column
    of the row too large by as much).  The library sums it in double precision: the hub's row stays at rounding level."""
    w = tg.scaled(tg.WORKLOADS["stress"], 4_700, chunk=2048)
    w = replace(w, mode=tg.GAT, dims=(33, 4), fanout=(0,), pool_slots=5_000, hub_count=1, gemm_mode=tg.GEMM_FP32, leaky_slope=0.0)
    g = tg.make_graph(w)
    hub = int(np.argmax(g.in_degree))
    assert g.in_degree[hub] > 4000
    model = tg.make_model(w, bias_scale=0.3)
    model.att_src = [(a * 3).astype(np.float32) for a in model.att_src]
    model.att_dst = [(a * 3).astype(np.float32) for a in model.att_dst]
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0, flags=flags)
    orc = run_oracle(w, g, model, x0)
    ref, mag = layer_on_input(w, model, orc, 0, x0)
    err = forward_error(lib["outs"][0], ref, mag)
    hub_err = forward_error(lib["outs"][0][hub:hub + 1], ref[hub:hub + 1], mag[hub:hub + 1])
    print("in-degree %d: forward error of the hub's row %.3e, of the layer %.3e" % (g.in_degree[hub], hub_err, err))
    # the CSR-order kernels add the hub's 8 000 weighted rows one by one in fp32 (2e-5 here); the grouped order pre-sums them
    assert err <= (TOL if flags else 5e-6), err


def test_gat_several_heads_in_one_context():
    """Heads weight their own column blocks; one pass over the topology serves all of them.  Checked against the oracle
    (one single-head evaluation per head, concatenated) and, head by head, against single-head contexts of this library
    built from the head's own columns."""
    import paper_2607_17374_b200 as tb
    w = tg.scaled(tg.WORKLOADS["large"], 30_000, chunk=2048)
    w = replace(w, mode=tg.GAT, dims=(64, 96, 32), fanout=(0, 4), pool_slots=20_000, hub_count=30, gat_heads=4)
    lib, orc = _check(w)                       # grouped scatter, eviction, hubs, a sampled layer
    assert lib["stats"][0]["evictions"] > 0
    _check(w, flags=4)                         # CSR-order scatter
    _check(replace(w, dims=(256, 128, 64), gat_heads=2, pool_slots=30_000), dense_output=True)
    # head by head: layer 0 of a 4-head context = four 1-head contexts on the head's columns
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.3)
    model.att_src = [(a * 4).astype(np.float32) for a in model.att_src]
    model.att_dst = [(a * 4).astype(np.float32) for a in model.att_dst]
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    d = w.dims[1] // w.gat_heads
    for hd in range(w.gat_heads):
        w1 = replace(w, dims=(w.dims[0], d), fanout=(0,), gat_heads=1)
        m1 = replace(tg.make_model(w1), W_neigh=[np.ascontiguousarray(model.W_neigh[0][:, hd * d:(hd + 1) * d])],
                     W_self=[np.ascontiguousarray(model.W_neigh[0][:, hd * d:(hd + 1) * d])],
                     bias=[np.ascontiguousarray(model.bias[0][hd * d:(hd + 1) * d])], act=(model.act[0],),
                     att_src=[np.ascontiguousarray(model.att_src[0][hd * d:(hd + 1) * d])],
                     att_dst=[np.ascontiguousarray(model.att_dst[0][hd * d:(hd + 1) * d])])
        one = run_library(w1, g, m1, x0)
        diff = np.abs(one["outs"][0] - lib["outs"][0][:, hd * d:(hd + 1) * d]).max()
        print("head %d: single-head context against the head's block of the 4-head context: max abs difference %.3e" % (hd, diff))
        assert diff <= 2e-5
    # widths that a head cannot own as whole float4 are refused
    with pytest.raises(tb.TaurusError):
        run_library(replace(w, dims=(64, 100, 32)), g, tg.make_model(replace(w, dims=(64, 100, 32))), x0)


def test_gat_call_order_and_arguments():
    import torch
    import paper_2607_17374_b200 as tb
    E = tb.ERROR_CODES
    w = replace(tg.WORKLOADS["tiny"], mode=tg.GAT, dims=(64, 32), fanout=(0,))
    g = tg.make_graph(w)
    model = tg.make_model(w)

    def code(fn):
        with pytest.raises(tb.TaurusError) as ei:
            fn()
        return ei.value.code

    args = (g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, tg.GAT, w.dims, model.W_neigh, model.W_self, model.bias, model.act,
            w.chunk, w.pool_slots, 0, w.fanout, w.seed, 0, g.V)
    assert code(lambda: tb.Context(*args)) == E["INVALID_ARG"]                                              # no attention vectors
    assert code(lambda: tb.Context(*args, tb.GEMM_BF16, 0, 0, 0.0, model.att_src, model.att_dst)) == E["UNSUPPORTED"]
    assert code(lambda: tb.Context(*args, 0, 0, 0, 0.0, model.att_src, model.att_dst, -0.5)) == E["INVALID_ARG"]
    ctx = tb.Context(*args, 0, 0, 0, 0.0, model.att_src, model.att_dst, 0.2)
    x = torch.from_numpy(tg.features(w.seed, 0, 0, g.V, 64)).cuda()
    hp = torch.empty((g.V, 32), device="cuda")
    ctx.layer_begin(0)
    assert code(lambda: ctx.push_chunk(0, w.chunk, hp[:w.chunk])) == E["ORDER"]                             # before passes 1 and 2
    assert code(lambda: ctx.gat_attention()) == E["ORDER"]                                                  # nothing projected yet
    assert code(lambda: ctx.gat_project_chunk(w.chunk, 2 * w.chunk, x[w.chunk:2 * w.chunk], hp[w.chunk:], 32)) == E["ORDER"]
    assert code(lambda: ctx.gat_project_chunk(0, w.chunk, x[:w.chunk], hp.cpu(), 32)) == E["INVALID_ARG"]   # host destination
    for s in range(0, g.V, w.chunk):
        ctx.gat_project_chunk(s, min(g.V, s + w.chunk), x[s:s + w.chunk], hp[s:], 32)
    ctx.gat_attention()
    assert code(lambda: ctx.gat_attention()) == E["ORDER"]
    assert code(lambda: ctx.gat_project_chunk(0, w.chunk, x[:w.chunk], hp, 32)) == E["ORDER"]
    ids = torch.empty(g.V, dtype=torch.int64, device="cuda")
    out = torch.empty((g.V, 32), device="cuda")
    n = 0
    for s in range(0, g.V, w.chunk):
        ctx.push_chunk(s, min(g.V, s + w.chunk), hp[s:s + w.chunk])
        n += ctx.drain_dense(out, 32, g.V, ids)
    assert n == g.V and ctx.layer_end()["completed"] == g.V
    # the other modes refuse the GAT calls
    w2 = replace(tg.WORKLOADS["tiny"], dims=(64, 32), fanout=(0,))
    m2 = tg.make_model(w2)
    c2 = tb.Context(g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, w2.mode, w2.dims, m2.W_neigh, m2.W_self, m2.bias, m2.act,
                    w2.chunk, w2.pool_slots)
    c2.layer_begin(0)
    assert code(lambda: c2.gat_attention()) == E["UNSUPPORTED"]
    ctx.destroy(); c2.destroy()
