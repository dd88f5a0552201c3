"""Layers that are abandoned half-way and begun again, and two contexts interleaved on one device: state left
over from the abandoned pass (pending counts, slots, evicted rows, graduation halves, open appends, GAT scalars)
must not leak into the next one."""
from dataclasses import replace

import numpy as np
import pytest

import taurus_gen as tg
from gpu_harness import check_accounting, row_error, run_oracle

pytestmark = pytest.mark.gpu


def make(w, **kw):
    import paper_2607_17374_b200 as tb
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.3)
    host_evict = 0 if w.pool_slots >= g.V - w.hub_count else g.V - w.hub_count
    ctx = tb.Context(g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                     model.act, w.chunk, w.pool_slots, w.hub_count, w.fanout, w.seed, host_evict, 2 * g.V, w.gemm_mode, 0, 0,
                     w.gin_eps, model.att_src, model.att_dst, w.leaky_slope, w.gat_heads)
    return g, model, ctx


def one_layer(ctx, w, g, feat, mode, runs=None, stop_after=None, hprime=None):
    """Runs layer 0 in the given output mode; stops after `stop_after` chunks when given.  Returns the dense output."""
    import torch
    dev = torch.device("cuda:0")
    V, d_out = g.V, w.dims[1]
    dense = torch.zeros((V, d_out), device=dev)
    ids = torch.empty(V, dtype=torch.int64, device=dev)
    plan = [(s, min(s + w.chunk, V)) for s in range(0, V, w.chunk)]
    ctx.layer_begin(0)
    src = feat
    if w.mode == tg.GAT:
        for i, (s, e) in enumerate(plan):
            if stop_after is not None and stop_after < 0 and i >= -stop_after:
                return None                                      # abandoned during pass 1
            ctx.gat_project_chunk(s, e, feat[s:e], hprime[s:e], d_out)
        ctx.gat_attention()
        src = hprime
    if mode == "dense":
        ctx.layer_set_dense_output(dense, d_out)
    elif mode == "runs":
        ctx.layer_set_run_output(runs)
    for i, (s, e) in enumerate(plan):
        if stop_after is not None and stop_after >= 0 and i >= stop_after:
            return None
        ctx.push_chunk(s, e, src[s:e])
        if mode == "drain":
            ctx.drain_dense(dense, d_out, V, ids)
    st = ctx.layer_end()
    if mode == "runs":
        for (s, e) in plan:
            runs.read_chunk(s, e, dense[s:e], d_out)
        torch.cuda.synchronize()
    return dense.cpu().numpy(), st, ctx.get_chunk_log(), ctx.get_vertex_array("reload_count")


@pytest.mark.parametrize("mode", ["drain", "dense", "runs"])
@pytest.mark.parametrize("model_mode", [tg.SAGE_MEAN, tg.GAT])
def test_abandoned_layer_then_clean_pass(mode, model_mode):
    import torch
    import paper_2607_17374_b200 as tb
    w = tg.scaled(tg.WORKLOADS["large"], 30_000, chunk=1024)
    w = replace(w, mode=model_mode, dims=(64, 48), fanout=(0,), pool_slots=12_000, hub_count=30)
    g, model, ctx = make(w)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    feat = torch.from_numpy(x0).cuda()
    hprime = torch.empty((g.V, 48), device="cuda")
    runs = tb.Runs(g.V, 48, 5, 2000, max_chunk_rows=w.chunk) if mode == "runs" else None
    orc = run_oracle(w, g, model, x0)
    assert orc["sims"][0].stats["evictions"] > 0
    for stop in ([-7, 11, 23] if model_mode == tg.GAT else [11, 23]):      # negative: abandoned during GAT pass 1
        assert one_layer(ctx, w, g, feat, mode, runs, stop_after=stop, hprime=hprime) is None
        if runs is not None:
            runs.reset()                                          # forget the abandoned pass's runs and its open append
    out, st, log, reloads = one_layer(ctx, w, g, feat, mode, runs, hprime=hprime)
    row, _, _ = row_error(out, orc["outs"][0])
    assert row <= 1e-4
    check_accounting(st, log, reloads, orc["sims"][0])
    ctx.destroy()


def test_two_contexts_interleaved():
    import torch
    wa = replace(tg.scaled(tg.WORKLOADS["large"], 20_000, chunk=1024), dims=(64, 128), fanout=(0,), pool_slots=12_000, hub_count=20)
    wb = replace(tg.scaled(tg.WORKLOADS["stress"], 16_000, chunk=512), dims=(96, 32), fanout=(0,), gemm_mode=tg.GEMM_FP32, pool_slots=9_000)
    ga, ma, ca = make(wa)
    gb, mb, cb = make(wb)
    xa, xb = tg.features(wa.seed, 0, 0, ga.V, 64), tg.features(wb.seed, 0, 0, gb.V, 96)
    fa, fb = torch.from_numpy(xa).cuda(), torch.from_numpy(xb).cuda()
    da, db = torch.zeros((ga.V, 128), device="cuda"), torch.zeros((gb.V, 32), device="cuda")
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    ca.layer_begin(0, sa); cb.layer_begin(0, sb)
    ca.layer_set_dense_output(da, 128); cb.layer_set_dense_output(db, 32)
    pa = [(s, min(s + wa.chunk, ga.V)) for s in range(0, ga.V, wa.chunk)]
    pb = [(s, min(s + wb.chunk, gb.V)) for s in range(0, gb.V, wb.chunk)]
    for i in range(max(len(pa), len(pb))):                       # alternate pushes of the two contexts on two streams
        if i < len(pa):
            ca.push_chunk(pa[i][0], pa[i][1], fa[pa[i][0]:pa[i][1]], sa)
        if i < len(pb):
            cb.push_chunk(pb[i][0], pb[i][1], fb[pb[i][0]:pb[i][1]], sb)
    sta, stb = ca.layer_end(), cb.layer_end()
    oa, ob = run_oracle(wa, ga, ma, xa), run_oracle(wb, gb, mb, xb)
    assert row_error(da.cpu().numpy(), oa["outs"][0])[0] <= 1e-4
    assert row_error(db.cpu().numpy(), ob["outs"][0])[0] <= 1e-4
    check_accounting(sta, ca.get_chunk_log(), ca.get_vertex_array("reload_count"), oa["sims"][0])
    check_accounting(stb, cb.get_chunk_log(), cb.get_vertex_array("reload_count"), ob["sims"][0])
    ca.destroy(); cb.destroy()
