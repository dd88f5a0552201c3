"""Drives libtaurus through its binding for the GPU parity tests and compares with the oracle."""
from __future__ import annotations

import numpy as np

import oracle
import taurus_gen as tg


def run_library(w, g, model, x0, *, drain_each_chunk=True, flags=0, host_features=False, drain_rows=None,
                host_evict_rows=None, chunk_plan=None, gemm_mode=None, dense_output=False, evict_policy=0, run_output=None):
    """Runs every layer of workload w on the GPU.  Returns per-layer outputs (float32 [V, d_out]), the ids each
    chunk completed, stats and chunk logs.  Layer l+1 streams layer l's drained output."""
    import torch
    import paper_2607_17374_b200 as tb

    dev = torch.device("cuda:0")
    V, L = g.V, w.L
    # rows evicted at once, plus the transient of one chunk (victims leave before that chunk's reloads return rows)
    host_evict = host_evict_rows if host_evict_rows is not None else (
        0 if w.pool_slots >= V - w.hub_count else V - w.hub_count)
    ctx = tb.Context(V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                     model.act, w.chunk, w.pool_slots, w.hub_count, w.fanout, w.seed, host_evict,
                     drain_rows or (2 * V if (dense_output or run_output) else V), w.gemm_mode if gemm_mode is None else gemm_mode, flags, evict_policy, w.gin_eps,
                     model.att_src, model.att_dst, w.leaky_slope, w.gat_heads)
    res = dict(outs=[], completed=[], stats=[], chunk_log=[], reload_count=[], masks=[], ctx=ctx)
    if host_features:
        feat = torch.from_numpy(np.ascontiguousarray(x0)).pin_memory()
    else:
        feat = torch.from_numpy(np.ascontiguousarray(x0)).to(dev)
    stream = torch.cuda.current_stream()
    prev_runs = None
    res["runs"] = []
    for l in range(L):
        d_out = w.dims[l + 1]
        if dense_output and host_features:
            dense = torch.zeros((V, d_out), dtype=torch.float32).pin_memory()
        else:
            dense = torch.zeros((V, d_out), dtype=torch.float32, device=dev)
        ids_buf = torch.empty(V, dtype=torch.int64, device=dev)
        ctx.layer_begin(l, stream)
        if w.fanout[l] > 0:
            res["masks"].append(ctx.get_edge_mask())
        else:
            res["masks"].append(None)
        res.setdefault("digests", []).append(ctx.get_sample_digest())
        per_chunk = []
        plan = chunk_plan or [(s, min(s + w.chunk, V)) for s in range(0, V, w.chunk)]
        if w.mode == tg.GAT:  # passes 1 and 2; pass 3 below streams the transformed rows instead of the features
            hprime = torch.empty((V, d_out), dtype=torch.float32, device=dev)
            for (s, e) in plan:
                if run_output and prev_runs is not None:
                    ctx.gat_project_chunk_from_runs(s, e, prev_runs, hprime[s:e], d_out, stream)
                else:
                    ctx.gat_project_chunk(s, e, feat[s:e], hprime[s:e], d_out, stream)
            ctx.gat_attention(stream)
            layer_in, feat = feat, (hprime.cpu().pin_memory() if host_features else hprime)
        if run_output:        # rows leave as sorted runs; layers after the first read their input back from runs
            P, R, kind = run_output
            runs = tb.Runs(V, d_out, P, R, store_rows=V, max_append_rows=V, max_chunk_rows=w.chunk, store_kind=kind)
            ctx.layer_set_run_output(runs)
            for (s, e) in plan:
                if prev_runs is None or w.mode == tg.GAT:      # GAT: pass 3 streams the transformed rows of pass 1
                    ctx.push_chunk(s, e, feat[s:e], stream)
                else:
                    ctx.push_chunk_from_runs(s, e, prev_runs, stream)
            per_chunk = None
        elif dense_output:    # the library places every finalised row itself; nothing to drain
            ctx.layer_set_dense_output(dense, d_out)
            for (s, e) in plan:
                ctx.push_chunk(s, e, feat[s:e], stream)
            assert ctx.drain_dense(dense, d_out, V, ids_buf) == 0
            per_chunk = None
        else:
            for (s, e) in plan:
                rc = ctx.push_chunk(s, e, feat[s:e], stream, raise_on_drain_full=False)
                if rc != 0:   # graduation buffer could overflow: drain, then push again
                    n = ctx.drain_dense(dense, d_out, V, ids_buf)
                    per_chunk.append(("drain", ids_buf[:n].cpu().numpy().copy()))
                    ctx.push_chunk(s, e, feat[s:e], stream)
                if drain_each_chunk:
                    n = ctx.drain_dense(dense, d_out, V, ids_buf)
                    per_chunk.append(ids_buf[:n].cpu().numpy().copy())
            n = ctx.drain_dense(dense, d_out, V, ids_buf)
            if n or not drain_each_chunk:
                per_chunk.append(("tail", ids_buf[:n].cpu().numpy().copy()))
        res["stats"].append(ctx.layer_end())
        if run_output:
            for (s, e) in [(s, min(s + w.chunk, V)) for s in range(0, V, w.chunk)]:
                runs.read_chunk(s, e, dense[s:e], d_out, stream)
            torch.cuda.synchronize()
            if prev_runs is not None:
                prev_runs.destroy()
            prev_runs = runs
            res["runs"].append(runs)
        res["chunk_log"].append(ctx.get_chunk_log())
        res["reload_count"].append(ctx.get_vertex_array("reload_count"))
        res["completed"].append(per_chunk)
        res["outs"].append(dense.cpu().numpy())
        feat = dense if (dense_output or not host_features) else dense.cpu().pin_memory()
    return res


def run_oracle(w, g, model, x0, evict_policy=0):
    """Oracle outputs for every layer plus the integer simulation per layer."""
    inl = oracle.build_in_lists(g.V, g.row_ptr, g.col_idx)
    din, dout = np.diff(inl.ptr), np.diff(g.row_ptr)
    hub = oracle.hub_set(g.in_degree, w.hub_count)
    h = x0.astype(np.float64)
    out = dict(outs=[], sims=[], msets=[], hub=hub, din=din, dout=dout)
    for l in range(w.L):
        ms = oracle.message_sets(inl, w.fanout[l], w.seed, l)
        if w.mode == tg.GAT:
            from oracle import gat
            h = gat.gat_layer_forward_heads(ms, h, model.W_neigh[l], model.att_src[l], model.att_dst[l], model.bias[l], model.act[l],
                                            w.gat_heads, w.leaky_slope)
        else:
            h = oracle.layer_forward(ms, w.mode, din, dout, h, model.W_neigh[l], model.W_self[l], model.bias[l], model.act[l],
                                     gin_eps=w.gin_eps)
        out["outs"].append(h)
        out["sims"].append(oracle.simulate(g.V, g.row_ptr, g.col_idx, ms, hub, w.chunk, w.pool_slots, evict_policy, w.seed))
        out["msets"].append(ms)
    return out


def layer_on_input(w, model, orc, l, h_in):
    """Layer l evaluated by the oracle on the rows h_in (those the library consumed for that layer).  Returns
    (ref, mag): ref is the layer's definition in fp64; mag is the same expression with every term replaced by its
    absolute value,  c_in sum c_out |h_u| |W_neigh| + c_self |h_v| |W_self| + |b|  (GAT: attention weights times
    |h_u| |W|): the sum of the magnitudes of everything that is added up for an output element."""
    ms = orc["msets"][l]
    h = np.asarray(h_in, dtype=np.float64)
    if w.mode == tg.GAT:
        from oracle import gat
        return gat.gat_layer_forward_heads(ms, h, model.W_neigh[l], model.att_src[l], model.att_dst[l], model.bias[l], model.act[l],
                                           w.gat_heads, w.leaky_slope, magnitude=True)
    ref = oracle.layer_forward(ms, w.mode, orc["din"], orc["dout"], h, model.W_neigh[l], model.W_self[l], model.bias[l], model.act[l],
                               gin_eps=w.gin_eps)
    mag = oracle.layer_forward(ms, w.mode, orc["din"], orc["dout"], np.abs(h), np.abs(model.W_neigh[l]), np.abs(model.W_self[l]),
                               np.abs(model.bias[l]), 0, gin_eps=w.gin_eps)   # 1 + eps > 0 for every eps the tests draw
    return ref, mag


def forward_error(got, ref, mag):
    """max over rows of ||g_v - r_v||_inf / ||mag_v||_inf: the error of a row measured against the magnitude of what
    was summed for it.  A computation that rounds every product and partial sum to a relative u ends below
    (number of terms) * u on this scale, whatever the cancellation in the row; a dropped, doubled or misplaced term
    ends near 1.  (The activation does not increase an error: |relu(a) - relu(b)| <= |a - b|.)"""
    diff = np.abs(got.astype(np.float64) - ref).max(axis=1)
    scale = np.abs(mag).max(axis=1)
    exact = scale == 0
    assert (diff[exact] == 0).all()          # nothing was summed: the row is exactly zero on both sides
    return float((diff[~exact] / scale[~exact]).max()) if (~exact).any() else 0.0


def row_error(got, ref):
    """max over rows of ||g_v - r_v||_inf / (||r_v||_inf + 1e-6), and the element-wise figures."""
    got = got.astype(np.float64)
    diff = np.abs(got - ref)
    row = diff.max(axis=1) / (np.abs(ref).max(axis=1) + 1e-6)
    elem = diff / (np.abs(ref) + 1e-6)
    return float(row.max()), float(elem.max()), elem


def check_accounting(lib_stats, lib_log, lib_reload, sim, completed_chunks=None):
    st = sim.stats
    for k_lib, k_or in [("evictions", "evictions"), ("reloads", "reloads"), ("max_reload_count", "max_reload_count"),
                        ("peak_occupancy", "peak_occupancy"), ("hub_messages", "hub_messages"),
                        ("total_messages", "total_messages"), ("hub_vertices", "hub_vertices"), ("completed", "completed"),
                        ("sum_hs", "sum_hs"), ("sum_ns", "sum_ns"), ("sum_ev", "sum_ev"), ("sum_gs", "sum_gs"),
                        ("free_slots", "free_end")]:
        assert lib_stats[k_lib] == st[k_or], (k_lib, lib_stats[k_lib], st[k_or])
    for k in ["hs", "ns", "ev", "gs", "need", "evicted", "reloaded", "completed", "occupancy"]:
        assert (lib_log[k] == sim.per_chunk[k]).all(), k
    assert (lib_reload == sim.reload_count).all()
    hist = np.bincount(np.minimum(sim.reload_count, 16), minlength=17)
    assert lib_stats["reload_histogram"] == hist.tolist()
    if completed_chunks is not None:
        for c, ids in enumerate(completed_chunks):
            want = np.flatnonzero(sim.complete_chunk == c)
            assert ids.size == want.size and (np.sort(ids) == want).all(), c
