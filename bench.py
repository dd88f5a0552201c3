"""Benchmark of the source-centric broadcast step (libtaurus) on synthetic graphs.

A step is one full pass of the hot path over the workload: every layer, every chunk (copy-in, projection,
classify, make-room, scatter, finalise, drain).  The metric is propagated edges per second (GTEPS,
self messages not counted) over the whole step.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload mid] [--impl ours|reference]

N > 1 (under torchrun): the path has no exchange step, so every rank runs an independent replica of the
workload on its own GPU ("replicas only", weak scaling); the value is the sum over ranks / max time.
--impl reference times the CPU oracle (a deliberately plain program) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import taurus_gen as tg  # noqa: E402


# DRAM bytes (read + write) per accumulator-row reduction of scatter_grouped_kernel<32,2>, from the ncu capture
# summarised in profiles/scatter_grouped_kernel_mid_1200k.md (2.67 GB per launch / 0.98 M groups).
SCATTER_TRAFFIC_PER_GROUP_BYTES = 2720.0


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=3)
    p.add_argument("--warmup", type=int, default=3)
    p.add_argument("--workload", default="mid")
    p.add_argument("--vertices", type=int, default=0, help="scale the workload to this many vertices (0 = full size)")
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--simt-gemm", action="store_true", help="use the plain FFMA projection kernel")
    p.add_argument("--no-grouping", action="store_true", help="CSR-order scatter for every chunk")
    p.add_argument("--project-first", action="store_true",
                   help="project every chunk before scattering it, also where the layer's input rows are narrower than its output rows")
    p.add_argument("--pool-fraction", type=float, default=0.0,
                   help="accumulator pool as a fraction of V (0 = the workload's own pool); below the peak active set it forces eviction")
    p.add_argument("--evict-policy", default="fewest", choices=["fewest", "fifo", "lru", "random"],
                   help="which IN_BUFFER rows leave first when the pool is full (the paper's policy and its ablation's alternatives)")
    p.add_argument("--model", default="", choices=["", "sage", "gcn", "gin", "gat"],
                   help="aggregation of every layer (default: the workload's); gat runs its three passes per layer")
    p.add_argument("--output", default="dense", choices=["dense", "runs-device", "runs-host"],
                   help="where a layer's rows go: a dense matrix in HBM (default), or sorted runs (in HBM / pinned host "
                        "memory) that the next layer reads back by merge-on-read")
    return p.parse_args()


def workload_of(args):
    w = tg.WORKLOADS[args.workload]
    if args.vertices:
        w = tg.scaled(w, args.vertices)
    if args.pool_fraction > 0:
        from dataclasses import replace
        w = replace(w, pool_slots=max(1, int(w.V * args.pool_fraction)))
    if args.model:
        from dataclasses import replace
        w = replace(w, mode={"sage": tg.SAGE_MEAN, "gcn": tg.GCN_SYM, "gin": tg.GIN_SUM, "gat": tg.GAT}[args.model],
                    gemm_mode=tg.GEMM_FP32 if args.model == "gat" else w.gemm_mode)
    return w


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples the SM clock and the throttle reasons while the timed region runs: through NVML every 10 ms
    when the bindings are importable (read-only queries), else through nvidia-smi every 200 ms."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    # NVML clocks-event reason bits
    BITS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.stop_flag = index, threading.Event()
        self.mhz, self.reasons, self.max_mhz, self.source = [], set(), None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible and all(x.strip().isdigit() for x in visible.split(",")):
                phys = int(visible.split(",")[index])
            self.nvml, self.handle = pynvml, pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM))
            self.source = "nvml"
        except Exception:
            self.nvml = None
            self.source = "nvidia-smi"

    def run(self):
        while not self.stop_flag.is_set():
            try:
                if self.nvml is not None:
                    self.mhz.append(float(self.nvml.nvmlDeviceGetClockInfo(self.handle, self.nvml.NVML_CLOCK_SM)))
                    bits = int(self.nvml.nvmlDeviceGetCurrentClocksEventReasons(self.handle)) \
                        if hasattr(self.nvml, "nvmlDeviceGetCurrentClocksEventReasons") \
                        else int(self.nvml.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle))
                    for name, bit in self.BITS.items():
                        if bits & bit:
                            self.reasons.add(name)
                else:
                    out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                    f = [x.strip() for x in out.strip().split(",")]
                    if len(f) >= 6:
                        self.mhz.append(float(f[0])); self.max_mhz = float(f[1])
                        for i, name in enumerate(["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]):
                            if f[2 + i].lower().startswith("active"):
                                self.reasons.add(name)
            except Exception:
                pass
            self.stop_flag.wait(0.01 if self.nvml is not None else 0.2)

    def summary(self):
        if not self.mhz:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=[], samples=0, source=self.source)
        mhz = sorted(self.mhz)
        return dict(sm_mhz=mhz[len(mhz) // 2], sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), samples=len(mhz),
                    source=self.source)


# ----------------------------------------------------------------------------------------------- reference arm / CPU baseline

def oracle_sample(w, g, budget_s=12.0, inl=None):
    """Times the oracle (as it stands) on a bounded destination sample of layer 0.  Returns (edges/s, info)."""
    import oracle
    t0 = time.time()
    inl = inl or oracle.build_in_lists(g.V, g.row_ptr, g.col_idx)
    t_inl = time.time() - t0
    ms = oracle.message_sets(inl, w.fanout[0], w.seed, 0)
    model = tg.make_model(w)
    rng = np.random.default_rng(0)
    n_dst = min(g.V, 4096)
    rate, used, edges, total_t = 0.0, 0, 0, 0.0
    x = tg.features(w.seed, 0, 0, g.V, w.dims[0]).astype(np.float64)
    din, dout = np.diff(inl.ptr), np.diff(g.row_ptr)
    while True:
        dst = np.sort(rng.choice(g.V, size=n_dst, replace=False)).astype(np.int64)
        t1 = time.time()
        oracle.layer_forward(ms, w.mode, din, dout, x, model.W_neigh[0], model.W_self[0], model.bias[0], model.act[0], dst)
        dt = time.time() - t1
        e = int(ms.m[dst].sum())
        edges += e; total_t += dt; used += n_dst
        rate = e / dt
        if total_t >= budget_s or n_dst >= g.V:
            break
        n_dst = int(min(g.V, max(n_dst * 2, n_dst * (budget_s - total_t) / max(dt, 1e-3) * 0.7)))
    info = dict(cores=oracle.cores_used(), kind="oracle",
                sample="layer 0 (%d -> %d), %d sampled destinations, %d in-edges pulled in %.1f s; in-list build %.1f s not counted"
                       % (w.dims[0], w.dims[1], used, edges, total_t, t_inl))
    return edges / total_t, info, inl


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = workload_of(args)
    g = tg.make_graph(w)
    inl = None
    for _ in range(max(args.warmup, 0) and 1):
        _, _, inl = oracle_sample(w, g, 2.0, inl)
    vals, info = [], None
    t0 = time.time()
    for _ in range(args.steps):
        v, info, inl = oracle_sample(w, g, 8.0, inl)
        vals.append(v)
    value = float(np.mean(vals)) / 1e9
    line = dict(impl="reference", metric="edges/sec per GNN layer (GTEPS)", value=value, unit="GTEPS", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=(time.time() - t0) * 1e3 / max(args.steps, 1),
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, V=g.V, E=g.E, dims=list(w.dims), l2="inputs larger than L2"),
                cpu_baseline=dict(value=value, unit="GTEPS", **info),
                e2e=dict(value=value, unit="GTEPS", h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- ranks

def max_over_ranks(ms: float, world: int, device=None) -> float:
    """Slowest rank's time: every rank runs an independent replica, the job is as slow as its slowest rank."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(units_per_rank_step: float, steps: int, world: int, ms_max: float) -> float:
    """Units all ranks processed / the slowest rank's time, in 1e9 units per second (weak scaling: replicas only)."""
    return world * units_per_rank_step * steps / (ms_max * 1e-3) / 1e9


# ----------------------------------------------------------------------------------------------- our arm

def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2607_17374_b200 as tb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    w = workload_of(args)
    g = tg.make_graph(w)
    model = tg.make_model(w)
    V, L = g.V, w.L
    chunks = [(s, min(s + w.chunk, V)) for s in range(0, V, w.chunk)]
    ctx_bound = V   # upper bound on the rows one chunk can complete
    # two graduation halves; badly ordered graphs complete a large share of V in the last chunks
    drain_rows = 2 * max(ctx_bound, w.chunk)
    host_evict = 0 if w.pool_slots >= V - w.hub_count else V - w.hub_count
    flags = (tb.FLAG_SIMT_GEMM if args.simt_gemm else 0) | (tb.FLAG_NO_GROUPING if args.no_grouping else 0) | \
        (tb.FLAG_PROJECT_FIRST if args.project_first else 0)
    pad4 = lambda x: (x + 3) // 4 * 4
    # the library's rule: a layer whose input rows are at most 3/4 as wide as its output rows aggregates input rows and
    # transforms the finished rows (SAGE: while its per-vertex store of input rows stays below 64 GiB)
    agg_first = [(not args.project_first) and 4 * pad4(w.dims[l]) <= 3 * pad4(w.dims[l + 1]) and
                 (w.mode != tg.SAGE_MEAN or V * pad4(w.dims[l]) * 4 <= (64 << 30)) for l in range(L)]
    ctx = tb.Context(V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                     model.act, w.chunk, w.pool_slots, w.hub_count, w.fanout, w.seed, host_evict, drain_rows, w.gemm_mode, flags,
                     {"fewest": 0, "fifo": 1, "lru": 2, "random": 3}[args.evict_policy], w.gin_eps, model.att_src, model.att_dst,
                     w.leaky_slope)
    gat = w.mode == tg.GAT
    use_runs = args.output != "dense"
    hprime = torch.zeros((V, max(w.dims[1:])), dtype=torch.float32, device=dev) if gat else None
    runs = None
    if use_runs:   # one run store per layer output: 16 id ranges, buffers of 32 768 rows
        kind = tb.RUNS_DEVICE if args.output == "runs-device" else tb.RUNS_HOST
        runs = [tb.Runs(V, w.dims[l + 1], 16, 32768, store_rows=V, max_append_rows=max(V, w.chunk), max_chunk_rows=w.chunk,
                        store_kind=kind) for l in range(L)]
    x_host = torch.empty((V, w.dims[0]), dtype=torch.float32).pin_memory()
    tg.features(w.seed, 0, 0, V, w.dims[0], out=x_host.numpy())
    x_dev = x_host.to(dev)
    dmax = max(w.dims[1:])
    dense_dev = [torch.zeros(V * dmax, dtype=torch.float32, device=dev) for _ in range(2)]
    out_dev = torch.zeros((V, w.dims[-1]), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    edges_per_layer = []
    groups_per_layer = []

    def step(feat0, final_out, collect_stats=False):
        """One pass over all layers.  feat0 is the layer-0 feature matrix (device for `value`, pinned host for e2e);
        intermediate layer outputs [V, dims[l+1]] stay in HBM (two ping-pong buffers) and are streamed by the next
        layer; the last layer's output goes to final_out (device for `value`, pinned host for e2e)."""
        feat = feat0
        for l in range(L):
            d_out = w.dims[l + 1]
            out = final_out if l == L - 1 else dense_dev[l % 2][:V * d_out].view(V, d_out)
            ctx.layer_begin(l, stream)
            src = feat
            if gat:    # passes 1 and 2: transformed rows and attention scalars, then the topology-only sweep
                hp = hprime.view(-1)[:V * d_out].view(V, d_out)
                for (s, e) in chunks:
                    if use_runs and l > 0:
                        ctx.gat_project_chunk_from_runs(s, e, runs[l - 1], hp[s:e], d_out, stream)
                    else:
                        ctx.gat_project_chunk(s, e, feat[s:e], hp[s:e], d_out, stream)
                ctx.gat_attention(stream)
                src = hp
            if use_runs:
                runs[l].reset()
                ctx.layer_set_run_output(runs[l])
                for (s, e) in chunks:
                    if l == 0 or gat:      # gat: pass 3 streams the transformed rows of pass 1
                        ctx.push_chunk(s, e, src[s:e], stream)
                    else:
                        ctx.push_chunk_from_runs(s, e, runs[l - 1], stream)
            else:
                ctx.layer_set_dense_output(out, d_out)   # finalised rows go straight to their place in the matrix
                for (s, e) in chunks:
                    ctx.push_chunk(s, e, src[s:e], stream)
            st = ctx.layer_end()
            if collect_stats:
                edges_per_layer.append(st["total_messages"])
                groups_per_layer.append(st["scatter_groups"])
            feat = out
        if use_runs:   # the result is read back from the last layer's runs in vertex order
            for (s, e) in chunks:
                runs[L - 1].read_chunk(s, e, final_out[s:e], w.dims[-1], stream)
        return feat

    # warm-up (also collects the per-layer message counts)
    barrier()
    for i in range(max(args.warmup, 1)):
        step(x_dev, out_dev, collect_stats=(i == 0))
    torch.cuda.synchronize()
    msgs_per_step = int(sum(edges_per_layer))

    # ---- device-resident timing
    sampler = ClockSampler(local)
    sampler.start()
    ctx.set_timing(True)
    launches0 = ctx.launch_count()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step(x_dev, out_dev)
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1)
    ctx.set_timing(False)
    launches = ctx.launch_count() - launches0
    sampler.stop_flag.set()
    sampler.join()
    phases = ctx.get_phase_ms()   # [pushes, 6]
    ms_max = max_over_ranks(ms, world, dev)
    value = whole_job_value(msgs_per_step, args.steps, world, ms_max)

    # ---- roofline of the dominant kernel (the scatter), from the events recorded inside the timed region
    n_push = len(chunks) * L * args.steps
    ph = phases[:n_push].reshape(args.steps, L, len(chunks), 6)
    scatter_ms = ph[..., 4]
    # Algorithmic bytes of the scatter: per accumulator-row reduction a read-modify-write of
    # the row (2 * 4 Hp) plus slot and pending-count words (8); per propagated edge its (destination, source)
    # words (8); per source its projected row read once (4 Hp) and its self message (row read 4 Hp + RMW 2 * 4 Hp + 8).
    # In CSR order a "group" is one edge.  The per-edge cold-miss model (12 + 2 * 4 Hp per edge) is kept beside it.
    layer_bytes, edge_model_bytes = [], []
    n_src = V
    acc_width = [pad4(w.dims[l]) if agg_first[l] else pad4(w.dims[l + 1]) for l in range(L)]   # floats per accumulator row
    for l in range(L):
        Wd = acc_width[l]
        self_row = not (agg_first[l] and w.mode == tg.SAGE_MEAN)   # aggregate-first SAGE adds its self term after the transform
        layer_bytes.append(groups_per_layer[l] * (8 * Wd + 8) + edges_per_layer[l] * 8 +
                           n_src * (4 * Wd + (12 * Wd if self_row else 0) + 8))
        edge_model_bytes.append(edges_per_layer[l] * (12 + 8 * Wd) + n_src * (4 * Wd + 8))
    alg_bytes_step = float(sum(layer_bytes))
    scatter_total_ms = float(scatter_ms.sum()) / args.steps
    pk = peaks()
    grouped = not args.no_grouping
    # The dominant kernel is the scatter instance with the largest total time: layers with the same accumulator width
    # run the same template instance.  `achieved` = its algorithmic bytes / its CUDA-event time; the other instances
    # are listed per layer, and the figure over all scatter launches is kept as all_scatter_gbs.
    per_layer_ms = [float(scatter_ms[:, l].sum()) / args.steps for l in range(L)]
    by_width = {}
    for l in range(L):
        by_width.setdefault(acc_width[l], []).append(l)
    dom_w = max(by_width, key=lambda k: sum(per_layer_ms[l] for l in by_width[k]))
    dom = by_width[dom_w]
    dom_ms = sum(per_layer_ms[l] for l in dom)
    dom_bytes = float(sum(layer_bytes[l] for l in dom))
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    kname = ("scatter_grouped_kernel" if grouped else "scatter_kernel") + " (accumulator rows of %d floats, layers %s)" % (dom_w, dom)
    roofline = dict(bound="hbm", kernel=kname, achieved=achieved,
                    peak=pk["hbm_gbs"], unit="GB/s", frac=achieved / pk["hbm_gbs"], peak_source=pk["source"],
                    traffic=SCATTER_TRAFFIC_PER_GROUP_BYTES * sum(groups_per_layer[l] for l in dom) / (len(dom) * len(chunks))
                    if grouped and dom_w == 256 else None,
                    traffic_note="ncu dram read+write per launch of the 256-float kernel, scaled by groups per launch "
                                 "(profiles/scatter_grouped_kernel_mid_1200k.md)" if grouped and dom_w == 256 else None,
                    launches_per_step=len(chunks) * len(dom), avg_launch_ms=dom_ms / (len(chunks) * len(dom)),
                    algorithmic_bytes_per_launch=dom_bytes / (len(chunks) * len(dom)),
                    share_of_step=dom_ms / (ms_max / args.steps),
                    all_scatter_gbs=alg_bytes_step / (scatter_total_ms * 1e-3) / 1e9,
                    edge_model_gbs=float(sum(edge_model_bytes)) / (scatter_total_ms * 1e-3) / 1e9,
                    per_layer=[dict(layer=l, scatter_ms=per_layer_ms[l],
                                    gbs=layer_bytes[l] / (per_layer_ms[l] * 1e-3) / 1e9,
                                    groups=int(groups_per_layer[l]), accumulator_floats=acc_width[l], aggregate_first=bool(agg_first[l]),
                                    gteps_scatter_only=edges_per_layer[l] / (per_layer_ms[l] * 1e-3) / 1e9)
                               for l in range(L)])
    phase_ms = dict(zip(["copy_in", "projection", "classify_select", "row_moves", "scatter", "finalise"],
                        [float(x) / args.steps for x in ph.sum(axis=(0, 1, 2))]))

    # ---- end to end through the C ABI with host buffers: every step streams the layer-0 features from pinned host
    # memory (one host -> device copy per chunk, inside push_chunk) and brings the last layer's rows back to pinned
    # host memory with one device -> host copy once the layer has ended (most vertices of this graph complete in the
    # last chunks of a layer, so there is nothing to overlap with inside the step; the library can also write finished
    # rows to pinned host memory itself, which is slower here because the copy engine moves rows faster than kernel
    # stores over PCIe).  That copy runs on a side stream out of one of two result buffers, so it overlaps the first
    # layer of the following step, as a serving loop would do; the timed region ends when the last copy has landed.
    # Intermediate layers stay in HBM, where they fit.
    e2e = None
    if not args.no_e2e:
        outs_dev = [out_dev, torch.zeros_like(out_dev)]
        outs_host = [torch.zeros((V, w.dims[-1]), dtype=torch.float32).pin_memory() for _ in range(2)]
        d2h_stream = torch.cuda.Stream()
        step_done = [torch.cuda.Event() for _ in range(2)]
        d2h_done = [torch.cuda.Event() for _ in range(2)]

        def e2e_step(i):
            b = i & 1
            stream.wait_event(d2h_done[b])            # the result buffer's previous copy has left
            step(x_host, outs_dev[b])
            step_done[b].record(stream)
            with torch.cuda.stream(d2h_stream):
                d2h_stream.wait_event(step_done[b])
                outs_host[b].copy_(outs_dev[b], non_blocking=True)
                d2h_done[b].record(d2h_stream)

        for b in range(2):
            d2h_done[b].record(stream)
        e2e_step(0)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(stream)
        for i in range(args.steps):
            e2e_step(i + 1)
        for b in range(2):
            stream.wait_event(d2h_done[b])
        e1.record(stream)
        barrier()
        wall = (time.time() - t0) * 1e3
        e2e_ms = max_over_ranks(max(e0.elapsed_time(e1), wall), world, dev)
        e2e = dict(value=whole_job_value(msgs_per_step, args.steps, world, e2e_ms), unit="GTEPS",
                   ms_per_step=e2e_ms / args.steps,
                   h2d_bytes_per_step=int(4 * V * w.dims[0]), d2h_bytes_per_step=int(4 * V * w.dims[-1]),
                   note="layer-0 features host -> device per chunk; last layer's rows device -> host in one copy per step on a "
                        "side stream, overlapping the next step's first layer; intermediate layers in HBM")
        out_host = outs_host
        del out_host

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not gat:
        v, info, _ = oracle_sample(w, g, 12.0)
        cpu = dict(value=v / 1e9, unit="GTEPS", **info)

    if rank == 0:
        line = dict(metric="edges/sec per GNN layer (GTEPS)", value=value, unit="GTEPS", n_gpus=world, steps=args.steps,
                    warmup=args.warmup, ms_per_step=ms_max / args.steps, higher_is_better=True, scaling="weak",
                    vs_baseline=None, dtype="f32", data="synthetic",
                    config=dict(workload=w.name, V=V, E=g.E, dims=list(w.dims), chunk=w.chunk, chunks_per_layer=len(chunks),
                                pool_slots=w.pool_slots, hub_count=w.hub_count, fanout=list(w.fanout),
                                mode=["sage_mean", "gcn_sym", "gin_sum", "gat"][w.mode], output=args.output, evict_policy=args.evict_policy,
                                messages_per_step=msgs_per_step,
                                l2="inputs larger than L2 (accumulators %.1f GB)" % (w.pool_slots * 4 * max(w.dims[1:]) / 1e9),
                                parallelism="replicas only" if world > 1 else "1 gpu",
                                layer_ms=[float(ph[:, l].sum()) / args.steps for l in range(L)], phase_ms=phase_ms),
                    clocks=sampler.summary(), roofline=roofline, e2e=e2e, cpu_baseline=cpu, gpu_launches=int(launches))
        print(json.dumps(line))
    for r in runs or []:
        r.destroy()
    ctx.destroy()
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
