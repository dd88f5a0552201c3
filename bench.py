"""Benchmark of the source-centric broadcast step (libtaurus) on synthetic graphs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload large] [--impl ours|reference]

The metric is propagated edges per second (GTEPS, self messages not counted).

Workloads whose accumulator pool holds every vertex ("mid", "tiny"): a step is one full pass of the hot path over
the workload, every layer and every chunk (copy-in, projection, classify, make-room, scatter, finalise, output).

Workloads with a bounded pool ("large", "sampled", "stress"; a full pass takes tens of seconds): a step is a
window of --window consecutive chunks of one layer pass in steady state.  The layer (--layer, default the first
hidden-to-hidden layer) is begun, --prefill chunks fill the pool (untimed), then W warm-up windows and K timed
windows follow in the same pass; every window ends with a drain of the rows it completed.  The layer's input rows
are generated rows of the right width (as the paper feeds later layers, whose real inputs it cannot materialise, with
stand-in rows of the same width, Sect. 4.2).  The full layer time is printed as an estimate from the timed windows, marked as such.

The default run times "large" (the eviction-bound configuration) and then "mid" as a secondary entry in the same
JSON line.  N > 1 (under torchrun): the path has no exchange step, so every rank runs an independent replica
("replicas only", weak scaling); value = sum over ranks / max time.  Every replica of "large" holds the 8 GB graph and
pins 65 GB of host memory for its evicted rows: N replicas need N times that on the node.
--impl reference times the CPU oracle (a deliberately plain program) on bounded destination samples of the workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time
from dataclasses import replace

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import taurus_gen as tg  # noqa: E402

METRIC = "edges/sec per GNN layer (GTEPS)"

# DRAM bytes (read + write) of the 256-float scatter_grouped_kernel instance per algorithmic byte, from the ncu capture
# summarised in profiles/scatter_grouped_kernel_mid_1200k.md (two launches: 2.691 and 2.721 GB measured against 2.143 and
# 2.164 GB algorithmic).  The figure belongs to the kernel source with the digest below (sha256 of csrc/kernels_group.cu,
# first 16 hex digits); when the source has changed since the capture the bench prints traffic = null instead of a
# stale number.
SCATTER_TRAFFIC_OVER_ALGORITHMIC = 1.257
SCATTER_CAPTURE_SOURCE = "85d27983976ae3e5"


def source_digest(name: str) -> str:
    path = os.path.join(ROOT, "paper_2607_17374_b200", "csrc", name)
    return hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=3)
    p.add_argument("--warmup", type=int, default=3)
    p.add_argument("--workload", default="large")
    p.add_argument("--secondary", default="mid", help="a second workload timed after the first and added to the JSON line "
                   "under 'secondary' (single-GPU runs only); 'none' switches it off")
    p.add_argument("--vertices", type=int, default=0, help="scale the workload to this many vertices (0 = full size)")
    p.add_argument("--chunk", type=int, default=0, help="sources per pushed chunk (0 = the workload's own, 65 536 for all but 'tiny')")
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--window", type=int, default=32, help="bounded-pool workloads: chunks per step")
    p.add_argument("--prefill", type=int, default=384, help="bounded-pool workloads: untimed chunks that fill the pool first")
    p.add_argument("--layer", type=int, default=1, help="bounded-pool workloads: the layer whose pass is timed")
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
                   help="where a layer's rows go: a dense matrix in HBM (full-pass workloads) or the caller's drain buffers (bounded-pool "
                        "workloads) by default, or sorted runs (in HBM / pinned host memory) that the next layer reads back by "
                        "merge-on-read")
    return p.parse_args()


def workload_of(args, name=None):
    w = tg.WORKLOADS[name or args.workload]
    if args.vertices:
        w = tg.scaled(w, args.vertices)
    if args.chunk > 0:
        w = replace(w, chunk=args.chunk)
    if args.pool_fraction > 0:
        w = replace(w, pool_slots=max(1, int(w.V * args.pool_fraction)))
    if args.model:
        w = replace(w, mode={"sage": tg.SAGE_MEAN, "gcn": tg.GCN_SYM, "gin": tg.GIN_SUM, "gat": tg.GAT}[args.model],
                    gemm_mode=tg.GEMM_FP32 if args.model == "gat" else w.gemm_mode)
    return w


def graph_of(args, w):
    """The workload's graph.  --chunk changes how the sources are cut into pushes, not the graph: the generator's band
    width stays the one of the workload's own chunk size."""
    base = tg.WORKLOADS[w.name.split("@")[0]]
    return tg.make_graph(replace(w, chunk=base.chunk) if args.chunk > 0 else w)


def plan_windows(n_chunks: int, K: int, W: int, window: int, prefill: int):
    """Chunks per window and untimed prefill chunks of one layer pass that has to hold the prefill and W + K windows: the
    where the pass is too short for what was asked, the prefill is cut to a quarter of it, then the window shrinks (a run with
    many steps times shorter windows), then the prefill again."""
    window, prefill = max(window, 1), max(prefill, 0)
    if prefill + (W + K) * window > n_chunks:
        prefill = min(prefill, n_chunks // 4)
    while prefill + (W + K) * window > n_chunks and window > 1:
        window -= 1
    prefill = max(0, min(prefill, n_chunks - (W + K) * window))
    if (W + K) * window > n_chunks:
        raise SystemExit("workload too small for %d windows" % (W + K))
    return window, prefill


def windowed(w) -> bool:
    """Bounded pool: rows can be evicted, and a step is a window of chunks."""
    return w.pool_slots < w.V - w.hub_count


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

    def finish(self):
        self.stop_flag.set()
        self.join()
        if not self.mhz:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=[], samples=0, source=self.source)
        mhz = sorted(self.mhz)
        return dict(sm_mhz=mhz[len(mhz) // 2], sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), samples=len(mhz),
                    source=self.source)


# ----------------------------------------------------------------------------------------------- reference arm / CPU baseline

class OracleSampler:
    """Times the oracle (as it stands) on bounded destination samples of a workload.

    One scan of the CSR collects the in-lists of all sampled destinations (not timed: it replaces the whole-graph
    in-list builder, which at 1.6 B edges would not fit the budget).  A batch is then timed as the oracle runs it:
    the layer's message sets (the sampler where the layer is sampled), the fp64 aggregation of the input rows, the fp64
    transform, bias and activation.  Layer l reads generated N(0,1) rows of its input width (layer 0: the workload's
    features), keyed by vertex; generating them is not timed."""

    def __init__(self, w, g, layers, n_batches, batch_dst):
        import oracle
        self.o, self.w, self.g, self.layers = oracle, w, g, list(layers)
        rng = np.random.default_rng(0)
        total = min(g.V, n_batches * batch_dst)
        t0 = time.time()
        self.dsts = np.sort(rng.choice(g.V, size=total, replace=False)).astype(np.int64)
        self.ptr, self.src, self.eid = oracle.subset_in_lists(g.V, g.row_ptr, g.col_idx, self.dsts)
        self.scan_s = time.time() - t0
        self.batches = [(i * total // n_batches, (i + 1) * total // n_batches) for i in range(n_batches)]
        self.model = tg.make_model(w)
        self.dout = np.diff(g.row_ptr)
        self.cores = oracle.cores_used()

    def run_batch(self, b):
        """Every listed layer on batch b.  Returns (in-edges pulled, seconds of oracle work)."""
        o, w, g = self.o, self.w, self.g
        lo, hi = self.batches[b % len(self.batches)]
        dsts = self.dsts[lo:hi]
        ptr = self.ptr[lo:hi + 1] - self.ptr[lo]
        src = self.src[self.ptr[lo]:self.ptr[hi]]
        eid = self.eid[self.ptr[lo]:self.ptr[hi]]
        edges, secs = 0, 0.0
        for l in self.layers:
            t0 = time.time()
            kp, ks, _ = (ptr, src, eid) if w.fanout[l] == 0 else o.subset_message_sets(ptr, src, eid, dsts, w.fanout[l], w.seed, l)
            need = np.unique(np.concatenate([ks, dsts]))
            t1 = time.time()
            h = tg.features_rows(w.seed, l, need, w.dims[l])          # inputs: not part of the oracle's work
            t2 = time.time()
            o.subset_forward(w.mode if w.mode != tg.GAT else o.SAGE_MEAN, dsts, kp, ks, g.in_degree[dsts], self.dout[dsts], need,
                             self.dout[need], h, self.model.W_neigh[l], self.model.W_self[l], self.model.bias[l], self.model.act[l])
            t3 = time.time()
            edges += int(kp[-1])
            secs += (t1 - t0) + (t3 - t2)
        return edges, secs

    def describe(self, batches_run, edges, secs):
        return dict(cores=self.cores, kind="oracle",
                    sample="layers %s, %d batch(es) of %d sampled destinations each (dims %s), %d in-edges pulled in %.1f s of oracle "
                           "work; one CSR scan for the sampled in-lists (%.1f s) and input-row generation not counted"
                           % (self.layers, batches_run, self.batches[0][1] - self.batches[0][0],
                              [(self.w.dims[l], self.w.dims[l + 1]) for l in self.layers], edges, secs, self.scan_s))


def batch_size_for(w, layers):
    """Destinations per batch: bounded by the fp64 input rows a batch gathers (about 3 GB)."""
    widest = max(w.dims[l] for l in layers)
    mean_deg = max(1.0, w.E / w.V)
    fan = [min(mean_deg, w.fanout[l]) if w.fanout[l] else mean_deg for l in layers]
    return int(max(1024, min(400_000, 3e9 / (8.0 * widest * (max(fan) + 1)))))


def timed_layers(args, w):
    return [min(max(args.layer, 0), w.L - 1)] if windowed(w) else list(range(w.L))


def cpu_baseline(args, w, g, budget_s=12.0):
    layers = timed_layers(args, w)
    smp = OracleSampler(w, g, layers, 8, batch_size_for(w, layers))
    edges, secs, n = 0, 0.0, 0
    while n < 8 and (n == 0 or secs < budget_s):
        e, s = smp.run_batch(n)
        edges += e; secs += s; n += 1
    return dict(value=edges / secs / 1e9, unit="GTEPS", **smp.describe(n, edges, secs))


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    w = workload_of(args)
    g = graph_of(args, w)
    layers = timed_layers(args, w)
    n = max(args.steps, 1) + max(args.warmup, 0)
    smp = OracleSampler(w, g, layers, min(n, 8), batch_size_for(w, layers))
    for i in range(max(args.warmup, 0)):
        smp.run_batch(i)
    edges, secs = 0, 0.0
    for i in range(args.steps):
        e, s = smp.run_batch(args.warmup + i)
        edges += e; secs += s
    value = edges / secs / 1e9
    info = smp.describe(args.steps, edges, secs)
    line = dict(impl="reference", metric=METRIC, value=value, unit="GTEPS", n_gpus=args.gpus, steps=args.steps, warmup=args.warmup,
                ms_per_step=secs * 1e3 / max(args.steps, 1), higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64",
                data="synthetic",
                config=dict(workload=w.name, V=g.V, E=g.E, dims=list(w.dims), layers_timed=layers, fanout=list(w.fanout),
                            step="one batch of sampled destinations through the listed layers",
                            l2="inputs larger than L2"),
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


class Env:
    """Device, rank and barrier of this process."""

    def __init__(self):
        import torch
        import torch.distributed as dist
        self.torch, self.dist = torch, dist
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.rank = int(os.environ.get("RANK", "0"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        if self.world > 1:
            dist.init_process_group("nccl", device_id=self.dev)

    def barrier(self):
        if self.world > 1:
            self.dist.barrier()
        self.torch.cuda.synchronize()

    def close(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def make_context(args, w, g, model, host_evict, drain_rows):
    import paper_2607_17374_b200 as tb
    flags = (tb.FLAG_SIMT_GEMM if args.simt_gemm else 0) | (tb.FLAG_NO_GROUPING if args.no_grouping else 0) | \
        (tb.FLAG_PROJECT_FIRST if args.project_first else 0)
    return tb.Context(g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                      model.act, w.chunk, w.pool_slots, w.hub_count, w.fanout, w.seed, host_evict, drain_rows, w.gemm_mode, flags,
                      {"fewest": 0, "fifo": 1, "lru": 2, "random": 3}[args.evict_policy], w.gin_eps, model.att_src, model.att_dst,
                      w.leaky_slope)


# per push, from taurus_get_phase_ms: seven consecutive spans of the compute stream, the chunk's own finalise (which, with a
# bounded pool, runs inside the NEXT chunk's fourth span) and the chunk's row transfers on the library's transfer stream
PHASES = ["copy_in", "projection", "classify_select", "transfer_wait_and_previous_finalise", "slot_handout", "scatter",
          "completion_list", "finalise", "row_transfers"]


def scatter_bytes(groups, edges, n_src, width, self_row):
    """Algorithmic bytes of the scatter: per accumulator-row reduction a read-modify-write of the row (2 * 4 width)
    plus slot and pending-count words (8); per propagated edge its (destination, source) words (8); per source its
    row read once (4 width) and its self message (row read 4 width + read-modify-write 2 * 4 width + 8)."""
    return groups * (8 * width + 8) + edges * 8 + n_src * (4 * width + (12 * width if self_row else 0) + 8)


def link_peaks(env, mb=256, reps=3):
    """Pinned-memory copy bandwidth of this machine, GB/s: host -> device alone, device -> host alone, and both at once on
    two streams (per direction).  Plain asynchronous copies of `mb` MB, best of `reps`."""
    torch = env.torch
    n = mb << 20
    h_in, h_out = torch.empty(n, dtype=torch.uint8).pin_memory(), torch.empty(n, dtype=torch.uint8).pin_memory()
    d_in, d_out = torch.empty(n, dtype=torch.uint8, device=env.dev), torch.zeros(n, dtype=torch.uint8, device=env.dev)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    best = [0.0, 0.0, 0.0]
    for _ in range(reps + 1):
        for mode in range(3):
            torch.cuda.synchronize()
            a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            a.record(s1)
            s2.wait_event(a)
            if mode in (0, 2):
                with torch.cuda.stream(s1):
                    d_in.copy_(h_in, non_blocking=True)
            if mode in (1, 2):
                with torch.cuda.stream(s2):
                    h_out.copy_(d_out, non_blocking=True)
            c.record(s2)
            s1.wait_event(c)
            b.record(s1)
            torch.cuda.synchronize()
            best[mode] = max(best[mode], n / (a.elapsed_time(b) * 1e-3) / 1e9)
    return dict(h2d_alone_gbs=best[0], d2h_alone_gbs=best[1], both_per_direction_gbs=best[2],
                how="cudaMemcpyAsync of %d MB pinned buffers, both directions at once on two streams, best of %d" % (mb, reps))


# ----------------------------------------------------------------------------------------------- bounded-pool workloads

def run_windowed(args, env, w):
    """Steps = windows of chunks of one layer pass in steady state (see the module docstring)."""
    import paper_2607_17374_b200 as tb
    torch, dev = env.torch, env.dev
    g = graph_of(args, w)
    model = tg.make_model(w)
    V, chunk = g.V, w.chunk
    chunks = [(s, min(s + chunk, V)) for s in range(0, V, chunk)]
    l = timed_layers(args, w)[0]
    d_in, d_out = w.dims[l], w.dims[l + 1]
    K, W = max(args.steps, 1), max(args.warmup, 0)
    window, prefill = plan_windows(len(chunks), K, W, args.window, args.prefill)
    cap = 3 * window * chunk                       # graduation buffer: drained once per window, earlier when it could overflow
    host_evict = min(V - w.hub_count, 56_000_000)   # rows evicted at once stay below this on the three bounded-pool workloads
    ctx = make_context(args, w, g, model, host_evict, cap)
    runs = None
    if args.output != "dense":
        # Finished rows leave as sorted runs (embedding writer of Sect. 3.7) instead of being drained: 64 id ranges with
        # partition buffers of 65 536 rows in HBM, the run store in HBM or in pinned host memory, sized for the rows the
        # pass can complete (the pass stops after the timed windows).
        n_used = prefill + (W + K) * window
        kind = tb.RUNS_DEVICE if args.output == "runs-device" else tb.RUNS_HOST
        runs = tb.Runs(V, w.dims[timed_layers(args, w)[0] + 1], 64, 65536, store_rows=min(V, int(1.25 * n_used * chunk) + 64 * 65536),
                       max_append_rows=cap, max_chunk_rows=chunk, store_kind=kind)
    agg_first, acc_width = ctx.layer_plan(l)
    R = 8                                          # distinct generated input chunks, reused in turn
    x_host = [torch.empty((chunk, d_in), dtype=torch.float32).pin_memory() for _ in range(R)]
    for i in range(R):
        tg.features(w.seed, l, i * chunk, (i + 1) * chunk, d_in, out=x_host[i].numpy())
    x_dev = [x.to(dev) for x in x_host]
    ids_dev = torch.empty(cap, dtype=torch.int64, device=dev)
    rows_dev = torch.empty((cap, d_out), dtype=torch.float32, device=dev)
    ids_host = torch.empty(cap, dtype=torch.int64).pin_memory()
    rows_host = torch.empty((cap, d_out), dtype=torch.float32).pin_memory()
    stream = torch.cuda.current_stream()
    link = link_peaks(env)
    pk = peaks()

    def run_chunks(c0, c1, feats, ids, rows, drain_every):
        """Chunks [c0, c1); a drain after every `drain_every` chunks.  Returns rows drained."""
        drained = 0
        for c in range(c0, c1):
            s, e = chunks[c]
            x = feats[c % R][: e - s]
            if runs is not None:                      # rows go to the run store on the library's output stream
                ctx.push_chunk(s, e, x, stream)
                continue
            if ctx.push_chunk(s, e, x, stream, raise_on_drain_full=False) != 0:
                drained += ctx.drain_completed(ids, rows, cap)
                ctx.push_chunk(s, e, x, stream)
            if (c - c0 + 1) % drain_every == 0:
                drained += ctx.drain_completed(ids, rows, cap)
        return drained

    def one_pass(feats, ids, rows, timing):
        """Prefill, warm-up windows, timed windows.  Returns (ms of the timed windows, stats before, stats after, rows drained,
        phase times, launches, clocks, wall ms)."""
        ctx.layer_begin(l, stream)
        if runs is not None:
            runs.reset()
            ctx.layer_set_run_output(runs)
        run_chunks(0, prefill, feats, ids, rows, window)
        if runs is None:
            ctx.drain_completed(ids, rows, cap)
        c = prefill
        run_chunks(c, c + W * window, feats, ids, rows, window)
        c += W * window
        st0 = ctx.get_stats()
        env.barrier()
        sampler = ClockSampler(env.local)
        sampler.start()
        if timing:
            ctx.set_timing(True)
        launches0 = ctx.launch_count()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        ev0.record(stream)
        drained = run_chunks(c, c + K * window, feats, ids, rows, window)
        ev1.record(stream)
        env.barrier()
        wall = (time.time() - t0) * 1e3
        ms = ev0.elapsed_time(ev1)
        launches = ctx.launch_count() - launches0
        clocks = sampler.finish()
        ph = None
        if timing:
            ph = ctx.get_phase_ms()
            ctx.set_timing(False)
        st1 = ctx.get_stats()
        if runs is not None:
            drained = st1["completed"] - st0["completed"]
        return ms, st0, st1, drained, ph, launches, clocks, wall

    # ---- inputs resident in HBM, rows drained into HBM
    ms, st0, st1, drained, ph, launches, clocks, _ = one_pass(x_dev, ids_dev, rows_dev, True)
    msgs = st1["total_messages"] - st0["total_messages"]
    evicted, reloaded = st1["evictions"] - st0["evictions"], st1["reloads"] - st0["reloads"]
    groups = st1["scatter_groups"] - st0["scatter_groups"]
    ms_max = max_over_ranks(ms, env.world, dev)
    value = whole_job_value(msgs / K, K, env.world, ms_max)
    phase = ph[: K * window].sum(axis=0).astype(np.float64)            # ms over the timed windows
    phase_ms = dict(zip(PHASES, [float(x) / K for x in phase]))
    row_bytes = 4 * acc_width
    move_s = phase[8] * 1e-3                                           # transfer kernels, timed on their own stream
    out_gbs, in_gbs = evicted * row_bytes / max(move_s, 1e-9) / 1e9, reloaded * row_bytes / max(move_s, 1e-9) / 1e9
    n_src = chunks[prefill + (W + K) * window - 1][1] - chunks[prefill + W * window][0]
    sc_bytes = scatter_bytes(groups, msgs, n_src, acc_width, not (agg_first and w.mode == tg.SAGE_MEAN))
    sc_s = phase[5] * 1e-3
    moves_share = phase[8] / ms
    # the dominant kernel: the row transfers between the pool and pinned host memory, bound by the host link
    # The link is full duplex: a launch cannot end before its busier direction has crossed, max(bytes out, bytes in) /
    # per-direction peak.  `achieved` is therefore the rate of the busier direction; both are listed.
    roofline = dict(bound="pcie", kernel="transfer_kernel (evicted rows out, reloaded rows in, %d-byte rows)" % row_bytes,
                    achieved=max(out_gbs, in_gbs), peak=link["both_per_direction_gbs"], unit="GB/s in the busier direction",
                    frac=max(out_gbs, in_gbs) / link["both_per_direction_gbs"], mean_of_directions_gbs=(out_gbs + in_gbs) / 2,
                    peak_source="measured in this run: " + link["how"],
                    device_to_host_gbs=out_gbs, host_to_device_gbs=in_gbs, link=link,
                    rows_out_per_step=evicted / K, rows_in_per_step=reloaded / K, launches_per_step=window,
                    avg_launch_ms=float(phase[8]) / (K * window), algorithmic_bytes_per_launch=max(evicted, reloaded) * row_bytes / (K * window),
                    algorithmic_bytes_note="rows of the busier direction x row bytes (counters of the library)",
                    share_of_step=float(moves_share),
                    share_note="the transfers run on their own stream beside the compute stream: their share of the step is how "
                               "much of the step the host link is busy",
                    traffic=None,
                    traffic_note="no counter capture at this size (110 GB resident); PCIe counters of the same kernel on a 1.5 M-vertex "
                                 "instance are in profiles/transfer_kernel_large_1500k.md")
    roofline_hbm = dict(bound="hbm", kernel="scatter_grouped_kernel (accumulator rows of %d floats)" % acc_width,
                        achieved=sc_bytes / sc_s / 1e9, peak=pk["hbm_gbs"], unit="GB/s", frac=sc_bytes / sc_s / 1e9 / pk["hbm_gbs"],
                        peak_source=pk["source"], groups_per_step=groups / K, avg_launch_ms=float(phase[5]) / (K * window),
                        algorithmic_bytes_per_launch=sc_bytes / (K * window), share_of_step=float(phase[5] / ms),

                        gteps_scatter_only=msgs / sc_s / 1e9)

    # ---- end to end through the C ABI with host buffers: every chunk's input rows come from pinned host memory (one
    # host -> device copy per chunk inside push_chunk) and every window's finished rows and ids are drained into pinned
    # host memory (taurus_drain_completed), all inside the timed region
    e2e = None
    if not args.no_e2e:
        ms2, s0, s1, drained2, _, _, _, wall2 = one_pass(x_host, ids_host, rows_host, False)
        msgs2 = s1["total_messages"] - s0["total_messages"]
        e2e_ms = max_over_ranks(max(ms2, wall2), env.world, dev)
        e2e = dict(value=whole_job_value(msgs2 / K, K, env.world, e2e_ms), unit="GTEPS", ms_per_step=e2e_ms / K,
                   h2d_bytes_per_step=int(4 * d_in * n_src / K), d2h_bytes_per_step=int(drained2 * (4 * d_out + 8) / K),
                   note="input rows of every chunk host -> device inside taurus_push_chunk; finished rows and ids device -> host "
                        "through taurus_drain_completed once per window; evicted rows travel over the same link")
    cpu = None
    if env.rank == 0 and env.world == 1 and not args.no_cpu_baseline and w.mode != tg.GAT:
        cpu = cpu_baseline(args, w, g)
    free, total = torch.cuda.mem_get_info()
    # `roofline` is the kernel with the larger share of the step: the row transfers where the pool is short of the active
    # set (large, sampled), the scatter where few rows move (stress); the other one is kept beside it
    # (a transfer launch that moves a few thousand rows is long only because its blocks wait for room on the SMs beside the
    # scatter: it counts as the dominant kernel only when the link is busy with bytes, here a quarter of its peak)
    other = {}
    if phase[8] >= phase[5] and max(out_gbs, in_gbs) >= 0.25 * link["both_per_direction_gbs"]:
        other["roofline_hbm"] = roofline_hbm
    else:
        other["roofline_pcie"] = roofline
        roofline = roofline_hbm
    line = dict(metric=METRIC, value=value, unit="GTEPS", n_gpus=env.world, steps=K, warmup=W, ms_per_step=ms_max / K,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="bf16" if w.gemm_mode == tg.GEMM_BF16 else "f32",
                data="synthetic",
                config=dict(workload=w.name, V=V, E=g.E, dims=list(w.dims), chunk=chunk, chunks_per_layer=len(chunks),
                            pool_slots=w.pool_slots, hub_count=w.hub_count, fanout=list(w.fanout),
                            mode=["sage_mean", "gcn_sym", "gin_sum", "gat"][w.mode], evict_policy=args.evict_policy, output=args.output,
                            step="window of %d chunks of layer %d (%d -> %d) in steady state; %d prefill chunks and %d warm-up windows "
                                 "before the timed ones, same layer pass; rows drained once per window" % (window, l, d_in, d_out, prefill, W),
                            layer=l, window_chunks=window, prefill_chunks=prefill, aggregate_first=bool(agg_first),
                            accumulator_floats=acc_width, messages_per_step=msgs / K, evictions_per_step=evicted / K,
                            reloads_per_step=reloaded / K, rows_drained_per_step=drained / K,
                            layer_time_estimate_ms=ms_max / (K * window) * len(chunks),
                            layer_time_note="extrapolated linearly from the timed windows to the layer's %d chunks" % len(chunks),
                            l2="inputs larger than L2 (pool %.1f GB, one chunk's rows %.0f MB)" %
                               (w.pool_slots * 4 * acc_width / 1e9, chunk * 4 * max(d_in, d_out) / 1e6),
                            device_memory_in_use_gb=(total - free) / 1e9,
                            parallelism="replicas only" if env.world > 1 else "1 gpu", phase_ms=phase_ms),
                clocks=clocks, roofline=roofline, e2e=e2e, cpu_baseline=cpu, gpu_launches=int(launches), **other)
    if runs is not None:
        runs.destroy()
    ctx.destroy()
    return line


# ----------------------------------------------------------------------------------------------- full-pass workloads

def run_full_pass(args, env, w):
    import paper_2607_17374_b200 as tb
    torch, dev, world, rank = env.torch, env.dev, env.world, env.rank
    g = graph_of(args, w)
    model = tg.make_model(w)
    V, L = g.V, w.L
    chunks = [(s, min(s + w.chunk, V)) for s in range(0, V, w.chunk)]
    # two graduation halves; badly ordered graphs complete a large share of V in the last chunks
    drain_rows = 2 * max(V, w.chunk)
    host_evict = 0 if w.pool_slots >= V - w.hub_count else V - w.hub_count
    ctx = make_context(args, w, g, model, host_evict, drain_rows)
    plan = [ctx.layer_plan(l) for l in range(L)]
    agg_first, acc_width = [p[0] for p in plan], [p[1] for p in plan]
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
    env.barrier()
    for i in range(max(args.warmup, 1)):
        step(x_dev, out_dev, collect_stats=(i == 0))
    torch.cuda.synchronize()
    msgs_per_step = int(sum(edges_per_layer))

    # ---- device-resident timing
    sampler = ClockSampler(env.local)
    sampler.start()
    # Inside the timed region the library records the two events around every scatter launch and nothing else: an
    # event after each of a push's phases costs about 2 us of the stream, 4-5 % of a step of 114 pushes.  The phase
    # split comes from one more, untimed step with all events on.
    ctx.set_timing(2)
    launches0 = ctx.launch_count()
    env.barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step(x_dev, out_dev)
    ev1.record(stream)
    env.barrier()
    ms = ev0.elapsed_time(ev1)
    ctx.set_timing(0)
    launches = ctx.launch_count() - launches0
    clocks = sampler.finish()
    phases = ctx.get_phase_ms()   # [pushes, 9], the scatter column only
    ctx.set_timing(1)
    step(x_dev, out_dev)
    torch.cuda.synchronize()
    ctx.set_timing(0)
    ph_all = ctx.get_phase_ms()[: len(chunks) * L].reshape(1, L, len(chunks), 9)
    ms_max = max_over_ranks(ms, world, dev)
    value = whole_job_value(msgs_per_step, args.steps, world, ms_max)

    # ---- roofline of the dominant kernel (the scatter), from the events recorded inside the timed region
    n_push = len(chunks) * L * args.steps
    ph = phases[:n_push].reshape(args.steps, L, len(chunks), 9)
    scatter_ms = ph[..., 5]
    # In CSR order a "group" is one edge.  The per-edge cold-miss model (12 + 2 * 4 width per edge) is kept beside it.
    layer_bytes, edge_model_bytes = [], []
    for l in range(L):
        Wd = acc_width[l]
        self_row = not (agg_first[l] and w.mode == tg.SAGE_MEAN)   # aggregate-first SAGE adds its self term after the transform
        layer_bytes.append(scatter_bytes(groups_per_layer[l], edges_per_layer[l], V, Wd, self_row))
        edge_model_bytes.append(edges_per_layer[l] * (12 + 8 * Wd) + V * (4 * Wd + 8))
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
    capture_valid = grouped and dom_w == 256 and source_digest("kernels_group.cu") == SCATTER_CAPTURE_SOURCE
    roofline = dict(bound="hbm", kernel=kname, achieved=achieved,
                    peak=pk["hbm_gbs"], unit="GB/s", frac=achieved / pk["hbm_gbs"], peak_source=pk["source"],
                    traffic=SCATTER_TRAFFIC_OVER_ALGORITHMIC * dom_bytes / (len(chunks) * len(dom)) if capture_valid else None,
                    traffic_note=("ncu dram read+write per launch of the 256-float kernel on a 1.2 M-vertex instance, scaled by the "
                                  "algorithmic bytes of a launch "
                                  "(profiles/scatter_grouped_kernel_mid_1200k.md)") if capture_valid else
                                 "no capture of this kernel source (profiles/scatter_grouped_kernel_mid_1200k.md names the source it measured)",
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
    phase_ms = dict(zip(PHASES, [float(x) for x in ph_all.sum(axis=(0, 1, 2))]))

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
        env.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.time()
        e0.record(stream)
        for i in range(args.steps):
            e2e_step(i + 1)
        for b in range(2):
            stream.wait_event(d2h_done[b])
        e1.record(stream)
        env.barrier()
        wall = (time.time() - t0) * 1e3
        e2e_ms = max_over_ranks(max(e0.elapsed_time(e1), wall), world, dev)
        e2e = dict(value=whole_job_value(msgs_per_step, args.steps, world, e2e_ms), unit="GTEPS",
                   ms_per_step=e2e_ms / args.steps,
                   h2d_bytes_per_step=int(4 * V * w.dims[0]), d2h_bytes_per_step=int(4 * V * w.dims[-1]),
                   note="layer-0 features host -> device per chunk; last layer's rows device -> host in one copy per step on a "
                        "side stream, overlapping the next step's first layer; intermediate layers in HBM")
        del outs_host

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not gat:
        cpu = cpu_baseline(args, w, g)

    line = dict(metric=METRIC, value=value, unit="GTEPS", n_gpus=world, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms_max / args.steps, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="bf16" if w.gemm_mode == tg.GEMM_BF16 else "f32", data="synthetic",
                config=dict(workload=w.name, V=V, E=g.E, dims=list(w.dims), chunk=w.chunk, chunks_per_layer=len(chunks),
                            pool_slots=w.pool_slots, hub_count=w.hub_count, fanout=list(w.fanout),
                            mode=["sage_mean", "gcn_sym", "gin_sum", "gat"][w.mode], output=args.output, evict_policy=args.evict_policy,
                            step="one pass over every layer and chunk of the workload",
                            messages_per_step=msgs_per_step,
                            l2="inputs larger than L2 (accumulators %.1f GB)" % (w.pool_slots * 4 * max(w.dims[1:]) / 1e9),
                            parallelism="replicas only" if world > 1 else "1 gpu",
                            phase_note="phase_ms, layer_ms and phase_ms_per_layer: one extra step after the timed ones with an event after "
                                       "every phase of every push (those events lengthen the step by 4-5 %, so the timed steps record "
                                       "only the events around the scatter launches that the roofline uses)",
                            layer_ms=[float(ph_all[:, l, :, :8].sum()) for l in range(L)], phase_ms=phase_ms,
                            phase_ms_per_layer=[dict(zip(PHASES, [round(float(x), 3) for x in ph_all[:, l].sum(axis=(0, 1))]))
                                                for l in range(L)]),
                clocks=clocks, roofline=roofline, e2e=e2e, cpu_baseline=cpu, gpu_launches=int(launches))
    for r in runs or []:
        r.destroy()
    ctx.destroy()
    return line


# Host and device memory (GB) a replica of a full-size bounded-pool workload takes in this bench: the graph, the pinned
# store of evicted rows (56 M rows of the timed layer's width) and the generator's temporaries; the pool, the grouped edge
# order and the in-lists on the device.
FULL_SIZE_NEEDS_GB = {"large": (90, 140), "sampled": (100, 150), "stress": (150, 150)}


def free_memory_gb(env):
    host_free = 0.0
    for ln in open("/proc/meminfo"):
        if ln.startswith("MemAvailable:"):
            host_free = int(ln.split()[1]) / 1e6
    return host_free, env.torch.cuda.mem_get_info()[0] / 1e9


def fallback_reason(args, env, w):
    """Why this box cannot hold the workload at full size (None when it can)."""
    base = w.name.split("@")[0]
    if args.vertices or args.pool_fraction > 0 or base not in FULL_SIZE_NEEDS_GB:
        return None
    host_need, dev_need = FULL_SIZE_NEEDS_GB[base]
    host_free, dev_free = free_memory_gb(env)
    if host_free < host_need * env.world or dev_free < dev_need:
        return ("'%s' at full size needs %d GB of host memory per replica (%d replicas) and %d GB of device memory; %.0f GB "
                "and %.0f GB are free here" % (base, host_need, env.world, dev_need, host_free, dev_free))
    return None


def run_ours(args):
    env = Env()
    w = workload_of(args)
    why = fallback_reason(args, env, w)
    if max_over_ranks(0.0 if why is None else 1.0, env.world, env.dev) > 0 and why is None:   # every rank takes the same road
        why = "another replica found too little memory for '%s' at full size" % w.name
    if why is not None and args.secondary not in ("none", ""):
        # the box cannot hold the configured workload: the secondary one becomes the line, and says so
        w = workload_of(args, args.secondary)
        line = run_windowed(args, env, w) if windowed(w) else run_full_pass(args, env, w)
        line["config"]["fallback"] = why
        if env.rank == 0:
            print(json.dumps(line))
        env.close()
        return
    line = run_windowed(args, env, w) if windowed(w) else run_full_pass(args, env, w)
    if args.secondary not in ("none", "", w.name.split("@")[0]) and env.world == 1:
        import gc
        gc.collect()
        env.torch.cuda.empty_cache()
        w2 = workload_of(args, args.secondary)
        line["secondary"] = {args.secondary: run_windowed(args, env, w2) if windowed(w2) else run_full_pass(args, env, w2)}
    if env.rank == 0:
        print(json.dumps(line))
    env.close()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
