"""ctypes binding of libtaurus: argument marshalling only.  Method names follow the C entry points
(taurus_graph_init -> Context(...), taurus_push_chunk -> Context.push_chunk, ...)."""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

SAGE_MEAN, GCN_SYM, GIN_SUM, GAT = 0, 1, 2, 3
GEMM_FP32, GEMM_BF16 = 0, 1
FLAG_SIMT_GEMM, FLAG_NO_GROUPING, FLAG_PROJECT_FIRST = 2, 4, 8
EVICT_FEWEST_PENDING, EVICT_FIFO, EVICT_LRU, EVICT_RANDOM = 0, 1, 2, 3
CHUNK_LOG_COLUMNS = ["hs", "ns", "ev", "gs", "need", "evicted", "reloaded", "completed", "occupancy"]
ERROR_CODES = {
    "OK": 0, "INVALID_ARG": -1, "ORDER": -2, "POOL_TOO_SMALL": -3, "HOST_STORE_FULL": -4, "DRAIN_FULL": -5,
    "CUDA": -6, "INTERNAL": -7, "NOMEM": -8, "UNSUPPORTED": -9, "RUN_STORE_FULL": -10, "RUNS_INCOMPLETE": -11,
}
RUNS_HOST, RUNS_DEVICE = 0, 1

_PKG = os.path.dirname(os.path.abspath(__file__))
_lib = None


def library_path() -> str:
    return os.path.join(_PKG, "libtaurus.so")


class TaurusError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = "%s failed: %d" % (where, code)
        if _lib is not None:
            msg += " (%s)" % _lib.taurus_strerror(code).decode()
        if detail:
            msg += ": " + detail
        super().__init__(msg)


class _Graph(ctypes.Structure):
    _fields_ = [("V", ctypes.c_int64), ("E", ctypes.c_int64), ("row_ptr", ctypes.c_void_p),
                ("col_idx", ctypes.c_void_p), ("in_degree", ctypes.c_void_p)]


class _Model(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("L", ctypes.c_int32), ("dims", ctypes.POINTER(ctypes.c_int32)),
                ("W_neigh", ctypes.POINTER(ctypes.c_void_p)), ("W_self", ctypes.POINTER(ctypes.c_void_p)),
                ("bias", ctypes.POINTER(ctypes.c_void_p)), ("act", ctypes.POINTER(ctypes.c_int32)),
                ("gemm_mode", ctypes.c_int32), ("gin_eps", ctypes.c_float),
                ("att_src", ctypes.POINTER(ctypes.c_void_p)), ("att_dst", ctypes.POINTER(ctypes.c_void_p)),
                ("leaky_slope", ctypes.c_float), ("gat_heads", ctypes.c_int32)]


class _Run(ctypes.Structure):
    _fields_ = [("chunk_sources", ctypes.c_int64), ("pool_slots", ctypes.c_int64), ("hub_count", ctypes.c_int64),
                ("fanout", ctypes.POINTER(ctypes.c_int32)), ("seed", ctypes.c_uint64),
                ("host_evict_rows", ctypes.c_int64), ("drain_rows", ctypes.c_int64), ("flags", ctypes.c_int32),
                ("evict_policy", ctypes.c_int32)]


class Stats(ctypes.Structure):
    _fields_ = [("evictions", ctypes.c_int64), ("reloads", ctypes.c_int64), ("max_reload_count", ctypes.c_int64),
                ("reload_histogram", ctypes.c_int64 * 17), ("peak_occupancy", ctypes.c_int64),
                ("hub_messages", ctypes.c_int64), ("total_messages", ctypes.c_int64), ("hub_vertices", ctypes.c_int64),
                ("completed", ctypes.c_int64), ("sum_hs", ctypes.c_int64), ("sum_ns", ctypes.c_int64),
                ("sum_ev", ctypes.c_int64), ("sum_gs", ctypes.c_int64), ("free_slots", ctypes.c_int64),
                ("chunks", ctypes.c_int64), ("scatter_groups", ctypes.c_int64)]

    def as_dict(self) -> dict:
        d = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            d[name] = list(v) if name == "reload_histogram" else int(v)
        return d


class _RunsConfig(ctypes.Structure):
    _fields_ = [("V", ctypes.c_int64), ("width", ctypes.c_int32), ("store_kind", ctypes.c_int32),
                ("partitions", ctypes.c_int64), ("partition_rows", ctypes.c_int64), ("store_rows", ctypes.c_int64),
                ("max_append_rows", ctypes.c_int64), ("max_chunk_rows", ctypes.c_int64)]


EXPORTS = [
    "taurus_graph_init", "taurus_layer_begin", "taurus_push_chunk", "taurus_drain_completed", "taurus_drain_dense",
    "taurus_layer_end", "taurus_get_stats", "taurus_get_chunk_log", "taurus_get_vertex_array",
    "taurus_get_sampled_edges", "taurus_get_edge_mask", "taurus_completion_bound", "taurus_launch_count", "taurus_get_layer_plan",
    "taurus_set_timing", "taurus_get_phase_ms", "taurus_destroy", "taurus_strerror", "taurus_last_cuda_error",
    "taurus_completion_counts_noalloc", "taurus_layer_set_dense_output", "taurus_reorder",
    "taurus_runs_create", "taurus_runs_append", "taurus_runs_flush", "taurus_runs_read_chunk", "taurus_runs_info",
    "taurus_runs_directory", "taurus_runs_get_run", "taurus_runs_reset", "taurus_runs_destroy",
    "taurus_layer_set_run_output", "taurus_push_chunk_from_runs", "taurus_gat_project_chunk", "taurus_gat_attention",
    "taurus_get_sample_digest", "taurus_gat_project_chunk_from_runs", "taurus_relabel_csr", "taurus_permute_rows",
]
NOALLOC_MAX_VERTICES = 4 * 1024 * 1024


def load_library():
    """Loads libtaurus.so.  Fails loudly when it has not been built: there is no fallback path."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError("libtaurus.so is missing at %s: build it with `python -m paper_2607_17374_b200.build` "
                           "(needs nvcc); this package has no CPU fallback" % path)
    lib = ctypes.CDLL(path)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
    lib.taurus_graph_init.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_Graph), ctypes.POINTER(_Model), ctypes.POINTER(_Run)]
    lib.taurus_layer_begin.argtypes = [vp, i32, vp]
    lib.taurus_push_chunk.argtypes = [vp, i64, i64, vp, vp]
    lib.taurus_drain_completed.argtypes = [vp, vp, vp, i64, ctypes.POINTER(i64)]
    lib.taurus_drain_dense.argtypes = [vp, vp, i64, vp, i64, ctypes.POINTER(i64)]
    lib.taurus_layer_end.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.taurus_layer_set_dense_output.argtypes = [vp, vp, i64]
    lib.taurus_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    lib.taurus_get_chunk_log.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
    lib.taurus_get_vertex_array.argtypes = [vp, i32, vp]
    lib.taurus_get_sampled_edges.argtypes = [vp, i32, i64, vp, vp, i32, ctypes.POINTER(i32)]
    lib.taurus_get_edge_mask.argtypes = [vp, vp]
    lib.taurus_get_sample_digest.argtypes = [vp, vp]
    lib.taurus_completion_bound.argtypes = [vp, i64, i64, ctypes.POINTER(i64)]
    lib.taurus_completion_counts_noalloc.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp]
    lib.taurus_reorder.argtypes = [i64, i64, vp, vp, vp, i32, vp, vp, vp, vp, vp]
    lib.taurus_runs_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(_RunsConfig)]
    lib.taurus_runs_append.argtypes = [vp, vp, vp, i64, i64, vp]
    lib.taurus_runs_flush.argtypes = [vp, vp]
    lib.taurus_runs_read_chunk.argtypes = [vp, i64, i64, vp, i64, vp]
    lib.taurus_runs_info.argtypes = [vp, ctypes.POINTER(i64), ctypes.POINTER(i64), ctypes.POINTER(i64)]
    lib.taurus_runs_directory.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
    lib.taurus_runs_get_run.argtypes = [vp, i64, vp, vp]
    lib.taurus_runs_reset.argtypes = [vp]
    lib.taurus_runs_destroy.argtypes = [vp]
    lib.taurus_runs_destroy.restype = None
    lib.taurus_layer_set_run_output.argtypes = [vp, vp]
    lib.taurus_push_chunk_from_runs.argtypes = [vp, i64, i64, vp, vp]
    lib.taurus_gat_project_chunk.argtypes = [vp, i64, i64, vp, vp, i64, vp]
    lib.taurus_gat_attention.argtypes = [vp, vp]
    lib.taurus_gat_project_chunk_from_runs.argtypes = [vp, i64, i64, vp, vp, i64, vp]
    lib.taurus_relabel_csr.argtypes = [i64, i64, vp, vp, vp, vp, vp, vp, vp]
    lib.taurus_permute_rows.argtypes = [i64, i32, vp, i64, vp, vp, i64, vp]
    lib.taurus_get_layer_plan.argtypes = [vp, ctypes.c_int32, vp, vp]
    lib.taurus_launch_count.argtypes = [vp]
    lib.taurus_launch_count.restype = i64
    lib.taurus_set_timing.argtypes = [vp, i32]
    lib.taurus_get_phase_ms.argtypes = [vp, vp, i64, ctypes.POINTER(i64)]
    lib.taurus_destroy.argtypes = [vp]
    lib.taurus_destroy.restype = None
    lib.taurus_strerror.argtypes = [ctypes.c_int]
    lib.taurus_strerror.restype = ctypes.c_char_p
    lib.taurus_last_cuda_error.restype = ctypes.c_char_p
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor, a numpy array, or a raw integer address."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if isinstance(x, np.ndarray):
        if not x.flags.c_contiguous:
            raise ValueError("array must be C-contiguous")
        return x.ctypes.data
    if hasattr(x, "data_ptr"):
        if not x.is_contiguous():
            raise ValueError("tensor must be contiguous")
        return x.data_ptr()
    raise TypeError("expected a torch tensor, a numpy array or an address, got %r" % type(x))


def _stream(s) -> Optional[int]:
    if s is None:
        return None
    return s if isinstance(s, int) else s.cuda_stream


def completion_counts_noalloc(V: int, E: int, row_ptr, col_idx, edge_mask, out_counts, out_bad_index, stream=None) -> int:
    """taurus_completion_counts_noalloc: per-64-source completion counts computed with the library's static
    scratch array, for callers that cannot allocate device memory.  Every array argument is a device tensor or
    address owned by the caller; returns the C return code (0 = enqueued)."""
    return int(load_library().taurus_completion_counts_noalloc(V, E, _ptr(row_ptr), _ptr(col_idx), _ptr(edge_mask),
                                                               _ptr(out_counts), _ptr(out_bad_index), _stream(stream)))


def reorder(V: int, E: int, row_ptr, col_idx, initial_rank=None, iterations: int = 5, stream=None):
    """taurus_reorder (Alg. 1).  Returns (rank int32 [V], positions float64 [V], J float64 [iterations + 1],
    span int64 [iterations + 1]) as numpy arrays."""
    rank = np.empty(V, np.int32)
    pos = np.empty(V, np.float64)
    J = np.zeros(iterations + 1, np.float64)
    span = np.zeros(iterations + 1, np.int64)
    rc = load_library().taurus_reorder(V, E, _ptr(row_ptr), _ptr(col_idx), _ptr(initial_rank), iterations, rank.ctypes.data,
                                       pos.ctypes.data, J.ctypes.data, span.ctypes.data, _stream(stream))
    if rc != 0:
        raise TaurusError(rc, "taurus_reorder")
    return rank, pos, J, span


def relabel_csr(V: int, E: int, row_ptr, col_idx, rank, stream=None):
    """taurus_relabel_csr.  Returns (row_ptr int64 [V+1], col_idx int32 [E], in_degree int32 [V]) as numpy arrays."""
    new_ptr = np.empty(V + 1, np.int64)
    new_col = np.empty(max(E, 1), np.int32)
    new_din = np.empty(V, np.int32)
    rc = load_library().taurus_relabel_csr(V, E, _ptr(row_ptr), _ptr(col_idx), _ptr(rank), new_ptr.ctypes.data, new_col.ctypes.data,
                                           new_din.ctypes.data, _stream(stream))
    if rc != 0:
        raise TaurusError(rc, "taurus_relabel_csr")
    return new_ptr, new_col[:E], new_din


def permute_rows(V: int, width: int, in_rows, ld_in: int, rank, out_rows, ld_out: int, stream=None):
    """taurus_permute_rows: out_rows[rank[v]] = in_rows[v] (device tensors)."""
    rc = load_library().taurus_permute_rows(V, width, _ptr(in_rows), ld_in, _ptr(rank), _ptr(out_rows), ld_out, _stream(stream))
    if rc != 0:
        raise TaurusError(rc, "taurus_permute_rows")


class Runs:
    """One taurus_runs: sorted runs of (vertex id, row) records and the merge-on-read chunk reader."""

    def __init__(self, V: int, width: int, partitions: int, partition_rows: int, store_rows: int = 0,
                 max_append_rows: int = 0, max_chunk_rows: int = 0, store_kind: int = RUNS_HOST):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        self.V, self.width = V, width
        cfg = _RunsConfig(V, width, store_kind, partitions, partition_rows, store_rows or V, max_append_rows or V,
                          max_chunk_rows or V)
        rc = self._lib.taurus_runs_create(ctypes.byref(self._h), ctypes.byref(cfg))
        if rc != 0:
            self._h = ctypes.c_void_p()
            raise TaurusError(rc, "taurus_runs_create", self._lib.taurus_last_cuda_error().decode())

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise TaurusError(rc, where, self._lib.taurus_last_cuda_error().decode() if rc == ERROR_CODES["CUDA"] else "")

    def append(self, ids, rows, ld: int, count: int, stream=None):
        self._check(self._lib.taurus_runs_append(self._h, _ptr(ids), _ptr(rows), ld, count, _stream(stream)), "taurus_runs_append")

    def flush(self, stream=None):
        self._check(self._lib.taurus_runs_flush(self._h, _stream(stream)), "taurus_runs_flush")

    def read_chunk(self, src_begin: int, src_end: int, out_rows, ld: int, stream=None):
        self._check(self._lib.taurus_runs_read_chunk(self._h, src_begin, src_end, _ptr(out_rows), ld, _stream(stream)),
                    "taurus_runs_read_chunk")

    def info(self) -> dict:
        a, b, c = ctypes.c_int64(0), ctypes.c_int64(0), ctypes.c_int64(0)
        self._check(self._lib.taurus_runs_info(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)), "taurus_runs_info")
        return {"runs": int(a.value), "stored_rows": int(b.value), "buffered_rows": int(c.value)}

    def directory(self) -> np.ndarray:
        """int64 [runs, 4]: id range, rows, first id, last id of every run in writing order."""
        n_runs = self.info()["runs"]
        out = np.zeros((max(n_runs, 1), 4), np.int64)
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_runs_directory(self._h, out.ctypes.data, n_runs, ctypes.byref(n)), "taurus_runs_directory")
        return out[:n.value].copy()

    def get_run(self, run: int, rows_in_run: int):
        ids = np.empty(rows_in_run, np.int64)
        rows = np.empty((rows_in_run, self.width), np.float32)
        self._check(self._lib.taurus_runs_get_run(self._h, run, ids.ctypes.data, rows.ctypes.data), "taurus_runs_get_run")
        return ids, rows

    def reset(self):
        self._check(self._lib.taurus_runs_reset(self._h), "taurus_runs_reset")

    def destroy(self):
        if self._h:
            self._lib.taurus_runs_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Context:
    """One taurus_ctx.  Every method is one C call; see include/taurus.h for the semantics."""

    def __init__(self, V: int, E: int, row_ptr, col_idx, in_degree, mode: int, dims: Sequence[int], W_neigh, W_self,
                 bias, act: Sequence[int], chunk_sources: int, pool_slots: int, hub_count: int = 0,
                 fanout: Optional[Sequence[int]] = None, seed: int = 1, host_evict_rows: int = 0, drain_rows: int = 0,
                 gemm_mode: int = GEMM_FP32, flags: int = 0, evict_policy: int = 0, gin_eps: float = 0.0,
                 att_src=None, att_dst=None, leaky_slope: float = 0.2, gat_heads: int = 1):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        L = len(dims) - 1
        self.V, self.E, self.L, self.dims = V, E, L, tuple(int(d) for d in dims)
        keep = [row_ptr, col_idx, in_degree, W_neigh, W_self, bias]
        g = _Graph(V, E, _ptr(row_ptr), _ptr(col_idx), _ptr(in_degree))
        c_dims = (ctypes.c_int32 * (L + 1))(*self.dims)
        c_act = (ctypes.c_int32 * L)(*[int(a) for a in act])
        c_wn = (ctypes.c_void_p * L)(*[_ptr(w) for w in W_neigh])
        c_ws = (ctypes.c_void_p * L)(*[_ptr(w) for w in W_self]) if W_self is not None else None
        c_b = (ctypes.c_void_p * L)(*[_ptr(b) for b in bias]) if bias is not None else None
        c_as = (ctypes.c_void_p * L)(*[_ptr(a) for a in att_src]) if att_src is not None else None
        c_ad = (ctypes.c_void_p * L)(*[_ptr(a) for a in att_dst]) if att_dst is not None else None
        keep += [att_src, att_dst]
        m = _Model(mode, L, c_dims, c_wn, c_ws, c_b, c_act, gemm_mode, gin_eps, c_as, c_ad, leaky_slope, gat_heads)
        c_f = (ctypes.c_int32 * L)(*[int(f) for f in fanout]) if fanout is not None else None
        r = _Run(chunk_sources, pool_slots, hub_count, c_f, seed, host_evict_rows, drain_rows or chunk_sources, flags, evict_policy)
        rc = self._lib.taurus_graph_init(ctypes.byref(self._h), ctypes.byref(g), ctypes.byref(m), ctypes.byref(r))
        del keep
        if rc != 0:
            self._h = ctypes.c_void_p()
            raise TaurusError(rc, "taurus_graph_init", self._lib.taurus_last_cuda_error().decode())
        self.layer = -1

    def _check(self, rc: int, where: str):
        if rc != 0:
            raise TaurusError(rc, where, self._lib.taurus_last_cuda_error().decode() if rc == ERROR_CODES["CUDA"] else "")

    def layer_begin(self, layer: int, stream=None):
        self._check(self._lib.taurus_layer_begin(self._h, layer, _stream(stream)), "taurus_layer_begin")
        self.layer = layer

    def push_chunk(self, src_begin: int, src_end: int, features, stream=None, raise_on_drain_full: bool = True) -> int:
        rc = self._lib.taurus_push_chunk(self._h, src_begin, src_end, _ptr(features), _stream(stream))
        if rc == ERROR_CODES["DRAIN_FULL"] and not raise_on_drain_full:
            return rc
        self._check(rc, "taurus_push_chunk")
        return rc

    def gat_project_chunk(self, src_begin: int, src_end: int, features, hprime_out, ld: int, stream=None):
        self._check(self._lib.taurus_gat_project_chunk(self._h, src_begin, src_end, _ptr(features), _ptr(hprime_out), ld,
                                                       _stream(stream)), "taurus_gat_project_chunk")

    def gat_project_chunk_from_runs(self, src_begin: int, src_end: int, runs: "Runs", hprime_out, ld: int, stream=None):
        self._check(self._lib.taurus_gat_project_chunk_from_runs(self._h, src_begin, src_end, runs._h, _ptr(hprime_out), ld,
                                                                 _stream(stream)), "taurus_gat_project_chunk_from_runs")

    def gat_attention(self, stream=None):
        self._check(self._lib.taurus_gat_attention(self._h, _stream(stream)), "taurus_gat_attention")

    def drain_completed(self, out_ids, out_rows, capacity_rows: int) -> int:
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_drain_completed(self._h, _ptr(out_ids), _ptr(out_rows), capacity_rows, ctypes.byref(n)),
                    "taurus_drain_completed")
        return int(n.value)

    def drain_dense(self, dense_rows, ld: int, capacity_rows: int, out_ids=None) -> int:
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_drain_dense(self._h, _ptr(dense_rows), ld, _ptr(out_ids), capacity_rows, ctypes.byref(n)),
                    "taurus_drain_dense")
        return int(n.value)

    def layer_set_dense_output(self, dense_rows, ld: int):
        self._check(self._lib.taurus_layer_set_dense_output(self._h, _ptr(dense_rows), ld), "taurus_layer_set_dense_output")

    def layer_set_run_output(self, runs: "Runs"):
        self._check(self._lib.taurus_layer_set_run_output(self._h, runs._h), "taurus_layer_set_run_output")

    def push_chunk_from_runs(self, src_begin: int, src_end: int, runs: "Runs", stream=None):
        self._check(self._lib.taurus_push_chunk_from_runs(self._h, src_begin, src_end, runs._h, _stream(stream)),
                    "taurus_push_chunk_from_runs")

    def layer_end(self) -> dict:
        s = Stats()
        self._check(self._lib.taurus_layer_end(self._h, ctypes.byref(s)), "taurus_layer_end")
        return s.as_dict()

    def get_stats(self) -> dict:
        s = Stats()
        self._check(self._lib.taurus_get_stats(self._h, ctypes.byref(s)), "taurus_get_stats")
        return s.as_dict()

    def get_chunk_log(self, capacity_chunks: int = 1 << 20) -> dict:
        out = np.zeros((capacity_chunks, len(CHUNK_LOG_COLUMNS)), np.int64)
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_get_chunk_log(self._h, out.ctypes.data, capacity_chunks, ctypes.byref(n)),
                    "taurus_get_chunk_log")
        return {k: out[:n.value, i].copy() for i, k in enumerate(CHUNK_LOG_COLUMNS)}

    def get_vertex_array(self, which: str) -> np.ndarray:
        idx = {"state": 0, "pending": 1, "reload_count": 2, "hub": 3}[which]
        out = np.empty(self.V, np.uint8 if idx in (0, 3) else np.int32)
        self._check(self._lib.taurus_get_vertex_array(self._h, idx, out.ctypes.data), "taurus_get_vertex_array")
        return out

    def get_sampled_edges(self, layer: int, dst: int, capacity: int = 1 << 16):
        eids = np.empty(capacity, np.int64)
        srcs = np.empty(capacity, np.int32)
        n = ctypes.c_int32(0)
        self._check(self._lib.taurus_get_sampled_edges(self._h, layer, dst, eids.ctypes.data, srcs.ctypes.data, capacity,
                                                       ctypes.byref(n)), "taurus_get_sampled_edges")
        k = min(n.value, capacity)
        return eids[:k].copy(), srcs[:k].copy(), int(n.value)

    def get_edge_mask(self) -> np.ndarray:
        words = np.empty((self.E + 31) // 32, np.uint32)
        self._check(self._lib.taurus_get_edge_mask(self._h, words.ctypes.data), "taurus_get_edge_mask")
        return words

    def get_sample_digest(self) -> np.ndarray:
        """uint64 [V, 2]: (sum, xor) of the mixed (source, CSR edge index) pairs of every vertex's propagated in-edges."""
        out = np.empty((self.V, 2), np.uint64)
        self._check(self._lib.taurus_get_sample_digest(self._h, out.ctypes.data), "taurus_get_sample_digest")
        return out

    def completion_bound(self, src_begin: int, src_end: int) -> int:
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_completion_bound(self._h, src_begin, src_end, ctypes.byref(n)), "taurus_completion_bound")
        return int(n.value)

    def layer_plan(self, layer: int):
        """(aggregate_first, floats per accumulator row) of a layer, as decided at init."""
        af, width = ctypes.c_int32(0), ctypes.c_int32(0)
        self._check(self._lib.taurus_get_layer_plan(self._h, layer, ctypes.addressof(af), ctypes.addressof(width)),
                    "taurus_get_layer_plan")
        return bool(af.value), int(width.value)

    def launch_count(self) -> int:
        return int(self._lib.taurus_launch_count(self._h))

    def set_timing(self, on):
        """False / 0: off; True / 1: events after every phase of a push; 2: events around the scatter only."""
        self._check(self._lib.taurus_set_timing(self._h, int(on)), "taurus_set_timing")

    def get_phase_ms(self, capacity_pushes: int = 16384) -> np.ndarray:
        """float32 [pushes, 9] (ms per recorded push): copy-in, projection, classify + victim selection, wait for the
        previous chunk's transfers + its finalise, slot hand-out, scatter, completion list, own finalise, row
        transfers over the host link (side stream)."""
        out = np.zeros((capacity_pushes, 9), np.float32)
        n = ctypes.c_int64(0)
        self._check(self._lib.taurus_get_phase_ms(self._h, out.ctypes.data, capacity_pushes, ctypes.byref(n)),
                    "taurus_get_phase_ms")
        return out[:n.value].copy()

    def destroy(self):
        if self._h:
            self._lib.taurus_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
