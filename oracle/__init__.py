"""CPU oracle for the layer-wise GNN step.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

A plain, slow, pull-based ("gather", Eq. 1-2) fp64 implementation of what the
CUDA library computes with source-centric broadcasts, plus an integer-only
simulator of the vertex state machine (Sect. 3.4-3.6) at chunk granularity.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import
this package; it shares no code with the CUDA path and never imports it.

The float side deliberately aggregates raw rows first and transforms afterwards
(Eq. 1 then Eq. 2), the opposite order from the CUDA path, so that the two
sides have no structure in common.

Pins (tests/test_oracle_*.py): dense-adjacency products, ring/star/complete
closed forms, constant-feature and linearity invariants, split vs concatenated
weights (SAGEConv paragraph of Sect. 3.9), sampler set properties and
uniformity, completion closed form vs simulator, active-set identity
(Sect. 3.8), a second independent simulator.  Nothing here is parity unpinned.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "taurus_oracle.c")
_SO = os.path.join(_HERE, "libtaurus_oracle.so")
_handle = None

SAGE_MEAN = 0
GCN_SYM = 1
GIN_SUM = 2

# eviction policies: the paper's (Sect. 3.5.3) and the alternatives of its ablation (Sect. 4.5)
EVICT_FEWEST_PENDING, EVICT_FIFO, EVICT_LRU, EVICT_RANDOM = 0, 1, 2, 3

# vertex states, Sect. 3.4
NOT_STARTED, IN_BUFFER, EVICTED, ON_GPU, COMPLETED = 0, 1, 2, 3, 4

STAT_KEYS = ["evictions", "reloads", "max_reload_count", "peak_occupancy", "hub_messages", "total_messages",
             "hub_vertices", "completed", "sum_hs", "sum_ns", "sum_ev", "sum_gs", "free_end", "bad_transitions"]
CHUNK_KEYS = ["hs", "ns", "ev", "gs", "need", "evicted", "reloaded", "completed", "occupancy"]


def build(force: bool = False) -> str:
    """Compile the oracle's C source with gcc (building the checker is not using it)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


def _lib():
    global _handle
    if _handle is None:
        lib = ctypes.CDLL(build())
        vp, i64, i32, u64 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32, ctypes.c_uint64
        lib.to_build_in_lists.argtypes = [i64, i64, vp, vp, vp, vp, vp]
        lib.to_sample_hash.restype = u64
        lib.to_sample_hash.argtypes = [u64, u64, u64, u64]
        lib.to_sample_positions.argtypes = [u64, i32, i64, i64, i32, vp]
        lib.to_message_sets.argtypes = [i64, vp, vp, vp, i32, u64, i32, vp, vp, vp, vp]
        lib.to_aggregate.argtypes = [i64, vp, vp, vp, vp, vp, i32, vp]
        lib.to_simulate.argtypes = [i64, vp, vp, vp, vp, vp, i64, i64, i32, u64, vp, vp, vp, vp, vp]
        lib.to_completion_rank_exact.argtypes = [i64, vp, vp, vp]
        lib.to_scan_in_edges.restype = i64
        lib.to_scan_in_edges.argtypes = [i64, vp, vp, vp, vp, vp, i64]
        lib.to_evict_hash.restype = ctypes.c_uint32
        lib.to_evict_hash.argtypes = [u64, u64, u64]
        _handle = lib
    return _handle


def cores_used() -> int:
    """Threads the OpenMP loops of the oracle run on."""
    n = os.environ.get("OMP_NUM_THREADS")
    return int(n) if n else len(os.sched_getaffinity(0))


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data


# ----------------------------------------------------------------------------- in-lists and message sets

@dataclass
class InLists:
    """In-neighbour lists (ascending source id, duplicates in CSR order)."""
    ptr: np.ndarray   # int64 [V+1]
    src: np.ndarray   # int32 [E]
    eid: np.ndarray   # int64 [E]  CSR edge index of each entry


def build_in_lists(V: int, row_ptr: np.ndarray, col: np.ndarray) -> InLists:
    E = int(row_ptr[V])
    ptr = np.empty(V + 1, np.int64)
    src = np.empty(E, np.int32)
    eid = np.empty(E, np.int64)
    rc = _lib().to_build_in_lists(V, E, _p(row_ptr), _p(col), _p(ptr), _p(src), _p(eid))
    if rc:
        raise MemoryError
    return InLists(ptr, src, eid)


def sample_positions(seed: int, layer: int, dst: int, din: int, fanout: int) -> np.ndarray:
    """In-list positions kept for dst (Sect. 3.9 sampling paragraph), in draw order."""
    n = din if (fanout <= 0 or din <= fanout) else fanout
    out = np.empty(max(n, 1), np.int64)
    rc = _lib().to_sample_positions(seed, layer, dst, din, fanout, _p(out))
    if rc:
        raise MemoryError
    return out[:n]


@dataclass
class MessageSets:
    """M(v) for every v for one layer: the propagated in-edges."""
    ptr: np.ndarray    # int64 [V+1]
    src: np.ndarray    # int32
    eid: np.ndarray    # int64 CSR edge index
    prop: Optional[np.ndarray]   # uint8 [E], 1 = propagated (None in exact mode = all)
    m: np.ndarray      # int32 [V]  |M(v)|


def message_sets(inl: InLists, fanout: int, seed: int, layer: int) -> MessageSets:
    V = inl.ptr.size - 1
    din = np.diff(inl.ptr)
    if fanout <= 0:
        return MessageSets(inl.ptr, inl.src, inl.eid, None, din.astype(np.int32))
    m = np.minimum(din, fanout)
    ptr = np.zeros(V + 1, np.int64)
    np.cumsum(m, out=ptr[1:])
    n = int(ptr[V])
    src = np.empty(n, np.int32)
    eid = np.empty(n, np.int64)
    prop = np.zeros(inl.src.size, np.uint8)
    rc = _lib().to_message_sets(V, _p(inl.ptr), _p(inl.src), _p(inl.eid), fanout, seed, layer,
                                _p(ptr), _p(src), _p(eid), _p(prop))
    if rc:
        raise MemoryError
    return MessageSets(ptr, src, eid, prop, m.astype(np.int32))


def sample_digest(ms: MessageSets) -> np.ndarray:
    """uint64 [V, 2]: per destination the sum (mod 2^64) and the xor of mix64(((u << 32) | e) + golden) over its
    propagated in-edges (source u, CSR edge index e); (0, 0) for an empty set.  A commutative fingerprint of M(v)
    (Sect. 3.9 sampling paragraph: the sampled set is a function of seed, layer and destination)."""
    M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
    with np.errstate(over="ignore"):
        x = ((ms.src.astype(np.uint64) << np.uint64(32)) | (ms.eid.astype(np.uint64) & np.uint64(0xFFFFFFFF))) + np.uint64(0x9E3779B97F4A7C15)
        x ^= x >> np.uint64(30); x = (x * np.uint64(0xBF58476D1CE4E5B9)) & M64
        x ^= x >> np.uint64(27); x = (x * np.uint64(0x94D049BB133111EB)) & M64
        x ^= x >> np.uint64(31)
        V = ms.m.size
        out = np.zeros((V, 2), np.uint64)
        nz = np.flatnonzero(ms.m > 0)
        if nz.size:
            out[nz, 0] = np.add.reduceat(x, ms.ptr[nz])
            out[nz, 1] = np.bitwise_xor.reduceat(x, ms.ptr[nz])
    return out


# ----------------------------------------------------------------------------- one layer, pull-based, fp64

def coefficients(mode: int, m: np.ndarray, din: np.ndarray, dout: np.ndarray, gin_eps: float = 0.0):
    """(c_out[V], c_in[V], c_self[V]) in fp64.

    SAGE-mean (Sect. 3.4 normalised message, SAGEConv paragraph of Sect. 3.9):
        c_out = 1, c_in = 1 / max(|M(v)|, 1), c_self = 1.
    GCN symmetric norm with the implicit self message every vertex aggregates (Sect. 3.8):
        c_out(u) = (dout(u) + 1)^-1/2, c_in(v) = (din(v) + 1)^-1/2, c_self = c_out * c_in,
        with the full-graph degrees also under sampling.
    GIN (sum aggregator; "GCN/GIN-style aggregation", Sect. 3.9; one of the models of Sect. 4.1):
        c_out = 1, c_in = 1, c_self = 1 + eps, with one shared weight.
    """
    V = m.size
    if mode == SAGE_MEAN:
        return np.ones(V), 1.0 / np.maximum(m.astype(np.float64), 1.0), np.ones(V)
    if mode == GIN_SUM:
        return np.ones(V), np.ones(V), np.full(V, 1.0 + gin_eps)
    c_out = (dout.astype(np.float64) + 1.0) ** -0.5
    c_in = (din.astype(np.float64) + 1.0) ** -0.5
    return c_out, c_in, c_out * c_in


def aggregate(ms: MessageSets, dst: np.ndarray, c_out: Optional[np.ndarray], h: np.ndarray) -> np.ndarray:
    """agg[i] = sum over u in M(dst[i]) of c_out[u] * h[u], fp64 (Eq. 1)."""
    h = np.ascontiguousarray(h, dtype=np.float64)
    dst = np.ascontiguousarray(dst, dtype=np.int64)
    agg = np.empty((dst.size, h.shape[1]), np.float64)
    co = None if c_out is None else np.ascontiguousarray(c_out, dtype=np.float64)
    _lib().to_aggregate(dst.size, _p(dst), _p(ms.ptr), _p(ms.src), _p(co), _p(h), h.shape[1], _p(agg))
    return agg


def layer_forward(ms: MessageSets, mode: int, din: np.ndarray, dout: np.ndarray, h: np.ndarray,
                  W_neigh: np.ndarray, W_self: np.ndarray, bias: np.ndarray, act: int,
                  dst: Optional[np.ndarray] = None, gin_eps: float = 0.0) -> np.ndarray:
    """out_v = act(c_in(v) * (agg_v @ W_neigh) + c_self(v) * (h_v @ W_self) + b) for v in dst (default: all), Eq. 1-2."""
    V = ms.m.size
    if dst is None:
        dst = np.arange(V, dtype=np.int64)
    c_out, c_in, c_self = coefficients(mode, ms.m, din, dout, gin_eps)
    h = np.asarray(h, dtype=np.float64)
    agg = aggregate(ms, dst, c_out if mode == GCN_SYM else None, h)
    Wn = np.asarray(W_neigh, dtype=np.float64)
    Ws = np.asarray(W_self, dtype=np.float64) if mode == SAGE_MEAN else Wn
    z = c_in[dst, None] * (agg @ Wn) + c_self[dst, None] * (h[dst] @ Ws) + np.asarray(bias, dtype=np.float64)[None, :]
    return np.maximum(z, 0.0) if act else z


# ----------------------------------------------------------------------------- a destination subset of a large graph
# Where the whole graph is out of reach, the same definition is evaluated for a listed subset of destinations:
# their in-lists come from one scan of the CSR, everything else is the code above.

def subset_in_lists(V: int, row_ptr: np.ndarray, col: np.ndarray, dsts: np.ndarray):
    """In-lists (ascending source id, duplicates in CSR order) of the sorted, distinct destinations dsts.
    Returns (ptr int64 [len(dsts) + 1], src int64, eid int64)."""
    dsts = np.asarray(dsts, dtype=np.int64)
    wanted = np.zeros(V, dtype=np.uint8)
    wanted[dsts] = 1
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int64)
    col = np.ascontiguousarray(col, dtype=np.int32)
    n = int(_lib().to_scan_in_edges(V, _p(row_ptr), _p(col), _p(wanted), None, None, 0))
    sel = np.empty(n, np.int64)                                # ascending CSR edge index = (source, position) order
    src = np.empty(n, np.int64)
    if int(_lib().to_scan_in_edges(V, _p(row_ptr), _p(col), _p(wanted), _p(sel), _p(src), n)) != n:
        raise MemoryError
    d = col[sel]
    order = np.argsort(d, kind="stable")
    sel, src, d = sel[order], src[order], d[order]
    ptr = np.zeros(dsts.size + 1, np.int64)
    np.cumsum(np.bincount(np.searchsorted(dsts, d), minlength=dsts.size), out=ptr[1:])
    return ptr, src, sel


def subset_message_sets(ptr: np.ndarray, src: np.ndarray, eid: np.ndarray, dsts: np.ndarray, fanout: int, seed: int, layer: int):
    """M(v) of the listed destinations from their in-lists: all entries, or the sampled positions (Sect. 3.9).
    Returns (keep_ptr, keep_src, keep_eid), kept entries in ascending in-list position."""
    keep_ptr, keep_src, keep_eid = [0], [], []
    for i, v in enumerate(dsts):
        lo, hi = int(ptr[i]), int(ptr[i + 1])
        p = np.sort(sample_positions(seed, layer, int(v), hi - lo, fanout))
        keep_src.append(src[lo:hi][p]); keep_eid.append(eid[lo:hi][p])
        keep_ptr.append(keep_ptr[-1] + p.size)
    cat = lambda xs: np.concatenate(xs) if xs else np.zeros(0, np.int64)
    return np.asarray(keep_ptr, np.int64), cat(keep_src), cat(keep_eid)


def subset_forward(mode: int, dsts: np.ndarray, keep_ptr: np.ndarray, keep_src: np.ndarray, din_dst: np.ndarray, dout_dst: np.ndarray,
                   need: np.ndarray, dout_need: np.ndarray, h_need: np.ndarray, W_neigh: np.ndarray, W_self: np.ndarray,
                   bias: np.ndarray, act: int, gin_eps: float = 0.0) -> np.ndarray:
    """Eq. 1-2 for the destinations dsts.  need = sorted distinct ids of every kept source and every destination,
    h_need their input rows, dout_need their out-degrees (GCN); din_dst / dout_dst the degrees of the destinations."""
    m = np.diff(keep_ptr).astype(np.int32)
    ms = MessageSets(keep_ptr, np.searchsorted(need, keep_src).astype(np.int32), None, None, m)
    c_out, c_in, c_self = coefficients(mode, m, din_dst, dout_dst, gin_eps)
    c_out_src = (dout_need.astype(np.float64) + 1.0) ** -0.5 if mode == GCN_SYM else None
    h = np.asarray(h_need, dtype=np.float64)
    agg = aggregate(ms, np.arange(dsts.size), c_out_src, h)
    Wn = np.asarray(W_neigh, dtype=np.float64)
    Ws = np.asarray(W_self, dtype=np.float64) if mode == SAGE_MEAN else Wn
    z = c_in[:, None] * (agg @ Wn) + c_self[:, None] * (h[np.searchsorted(need, dsts)] @ Ws) + np.asarray(bias, dtype=np.float64)[None, :]
    return np.maximum(z, 0.0) if act else z


def forward(V: int, row_ptr: np.ndarray, col: np.ndarray, x: np.ndarray, mode: int, W_neigh: Sequence[np.ndarray],
            W_self: Sequence[np.ndarray], bias: Sequence[np.ndarray], act: Sequence[int],
            fanout: Sequence[int], seed: int, inl: Optional[InLists] = None, gin_eps: float = 0.0) -> List[np.ndarray]:
    """All layers; layer l+1 consumes this oracle's own fp64 output of layer l.  Returns every layer's output."""
    inl = inl or build_in_lists(V, row_ptr, col)
    din = np.diff(inl.ptr)
    dout = np.diff(row_ptr)
    h = np.asarray(x, dtype=np.float64)
    outs = []
    for l in range(len(W_neigh)):
        ms = message_sets(inl, fanout[l], seed, l)
        h = layer_forward(ms, mode, din, dout, h, W_neigh[l], W_self[l], bias[l], act[l], gin_eps=gin_eps)
        outs.append(h)
    return outs


# ----------------------------------------------------------------------------- integer side

def hub_set(in_degree: np.ndarray, hub_count: int) -> np.ndarray:
    """uint8 [V] flag of the hub_count vertices largest by (-in_degree, id) (GPU store, Sect. 3.5.1)."""
    V = in_degree.size
    flag = np.zeros(V, np.uint8)
    if hub_count > 0:
        order = np.lexsort((np.arange(V), -in_degree.astype(np.int64)))
        flag[order[:hub_count]] = 1
    return flag


def complete_chunk_closed_form(ms: MessageSets, chunk_sources: int) -> np.ndarray:
    """Chunk in which v completes: floor(max(v, max M(v)) / chunk), from c(v) = max rank of the in-neighbours (Sect. 3.8)."""
    V = ms.m.size
    last = np.arange(V, dtype=np.int64)
    nz = np.flatnonzero(ms.m > 0)
    if nz.size:
        mx = np.maximum.reduceat(ms.src.astype(np.int64), ms.ptr[nz])
        last[nz] = np.maximum(last[nz], mx)
    return (last // chunk_sources).astype(np.int32)


def completion_rank_exact(V: int, row_ptr: np.ndarray, col: np.ndarray) -> np.ndarray:
    """max(v, largest in-neighbour of v) for every v of an exact layer, straight from the CSR (no in-lists needed): the
    rank whose chunk completes v (Sect. 3.8, c(v))."""
    rank = np.empty(V, np.int32)
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int64)
    col = np.ascontiguousarray(col, dtype=np.int32)
    _lib().to_completion_rank_exact(V, _p(row_ptr), _p(col), _p(rank))
    return rank


def first_touch_chunk(ms: MessageSets, chunk_sources: int) -> np.ndarray:
    """Chunk in which v becomes active: floor(min(v, min M(v)) / chunk), from a(v) (Sect. 3.8)."""
    V = ms.m.size
    first = np.arange(V, dtype=np.int64)
    nz = np.flatnonzero(ms.m > 0)
    if nz.size:
        mn = np.minimum.reduceat(ms.src.astype(np.int64), ms.ptr[nz])
        first[nz] = np.minimum(first[nz], mn)
    return (first // chunk_sources).astype(np.int32)


@dataclass
class SimResult:
    stats: dict
    complete_chunk: np.ndarray   # int32 [V]
    reload_count: np.ndarray     # int32 [V]
    per_chunk: dict              # name -> int64 [n_chunks]
    last_evict_chunk: np.ndarray  # int32 [V], -1 = never evicted
    rc: int


def simulate(V: int, row_ptr: np.ndarray, col: np.ndarray, ms: MessageSets, is_hub: np.ndarray,
             chunk_sources: int, pool_slots: int, policy: int = EVICT_FEWEST_PENDING, seed: int = 0) -> SimResult:
    """Chunk-granular state machine (Sect. 3.4-3.6).  rc: 0 ok, -2/-3 pool too small."""
    n_chunks = (V + chunk_sources - 1) // chunk_sources
    stats = np.zeros(len(STAT_KEYS), np.int64)
    cc = np.empty(V, np.int32)
    rcount = np.empty(V, np.int32)
    per = np.zeros((n_chunks, len(CHUNK_KEYS)), np.int64)
    evlog = np.empty(V, np.int32)
    m = np.ascontiguousarray(ms.m, dtype=np.int32)
    hub = np.ascontiguousarray(is_hub, dtype=np.uint8)
    rc = _lib().to_simulate(V, _p(row_ptr), _p(col), _p(ms.prop), _p(m), _p(hub), chunk_sources, pool_slots, policy, seed,
                            _p(stats), _p(cc), _p(rcount), _p(per), _p(evlog))
    if rc == -1:
        raise MemoryError
    return SimResult({k: int(stats[i]) for i, k in enumerate(STAT_KEYS)}, cc, rcount,
                     {k: per[:, i].copy() for i, k in enumerate(CHUNK_KEYS)}, evlog, rc)


# ----------------------------------------------------------------------------- topology-aware reordering (Sect. 3.8)

def _in_sums(V: int, row_ptr: np.ndarray, col: np.ndarray, per_source: np.ndarray) -> np.ndarray:
    """sum over in-edges (u -> v) of per_source[u], for every v (edges visited in CSR order)."""
    src = np.repeat(np.arange(V), np.diff(row_ptr))
    return np.bincount(col, weights=per_source[src], minlength=V)


def _out_sums(V: int, row_ptr: np.ndarray, col: np.ndarray, per_dst: np.ndarray) -> np.ndarray:
    """sum over out-edges (w -> v) of per_dst[v], for every w."""
    src = np.repeat(np.arange(V), np.diff(row_ptr))
    return np.bincount(src, weights=per_dst[col], minlength=V)


def reorder_step(V: int, row_ptr: np.ndarray, col: np.ndarray, r: np.ndarray):
    """One iteration of Alg. 1 on real-valued positions r.  Every vertex also aggregates its own self message,
    so d(v) = in_degree(v) + 1 >= 1 and v belongs to its own in- and out-neighbourhood (Sect. 3.8).

        mu(v) = (r(v) + sum_{u -> v} r(u)) / d(v)
        r'(w) = (mu(w)/d(w) + sum_{w -> v} mu(v)/d(v)) / (1/d(w) + sum_{w -> v} 1/d(v))

    Returns (mu, r')."""
    r = np.asarray(r, dtype=np.float64)
    d = np.bincount(col, minlength=V).astype(np.float64) + 1.0
    mu = (r + _in_sums(V, row_ptr, col, r)) / d
    num = mu / d + _out_sums(V, row_ptr, col, mu / d)
    den = 1.0 / d + _out_sums(V, row_ptr, col, 1.0 / d)
    return mu, num / den


def dispersion_J(V: int, row_ptr: np.ndarray, col: np.ndarray, r: np.ndarray, mu: np.ndarray) -> float:
    """J(r, mu) = sum_v 1/d(v) * sum_{u in N^-(v) + self} (r(u) - mu(v))^2  (Sect. 3.8)."""
    d = np.bincount(col, minlength=V).astype(np.float64) + 1.0
    src = np.repeat(np.arange(V), np.diff(row_ptr))
    per_edge = (r[src] - mu[col]) ** 2 / d[col]
    return float(per_edge.sum() + ((r - mu) ** 2 / d).sum())


def total_span(V: int, row_ptr: np.ndarray, col: np.ndarray, rank: np.ndarray) -> int:
    """C(pi) = sum_v (max - min) of the processing ranks over v's in-neighbours and v itself (Sect. 3.8)."""
    rank = np.asarray(rank, dtype=np.int64)
    src = np.repeat(np.arange(V), np.diff(row_ptr))
    hi, lo = rank.copy(), rank.copy()
    np.maximum.at(hi, col, rank[src])
    np.minimum.at(lo, col, rank[src])
    return int((hi - lo).sum())


def relabel_csr(V: int, row_ptr: np.ndarray, col: np.ndarray, rank: np.ndarray):
    """The graph with vertex v renamed rank[v] (Sect. 3.8, topology relabelling): row rank[u] = the out-edges of u in
    their original order, destinations renamed.  Returns (row_ptr, col, in_degree)."""
    rank = np.asarray(rank, dtype=np.int64)
    old_of_new = np.empty(V, np.int64)
    old_of_new[rank] = np.arange(V)
    deg = np.diff(row_ptr)
    new_ptr = np.zeros(V + 1, np.int64)
    np.cumsum(deg[old_of_new], out=new_ptr[1:])
    new_col = np.empty(int(row_ptr[V]), np.int32)
    for nu in range(V):
        u = old_of_new[nu]
        new_col[new_ptr[nu]:new_ptr[nu + 1]] = rank[col[row_ptr[u]:row_ptr[u + 1]]]
    return new_ptr, new_col, np.bincount(new_col, minlength=V).astype(np.int32)


def ranks_of(r: np.ndarray) -> np.ndarray:
    """pi = ArgSort(r), ties by vertex id; returned as the rank of every vertex."""
    order = np.argsort(r, kind="stable")
    rank = np.empty(r.size, np.int64)
    rank[order] = np.arange(r.size)
    return rank


def reorder(V: int, row_ptr: np.ndarray, col: np.ndarray, initial_rank: Optional[np.ndarray] = None, iterations: int = 5):
    """Alg. 1: r <- pi0; repeat (mu, r) updates; pi <- ArgSort(r).  Returns (rank, history) where history holds,
    for the initial ordering and after every iteration, (J, C(pi))."""
    r = np.arange(V, dtype=np.float64) if initial_rank is None else np.asarray(initial_rank, dtype=np.float64)
    rank = ranks_of(r)

    def measures(rank):
        # J is evaluated on the ordering itself (positions = ranks, centres = their optimum), so that its values
        # are comparable across iterations although the real-valued positions contract
        pos = rank.astype(np.float64)
        mu_pos, _ = reorder_step(V, row_ptr, col, pos)
        return dispersion_J(V, row_ptr, col, pos, mu_pos), total_span(V, row_ptr, col, rank)

    hist = [measures(rank)]
    for _ in range(iterations):
        _, r = reorder_step(V, row_ptr, col, r)
        rank = ranks_of(r)
        hist.append(measures(rank))
    return rank, hist, r
