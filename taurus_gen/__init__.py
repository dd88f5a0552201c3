"""Seeded synthetic inputs: graphs, feature rows, weights, and the workload table.

This package defines the *problem* only (what graph, what features, what
weights, what run parameters).  It contains none of the method's arithmetic and
is the only code shared by the CPU oracle's tests and the CUDA library's tests.
The C source next to this file is compiled with gcc on first use.
"""
from __future__ import annotations

import ctypes
import math
import os
import subprocess
from dataclasses import dataclass, field, replace
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_SO = os.path.join(_HERE, "libtaurus_gen.so")
_lib_handle = None


def build(force: bool = False) -> str:
    """Compile gen.c into libtaurus_gen.so (skipped when the library is newer than its source)."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _SO)
    return _SO


class _Params(ctypes.Structure):
    _fields_ = [
        ("seed", ctypes.c_uint64), ("V", ctypes.c_int64), ("alpha", ctypes.c_double),
        ("kappa", ctypes.c_double), ("d_max", ctypes.c_int64), ("dst_mode", ctypes.c_int32),
        ("lam", ctypes.c_double), ("local_B", ctypes.c_double), ("beta", ctypes.c_double),
        ("r0", ctypes.c_double), ("perm_a", ctypes.c_int64), ("perm_b", ctypes.c_int64),
    ]


def _lib():
    global _lib_handle
    if _lib_handle is None:
        lib = ctypes.CDLL(build())
        P = ctypes.POINTER(_Params)
        vp = ctypes.c_void_p
        lib.tg_hash64.restype = ctypes.c_uint64
        lib.tg_hash64.argtypes = [ctypes.c_uint64] * 4
        lib.tg_calibrate_kappa.restype = ctypes.c_double
        lib.tg_calibrate_kappa.argtypes = [P, ctypes.c_int64]
        lib.tg_out_degrees.argtypes = [P, vp]
        lib.tg_fill_directed.argtypes = [P, vp, vp]
        lib.tg_fill_symmetric.argtypes = [P, vp, vp, vp]
        lib.tg_in_degrees.argtypes = [ctypes.c_int64, ctypes.c_int64, vp, vp]
        lib.tg_features.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int64, ctypes.c_int64,
                                    ctypes.c_int32, ctypes.c_int64, vp]
        lib.tg_features_rows.argtypes = [ctypes.c_uint64, ctypes.c_uint64, vp, ctypes.c_int64, ctypes.c_int32,
                                         ctypes.c_int64, vp]
        lib.tg_weights.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int32,
                                   ctypes.c_int32, vp]
        lib.tg_zipf_top_mass.restype = ctypes.c_double
        lib.tg_zipf_top_mass.argtypes = [ctypes.c_double] * 3
        _lib_handle = lib
    return _lib_handle


def hash64(seed: int, tag: int, i: int, j: int) -> int:
    return int(_lib().tg_hash64(seed, tag, i, j))


# ----------------------------------------------------------------------------- workloads

SAGE_MEAN = 0
GCN_SYM = 1
GIN_SUM = 2
GAT = 3
GEMM_FP32 = 0
GEMM_BF16 = 1


@dataclass(frozen=True)
class Workload:
    """One synthetic workload: graph shape, model and run parameters."""
    name: str
    V: int
    E: int                      # target edge count (the realised count is within 0.1 %)
    alpha: float                # out-degree power-law exponent
    d_max: int                  # cap on the out-degree weight
    dst_mode: int               # 0 uniform, 1 local + hub-Zipf
    lam: float                  # share of local destinations (mode 1)
    top_in: int                 # target for the largest in-degree (mode 1)
    symmetric: bool
    dims: Tuple[int, ...]       # F, hidden..., out
    mode: int                   # SAGE_MEAN, GCN_SYM, GIN_SUM or GAT
    chunk: int                  # sources per pushed chunk
    pool_slots: int             # accumulator slot pool capacity
    hub_count: int              # vertices pinned in the GPU-resident store
    fanout: Tuple[int, ...]     # per layer, 0 = exact
    gemm_mode: int = GEMM_FP32
    seed: int = 1
    gin_eps: float = 0.0        # GIN_SUM only: the self weight is 1 + gin_eps
    leaky_slope: float = 0.2    # GAT only: negative slope of the LeakyReLU on the attention scores
    gat_heads: int = 1          # GAT only: attention heads; head i owns columns [i d, (i + 1) d) of every layer's output

    @property
    def L(self) -> int:
        return len(self.dims) - 1

    @property
    def act(self) -> Tuple[int, ...]:
        """ReLU on every layer but the last."""
        return tuple([1] * (self.L - 1) + [0])


# The five configurations.  The graphs of the paper's Table 1 are not available;
# these are seeded stand-ins of the same shapes.
WORKLOADS = {
    "tiny": Workload("tiny", 10_000, 100_000, 2.1, 10_000, 0, 0.0, 0, False, (64, 64, 16), SAGE_MEAN,
                     1024, 10_000, 0, (0, 0)),
    "mid": Workload("mid", 2_450_000, 124_000_000, 2.1, 20_000, 1, 0.5, 20_000, True, (100, 256, 256, 47),
                    SAGE_MEAN, 65_536, 2_450_000, 0, (0, 0, 0)),
    "large": Workload("large", 111_000_000, 1_600_000_000, 2.0, 100_000, 1, 0.5, 100_000, False,
                      (128, 256, 256, 256), SAGE_MEAN, 65_536, 20_000_000, 111_000, (0, 0, 0)),
    "sampled": Workload("sampled", 111_000_000, 1_600_000_000, 2.0, 100_000, 1, 0.5, 100_000, False,
                        (128, 256, 256, 256), SAGE_MEAN, 65_536, 20_000_000, 111_000, (15, 10, 5)),
    "stress": Workload("stress", 269_000_000, 4_000_000_000, 1.8, 2_000_000, 1, 0.5, 2_000_000, False,
                       (512, 256, 256), GCN_SYM, 65_536, 40_000_000, 269_000, (0, 0), GEMM_BF16),
}


def scaled(w: Workload, V: int, chunk: Optional[int] = None, name: Optional[str] = None) -> Workload:
    """The same workload shape at a smaller vertex count (edges, pool, hubs and degree caps scale along)."""
    f = V / w.V
    return replace(
        w, name=name or "%s@%d" % (w.name, V), V=V, E=max(V, int(round(w.E * f))),
        d_max=max(16, int(w.d_max * f ** 0.5)), top_in=max(16, int(w.top_in * f ** 0.5)) if w.top_in else 0,
        pool_slots=max(1, int(math.ceil(w.pool_slots * f))), hub_count=int(math.ceil(w.hub_count * f)),
        chunk=chunk or w.chunk)


@dataclass
class Graph:
    V: int
    E: int
    row_ptr: np.ndarray      # int64 [V+1]
    col_idx: np.ndarray      # int32 [E]
    in_degree: np.ndarray    # int32 [V]
    params: dict = field(default_factory=dict)


def _coprime_multiplier(V: int) -> int:
    a = max(1, int(V * 0.6180339887498949)) | 1
    while math.gcd(a, V) != 1:
        a += 2
    return a


def _solve_r0(beta: float, V: int, hub_edges: float, top_in: float) -> float:
    """Shift r0 of the rank law so that rank 0 expects top_in of the hub_edges hub-directed edges."""
    lib = _lib()
    target = min(0.5, top_in / max(hub_edges, 1.0))
    lo, hi = 1e-6, float(V) * 10
    for _ in range(200):
        mid = math.sqrt(lo * hi)
        if lib.tg_zipf_top_mass(beta, mid, float(V)) > target:
            lo = mid
        else:
            hi = mid
    return math.sqrt(lo * hi)


def make_graph(w: Workload) -> Graph:
    """Build the CSR out-edge graph of workload w (deterministic in w.seed)."""
    lib = _lib()
    V = w.V
    E_gen = w.E // 2 if w.symmetric else w.E
    beta = 1.0 / (w.alpha - 1.0)
    chunk_B = 4.0 * w.chunk
    r0 = 1.0
    if w.dst_mode == 1:
        r0 = _solve_r0(beta, V, (1.0 - w.lam) * E_gen, float(w.top_in) * (0.5 if w.symmetric else 1.0))
    p = _Params(w.seed, V, w.alpha, 1.0, w.d_max, w.dst_mode, w.lam, chunk_B, beta, r0,
                _coprime_multiplier(V), (w.seed * 7919 + 13) % V)
    p.kappa = lib.tg_calibrate_kappa(ctypes.byref(p), E_gen)
    gen_ptr = np.empty(V + 1, dtype=np.int64)
    lib.tg_out_degrees(ctypes.byref(p), gen_ptr.ctypes.data)
    Eg = int(gen_ptr[V])
    if w.symmetric:
        row_ptr = np.empty(V + 1, dtype=np.int64)
        col = np.empty(2 * Eg, dtype=np.int32)
        rc = lib.tg_fill_symmetric(ctypes.byref(p), gen_ptr.ctypes.data, row_ptr.ctypes.data, col.ctypes.data)
        if rc != 0:
            raise MemoryError("tg_fill_symmetric")
    else:
        row_ptr = gen_ptr
        col = np.empty(Eg, dtype=np.int32)
        lib.tg_fill_directed(ctypes.byref(p), row_ptr.ctypes.data, col.ctypes.data)
    E = int(row_ptr[V])
    din = np.empty(V, dtype=np.int32)
    lib.tg_in_degrees(V, E, col.ctypes.data, din.ctypes.data)
    return Graph(V, E, row_ptr, col, din, dict(kappa=p.kappa, r0=r0, beta=beta, perm_a=p.perm_a, perm_b=p.perm_b))


def features(seed: int, layer_tag: int, v_begin: int, v_end: int, F: int, out: Optional[np.ndarray] = None,
             ld: Optional[int] = None) -> np.ndarray:
    """fp32 N(0,1) feature rows [v_begin, v_end) x F, keyed (seed, layer_tag, v, column)."""
    n = v_end - v_begin
    ld = ld or F
    if out is None:
        out = np.zeros((n, ld), dtype=np.float32) if ld != F else np.empty((n, F), dtype=np.float32)
    assert out.dtype == np.float32 and out.flags.c_contiguous and out.size >= n * ld
    _lib().tg_features(seed, layer_tag, v_begin, v_end, F, ld, out.ctypes.data)
    return out


def features_rows(seed: int, layer_tag: int, ids: np.ndarray, F: int) -> np.ndarray:
    """Feature rows of the listed vertices, [len(ids), F] fp32 (same values as features())."""
    ids = np.ascontiguousarray(ids, dtype=np.int64)
    out = np.empty((ids.size, F), dtype=np.float32)
    _lib().tg_features_rows(seed, layer_tag, ids.ctypes.data, ids.size, F, F, out.ctypes.data)
    return out


def weights(seed: int, layer: int, which: int, rows: int, cols: int) -> np.ndarray:
    """Xavier-uniform fp32 [rows x cols]; which = 0 neighbour weight, 1 self weight."""
    out = np.empty((rows, cols), dtype=np.float32)
    _lib().tg_weights(seed, layer, which, rows, cols, out.ctypes.data)
    return out


@dataclass
class Model:
    mode: int
    dims: Tuple[int, ...]
    W_neigh: list
    W_self: list
    bias: list
    act: Tuple[int, ...]
    att_src: Optional[list] = None   # GAT only: per layer, dims[l+1] floats
    att_dst: Optional[list] = None


def make_model(w: Workload, bias_scale: float = 0.0) -> Model:
    """Weights of workload w: dims[l] x dims[l+1] row-major, Xavier-uniform; bias zero unless bias_scale > 0."""
    Wn, Ws, b = [], [], []
    for l in range(w.L):
        Wn.append(weights(w.seed, l, 0, w.dims[l], w.dims[l + 1]))
        Ws.append(weights(w.seed, l, 1, w.dims[l], w.dims[l + 1]) if w.mode == SAGE_MEAN else Wn[-1])
        if bias_scale > 0:
            b.append((weights(w.seed, l, 2, 1, w.dims[l + 1])[0] * bias_scale).astype(np.float32))
        else:
            b.append(np.zeros(w.dims[l + 1], dtype=np.float32))
    att_s = att_d = None
    if w.mode == GAT:      # attention vectors drawn like weight columns (which = 3 and 4)
        att_s = [weights(w.seed, l, 3, w.dims[l + 1], 1)[:, 0].copy() for l in range(w.L)]
        att_d = [weights(w.seed, l, 4, w.dims[l + 1], 1)[:, 0].copy() for l in range(w.L)]
    return Model(w.mode, w.dims, Wn, Ws, b, w.act, att_s, att_d)
