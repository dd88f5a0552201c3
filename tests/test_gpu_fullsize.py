"""Parity at the size and in the launch configuration bench.py times (workload "mid", dense-output mode),
and the other workloads' shapes at the largest sizes the oracle still finishes in well under a minute."""
import os
from dataclasses import replace

import numpy as np
import pytest

import taurus_gen as tg
from gpu_harness import check_accounting, row_error, run_library, run_oracle

pytestmark = pytest.mark.gpu


def _check(w, tol, **kw):
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.2)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0, dense_output=True, **kw)
    orc = run_oracle(w, g, model, x0)
    for l in range(w.L):
        row, elem_max, elem = row_error(lib["outs"][l], orc["outs"][l])
        print("%s layer %d: row-wise %.3e  element-wise max %.3e  elements over %.0e: %d of %d" %
              (w.name, l, row, elem_max, tol, int((elem > tol).sum()), elem.size))
        assert row <= tol
        assert orc["sims"][l].rc == 0
        check_accounting(lib["stats"][l], lib["chunk_log"][l], lib["reload_count"][l], orc["sims"][l], None)
    return lib, orc


def test_mid_workload_at_full_size():
    """V = 2.45 M, E = 124 M, 100 -> 256 -> 256 -> 47, chunk 65 536, pool = V: every output row of every layer
    against the oracle, and the integer accounting."""
    _check(tg.WORKLOADS["mid"], 1e-4)


def test_large_shape_with_eviction_and_hubs():
    """'large' at V = 1.5 M (E = 21.6 M): pool of 18 % of V, top 0.1 % pinned, heavy eviction over pinned host rows."""
    w = tg.scaled(tg.WORKLOADS["large"], 1_500_000, chunk=65_536)
    w = replace(w, pool_slots=int(w.pool_slots * 2.5))      # the scaled graph has a wider active set than the full one
    lib, orc = _check(w, 1e-4)
    assert lib["stats"][0]["evictions"] > 100_000


def test_sampled_shape():
    w = tg.scaled(tg.WORKLOADS["sampled"], 1_500_000, chunk=65_536)
    w = replace(w, pool_slots=int(w.pool_slots * 2.5))
    g = tg.make_graph(w)
    lib, orc = _check(w, 1e-4)
    ctx = lib["ctx"]
    rng = np.random.default_rng(0)
    dsts = np.concatenate([np.argsort(-g.in_degree)[:16], rng.integers(0, g.V, 2000)])
    for l in range(w.L):      # sampled edge sets, bit-exact
        ms = orc["msets"][l]
        for dst in dsts:
            eids, srcs, n = ctx.get_sampled_edges(l, int(dst))
            assert n == ms.m[dst] and (eids == ms.eid[ms.ptr[dst]:ms.ptr[dst + 1]]).all()


def test_stress_shape_gcn_bf16():
    w = tg.scaled(tg.WORKLOADS["stress"], 1_000_000, chunk=65_536)
    w = replace(w, pool_slots=int(w.pool_slots * 4))
    _check(w, 2e-2)
