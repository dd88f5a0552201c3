"""GPU parity: libtaurus (through the C ABI) against the fp64 pull-based oracle on the same seeded inputs."""
import numpy as np
import pytest

import taurus_gen as tg
from gpu_harness import check_accounting, row_error, run_library, run_oracle

pytestmark = pytest.mark.gpu

FP32_TOL = 1e-4   # max over rows of ||g - r||_inf / (||r||_inf + 1e-6), fp32 path
BF16_TOL = 2e-2


def _compare_layers(lib, orc, tol):
    for l, (got, ref) in enumerate(zip(lib["outs"], orc["outs"])):
        row, elem_max, elem = row_error(got, ref)
        over = int((elem > tol).sum())
        print("layer %d: row-wise %.3e  element-wise max %.3e  elements over %.0e: %d of %d" %
              (l, row, elem_max, tol, over, elem.size))
        assert row <= tol, (l, row)


def test_tiny_config_two_layers_exact():
    w = tg.WORKLOADS["tiny"]
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.5)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0)
    orc = run_oracle(w, g, model, x0)
    _compare_layers(lib, orc, FP32_TOL)
    for l in range(w.L):
        check_accounting(lib["stats"][l], lib["chunk_log"][l], lib["reload_count"][l], orc["sims"][l], lib["completed"][l])
