"""Seeded random configurations (mode, widths, chunk size, pool, hubs, fanouts, kernel choices, output mode) through
the C ABI against the oracle: outputs within the fp32 bound, accounting and completion sets bit-exact."""
import os
from dataclasses import replace

import numpy as np
import pytest

import oracle
import taurus_gen as tg
from gpu_harness import check_accounting, forward_error, layer_on_input, row_error, run_library, run_oracle

pytestmark = pytest.mark.gpu


_SCALE = int(os.environ.get("TAURUS_FUZZ_SCALE", "1"))      # multiplies the vertex counts drawn (400 .. 6 000)


def random_config(seed):
    rng = np.random.default_rng(1000 + seed)
    base = ["tiny", "mid", "large", "stress"][int(rng.integers(0, 4))]
    V = int(rng.integers(400, 6000)) * _SCALE
    chunk = int(rng.choice([64, 100, 128, 257, 512, 1000, 2048]))
    w = tg.scaled(tg.WORKLOADS[base], V, chunk=chunk)
    L = int(rng.integers(1, 4))
    widths = [1, 3, 4, 7, 16, 20, 32, 33, 47, 48, 64, 100, 128, 130, 256, 300]
    dims = tuple(int(rng.choice(widths)) for _ in range(L + 1))
    mode = int(rng.choice([tg.SAGE_MEAN, tg.GCN_SYM, tg.GIN_SUM, tg.GAT]))
    fanout = tuple(int(rng.choice([0, 0, 1, 2, 5, 9])) for _ in range(L))
    hub_count = int(rng.choice([0, 0, 1, 7, V // 50, V // 3]))
    heads = 1
    if mode == tg.GAT:     # several heads where every layer's output width splits into whole float4 per head
        ok = [hd for hd in (1, 1, 2, 4, 8) if all(d % (4 * hd) == 0 for d in dims[1:])]
        heads = int(rng.choice(ok)) if ok else 1
    w = replace(w, dims=dims, mode=mode, fanout=fanout, hub_count=hub_count, gemm_mode=tg.GEMM_FP32, gin_eps=float(rng.uniform(-0.5, 0.5)),
                leaky_slope=float(rng.choice([0.0, 0.2, 1.0])), seed=int(rng.integers(1, 1 << 30)), gat_heads=heads)
    g = tg.make_graph(w)
    # a pool between "just feasible" and "never evicts": grow it until the oracle's simulator accepts every layer
    inl = oracle.build_in_lists(g.V, g.row_ptr, g.col_idx)
    hub = oracle.hub_set(g.in_degree, hub_count)
    policy = int(rng.integers(0, 4))
    pool = max(1, int(g.V * rng.uniform(0.05, 1.1)))
    while True:
        ok = True
        for l in range(L):
            ms = oracle.message_sets(inl, fanout[l], w.seed, l)
            if oracle.simulate(g.V, g.row_ptr, g.col_idx, ms, hub, chunk, pool, policy, w.seed).rc != 0:
                ok = False
                break
        if ok:
            break
        pool = int(pool * 1.3) + 1
    w = replace(w, pool_slots=pool)
    kw = dict(flags=int(rng.choice([0, 0, 0, 2, 4, 6, 8, 10, 12])), evict_policy=policy)   # 8: always project first
    if mode != tg.GAT and L <= 2 and rng.integers(0, 8) == 0:
        kw["gemm_mode"] = tg.GEMM_BF16          # bf16 operands, fp32 accumulate
    out_mode = int(rng.integers(0, 6))
    if out_mode == 4:                          # layers chained through sorted runs
        import paper_2607_17374_b200 as tb
        kw["run_output"] = (int(rng.choice([1, 3, 16])), int(rng.choice([1, 50, 4000])) if g.V < 1500 else int(rng.choice([50, 4000])),
                            tb.RUNS_HOST if rng.integers(0, 2) else tb.RUNS_DEVICE)
    elif out_mode == 5:                        # pushes that are not cells of the chunk grid (CSR-order kernels), small graduation buffer
        cuts = sorted(set([0, g.V] + [int(x) for x in rng.integers(1, g.V, size=int(rng.integers(1, 12)))]))
        plan = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            while b - a > chunk:
                plan.append((a, a + chunk)); a += chunk
            plan.append((a, b))
        kw["chunk_plan"] = plan
        kw["drain_each_chunk"] = bool(rng.integers(0, 2))
        w = replace(w, pool_slots=g.V)         # the simulator works on the chunk grid: no eviction, outputs and sets only
    if out_mode == 1:
        kw["dense_output"] = True
    elif out_mode == 2:
        kw["dense_output"] = True
        kw["host_features"] = True
    elif out_mode == 3:
        kw["drain_each_chunk"] = False
    return w, g, kw


_FIRST = int(os.environ.get("TAURUS_FUZZ_FIRST", "0"))        # first seed of the sweep


@pytest.mark.parametrize("seed", range(_FIRST, _FIRST + int(os.environ.get("TAURUS_FUZZ_SEEDS", "32"))))   # more seeds: set TAURUS_FUZZ_SEEDS
def test_random_configuration(seed):
    w, g, kw = random_config(seed)
    print("config %d: %s V=%d E=%d mode=%d heads=%d dims=%s chunk=%d pool=%d hubs=%d fanout=%s %s" %
          (seed, w.name, g.V, g.E, w.mode, w.gat_heads, w.dims, w.chunk, w.pool_slots, w.hub_count, w.fanout, kw))
    model = tg.make_model(w, bias_scale=0.3)
    if w.mode == tg.GAT:
        model.att_src = [(a * 3).astype(np.float32) for a in model.att_src]
        model.att_dst = [(a * 3).astype(np.float32) for a in model.att_dst]
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0, **kw)
    orc = run_oracle(w, g, model, x0, kw["evict_policy"])
    for l in range(w.L):
        row, elem_max, _ = row_error(lib["outs"][l], orc["outs"][l])
        # One gate for every width and mode: the layer as the oracle evaluates it on the very rows the library consumed
        # (its own previous output, so that earlier layers' errors are not counted twice), and the error of each row
        # measured against the magnitude of what was summed for it.  tol is the stated 1e-4 (fp32) / 2e-2 (bf16 operands).
        bf16 = kw.get("gemm_mode") == tg.GEMM_BF16 and not (kw["flags"] & 2)
        tol = 2e-2 if bf16 else 1e-4
        ref, mag = layer_on_input(w, model, orc, l, x0 if l == 0 else lib["outs"][l - 1])
        fwd = forward_error(lib["outs"][l], ref, mag)
        print("layer %d: forward error %.3e of the summed magnitude; against the chained oracle: row-wise %.3e, element-wise max %.3e"
              % (l, fwd, row, elem_max))
        assert fwd <= tol, (l, fwd, row, elem_max)
        assert orc["sims"][l].rc == 0 or kw.get("chunk_plan")
        assert np.array_equal(lib["digests"][l], oracle.sample_digest(orc["msets"][l]))   # the propagated in-edge sets, all V
        completed = lib["completed"][l]
        per_chunk = completed if (completed and kw.get("drain_each_chunk", True) and not kw.get("dense_output")
                                  and not kw.get("chunk_plan")) else None
        if per_chunk is not None and any(isinstance(c, tuple) for c in per_chunk):
            per_chunk = None
        if kw.get("chunk_plan"):
            assert lib["stats"][l]["completed"] == g.V and lib["stats"][l]["total_messages"] == int(orc["msets"][l].m.sum())
        else:
            check_accounting(lib["stats"][l], lib["chunk_log"][l], lib["reload_count"][l], orc["sims"][l], per_chunk)
