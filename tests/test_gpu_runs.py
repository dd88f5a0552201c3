"""Output side on the GPU (sorted runs, merge-on-read; Sect. 3.3 and 3.7) against the oracle's writer and reader."""
import dataclasses

import numpy as np
import pytest

import taurus_gen as tg
from oracle import run_store as rs

from gpu_harness import row_error, run_oracle

pytestmark = pytest.mark.gpu


def rows_for(ids, width, salt=0.0):
    ids = np.asarray(ids, dtype=np.int64)
    return (np.sin(ids[:, None] * 0.37 + np.arange(width)[None, :] * 1.3 + salt) * 100).astype(np.float32)


def compare_with_oracle(runs, w, width):
    """Per id range, the sequence of runs must be the oracle's: same sizes, ids and rows, bit for bit."""
    d = runs.directory()
    assert d.shape[0] == len(w.runs)
    seen = {p: 0 for p in range(w.partitions)}
    want = {p: w.runs_of(p) for p in range(w.partitions)}
    for f in range(d.shape[0]):
        p, n, first, last = (int(x) for x in d[f])
        ref = want[p][seen[p]]
        seen[p] += 1
        assert (n, first, last) == (ref.n,) + ref.id_range
        ids, rows = runs.get_run(f, n)
        assert np.array_equal(ids, ref.ids)
        assert np.array_equal(rows, ref.rows)
    assert all(seen[p] == len(want[p]) for p in seen)


@pytest.mark.parametrize("kind", ["host", "device"])
@pytest.mark.parametrize("V,P,R,width,ld", [(5000, 4, 300, 20, 24), (4099, 7, 64, 64, 64), (1000, 1, 5000, 3, 3), (777, 16, 1, 8, 8)])
def test_writer_and_reader_match_the_oracle(kind, V, P, R, width, ld):
    import torch
    import paper_2607_17374_b200 as tb
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(V + P)
    order = rng.permutation(V).astype(np.int64)
    runs = tb.Runs(V, width, P, R, store_kind=tb.RUNS_HOST if kind == "host" else tb.RUNS_DEVICE)
    w = rs.RunWriter(V, P, R, width)
    # appends of mixed sizes: single rows, a burst much larger than one buffer load, empty ones
    cuts = sorted(min(V, c) for c in [0, 1, 2, 2, 40, 40 + 6 * R + 11, V // 2 + 40, V])
    for a, b in zip(cuts[:-1], cuts[1:]):
        ids = order[a:b]
        rows = np.zeros((b - a, ld), np.float32)
        rows[:, :width] = rows_for(ids, width)
        rows[:, width:] = -7.0                      # padding columns must not be stored
        w.append(ids, rows[:, :width])
        if b > a:
            runs.append(torch.from_numpy(ids).to(dev), torch.from_numpy(rows).to(dev), ld, b - a)
        else:
            runs.append(None, None, ld, 0)
    runs.flush()
    w.flush()
    info = runs.info()
    assert info == {"runs": len(w.runs), "stored_rows": V, "buffered_rows": 0}
    compare_with_oracle(runs, w, width)
    # merge-on-read, several chunk sizes including ragged tails and chunks that straddle id ranges
    dense = rows_for(np.arange(V), width)
    for chunk in (1, 37, w.range_ids, w.range_ids + 13, V):
        if V // chunk > 600:
            continue
        out_ld = width + 4
        for s in range(0, V, chunk):
            e = min(V, s + chunk)
            out = torch.full((e - s, out_ld), -1.0, device=dev)
            runs.read_chunk(s, e, out, out_ld)
            got = out.cpu().numpy()
            ref_ids, ref_rows = rs.read_chunk(w.runs, s, e, width)
            assert ref_ids.tolist() == list(range(s, e))
            assert np.array_equal(got[:, :width], ref_rows)
            assert np.array_equal(ref_rows, dense[s:e])
            assert (got[:, width:] == -1.0).all()
    runs.destroy()


def test_pinned_host_rows_and_reset():
    import torch
    import paper_2607_17374_b200 as tb
    dev = torch.device("cuda:0")
    V, width = 3000, 16
    runs = tb.Runs(V, width, 3, 256)
    for salt in (0.0, 1.0):                          # the object is reused for the next layer's output
        order = np.random.default_rng(int(salt) + 9).permutation(V).astype(np.int64)
        ids = torch.from_numpy(order).pin_memory()
        rows = torch.from_numpy(rows_for(order, width, salt)).pin_memory()
        runs.append(ids, rows, width, V)
        runs.flush()
        out = torch.empty((V, width), device=dev)
        runs.read_chunk(0, V, out, width)
        assert np.array_equal(out.cpu().numpy(), rows_for(np.arange(V), width, salt))
        runs.reset()
        assert runs.info() == {"runs": 0, "stored_rows": 0, "buffered_rows": 0}
    runs.destroy()


def test_error_paths():
    import torch
    import paper_2607_17374_b200 as tb
    E = tb.ERROR_CODES
    dev = torch.device("cuda:0")
    V, width = 1000, 8
    runs = tb.Runs(V, width, 2, 100, store_rows=600, max_append_rows=500, max_chunk_rows=400)
    ids = np.arange(V, dtype=np.int64)
    rows = rows_for(ids, width)
    d_ids, d_rows = torch.from_numpy(ids).to(dev), torch.from_numpy(rows).to(dev)
    out = torch.zeros((400, width), device=dev)

    def code(fn):
        with pytest.raises(tb.TaurusError) as ei:
            fn()
        return ei.value.code

    assert code(lambda: runs.append(d_ids, d_rows, width, 501)) == E["INVALID_ARG"]          # beyond max_append_rows
    assert code(lambda: runs.append(ids, rows, width, 10)) == E["INVALID_ARG"]               # pageable host memory
    assert code(lambda: runs.append(d_ids, d_rows, width - 1, 10)) == E["INVALID_ARG"]       # ld below the width
    bad = d_ids[:10].clone()
    bad[3] = V
    assert code(lambda: runs.append(bad, d_rows, width, 10)) == E["INVALID_ARG"]             # id outside [0, V)
    assert runs.info() == {"runs": 0, "stored_rows": 0, "buffered_rows": 0}                  # ... and nothing was appended
    runs.append(d_ids, d_rows, width, 250)                                                    # ids 0..249: two runs, 50 buffered
    assert runs.info() == {"runs": 2, "stored_rows": 200, "buffered_rows": 50}
    assert code(lambda: runs.read_chunk(0, 250, out, width)) == E["RUNS_INCOMPLETE"]         # 50 rows are not flushed yet
    runs.read_chunk(0, 200, out, width)
    assert np.array_equal(out[:200].cpu().numpy(), rows[:200])
    runs.flush()
    runs.read_chunk(0, 250, out, width)
    assert code(lambda: runs.read_chunk(0, 251, out, width)) == E["RUNS_INCOMPLETE"]         # vertex 250 was never written
    assert code(lambda: runs.read_chunk(0, 401, out, width)) == E["INVALID_ARG"]             # beyond max_chunk_rows
    assert code(lambda: runs.read_chunk(0, 10, out.cpu(), width)) == E["INVALID_ARG"]        # host destination
    before = runs.info()
    assert code(lambda: runs.append(d_ids[500:], d_rows[500:], width, 400)) == E["RUN_STORE_FULL"]   # 250 + 400 > 600
    assert runs.info() == before
    runs.destroy()


def check_run_structure(runs, V, P, R):
    """What holds whatever order the vertices of a chunk completed in: every run sorted and inside its id range,
    all runs of a range full except its last, every vertex in exactly one run."""
    d = runs.directory()
    range_ids = -(-V // P)
    seen = np.zeros(V, np.int32)
    last_of = {}
    for f in range(d.shape[0]):
        p, n, first, last = (int(x) for x in d[f])
        ids, _ = runs.get_run(f, n)
        assert np.all(np.diff(ids) > 0) and ids[0] == first and ids[-1] == last
        assert first >= p * range_ids and last < min(V, (p + 1) * range_ids)
        assert 1 <= n <= R
        if p in last_of:
            assert last_of[p] == R            # an earlier run of this range was short
        last_of[p] = n
        seen[ids] += 1
    assert (seen == 1).all()
    per_range = np.bincount(np.arange(V) // range_ids, minlength=P)
    assert d.shape[0] == sum(-(-int(c) // R) for c in per_range)


@pytest.mark.parametrize("kind", ["host", "device"])
def test_layers_chained_through_runs(kind):
    """Run-output mode: each layer's rows leave as sorted runs and the next layer streams them back by
    merge-on-read (no dense V x H array in between); outputs and accounting equal the oracle's."""
    import paper_2607_17374_b200 as tb
    from gpu_harness import check_accounting, run_library
    k = tb.RUNS_HOST if kind == "host" else tb.RUNS_DEVICE
    w = tg.scaled(tg.WORKLOADS["large"], 60_000, chunk=1024)
    w = dataclasses.replace(w, dims=(128, 256, 64, 20), fanout=(0, 0, 0), pool_slots=16_000, hub_count=60)
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.3)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    P, R = 7, 2500
    lib = run_library(w, g, model, x0, run_output=(P, R, k))
    orc = run_oracle(w, g, model, x0)
    for l in range(w.L):
        row, elem_max, _ = row_error(lib["outs"][l], orc["outs"][l])
        print("layer %d via runs: row-wise %.3e element-wise max %.3e" % (l, row, elem_max))
        assert row <= 1e-4
        assert orc["sims"][l].rc == 0
        check_accounting(lib["stats"][l], lib["chunk_log"][l], lib["reload_count"][l], orc["sims"][l])
    check_run_structure(lib["runs"][-1], g.V, P, R)
    assert lib["stats"][0]["evictions"] > 1000


def test_run_output_mid_shape_ragged():
    import paper_2607_17374_b200 as tb
    from gpu_harness import run_library
    w = tg.scaled(tg.WORKLOADS["mid"], 30_011, chunk=4096)      # widths 100 -> 256 -> 256 -> 47, ragged last chunk
    g = tg.make_graph(w)
    model = tg.make_model(w, bias_scale=0.3)
    x0 = tg.features(w.seed, 0, 0, g.V, w.dims[0])
    lib = run_library(w, g, model, x0, run_output=(3, 1000, tb.RUNS_HOST), host_features=True)
    orc = run_oracle(w, g, model, x0)
    for l in range(w.L):
        row, _, _ = row_error(lib["outs"][l], orc["outs"][l])
        assert row <= 1e-4, (l, row)
    check_run_structure(lib["runs"][-1], g.V, 3, 1000)


def test_run_output_argument_checks():
    import torch
    import paper_2607_17374_b200 as tb
    E = tb.ERROR_CODES
    w = dataclasses.replace(tg.WORKLOADS["tiny"], dims=(64, 32, 8))
    g = tg.make_graph(w)
    model = tg.make_model(w)
    ctx = tb.Context(g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                     model.act, w.chunk, w.pool_slots, 0, w.fanout, w.seed, 0, 2 * g.V)
    x = torch.from_numpy(tg.features(w.seed, 0, 0, g.V, 64)).cuda()

    def code(fn):
        with pytest.raises(tb.TaurusError) as ei:
            fn()
        return ei.value.code

    good = tb.Runs(g.V, 32, 4, 500, max_chunk_rows=w.chunk)
    assert code(lambda: ctx.layer_set_run_output(good)) == E["ORDER"]                      # no layer begun
    ctx.layer_begin(0)
    assert code(lambda: ctx.layer_set_run_output(tb.Runs(g.V, 31, 4, 500))) == E["INVALID_ARG"]          # wrong width
    assert code(lambda: ctx.layer_set_run_output(tb.Runs(g.V, 32, 4, 500, max_append_rows=10))) == E["INVALID_ARG"]
    ctx.layer_set_run_output(good)
    for s in range(0, g.V, w.chunk):
        ctx.push_chunk(s, min(g.V, s + w.chunk), x[s:s + w.chunk])
    ctx.layer_end()
    ctx.layer_begin(1)
    out = tb.Runs(g.V, 8, 2, 300, max_chunk_rows=w.chunk)
    ctx.layer_set_run_output(out)
    assert code(lambda: ctx.push_chunk_from_runs(0, w.chunk, out)) == E["INVALID_ARG"]    # reading what is being written
    empty = tb.Runs(g.V, 32, 4, 500, max_chunk_rows=w.chunk)
    assert code(lambda: ctx.push_chunk_from_runs(0, w.chunk, empty)) == E["RUNS_INCOMPLETE"]
    for s in range(0, g.V, w.chunk):                                                       # the failed calls changed nothing
        ctx.push_chunk_from_runs(s, min(g.V, s + w.chunk), good)
    st = ctx.layer_end()
    assert st["completed"] == g.V and out.info()["stored_rows"] == g.V
    ctx.destroy()


@pytest.mark.parametrize("seed", range(24))
def test_random_writer_reader_configurations(seed):
    """Random V / ranges / buffer sizes / widths / append sizes (more ranges than vertices, one-row buffers, wide
    rows, partial layers) against the oracle's writer and reader."""
    import torch
    import paper_2607_17374_b200 as tb
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(500 + seed)
    V = int(rng.choice([1, 2, 17, 300, 1000, 4097, 20000]))
    P = int(rng.choice([1, 2, 3, 16, 100, 1024]))
    R = int(rng.choice([1, 2, 7, 64, 1000, 50000]))
    if V // max(1, min(P, V)) > 400 * R:          # keep the number of runs (each a few launches) bounded
        R = max(R, V // (400 * P) + 1)
    width = int(rng.choice([1, 3, 4, 12, 64, 257, 1024])) if V <= 4097 else int(rng.choice([1, 4, 12, 64]))
    ld = width + int(rng.choice([0, 0, 1, 4]))
    kind = tb.RUNS_HOST if rng.integers(0, 2) else tb.RUNS_DEVICE
    present = rng.permutation(V)[:max(1, int(V * rng.choice([1.0, 1.0, 0.6])))].astype(np.int64)   # sometimes a partial layer
    runs = tb.Runs(V, width, P, R, store_kind=kind)
    w = rs.RunWriter(V, P, R, width)
    at = 0
    while at < present.size:
        n = int(min(present.size - at, rng.choice([1, 3, 50, 1000, V])))
        ids = present[at:at + n]
        rows = np.full((n, ld), -3.0, np.float32)
        rows[:, :width] = rows_for(ids, width)
        w.append(ids, rows[:, :width])
        runs.append(torch.from_numpy(ids).to(dev), torch.from_numpy(rows).to(dev), ld, n)
        at += n
    runs.flush(); w.flush()
    assert runs.info() == {"runs": len(w.runs), "stored_rows": int(present.size), "buffered_rows": 0}
    compare_with_oracle(runs, w, width)
    have = np.zeros(V, bool)
    have[present] = True
    chunk = int(rng.choice([1, 5, 64, 1000, V]))
    chunk = max(chunk, V // 200 + 1)
    for s in range(0, V, chunk):
        e = min(V, s + chunk)
        out = torch.full((e - s, width), -1.0, device=dev)
        if have[s:e].all():
            runs.read_chunk(s, e, out, width)
            ref_ids, ref_rows = rs.read_chunk(w.runs, s, e, width)
            assert ref_ids.tolist() == list(range(s, e)) and np.array_equal(out.cpu().numpy(), ref_rows)
        else:
            with pytest.raises(tb.TaurusError) as ei:
                runs.read_chunk(s, e, out, width)
            assert ei.value.code == tb.ERROR_CODES["RUNS_INCOMPLETE"]
            assert (out == -1.0).all()
    runs.destroy()
