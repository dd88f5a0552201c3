"""Pins of the oracle's output side (sorted runs, merge-on-read) against what Sect. 3.3 / 3.7 fix."""
import os

import numpy as np
import pytest

from oracle import run_store as rs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "runs_example.txt")


def rows_for(ids, width):
    ids = np.asarray(ids, dtype=np.int64)
    return (ids[:, None] * 16 + np.arange(width)[None, :]).astype(np.float32)


def parse_golden():
    out = {"runs": [], "bounds": []}
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "V":
            out.update(V=int(t[1]), P=int(t[3]), R=int(t[5]))
        elif t[0] == "arrival":
            out["arrival"] = [int(x) for x in t[1:]]
        elif t[0] == "run":
            out["runs"].append((int(t[1]), [int(x) for x in t[2:]]))
        elif t[0] == "chunk":
            out["chunk"] = (int(t[1]), int(t[2]))
        elif t[0] == "bounds":
            out["bounds"].append((int(t[1]), int(t[2])))
        elif t[0] == "merged":
            out["merged"] = [int(x) for x in t[1:]]
    return out


def test_hand_worked_example():
    g = parse_golden()
    w = rs.RunWriter(g["V"], g["P"], g["R"], width=2)
    # one row at a time, as the writer receives them
    for vid in g["arrival"]:
        w.append([vid], rows_for([vid], 2))
    w.flush()
    assert [(r.partition, r.ids.tolist()) for r in w.runs] == g["runs"]
    s, e = g["chunk"]
    assert [rs.search_bounds(r.ids, s, e) for r in w.runs] == g["bounds"]
    ids, rows = rs.read_chunk(w.runs, s, e, 2)
    assert ids.tolist() == g["merged"]
    assert np.array_equal(rows, rows_for(g["merged"], 2))


@pytest.mark.parametrize("V,P,R,batch", [(1000, 4, 64, 37), (1000, 7, 1, 1000), (513, 3, 500, 5), (64, 64, 2, 9), (100, 1, 1000, 13)])
def test_merge_on_read_equals_global_sort(V, P, R, batch):
    """Reading every chunk back gives the same matrix as one external sort of all (id, row) records."""
    rng = np.random.default_rng(V * 31 + P)
    order = rng.permutation(V)
    width = 3
    w = rs.RunWriter(V, P, R, width)
    for i in range(0, V, batch):
        ids = order[i:i + batch]
        w.append(ids, rows_for(ids, width))
    w.flush()
    # the definition: sort all records by id
    allrows = rows_for(order, width)
    perm = np.argsort(order, kind="stable")
    dense = allrows[perm]
    for chunk in (1, 17, 100, V):
        got = []
        for s in range(0, V, chunk):
            e = min(V, s + chunk)
            ids, rows = rs.read_chunk(w.runs, s, e, width)
            assert ids.tolist() == list(range(s, e))
            got.append(rows)
        assert np.array_equal(np.concatenate(got), dense)


def test_run_structure():
    V, P, R = 2000, 6, 50
    rng = np.random.default_rng(5)
    order = rng.permutation(V)
    w = rs.RunWriter(V, P, R, 1)
    w.append(order, rows_for(order, 1))
    w.flush()
    per_range = np.bincount(order // w.range_ids, minlength=P)
    assert len(w.runs) == sum(-(-int(n) // R) for n in per_range)
    for p in range(P):
        runs = w.runs_of(p)
        for k, r in enumerate(runs):
            assert np.all(np.diff(r.ids) > 0)
            assert r.ids[0] >= p * w.range_ids and r.ids[-1] < min(V, (p + 1) * w.range_ids)
            assert r.n == R or k == len(runs) - 1            # only the flush at the end of the layer writes a short run
        # run k of a range holds arrivals k*R .. (k+1)*R - 1 of that range, whatever the other ranges did
        arrivals = [int(v) for v in order if v // w.range_ids == p]
        for k, r in enumerate(runs):
            assert sorted(arrivals[k * R:(k + 1) * R]) == r.ids.tolist()


def test_partial_layer_reads_only_what_was_written():
    w = rs.RunWriter(20, 2, 4, 1)
    w.append([3, 11, 7], rows_for([3, 11, 7], 1))
    w.flush()
    ids, rows = rs.read_chunk(w.runs, 0, 10, 1)
    assert ids.tolist() == [3, 7] and rows[:, 0].tolist() == [48.0, 112.0]
    ids, _ = rs.read_chunk(w.runs, 12, 20, 1)
    assert ids.size == 0


def test_search_bounds_edges():
    ids = np.array([4, 6, 9, 15])
    assert rs.search_bounds(ids, 0, 4) == (0, 0)
    assert rs.search_bounds(ids, 4, 5) == (0, 1)
    assert rs.search_bounds(ids, 5, 15) == (1, 3)
    assert rs.search_bounds(ids, 15, 16) == (3, 4)
    assert rs.search_bounds(ids, 16, 99) == (4, 4)
    # against the library routine on random sorted arrays
    rng = np.random.default_rng(0)
    for _ in range(50):
        a = np.unique(rng.integers(0, 200, size=40))
        s, e = sorted(rng.integers(0, 220, size=2).tolist())
        assert rs.search_bounds(a, s, e) == (int(np.searchsorted(a, s, "left")), int(np.searchsorted(a, e, "left")))
