"""taurus_reorder (Alg. 1, Sect. 3.8) against the oracle."""
import numpy as np
import pytest

import oracle
import taurus_gen as tg

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,V,scramble", [("large", 60_000, True), ("mid", 30_011, False), ("tiny", 10_000, True)])
def test_reorder_matches_the_oracle(name, V, scramble):
    import paper_2607_17374_b200 as tb
    w = tg.WORKLOADS[name] if V == tg.WORKLOADS[name].V else tg.scaled(tg.WORKLOADS[name], V, chunk=1024)
    g = tg.make_graph(w)
    init = np.random.default_rng(0).permutation(g.V).astype(np.int32) if scramble else None
    rank, pos, J, span = tb.reorder(g.V, g.E, g.row_ptr, g.col_idx, init, 5)
    o_rank, hist, o_pos = oracle.reorder(g.V, g.row_ptr, g.col_idx, init, 5)
    # positions: same arithmetic up to the summation order
    np.testing.assert_allclose(pos, o_pos, rtol=1e-11, atol=1e-9)
    # the order is a permutation, and sorts the oracle's positions (where positions nearly tie, either order is valid)
    assert np.array_equal(np.sort(rank), np.arange(g.V))
    by_rank = np.empty(g.V, np.int64); by_rank[rank] = np.arange(g.V)
    gaps = np.diff(o_pos[by_rank])
    assert gaps.min() >= -1e-9 * max(1.0, np.abs(o_pos).max())
    agree = float((rank == o_rank).mean())
    print("%s: ranks identical for %.4f of the vertices; span %d -> %d; J %.4g -> %.4g" % (w.name, agree, span[0], span[-1], J[0], J[-1]))
    assert agree > 0.999
    for it in range(6):
        assert abs(span[it] - hist[it][1]) <= 2e-4 * hist[it][1]      # equal unless near-ties were ordered differently
        assert abs(J[it] - hist[it][0]) <= 1e-6 * hist[it][0]
    if agree == 1.0:
        assert [int(x) for x in span] == [h[1] for h in hist]
    if scramble:
        assert span[-1] < span[0]


def test_reorder_rejects_bad_input():
    import paper_2607_17374_b200 as tb
    w = tg.WORKLOADS["tiny"]
    g = tg.make_graph(w)
    bad = g.col_idx.copy(); bad[5] = g.V + 3
    with pytest.raises(tb.TaurusError) as ei:
        tb.reorder(g.V, g.E, g.row_ptr, bad, None, 1)
    assert ei.value.code == tb.ERROR_CODES["INVALID_ARG"]
