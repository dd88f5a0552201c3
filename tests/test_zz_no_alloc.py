"""The allocation-free entry point against the regular one.

taurus_completion_counts_noalloc serves callers that may not allocate device memory while they run (the GPU's
memory already belongs to a framework allocator, or an allocation would stall a latency-bound loop).  It must
return exactly what taurus_layer_begin computes for taurus_completion_bound.  The scratch array is shared by all
calls and keeps old contents, so the check is made on two calls in a row over different graphs, the second one
smaller, which would expose stale entries."""
import numpy as np
import pytest

import taurus_gen as tg

pytestmark = pytest.mark.gpu


def _counts_from_context(w, g, layer):
    """Per-64-source completion counts through the existing entry points (layer_begin + completion_bound)."""
    import paper_2607_17374_b200 as tb
    model = tg.make_model(w)
    ctx = tb.Context(g.V, g.E, g.row_ptr, g.col_idx, g.in_degree, w.mode, w.dims, model.W_neigh, model.W_self, model.bias,
                     model.act, w.chunk, w.pool_slots, w.hub_count, w.fanout, w.seed, 0, g.V, 0, 0)
    ctx.layer_begin(layer)
    nb = (g.V + 63) // 64
    counts = np.array([ctx.completion_bound(64 * b, min(64 * b + 64, g.V)) for b in range(nb)], dtype=np.int64)
    mask = ctx.get_edge_mask() if w.fanout[layer] > 0 else None
    ctx.destroy()
    return counts, mask


def _counts_noalloc(g, mask, check_free=False):
    import torch
    import paper_2607_17374_b200 as tb
    dev = torch.device("cuda:0")
    row_ptr = torch.from_numpy(g.row_ptr).to(dev)
    col = torch.from_numpy(g.col_idx).to(dev)
    d_mask = torch.from_numpy(mask.view(np.int32)).to(dev) if mask is not None else None
    out = torch.full(((g.V + 63) // 64,), -7, dtype=torch.int32, device=dev)   # the call must clear its output
    bad = torch.full((1,), -7, dtype=torch.int32, device=dev)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    rc = tb.completion_counts_noalloc(g.V, g.E, row_ptr, col, d_mask, out, bad, torch.cuda.current_stream())
    assert rc == 0
    torch.cuda.synchronize()
    if check_free:   # once the module is resident, a call leaves the device's free memory untouched
        assert torch.cuda.mem_get_info()[0] == free_before
    assert int(bad.item()) == 0
    return out.cpu().numpy().astype(np.int64)


def test_noalloc_matches_layer_begin_on_two_calls_in_a_row():
    from dataclasses import replace
    big = replace(tg.scaled(tg.WORKLOADS["sampled"], 40_000, chunk=2048), dims=(16, 8, 8, 8), pool_slots=40_000, hub_count=0)
    small = replace(tg.WORKLOADS["tiny"], dims=(16, 8, 8))
    g_big, g_small = tg.make_graph(big), tg.make_graph(small)
    want_big, mask_big = _counts_from_context(big, g_big, 1)        # a sampled layer: the edge mask matters
    want_small, mask_small = _counts_from_context(small, g_small, 0)   # exact layer: no mask
    assert mask_big is not None and mask_small is None
    got_big = _counts_noalloc(g_big, mask_big)
    got_small = _counts_noalloc(g_small, mask_small, check_free=True)   # second call, fewer vertices, same scratch
    assert (got_big == want_big).all()
    assert (got_small == want_small).all()
    assert got_big.sum() == g_big.V and got_small.sum() == g_small.V
    # and against the oracle's closed form of the completion rank, max(v, largest propagated in-neighbour), per 64 ranks
    import oracle
    for g, w, layer, got in [(g_big, big, 1, got_big), (g_small, small, 0, got_small)]:
        ms = oracle.message_sets(oracle.build_in_lists(g.V, g.row_ptr, g.col_idx), w.fanout[layer], w.seed, layer)
        want = np.bincount(oracle.complete_chunk_closed_form(ms, 64), minlength=(g.V + 63) // 64)
        assert (got == want).all()
    # and once more in the other order
    assert (_counts_noalloc(g_big, mask_big) == want_big).all()


def test_noalloc_flags_malformed_row_offsets_without_reading_past_the_edges():
    """Row offsets that leave [0, E] or run backwards are reported and cut to the valid part; a graph without edges and
    a null destination array is fine."""
    import torch
    import paper_2607_17374_b200 as tb
    dev = torch.device("cuda:0")
    g = tg.make_graph(tg.WORKLOADS["tiny"])

    def call(row_ptr, E, col):
        out = torch.zeros(((g.V + 63) // 64,), dtype=torch.int32, device=dev)
        bad = torch.zeros((1,), dtype=torch.int32, device=dev)
        assert tb.completion_counts_noalloc(g.V, E, torch.from_numpy(row_ptr).to(dev), col, None, out, bad) == 0
        torch.cuda.synchronize()
        return out.cpu().numpy().astype(np.int64), int(bad.item())

    col = torch.from_numpy(g.col_idx).to(dev)
    counts, bad = call(g.row_ptr, g.E, col)
    assert bad == 0 and counts.sum() == g.V
    # the caller says E is smaller than the offsets claim: rows are cut at E (the array still holds g.E entries)
    counts, bad = call(g.row_ptr, g.E - 1000, col)
    assert bad == 1 and counts.sum() == g.V
    backwards = g.row_ptr.copy()
    backwards[100] = backwards[101] + 5
    assert call(backwards, g.E, col)[1] == 1
    negative = g.row_ptr.copy()
    negative[0] = -3
    assert call(negative, g.E, col)[1] == 1
    # no edges at all: every vertex completes with its own chunk
    counts, bad = call(np.zeros(g.V + 1, np.int64), 0, None)
    assert bad == 0 and (counts[:-1] == 64).all() and counts.sum() == g.V


def test_noalloc_rejects_sizes_beyond_the_static_scratch():
    import torch
    import paper_2607_17374_b200 as tb
    d = torch.zeros(4, dtype=torch.int64, device="cuda:0")
    rc = tb.completion_counts_noalloc(tb.NOALLOC_MAX_VERTICES + 1, 0, d, d, None, d, d)
    assert rc == tb.ERROR_CODES["UNSUPPORTED"]
