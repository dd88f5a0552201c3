"""Pins for the neighbour sampler (Sect. 3.9, sampling paragraph): set properties that any
correct without-replacement draw must have, uniformity, and the frozen hash values."""
import os

import numpy as np
import pytest

import oracle
from helpers import random_multigraph

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "sample_hash.txt")


def test_positions_are_distinct_in_range_and_of_the_right_count():
    for din in (1, 2, 5, 16, 17, 100, 1000):
        for fanout in (1, 5, 15, 16):
            pos = oracle.sample_positions(7, 2, 123, din, fanout)
            assert pos.size == min(din, fanout)
            assert np.unique(pos).size == pos.size
            assert pos.min() >= 0 and pos.max() < din


def test_fanout_at_least_degree_keeps_every_in_edge():
    V, E = 100, 800
    row_ptr, col = random_multigraph(V, E, 0)
    inl = oracle.build_in_lists(V, row_ptr, col)
    big = int(np.diff(inl.ptr).max())
    ms = oracle.message_sets(inl, big, 3, 0)
    assert (ms.prop == 1).all()
    assert (ms.ptr == inl.ptr).all() and (ms.src == inl.src).all() and (ms.eid == inl.eid).all()


def test_repeatable_and_layers_and_seeds_differ():
    a = oracle.sample_positions(1, 0, 55, 500, 10)
    assert (a == oracle.sample_positions(1, 0, 55, 500, 10)).all()
    assert not (a == oracle.sample_positions(1, 1, 55, 500, 10)).all()
    assert not (a == oracle.sample_positions(2, 0, 55, 500, 10)).all()
    assert not (a == oracle.sample_positions(1, 0, 56, 500, 10)).all()


def test_sampled_sources_are_a_sub_multiset_of_the_in_list():
    V, E, fanout = 50, 2000, 7
    row_ptr, col = random_multigraph(V, E, 1)
    inl = oracle.build_in_lists(V, row_ptr, col)
    ms = oracle.message_sets(inl, fanout, 9, 1)
    assert int(ms.prop.sum()) == int(np.minimum(np.diff(inl.ptr), fanout).sum())
    for v in range(V):
        full = set(inl.eid[inl.ptr[v]:inl.ptr[v + 1]].tolist())
        got = ms.eid[ms.ptr[v]:ms.ptr[v + 1]].tolist()
        assert len(set(got)) == len(got) == min(len(full), fanout)
        assert set(got) <= full
        assert (col[got] == v).all()


def test_position_frequencies_are_uniform():
    """Chi-square on a degree-32 vertex, fanout 8, over 4000 seeds: every position is kept with probability 1/4."""
    din, fanout, trials = 32, 8, 4000
    counts = np.zeros(din)
    for seed in range(trials):
        counts[oracle.sample_positions(seed, 0, 17, din, fanout)] += 1
    expect = trials * fanout / din
    chi2 = ((counts - expect) ** 2 / expect).sum() / (1 - fanout / din)   # hypergeometric variance correction
    assert chi2 < 61.1   # 99.9 % quantile of chi-square with 31 degrees of freedom


def test_first_draw_is_uniform_over_a_large_degree():
    """The first kept position is floor(h * din / 2^64): its mean over seeds sits at din / 2."""
    din = 1_000_003
    first = np.array([oracle.sample_positions(s, 3, 99, din, 1)[0] for s in range(3000)], dtype=np.float64)
    assert abs(first.mean() / din - 0.5) < 4 * (1 / 12 ** 0.5) / 3000 ** 0.5


def test_frozen_hash_values():
    """The (seed, layer, dst, k) hash is part of the definition of the sampled sets; its values are frozen
    in tests/golden/sample_hash.txt (written by tests/golden/make_sample_hash.py from the oracle)."""
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) >= 16
    for seed, layer, dst, k, h in rows:
        assert oracle._lib().to_sample_hash(int(seed), int(layer), int(dst), int(k)) == int(h, 16)


def test_sample_digest_against_python_integers_and_its_invariances():
    """The digest is the plain definition (checked with Python's unbounded integers), does not depend on the order
    of the entries, and changes when one kept edge is exchanged for another."""
    rng = np.random.default_rng(12)
    V, E = 60, 700
    src = np.sort(rng.integers(0, V, E))
    col = rng.integers(0, V, E).astype(np.int32)
    row_ptr = np.zeros(V + 1, np.int64)
    np.cumsum(np.bincount(src, minlength=V), out=row_ptr[1:])
    inl = oracle.build_in_lists(V, row_ptr, col)
    for fanout in (0, 4):
        ms = oracle.message_sets(inl, fanout, 5, 1)
        d = oracle.sample_digest(ms)

        def mix(u, e):
            m = (1 << 64) - 1
            x = (((u << 32) | e) + 0x9E3779B97F4A7C15) & m
            x ^= x >> 30; x = (x * 0xBF58476D1CE4E5B9) & m
            x ^= x >> 27; x = (x * 0x94D049BB133111EB) & m
            x ^= x >> 31
            return x
        for v in range(V):
            hs = [mix(int(ms.src[k]), int(ms.eid[k])) for k in range(ms.ptr[v], ms.ptr[v + 1])]
            s, x = 0, 0
            for h in hs:
                s = (s + h) & ((1 << 64) - 1)
                x ^= h
            assert (int(d[v, 0]), int(d[v, 1])) == (s, x)
        # order of the entries inside a list does not matter
        perm = np.concatenate([ms.ptr[v] + rng.permutation(ms.ptr[v + 1] - ms.ptr[v]) for v in range(V)]).astype(np.int64)
        shuffled = oracle.MessageSets(ms.ptr, ms.src[perm], ms.eid[perm], ms.prop, ms.m)
        assert np.array_equal(oracle.sample_digest(shuffled), d)
    exact, sampled = oracle.message_sets(inl, 0, 5, 1), oracle.message_sets(inl, 4, 5, 1)
    de, ds = oracle.sample_digest(exact), oracle.sample_digest(sampled)
    big = np.diff(inl.ptr) > 4
    assert big.any() and (de[big] != ds[big]).any(axis=1).all()       # a thinned list has another digest
    assert np.array_equal(de[~big], ds[~big])                          # lists that were kept whole have the same
    other = oracle.sample_digest(oracle.message_sets(inl, 4, 6, 1))   # another seed keeps other edges somewhere
    assert not np.array_equal(other, ds)
