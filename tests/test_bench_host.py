"""Host-side arithmetic of bench.py that needs no GPU: the window plan of the bounded-pool workloads, the algorithmic
bytes of a scatter launch, which workloads are timed in windows, and the fallback when a box cannot hold a workload."""
import os
import sys
import types

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
import taurus_gen as tg  # noqa: E402


def test_window_plan_holds_prefill_and_every_window_in_one_pass():
    assert bench.plan_windows(1694, 20, 5, 32, 384) == (32, 384)          # the default run on 'large'
    window, prefill = bench.plan_windows(1694, 50, 5, 32, 384)             # more steps: shorter windows, same prefill
    assert window == 23 and prefill == 384 and prefill + 55 * window <= 1694 and prefill + 55 * (window + 1) > 1694
    assert bench.plan_windows(100, 3, 1, 32, 384) == (18, 25)              # a short pass: a quarter of it fills the pool
    assert bench.plan_windows(10, 8, 2, 32, 5) == (1, 0)
    assert bench.plan_windows(23, 2, 1, 4, 8) == (4, 8)                    # fits as asked: nothing changes
    with pytest.raises(SystemExit):
        bench.plan_windows(9, 8, 2, 32, 0)


def test_scatter_bytes_by_hand():
    # 10 groups, 25 edges, 4 sources, accumulator rows of 8 floats: a read-modify-write of 32 bytes and an 8-byte record
    # per group, 8 bytes per edge, per source its projected row (32), its self row (96 with the self columns) and 8 bytes
    assert bench.scatter_bytes(10, 25, 4, 8, True) == 10 * (64 + 8) + 25 * 8 + 4 * (32 + 96 + 8)
    assert bench.scatter_bytes(10, 25, 4, 8, False) == 10 * (64 + 8) + 25 * 8 + 4 * (32 + 8)


def test_which_workloads_are_timed_in_windows():
    assert not bench.windowed(tg.WORKLOADS["mid"]) and not bench.windowed(tg.WORKLOADS["tiny"])
    for name in ("large", "sampled", "stress"):
        assert bench.windowed(tg.WORKLOADS[name])


def test_fallback_when_the_box_cannot_hold_the_workload(monkeypatch):
    args = types.SimpleNamespace(vertices=0, pool_fraction=0.0)
    env = types.SimpleNamespace(world=1)
    monkeypatch.setattr(bench, "free_memory_gb", lambda e: (200.0, 180.0))
    assert bench.fallback_reason(args, env, tg.WORKLOADS["large"]) is None
    assert bench.fallback_reason(args, env, tg.WORKLOADS["mid"]) is None
    env.world = 4                                                          # four replicas share the host memory
    assert "4 replicas" in bench.fallback_reason(args, env, tg.WORKLOADS["large"])
    env.world = 1
    monkeypatch.setattr(bench, "free_memory_gb", lambda e: (200.0, 79.0))   # a smaller GPU
    assert "device memory" in bench.fallback_reason(args, env, tg.WORKLOADS["large"])
    args.vertices = 1_500_000                                              # a scaled instance always fits
    assert bench.fallback_reason(args, env, tg.WORKLOADS["large"]) is None
