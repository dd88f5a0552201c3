"""CPU oracle for the output side of a layer: sorted runs and merge-on-read.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.

Follows the embedding writer (Sect. 3.7) and the graph reader (Sect. 3.3) step by step, one row at a time:

* writer: the vertex-id space is cut into fixed ranges; a finished row goes to the buffer of its range in
  arrival order; a buffer that reaches its capacity is sorted by vertex id and leaves as one sorted run; runs
  are never merged; at the end of the layer every non-empty buffer leaves as a (short) run;
* reader: for a chunk of ids [s, e) every run that overlaps it contributes the rows between two binary
  searches (first id >= s, first id >= e), and the contributions are merged by vertex id into the chunk
  matrix in vertex order.

Plain Python and numpy; no blocking, no device, nothing shared with the CUDA path.

Pins (tests/test_oracle_runs.py): a hand-worked example (tests/golden/runs_example.txt); the merged chunks of
a whole layer equal one global sort by id (the external merge sort that merge-on-read replaces), for any
arrival order, capacity and partition count; every run is sorted, stays inside its range and holds at most
the capacity; the number of runs is sum over ranges of ceil(rows / capacity); a chunk that a run only touches
at its ends gets exactly the rows the two searches delimit.  Nothing here is parity unpinned.
"""
from __future__ import annotations

import heapq
from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np


@dataclass
class Run:
    """One sorted run: ids I_f (ascending), rows X_f, inside the id range of `partition`."""
    partition: int
    ids: np.ndarray
    rows: np.ndarray

    @property
    def n(self) -> int:
        return int(self.ids.shape[0])

    @property
    def id_range(self) -> Tuple[int, int]:
        return int(self.ids[0]), int(self.ids[-1])


@dataclass
class RunWriter:
    """Range-partitioning writer of Sect. 3.7 (partition buffers of `partition_rows` rows)."""
    V: int
    partitions: int
    partition_rows: int
    width: int
    runs: List[Run] = field(default_factory=list)

    def __post_init__(self):
        if self.V < 1 or self.partitions < 1 or self.partition_rows < 1:
            raise ValueError("bad run writer configuration")
        self.range_ids = -(-self.V // self.partitions)          # ids per range, the last range may be short
        self._buf: Dict[int, List[Tuple[int, np.ndarray]]] = {p: [] for p in range(self.partitions)}

    def partition_of(self, vid: int) -> int:
        return vid // self.range_ids

    def _emit(self, p: int) -> None:
        held = self._buf[p]
        if not held:
            return
        held.sort(key=lambda t: t[0])                            # sort the buffered rows by vertex id
        ids = np.array([t[0] for t in held], dtype=np.int64)
        rows = np.stack([t[1] for t in held]).astype(np.float32)
        self.runs.append(Run(p, ids, rows))
        self._buf[p] = []

    def append(self, ids, rows) -> None:
        """Rows arrive in graduation order, not vertex order."""
        rows = np.asarray(rows, dtype=np.float32).reshape(len(ids), self.width)
        for i, vid in enumerate(ids):
            vid = int(vid)
            if not 0 <= vid < self.V:
                raise ValueError("vertex id out of range")
            p = self.partition_of(vid)
            self._buf[p].append((vid, rows[i].copy()))
            if len(self._buf[p]) == self.partition_rows:        # buffer full: sort and flush as a run
                self._emit(p)

    def flush(self) -> None:
        for p in range(self.partitions):
            self._emit(p)

    def runs_of(self, p: int) -> List[Run]:
        """Runs of one range in the order they were written."""
        return [r for r in self.runs if r.partition == p]


def search_bounds(run_ids: np.ndarray, s: int, e: int) -> Tuple[int, int]:
    """l = min{i : I[i] >= s}, r = min{i : I[i] >= e} (both n when no such i), by bisection."""
    def first_at_least(x: int) -> int:
        lo, hi = 0, int(run_ids.shape[0])
        while lo < hi:
            mid = (lo + hi) // 2
            if int(run_ids[mid]) >= x:
                hi = mid
            else:
                lo = mid + 1
        return lo
    return first_at_least(s), first_at_least(e)


def read_chunk(runs: List[Run], s: int, e: int, width: int):
    """Merge-on-read: the chunk matrix for ids [s, e) in vertex order, plus the ids found.

    Each overlapping run yields its slice [l, r); the slices are merged by vertex id with a k-way merge.
    Returns (ids, rows); ids has e - s entries exactly when every vertex of the chunk was written once.
    """
    slices = []
    for f, run in enumerate(runs):
        if run.n == 0:
            continue
        first, last = run.id_range
        if last < s or first >= e:
            continue
        l, r = search_bounds(run.ids, s, e)
        if r > l:
            slices.append([(int(run.ids[i]), f, i) for i in range(l, r)])
    merged = list(heapq.merge(*slices))
    ids = np.array([m[0] for m in merged], dtype=np.int64)
    rows = np.zeros((len(merged), width), dtype=np.float32)
    for k, (_, f, i) in enumerate(merged):
        rows[k] = runs[f].rows[i]
    return ids, rows


def directory(writer: RunWriter):
    """Per range, the list of (n, first id, last id) of its runs in writing order."""
    return {p: [(r.n,) + r.id_range for r in writer.runs_of(p)] for p in range(writer.partitions)}
