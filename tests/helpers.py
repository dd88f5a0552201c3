"""Small graph builders shared by the tests (no method arithmetic)."""
import numpy as np


def csr_from_edges(V, edges):
    """CSR (row_ptr int64, col int32) from a list of (u, v); per-source order follows the list order."""
    edges = list(edges)
    deg = np.zeros(V, np.int64)
    for u, _ in edges:
        deg[u] += 1
    row_ptr = np.zeros(V + 1, np.int64)
    np.cumsum(deg, out=row_ptr[1:])
    cur = row_ptr[:-1].copy()
    col = np.zeros(len(edges), np.int32)
    for u, v in edges:
        col[cur[u]] = v
        cur[u] += 1
    return row_ptr, col


def random_multigraph(V, E, seed, self_loops=True):
    rng = np.random.default_rng(seed)
    u = rng.integers(0, V, E)
    v = rng.integers(0, V, E)
    # force some duplicates and self-loops
    if E >= 8:
        u[1], v[1] = u[0], v[0]
        u[3], v[3] = u[2], v[2]
        if self_loops:
            v[5] = u[5]
    return csr_from_edges(V, zip(u.tolist(), v.tolist()))


def dense_adjacency(V, row_ptr, col):
    """A[v, u] = number of edges u -> v."""
    A = np.zeros((V, V), np.float64)
    for u in range(V):
        for e in range(row_ptr[u], row_ptr[u + 1]):
            A[col[e], u] += 1.0
    return A
