"""B200-native source-centric broadcast step for layer-wise GNN inference (libtaurus).

The product is the CUDA library behind include/taurus.h; this package is its thin ctypes binding.
There is no CPU fallback: importing the binding works anywhere, but every call needs the compiled
library (python -m paper_2607_17374_b200.build) and a CUDA device.
"""
from .binding import (  # noqa: F401
    Context, Runs, RUNS_HOST, RUNS_DEVICE, TaurusError, Stats, library_path, load_library, completion_counts_noalloc, NOALLOC_MAX_VERTICES, reorder, relabel_csr, permute_rows,
    SAGE_MEAN, GCN_SYM, GIN_SUM, GAT, GEMM_FP32, GEMM_BF16, FLAG_SIMT_GEMM, FLAG_NO_GROUPING, FLAG_PROJECT_FIRST, EVICT_FEWEST_PENDING, EVICT_FIFO, EVICT_LRU, EVICT_RANDOM, CHUNK_LOG_COLUMNS, ERROR_CODES,
)
