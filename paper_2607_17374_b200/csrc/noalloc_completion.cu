// taurus_completion_counts_noalloc: the completion-count histogram of taurus_layer_begin for callers that
// must not allocate.  Its only scratch is the file-scope device array below.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "taurus.h"

#define NOALLOC_MAX_DEVICES 64

// Scratch: the completion rank of every vertex.  Lives in the library image, so every GPU that loads
// libtaurus holds these 16 MiB until the process exits.  Shared by all calls; each call rewrites
// entries [0, V) before reading them.
static __device__ __align__(256) int32_t g_completion_rank[TAURUS_NOALLOC_MAX_VERTICES];

// In host code g_completion_rank is only a handle for the runtime, not an address a kernel can use:
// the real device address is looked up once per device and kept here.
static int32_t* g_rank_addr[NOALLOC_MAX_DEVICES] = {nullptr};
static std::mutex g_rank_mutex;

static __global__ void na_rank_init_kernel(long long V, int32_t* rank) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) rank[v] = (int32_t)v;
}

// A row range that leaves [0, E] or runs backwards is reported through *bad and clamped, so that neither the
// destination array nor the edge mask is ever read outside its E entries.
static __global__ void na_rank_max_kernel(long long V, long long E, const long long* row_ptr, const int32_t* col, const uint32_t* mask,
                                          int32_t* rank, int* bad) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int lane = threadIdx.x & 31;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    long long b = row_ptr[u], e = row_ptr[u + 1];
    if (b < 0 || e > E || b > e) {
      if (lane == 0) *bad = 1;
      b = b < 0 ? 0 : b;
      e = e > E ? E : e;
    }
    for (long long k = b + lane; k < e; k += 32) {
      if (mask != nullptr && !((mask[k >> 5] >> (k & 31)) & 1u)) continue;
      int v = col[k];
      if (v < 0 || v >= V) { *bad = 1; continue; }   // never index the scratch out of range
      atomicMax(&rank[v], (int32_t)u);
    }
  }
}

static __global__ void na_rank_hist_kernel(long long V, const int32_t* rank, int32_t* counts) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) atomicAdd(&counts[rank[v] >> 6], 1);
}

extern "C" int taurus_completion_counts_noalloc(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx,
                                                const uint32_t* edge_mask, int32_t* out_counts, int32_t* out_bad_index,
                                                void* cuda_stream) {
  if (V < 1 || E < 0 || !row_ptr || (E > 0 && !col_idx) || !out_counts || !out_bad_index) return TAURUS_ERR_INVALID_ARG;
  if (V > TAURUS_NOALLOC_MAX_VERTICES) return TAURUS_ERR_UNSUPPORTED;   // the static scratch holds no more
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) { cudaGetLastError(); return TAURUS_ERR_CUDA; }
  int32_t* rank = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_rank_mutex);
    if (g_rank_addr[dev] == nullptr) {   // first call on this device: resolve the symbol with this device current
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_completion_rank) != cudaSuccess || p == nullptr) { cudaGetLastError(); return TAURUS_ERR_CUDA; }
      g_rank_addr[dev] = static_cast<int32_t*>(p);
    }
    rank = g_rank_addr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const long long blocks64 = (V + 63) / 64;
  if (cudaMemsetAsync(out_counts, 0, (size_t)blocks64 * sizeof(int32_t), st) != cudaSuccess ||
      cudaMemsetAsync(out_bad_index, 0, sizeof(int32_t), st) != cudaSuccess) { cudaGetLastError(); return TAURUS_ERR_CUDA; }
  const int grid = 148 * 8;
  na_rank_init_kernel<<<grid, 256, 0, st>>>(V, rank);
  na_rank_max_kernel<<<grid, 256, 0, st>>>(V, E, reinterpret_cast<const long long*>(row_ptr), col_idx, edge_mask, rank, out_bad_index);
  na_rank_hist_kernel<<<grid, 256, 0, st>>>(V, rank, out_counts);
  if (cudaGetLastError() != cudaSuccess) return TAURUS_ERR_CUDA;
  return TAURUS_OK;
}
