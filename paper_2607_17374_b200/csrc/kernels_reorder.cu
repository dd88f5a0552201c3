// Topology-aware reordering (Alg. 1, Sect. 3.8): positions r, locality centres mu, new order = ArgSort(r).
// Both update rules are evaluated pull-based in fp64 with one warp per vertex (in-lists for mu, CSR rows for r),
// so no floating-point atomics take part in the positions; the order is a stable radix sort of r (ties by
// vertex id).  The dispersion J and the total span C(pi) are reported for the initial order and after every
// iteration, both measured on the ordering itself (positions = ranks).
#include <cub/cub.cuh>

#include <vector>

#include "taurus.h"

#define FULL 0xffffffffu

namespace {

__device__ __forceinline__ int lane() { return threadIdx.x & 31; }
__device__ __forceinline__ double warp_sum(double x) {
  for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(FULL, x, o);
  return x;
}

__global__ void ro_degree_kernel(long long E, const int32_t* col, long long V, int32_t* din, int* bad) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < E; e += stride) {
    int v = col[e];
    if (v < 0 || v >= V) *bad = 1; else atomicAdd(&din[v], 1);
  }
}
__global__ void ro_src_kernel(long long V, const long long* row_ptr, int32_t* src_of_edge) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps)
    for (long long k = row_ptr[u] + lane(); k < row_ptr[u + 1]; k += 32) src_of_edge[k] = (int32_t)u;
}
__global__ void ro_widen_kernel(long long V, const int32_t* din, long long* ptr) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v <= V; v += stride) ptr[v] = v < V ? din[v] : 0;
}
__global__ void ro_init_kernel(long long V, const int32_t* initial_rank, double* r) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride)
    r[v] = initial_rank ? (double)initial_rank[v] : (double)v;
}

// mu(v) = (r(v) + sum_{u -> v} r(u)) / d(v), d = in-degree + 1 (every vertex aggregates a self message);
// also w1 = mu / d and w2 = 1 / d, the two terms each out-neighbourhood sums.
__global__ void ro_mu_kernel(long long V, const long long* in_ptr, const int32_t* in_src, const double* r, double* mu,
                             double* w1, double* w2) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long v = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; v < V; v += warps) {
    const long long b = in_ptr[v], e = in_ptr[v + 1];
    double s = 0.0;
    for (long long p = b + lane(); p < e; p += 32) s += r[in_src[p]];
    s = warp_sum(s);
    if (lane() == 0) {
      const double d = (double)(e - b) + 1.0;
      const double m = (r[v] + s) / d;
      mu[v] = m;
      if (w1) { w1[v] = m / d; w2[v] = 1.0 / d; }
    }
  }
}
// r(w) = (mu(w)/d(w) + sum_{w -> v} mu(v)/d(v)) / (1/d(w) + sum_{w -> v} 1/d(v))
__global__ void ro_r_kernel(long long V, const long long* row_ptr, const int32_t* col, const double* w1, const double* w2, double* r) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < V; w += warps) {
    double num = 0.0, den = 0.0;
    for (long long k = row_ptr[w] + lane(); k < row_ptr[w + 1]; k += 32) { const int v = col[k]; num += w1[v]; den += w2[v]; }
    num = warp_sum(num); den = warp_sum(den);
    if (lane() == 0) r[w] = (w1[w] + num) / (w2[w] + den);
  }
}
__global__ void ro_iota_kernel(long long V, int32_t* ids) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) ids[v] = (int32_t)v;
}
__global__ void ro_rank_kernel(long long V, const int32_t* order, int32_t* rank, double* pos) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < V; i += stride) {
    rank[order[i]] = (int32_t)i;
    pos[order[i]] = (double)i;
  }
}
// J = sum_v 1/d(v) * sum over v's in-neighbours and v itself of (pos(u) - mu(v))^2; span = sum_v (max - min) of ranks.
__global__ void ro_measure_kernel(long long V, const long long* in_ptr, const int32_t* in_src, const double* pos, const double* mu,
                                  const int32_t* rank, double* J, unsigned long long* span) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  double jsum = 0.0;
  unsigned long long ssum = 0;
  for (long long v = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; v < V; v += warps) {
    const long long b = in_ptr[v], e = in_ptr[v + 1];
    const double m = mu[v];
    double s = 0.0;
    int lo = rank[v], hi = rank[v];
    for (long long p = b + lane(); p < e; p += 32) {
      const int u = in_src[p];
      const double dlt = pos[u] - m;
      s += dlt * dlt;
      const int ru = rank[u];
      lo = ru < lo ? ru : lo; hi = ru > hi ? ru : hi;
    }
    s = warp_sum(s);
    for (int o = 16; o; o >>= 1) {
      int l2 = __shfl_xor_sync(FULL, lo, o), h2 = __shfl_xor_sync(FULL, hi, o);
      lo = l2 < lo ? l2 : lo; hi = h2 > hi ? h2 : hi;
    }
    if (lane() == 0) {
      const double dv = pos[v] - m;
      jsum += (s + dv * dv) / ((double)(e - b) + 1.0);
      ssum += (unsigned long long)(hi - lo);
    }
  }
  if (lane() == 0) {
    if (jsum != 0.0) atomicAdd(J, jsum);
    if (ssum) atomicAdd(span, ssum);
  }
}

struct Buffers {
  std::vector<void*> ptrs;
  ~Buffers() { for (void* p : ptrs) cudaFree(p); }
  template <class T> T* get(size_t n) {
    void* p = nullptr;
    if (cudaMalloc(&p, (n > 0 ? n : 1) * sizeof(T)) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    ptrs.push_back(p);
    return static_cast<T*>(p);
  }
};

}  // namespace

extern "C" int taurus_reorder(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx, const int32_t* initial_rank,
                              int32_t iterations, int32_t* out_rank, double* out_positions, double* out_J, int64_t* out_span,
                              void* cuda_stream) {
  if (V < 1 || V >= (1ll << 31) || E < 0 || E >= (1ll << 32) || !row_ptr || (E > 0 && !col_idx) || !out_rank || iterations < 0 ||
      iterations > 1000)
    return TAURUS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int sms = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = sms * 8;
  Buffers B;
  long long* d_row = B.get<long long>((size_t)V + 1);
  int32_t* d_col = B.get<int32_t>((size_t)E);
  int32_t* d_din = B.get<int32_t>((size_t)V);
  int32_t* d_init = initial_rank ? B.get<int32_t>((size_t)V) : nullptr;
  long long* d_inptr = B.get<long long>((size_t)V + 1);
  int32_t* d_insrc = B.get<int32_t>((size_t)E);
  int32_t* d_srcedge = B.get<int32_t>((size_t)E);
  int32_t* d_keys = B.get<int32_t>((size_t)E);
  double* d_r = B.get<double>((size_t)V);
  double* d_rsorted = B.get<double>((size_t)V);
  double* d_mu = B.get<double>((size_t)V);
  double* d_w1 = B.get<double>((size_t)V);
  double* d_w2 = B.get<double>((size_t)V);
  double* d_pos = B.get<double>((size_t)V);
  int32_t* d_ids = B.get<int32_t>((size_t)V);
  int32_t* d_order = B.get<int32_t>((size_t)V);
  int32_t* d_rank = B.get<int32_t>((size_t)V);
  double* d_J = B.get<double>(1);
  unsigned long long* d_span = B.get<unsigned long long>(1);
  int* d_bad = B.get<int>(1);
  if (!d_row || !d_col || !d_din || (initial_rank && !d_init) || !d_inptr || !d_insrc || !d_srcedge || !d_keys || !d_r ||
      !d_rsorted || !d_mu || !d_w1 || !d_w2 || !d_pos || !d_ids || !d_order || !d_rank || !d_J || !d_span || !d_bad)
    return TAURUS_ERR_NOMEM;
#define RO(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return TAURUS_ERR_CUDA; } } while (0)
  RO(cudaMemcpyAsync(d_row, row_ptr, (size_t)(V + 1) * sizeof(long long), cudaMemcpyDefault, st));
  if (E > 0) RO(cudaMemcpyAsync(d_col, col_idx, (size_t)E * sizeof(int32_t), cudaMemcpyDefault, st));
  if (initial_rank) RO(cudaMemcpyAsync(d_init, initial_rank, (size_t)V * sizeof(int32_t), cudaMemcpyDefault, st));
  RO(cudaMemsetAsync(d_din, 0, (size_t)V * sizeof(int32_t), st));
  RO(cudaMemsetAsync(d_bad, 0, sizeof(int), st));
  // in-lists: in-degrees, their prefix sums, sources sorted (stably) by destination
  ro_degree_kernel<<<grid, 256, 0, st>>>(E, d_col, V, d_din, d_bad);
  ro_widen_kernel<<<grid, 256, 0, st>>>(V, d_din, d_inptr);
  ro_src_kernel<<<grid, 256, 0, st>>>(V, d_row, d_srcedge);
  int end_bit = 1;
  while (end_bit < 31 && (1ll << end_bit) < V) ++end_bit;
  size_t t1 = 0, t2 = 0, t3 = 0;
  cub::DeviceScan::ExclusiveSum(nullptr, t1, d_inptr, d_inptr, V + 1, st);
  if (E > 0) cub::DeviceRadixSort::SortPairs(nullptr, t2, d_col, d_keys, d_srcedge, d_insrc, E, 0, end_bit, st);
  cub::DeviceRadixSort::SortPairs(nullptr, t3, d_r, d_rsorted, d_ids, d_order, V, 0, 64, st);
  size_t tmp_bytes = t1 > t2 ? t1 : t2;
  if (t3 > tmp_bytes) tmp_bytes = t3;
  void* d_tmp = B.get<char>(tmp_bytes);
  if (!d_tmp) return TAURUS_ERR_NOMEM;
  size_t tb = tmp_bytes;
  RO(cub::DeviceScan::ExclusiveSum(d_tmp, tb, d_inptr, d_inptr, V + 1, st));
  if (E > 0) { tb = tmp_bytes; RO(cub::DeviceRadixSort::SortPairs(d_tmp, tb, d_col, d_keys, d_srcedge, d_insrc, E, 0, end_bit, st)); }
  int bad = 0;
  RO(cudaMemcpyAsync(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, st));
  RO(cudaStreamSynchronize(st));
  if (bad) return TAURUS_ERR_INVALID_ARG;

  ro_init_kernel<<<grid, 256, 0, st>>>(V, d_init, d_r);
  ro_iota_kernel<<<grid, 256, 0, st>>>(V, d_ids);
  std::vector<double> J((size_t)iterations + 1, 0.0);
  std::vector<unsigned long long> span((size_t)iterations + 1, 0);
  for (int it = 0; it <= iterations; ++it) {
    if (it > 0) {   // one iteration of the update rules on the real-valued positions
      ro_mu_kernel<<<grid, 256, 0, st>>>(V, d_inptr, d_insrc, d_r, d_mu, d_w1, d_w2);
      ro_r_kernel<<<grid, 256, 0, st>>>(V, d_row, d_col, d_w1, d_w2, d_r);
    }
    // pi = ArgSort(r), ties by vertex id
    tb = tmp_bytes;
    RO(cub::DeviceRadixSort::SortPairs(d_tmp, tb, d_r, d_rsorted, d_ids, d_order, V, 0, 64, st));
    ro_rank_kernel<<<grid, 256, 0, st>>>(V, d_order, d_rank, d_pos);
    if (out_J || out_span) {   // J and C(pi) of this ordering (positions = ranks, centres = their optimum)
      RO(cudaMemsetAsync(d_J, 0, sizeof(double), st));
      RO(cudaMemsetAsync(d_span, 0, sizeof(unsigned long long), st));
      ro_mu_kernel<<<grid, 256, 0, st>>>(V, d_inptr, d_insrc, d_pos, d_mu, nullptr, nullptr);
      ro_measure_kernel<<<grid, 256, 0, st>>>(V, d_inptr, d_insrc, d_pos, d_mu, d_rank, d_J, d_span);
      RO(cudaMemcpyAsync(&J[(size_t)it], d_J, sizeof(double), cudaMemcpyDeviceToHost, st));
      RO(cudaMemcpyAsync(&span[(size_t)it], d_span, sizeof(unsigned long long), cudaMemcpyDeviceToHost, st));
    }
  }
  RO(cudaMemcpyAsync(out_rank, d_rank, (size_t)V * sizeof(int32_t), cudaMemcpyDefault, st));
  if (out_positions) RO(cudaMemcpyAsync(out_positions, d_r, (size_t)V * sizeof(double), cudaMemcpyDefault, st));
  RO(cudaStreamSynchronize(st));
  RO(cudaGetLastError());
  for (int it = 0; it <= iterations; ++it) {
    if (out_J) out_J[it] = J[(size_t)it];
    if (out_span) out_span[it] = (int64_t)span[(size_t)it];
  }
#undef RO
  return TAURUS_OK;
}

// ------------------------------------------------------------------------------------------------ relabelling
// Applying an ordering (Sect. 3.8: topology relabelling and feature relabelling): vertex v becomes rank[v].
namespace {

__global__ void rl_check_kernel(long long V, const int32_t* __restrict__ rank, int32_t* __restrict__ seen, int* bad) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) {
    const int r = rank[v];
    if (r < 0 || r >= V || atomicAdd(&seen[r], 1) != 0) *bad = 1;   // not a permutation of [0, V)
  }
}
__global__ void rl_degree_kernel(long long V, const long long* __restrict__ row_ptr, const int32_t* __restrict__ rank,
                                 long long* __restrict__ new_ptr) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v <= V; v += stride) {
    if (v < V) new_ptr[rank[v]] = row_ptr[v + 1] - row_ptr[v];
    else new_ptr[V] = 0;
  }
}
// row rank[u] of the output = the out-edges of u in their original order, destinations renamed
__global__ void rl_edges_kernel(long long V, const long long* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                const int32_t* __restrict__ rank, const long long* __restrict__ new_ptr, int32_t* __restrict__ new_col,
                                int32_t* __restrict__ new_din, int* bad) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    const long long b = row_ptr[u], n = row_ptr[u + 1] - b, nb = new_ptr[rank[u]];
    for (long long k = lane(); k < n; k += 32) {
      const int v = col[b + k];
      if (v < 0 || v >= V) { *bad = 1; continue; }
      const int nv = rank[v];
      new_col[nb + k] = nv;
      if (new_din) atomicAdd(&new_din[nv], 1);
    }
  }
}
__global__ void rl_rows_kernel(long long V, int width, const float* __restrict__ in, long long ld_in, const int32_t* __restrict__ rank,
                               float* __restrict__ out, long long ld_out) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long v = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; v < V; v += warps) {
    const float* src = in + (size_t)v * ld_in;
    float* dst = out + (size_t)rank[v] * ld_out;
    for (int k = lane(); k < width; k += 32) dst[k] = src[k];
  }
}

}  // namespace

extern "C" int taurus_relabel_csr(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx, const int32_t* rank,
                                  int64_t* out_row_ptr, int32_t* out_col_idx, int32_t* out_in_degree, void* cuda_stream) {
  if (V < 1 || V >= (1ll << 31) || E < 0 || E >= (1ll << 32) || !row_ptr || (E > 0 && (!col_idx || !out_col_idx)) || !rank || !out_row_ptr)
    return TAURUS_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int sms = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int grid = sms * 8;
  Buffers B;
  long long* d_row = B.get<long long>((size_t)V + 1);
  int32_t* d_col = B.get<int32_t>((size_t)E);
  int32_t* d_rank = B.get<int32_t>((size_t)V);
  int32_t* d_seen = B.get<int32_t>((size_t)V);
  long long* d_nptr = B.get<long long>((size_t)V + 1);
  int32_t* d_ncol = B.get<int32_t>((size_t)E);
  int32_t* d_ndin = out_in_degree ? B.get<int32_t>((size_t)V) : nullptr;
  int* d_bad = B.get<int>(1);
  size_t tb = 0;
  cub::DeviceScan::ExclusiveSum(nullptr, tb, d_nptr, d_nptr, V + 1, st);
  void* d_tmp = B.get<char>(tb);
  if (!d_row || !d_col || !d_rank || !d_seen || !d_nptr || !d_ncol || (out_in_degree && !d_ndin) || !d_bad || !d_tmp) return TAURUS_ERR_NOMEM;
#define RL(call) do { if ((call) != cudaSuccess) { cudaGetLastError(); return TAURUS_ERR_CUDA; } } while (0)
  RL(cudaMemcpyAsync(d_row, row_ptr, (size_t)(V + 1) * sizeof(long long), cudaMemcpyDefault, st));
  if (E > 0) RL(cudaMemcpyAsync(d_col, col_idx, (size_t)E * sizeof(int32_t), cudaMemcpyDefault, st));
  RL(cudaMemcpyAsync(d_rank, rank, (size_t)V * sizeof(int32_t), cudaMemcpyDefault, st));
  RL(cudaMemsetAsync(d_seen, 0, (size_t)V * sizeof(int32_t), st));
  RL(cudaMemsetAsync(d_bad, 0, sizeof(int), st));
  if (d_ndin) RL(cudaMemsetAsync(d_ndin, 0, (size_t)V * sizeof(int32_t), st));
  rl_check_kernel<<<grid, 256, 0, st>>>(V, d_rank, d_seen, d_bad);
  int bad = 0;
  RL(cudaMemcpyAsync(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, st));
  RL(cudaStreamSynchronize(st));
  if (bad) return TAURUS_ERR_INVALID_ARG;      // before any index derived from rank is used as an address
  rl_degree_kernel<<<grid, 256, 0, st>>>(V, d_row, d_rank, d_nptr);
  RL(cub::DeviceScan::ExclusiveSum(d_tmp, tb, d_nptr, d_nptr, V + 1, st));
  rl_edges_kernel<<<grid, 256, 0, st>>>(V, d_row, d_col, d_rank, d_nptr, d_ncol, d_ndin, d_bad);
  RL(cudaMemcpyAsync(&bad, d_bad, sizeof(int), cudaMemcpyDeviceToHost, st));
  RL(cudaMemcpyAsync(out_row_ptr, d_nptr, (size_t)(V + 1) * sizeof(long long), cudaMemcpyDefault, st));
  if (E > 0) RL(cudaMemcpyAsync(out_col_idx, d_ncol, (size_t)E * sizeof(int32_t), cudaMemcpyDefault, st));
  if (out_in_degree) RL(cudaMemcpyAsync(out_in_degree, d_ndin, (size_t)V * sizeof(int32_t), cudaMemcpyDefault, st));
  RL(cudaStreamSynchronize(st));
  RL(cudaGetLastError());
  return bad ? TAURUS_ERR_INVALID_ARG : TAURUS_OK;
#undef RL
}

extern "C" int taurus_permute_rows(int64_t V, int32_t width, const float* in_rows, int64_t ld_in, const int32_t* rank, float* out_rows,
                                   int64_t ld_out, void* cuda_stream) {
  if (V < 1 || V >= (1ll << 31) || width < 1 || !in_rows || !rank || !out_rows || ld_in < width || ld_out < width || in_rows == out_rows)
    return TAURUS_ERR_INVALID_ARG;
  cudaPointerAttributes a_in, a_out, a_rank;
  if (cudaPointerGetAttributes(&a_in, in_rows) != cudaSuccess || cudaPointerGetAttributes(&a_out, out_rows) != cudaSuccess ||
      cudaPointerGetAttributes(&a_rank, rank) != cudaSuccess || a_in.type != cudaMemoryTypeDevice || a_out.type != cudaMemoryTypeDevice ||
      a_rank.type != cudaMemoryTypeDevice) {
    cudaGetLastError();
    return TAURUS_ERR_INVALID_ARG;             // device memory only: the matrices are too large to stage
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int sms = 148, dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  rl_rows_kernel<<<sms * 8, 256, 0, st>>>(V, width, in_rows, ld_in, rank, out_rows, ld_out);
  return cudaGetLastError() == cudaSuccess ? TAURUS_OK : TAURUS_ERR_CUDA;
}
