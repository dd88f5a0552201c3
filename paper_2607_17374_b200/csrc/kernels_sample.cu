// Fanout sampling (S0; Sect. 3.9, "Sampling-based Inference"): per layer, keep at most `fanout` in-edges
// of every destination and suppress the rest through an edge mask over the CSR.
//
// The kept set is a function of (seed, layer, dst) only: a partial Fisher-Yates shuffle over the
// destination's in-list positions 0..din-1, step k swapping entry k with entry
// k + floor(hash(seed, layer, dst, k) * (din - k) / 2^64); the first `fanout` entries are kept.
// The in-list order is ascending source id with equal sources in CSR order, i.e. ascending CSR edge index,
// which a stable sort of the edges by destination provides.
#include <cub/cub.cuh>

#include "taurus_internal.h"

// 64-bit finaliser and absorb step of the sampling hash; constants are part of the sampler's definition.
static __host__ __device__ __forceinline__ unsigned long long smp_mix(unsigned long long x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27; x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}
static __host__ __device__ __forceinline__ unsigned long long smp_absorb(unsigned long long h, unsigned long long x) {
  return smp_mix(h ^ (0x9E3779B97F4A7C15ull * (x + 1ull)));
}
static __device__ __forceinline__ unsigned long long smp_hash_prefix(unsigned long long seed, unsigned long long layer,
                                                                     unsigned long long dst) {
  unsigned long long h = 0x243F6A8885A308D3ull;
  h = smp_absorb(h, seed);
  h = smp_absorb(h, layer);
  return smp_absorb(h, dst);
}

// Kept positions of one destination with din > fanout, written to pos[0..fanout).  The virtual array
// a[i] = i is represented by its first `fanout` entries plus a short list of displaced far entries.
static __device__ void sample_positions(unsigned long long seed, int layer, long long dst, int din, int fanout, int* pos) {
  int far_idx[TAURUS_MAX_FANOUT], far_val[TAURUS_MAX_FANOUT];
  int n_far = 0;
  for (int k = 0; k < fanout; ++k) pos[k] = k;
  const unsigned long long hp = smp_hash_prefix(seed, (unsigned long long)layer, (unsigned long long)dst);
  for (int k = 0; k < fanout; ++k) {
    unsigned long long h = smp_absorb(hp, (unsigned long long)k);
    int j = k + (int)__umul64hi(h, (unsigned long long)(din - k));
    if (j < fanout) {
      int t = pos[k]; pos[k] = pos[j]; pos[j] = t;
    } else {
      int f = 0;
      while (f < n_far && far_idx[f] != j) ++f;
      if (f == n_far) { far_idx[n_far] = j; far_val[n_far] = j; ++n_far; }
      int t = pos[k]; pos[k] = far_val[f]; far_val[f] = t;
    }
  }
}

__global__ void sample_mask_kernel(long long V, const int32_t* din, const long long* csc_ptr, const uint32_t* csc_eid,
                                   unsigned long long seed, int layer, int fanout, uint32_t* mask) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) {
    int d = din[v];
    long long base = csc_ptr[v];
    if (d <= fanout) {
      for (int p = 0; p < d; ++p) {
        uint32_t e = csc_eid[base + p];
        atomicOr(&mask[e >> 5], 1u << (e & 31));
      }
    } else {
      int pos[TAURUS_MAX_FANOUT];
      sample_positions(seed, layer, v, d, fanout, pos);
      for (int k = 0; k < fanout; ++k) {
        uint32_t e = csc_eid[base + pos[k]];
        atomicOr(&mask[e >> 5], 1u << (e & 31));
      }
    }
  }
}

void launch_sample_mask(taurus_ctx* c, int layer, cudaStream_t st) {
  size_t words = (size_t)((c->E + 31) / 32);
  cudaMemsetAsync(c->d_mask, 0, words * sizeof(uint32_t), st);
  sample_mask_kernel<<<c->sm_count * 8, 128, 0, st>>>(c->V, c->d_din, c->d_csc_ptr, c->d_csc_eid, c->seed, layer,
                                                      c->fanout[layer], c->d_mask);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ in-edge order
__global__ void iota_kernel(long long n, uint32_t* out) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = (uint32_t)i;
}
__global__ void widen_kernel(long long n, const int32_t* in, long long* out) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) out[i] = in[i];
}

// csc_ptr = exclusive prefix sums of the in-degrees; csc_eid = CSR edge indices sorted (stably) by destination.
int build_in_edge_order(taurus_ctx* c) {
  const long long V = c->V, E = c->E;
  int32_t* keys_out = nullptr;
  uint32_t* vals_in = nullptr;
  void* tmp = nullptr;
  size_t tmp_bytes = 0, scan_bytes = 0;
  int rc = 0;
  int end_bit = 1;
  while (end_bit < 31 && (1ll << end_bit) < V) ++end_bit;
  do {
    if (cudaMalloc(&c->d_csc_ptr, (size_t)(V + 1) * sizeof(long long)) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    if (cudaMalloc(&c->d_csc_eid, (size_t)(E > 0 ? E : 1) * sizeof(uint32_t)) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    // prefix sums: widen to 64 bit first (in place in csc_ptr), then scan
    widen_kernel<<<c->sm_count * 8, 256>>>(V, c->d_din, c->d_csc_ptr);
    cudaMemset(c->d_csc_ptr + V, 0, sizeof(long long));
    cub::DeviceScan::ExclusiveSum(nullptr, scan_bytes, c->d_csc_ptr, c->d_csc_ptr, V + 1);
    if (E > 0) {
      if (cudaMalloc(&keys_out, (size_t)E * sizeof(int32_t)) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
      if (cudaMalloc(&vals_in, (size_t)E * sizeof(uint32_t)) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
      cub::DeviceRadixSort::SortPairs(nullptr, tmp_bytes, c->d_col, keys_out, vals_in, c->d_csc_eid, E, 0, end_bit);
    }
    if (scan_bytes > tmp_bytes) tmp_bytes = scan_bytes;
    if (cudaMalloc(&tmp, tmp_bytes > 0 ? tmp_bytes : 16) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    size_t b = tmp_bytes;
    if (cub::DeviceScan::ExclusiveSum(tmp, b, c->d_csc_ptr, c->d_csc_ptr, V + 1) != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
    if (E > 0) {
      iota_kernel<<<c->sm_count * 8, 256>>>(E, vals_in);
      b = tmp_bytes;
      if (cub::DeviceRadixSort::SortPairs(tmp, b, c->d_col, keys_out, vals_in, c->d_csc_eid, E, 0, end_bit) != cudaSuccess) {
        rc = TAURUS_ERR_CUDA; break;
      }
    }
    if (cudaDeviceSynchronize() != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
  } while (0);
  cudaFree(keys_out); cudaFree(vals_in); cudaFree(tmp);
  c->launches += 2;
  return rc;
}

// csc_ptr alone (the in-list sources are then filled from the grouped edge order, chunk by chunk).
int build_csc_ptr(taurus_ctx* c) {
  const long long V = c->V;
  void* tmp = nullptr;
  size_t scan_bytes = 0;
  int rc = TAURUS_OK;
  do {
    if (cudaMalloc(&c->d_csc_ptr, (size_t)(V + 1) * sizeof(long long)) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    widen_kernel<<<c->sm_count * 8, 256>>>(V, c->d_din, c->d_csc_ptr);
    cudaMemset(c->d_csc_ptr + V, 0, sizeof(long long));
    cub::DeviceScan::ExclusiveSum(nullptr, scan_bytes, c->d_csc_ptr, c->d_csc_ptr, V + 1);
    if (cudaMalloc(&tmp, scan_bytes > 0 ? scan_bytes : 16) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    if (cub::DeviceScan::ExclusiveSum(tmp, scan_bytes, c->d_csc_ptr, c->d_csc_ptr, V + 1) != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
    if (cudaDeviceSynchronize() != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
  } while (0);
  cudaFree(tmp);
  c->launches += 1;
  return rc;
}

// Source of every in-list entry from its CSR edge index: the row whose range holds the index.
__global__ void csc_src_from_eid_kernel(long long E, long long V, const long long* __restrict__ row_ptr, const uint32_t* __restrict__ csc_eid,
                                        int32_t* __restrict__ csc_src) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < E; i += stride) {
    const long long e = csc_eid[i];
    long long lo = 0, hi = V;   // largest u with row_ptr[u] <= e
    while (hi - lo > 1) { const long long mid = (lo + hi) >> 1; if (row_ptr[mid] <= e) lo = mid; else hi = mid; }
    csc_src[i] = (int32_t)lo;
  }
}

int build_csc_src_from_eid(taurus_ctx* c) {
  if (c->E > 0) csc_src_from_eid_kernel<<<c->sm_count * 16, 256>>>(c->E, c->V, c->d_row_ptr, c->d_csc_eid, c->d_csc_src);
  c->launches += 1;
  return cudaDeviceSynchronize() == cudaSuccess ? TAURUS_OK : TAURUS_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------ inspection
// One block: the kept edges of one destination, ascending edge index, with their sources.
__global__ void sampled_edges_kernel(long long dst, const int32_t* din, const long long* csc_ptr, const uint32_t* csc_eid,
                                     const long long* row_ptr, long long V, unsigned long long seed, int layer, int fanout,
                                     long long* out_eid, int32_t* out_src, int cap, int* out_n) {
  __shared__ int pos[TAURUS_MAX_FANOUT];
  __shared__ int n;
  const int d = din[dst];
  const long long base = csc_ptr[dst];
  if (threadIdx.x == 0) {
    if (fanout <= 0 || d <= fanout) n = d;
    else {
      sample_positions(seed, layer, dst, d, fanout, pos);
      for (int i = 1; i < fanout; ++i) {   // insertion sort: ascending position = ascending edge index
        int x = pos[i], j = i - 1;
        while (j >= 0 && pos[j] > x) { pos[j + 1] = pos[j]; --j; }
        pos[j + 1] = x;
      }
      n = fanout;
    }
    *out_n = n;
  }
  __syncthreads();
  const bool all = fanout <= 0 || d <= fanout;
  for (int i = threadIdx.x; i < n && i < cap; i += blockDim.x) {
    long long e = csc_eid[base + (all ? i : pos[i])];
    long long lo = 0, hi = V;   // source: largest u with row_ptr[u] <= e
    while (hi - lo > 1) { long long mid = (lo + hi) >> 1; if (row_ptr[mid] <= e) lo = mid; else hi = mid; }
    out_eid[i] = e;
    out_src[i] = (int32_t)lo;
  }
}

int sampled_edges_of(taurus_ctx* c, int layer, long long dst, long long* out_eids, int32_t* out_src, int cap, int* n) {
  long long* d_e = nullptr; int32_t* d_s = nullptr; int* d_n = nullptr;
  int rc = TAURUS_OK;
  size_t cap1 = cap > 0 ? cap : 1;
  if (cudaMalloc(&d_e, cap1 * sizeof(long long)) != cudaSuccess || cudaMalloc(&d_s, cap1 * sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&d_n, sizeof(int)) != cudaSuccess) {
    rc = TAURUS_ERR_NOMEM;
  } else {
    sampled_edges_kernel<<<1, 256>>>(dst, c->d_din, c->d_csc_ptr, c->d_csc_eid, c->d_row_ptr, c->V, c->seed, layer,
                                     c->fanout[layer], d_e, d_s, cap, d_n);
    c->launches += 1;
    if (cudaMemcpy(n, d_n, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) rc = TAURUS_ERR_CUDA;
    else {
      int m = *n < cap ? *n : cap;
      if (m > 0 && (cudaMemcpy(out_eids, d_e, (size_t)m * sizeof(long long), cudaMemcpyDeviceToHost) != cudaSuccess ||
                    cudaMemcpy(out_src, d_s, (size_t)m * sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess))
        rc = TAURUS_ERR_CUDA;
    }
  }
  cudaFree(d_e); cudaFree(d_s); cudaFree(d_n);
  return rc;
}

// Digest of every destination's propagated in-edges: commutative sum and xor of a 64-bit mix of (source, CSR
// edge index), accumulated push-based with one warp per source row.
__global__ void sample_digest_kernel(long long V, const long long* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                     const uint32_t* __restrict__ mask, unsigned long long* __restrict__ digest) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int lane = threadIdx.x & 31;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    for (long long e = row_ptr[u] + lane; e < row_ptr[u + 1]; e += 32) {
      if (mask && !((mask[e >> 5] >> (e & 31)) & 1u)) continue;
      unsigned long long x = (((unsigned long long)u << 32) | (unsigned long long)(e & 0xffffffffll)) + 0x9E3779B97F4A7C15ull;
      x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
      x ^= x >> 27; x *= 0x94D049BB133111EBull;
      x ^= x >> 31;
      const long long v = col[e];
      atomicAdd(&digest[2 * v], x);
      atomicXor(&digest[2 * v + 1], x);
    }
  }
}

void launch_sample_digest(taurus_ctx* c, unsigned long long* d_digest, cudaStream_t st) {
  sample_digest_kernel<<<c->sm_count * 8, 256, 0, st>>>(c->V, c->d_row_ptr, c->d_col, c->d_mask_cur, d_digest);
  c->launches += 1;
}
