// Output side of a layer: range-partitioned sorted runs (embedding writer, Sect. 3.7) and merge-on-read
// (graph reader, Sect. 3.3).
//
// Writer.  One append runs in two phases.  Phase 1 (device): every row gets the number of its id range as a
// key, a stable radix sort of (key, position) groups the rows by range in arrival order, and the per-range
// counts go to pinned host memory.  Phase 2 (host plans, device moves): with the counts known the host cuts
// each range's rows into what still fits its partition buffer, what fills the next buffer load, and so on;
// each pass moves one such piece per range (one launch for all ranges) and then sorts and flushes the
// buffers that are full: their ids are collected, radix-sorted together with the buffer positions as payload
// (the ranges are contiguous in id, so one sort leaves them range after range), and one gather writes ids and
// rows of the runs sequentially into the run store (directly over PCIe when the store is pinned host memory).  Because the grouping sort is stable, run k of a range holds that range's arrivals
// k R .. (k + 1) R - 1 whatever the other ranges did.
//
// Reader.  The ids of all runs live in pinned host memory; for a chunk [s, e) the host bisects each
// overlapping run (first id >= s, first id >= e), issues one contiguous copy per run slice into a device
// staging area, and one kernel places every staged row at (id - s): the k-way merge by vertex id, which for
// ids that occur once is a placement.
#include <cub/cub.cuh>

#include <algorithm>
#include <vector>

#include "taurus.h"
#include "taurus_internal.h"

namespace {

struct RunRec { long long partition, offset, n; };
struct MoveSeg { long long src, n, dst; };   // src: position in the grouped index list; dst: row of the partition buffers

constexpr int SEG_RING = 8;

__device__ __forceinline__ int rs_lane() { return threadIdx.x & 31; }

__device__ __forceinline__ void copy_row(float* __restrict__ dst, const float* __restrict__ src, int width) {
  if ((((uintptr_t)dst | (uintptr_t)src) & 15) == 0 && (width & 3) == 0) {
    for (int k = rs_lane(); k < (width >> 2); k += 32) reinterpret_cast<float4*>(dst)[k] = reinterpret_cast<const float4*>(src)[k];
  } else {
    for (int k = rs_lane(); k < width; k += 32) dst[k] = src[k];
  }
}

// key[i] = id range of row i (P for positions past the row count), idx[i] = i; cnt[0..P) = rows per range,
// cnt[P] = rows seen, cnt[P + 1] = rows with an id outside [0, V) or a count beyond the bound.
__global__ void rs_key_kernel(const long long* __restrict__ ids, long long n_bound, const long long* d_count, long long count_host,
                              long long V, long long range_ids, int P, int32_t* __restrict__ key, int32_t* __restrict__ idx,
                              long long* __restrict__ cnt) {
  extern __shared__ unsigned int sh[];
  for (int t = threadIdx.x; t < P + 2; t += blockDim.x) sh[t] = 0;
  __syncthreads();
  long long count = d_count ? *d_count : count_host;
  if (count > n_bound) {
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicAdd((unsigned long long*)&cnt[P + 1], 1ull);
    count = n_bound;
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_bound; i += stride) {
    int k = P;
    if (i < count) {
      const long long id = ids[i];
      if (id < 0 || id >= V) atomicAdd(&sh[P + 1], 1u);
      else { k = (int)(id / range_ids); atomicAdd(&sh[k], 1u); }
    }
    key[i] = k;
    idx[i] = (int32_t)i;
  }
  __syncthreads();
  for (int t = threadIdx.x; t < P + 2; t += blockDim.x)
    if (t != P && sh[t]) atomicAdd((unsigned long long*)&cnt[t], (unsigned long long)sh[t]);
  if (blockIdx.x == 0 && threadIdx.x == 0) cnt[P] = count;
}

// One piece per range: rows idx_s[src .. src + n) of the append go to partition-buffer rows dst .. dst + n.
__global__ void rs_move_kernel(const MoveSeg* __restrict__ segs, const int32_t* __restrict__ idx_s, const long long* __restrict__ ids,
                               const float* __restrict__ rows, long long ld, int width, int32_t* __restrict__ pids,
                               float* __restrict__ prows) {
  const MoveSeg sg = segs[blockIdx.y];
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < sg.n; i += warps) {
    const long long r = idx_s[sg.src + i];
    if (rs_lane() == 0) pids[sg.dst + i] = (int32_t)ids[r];
    copy_row(prows + (size_t)(sg.dst + i) * width, rows + (size_t)r * ld, width);
  }
}

// Buffers that leave together: ids of piece q go to fkeys[dst ..], their partition-buffer row numbers to fvals[dst ..].
__global__ void rs_collect_kernel(const MoveSeg* __restrict__ segs, const int32_t* __restrict__ pids, int32_t* __restrict__ fkeys,
                                  int32_t* __restrict__ fvals) {
  const MoveSeg sg = segs[blockIdx.y];
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < sg.n; i += stride) {
    fkeys[sg.dst + i] = pids[sg.src + i];
    fvals[sg.dst + i] = (int32_t)(sg.src + i);
  }
}

// Writes sorted runs: ids and rows in id order, sequentially, into the store (the id ranges are contiguous, so
// buffers sorted together come out range after range).
__global__ void rs_gather_kernel(long long n, const int32_t* __restrict__ sid, const int32_t* __restrict__ sidx,
                                 const float* __restrict__ prows, int width, int32_t* __restrict__ run_ids,
                                 float* __restrict__ run_rows) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
    if (rs_lane() == 0) run_ids[i] = sid[i];
    copy_row(run_rows + (size_t)i * width, prows + (size_t)sidx[i] * width, width);
  }
}

// Merge by vertex id: staged row i belongs at row (id - s) of the chunk matrix.
__global__ void rs_place_kernel(long long n, const int32_t* __restrict__ sid, const float* __restrict__ srows, int width,
                                long long s, float* __restrict__ out, long long ld) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps)
    copy_row(out + (size_t)(sid[i] - s) * ld, srows + (size_t)i * width, width);
}

// The same for a store in device memory: slice q of the chunk (rows src .. src + n of the store, their ids staged
// at dst ..) is read in place, without a staging copy of the rows.
__global__ void rs_place_slices_kernel(const MoveSeg* __restrict__ segs, const int32_t* __restrict__ sid, const float* __restrict__ store,
                                       int width, long long s, float* __restrict__ out, long long ld) {
  const MoveSeg sg = segs[blockIdx.y];
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < sg.n; i += warps)
    copy_row(out + (size_t)(sid[sg.dst + i] - s) * ld, store + (size_t)(sg.src + i) * width, width);
}

int bits_for(long long values) {   // bits needed to tell `values` different keys apart
  int b = 1;
  while ((1ll << b) < values) ++b;
  return b;
}

}  // namespace

struct taurus_runs {
  int device = 0, width = 0, kind = 0, part_bits = 1, id_bits = 1, sm_count = 148;
  long long V = 0, P = 0, R = 0, range_ids = 0, store_rows = 0, max_append = 0, max_chunk = 0;
  // partition buffers
  int32_t* d_pids = nullptr;
  float* d_prows = nullptr;
  std::vector<long long> fill;
  // run store
  float* store_dev = nullptr;    // what kernels write: device memory, or the device alias of store_host
  float* store_host = nullptr;   // pinned + mapped (host kind only)
  int32_t* h_ids = nullptr;      // ids of all runs, pinned + mapped
  int32_t* d_ids = nullptr;      // device alias of h_ids
  long long store_top = 0;
  std::vector<RunRec> dir;
  std::vector<std::vector<int>> by_part;
  // append scratch
  int32_t *d_key = nullptr, *d_key_s = nullptr, *d_idx = nullptr, *d_idx_s = nullptr;
  long long* d_cnt = nullptr;
  long long* h_cnt = nullptr;    // pinned
  MoveSeg* d_segs = nullptr;     // SEG_RING tables of P pieces
  MoveSeg* h_segs = nullptr;     // pinned
  cudaEvent_t seg_done[SEG_RING] = {nullptr};
  bool seg_used[SEG_RING] = {false};
  long long seg_seq = 0;
  // flush scratch
  int32_t *d_fkeys = nullptr, *d_fvals = nullptr, *d_sid = nullptr, *d_sidx = nullptr;   // [flush_cap]
  long long flush_cap = 0;       // most rows sorted in one go
  void* d_tmp = nullptr;
  size_t tmp_bytes = 0;
  // read staging
  float* d_stage_rows = nullptr;
  int32_t* d_stage_ids = nullptr;
  cudaEvent_t cnt_ready = nullptr, write_done = nullptr, stage_free = nullptr;
  bool stage_used = false, dirty = false, pending = false;
  // the append whose phase 2 has not run yet
  const long long* p_ids = nullptr;
  const float* p_rows = nullptr;
  long long p_ld = 0;
  long long launches = 0;
};

#define RCU(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { taurus_note_cuda_error(e_, #call); return TAURUS_ERR_CUDA; } } while (0)

template <class T>
static int rs_alloc(T** p, size_t count) {
  *p = nullptr;
  cudaError_t e = cudaMalloc((void**)p, (count ? count : 1) * sizeof(T));
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return TAURUS_ERR_NOMEM; }
  if (e != cudaSuccess) { taurus_note_cuda_error(e, "cudaMalloc"); return TAURUS_ERR_CUDA; }
  return TAURUS_OK;
}
template <class T>
static int rs_pinned(T** p, size_t count) {
  *p = nullptr;
  cudaError_t e = cudaHostAlloc((void**)p, (count ? count : 1) * sizeof(T), cudaHostAllocMapped);
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return TAURUS_ERR_NOMEM; }
  if (e != cudaSuccess) { taurus_note_cuda_error(e, "cudaHostAlloc"); return TAURUS_ERR_CUDA; }
  return TAURUS_OK;
}
#define RALLOC(p, n) do { int rc_ = rs_alloc(&(p), (size_t)(n)); if (rc_) { taurus_runs_destroy(r); return rc_; } } while (0)
#define RPINNED(p, n) do { int rc_ = rs_pinned(&(p), (size_t)(n)); if (rc_) { taurus_runs_destroy(r); return rc_; } } while (0)

extern "C" void taurus_runs_destroy(taurus_runs* r) {
  if (!r) return;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(r->device);
  cudaDeviceSynchronize();
  cudaFree(r->d_pids); cudaFree(r->d_prows);
  if (r->kind == TAURUS_RUNS_HOST) cudaFreeHost(r->store_host); else cudaFree(r->store_dev);
  cudaFreeHost(r->h_ids); cudaFreeHost(r->h_cnt); cudaFreeHost(r->h_segs);
  cudaFree(r->d_key); cudaFree(r->d_key_s); cudaFree(r->d_idx); cudaFree(r->d_idx_s); cudaFree(r->d_cnt); cudaFree(r->d_segs);
  cudaFree(r->d_fkeys); cudaFree(r->d_fvals); cudaFree(r->d_sid); cudaFree(r->d_sidx); cudaFree(r->d_tmp);
  cudaFree(r->d_stage_rows); cudaFree(r->d_stage_ids);
  for (int i = 0; i < SEG_RING; ++i) if (r->seg_done[i]) cudaEventDestroy(r->seg_done[i]);
  if (r->cnt_ready) cudaEventDestroy(r->cnt_ready);
  if (r->write_done) cudaEventDestroy(r->write_done);
  if (r->stage_free) cudaEventDestroy(r->stage_free);
  cudaGetLastError();
  cudaSetDevice(prev);
  delete r;
}

extern "C" int taurus_runs_create(taurus_runs** out, const taurus_runs_config* cfg) {
  if (!out || !cfg) return TAURUS_ERR_INVALID_ARG;
  if (cfg->V < 1 || cfg->V >= (1ll << 31) || cfg->width < 1 || cfg->width > TAURUS_MAX_DIM || cfg->partitions < 1 ||
      cfg->partitions > 1024 || cfg->partition_rows < 1 || cfg->partition_rows >= (1ll << 31) || cfg->store_rows < 1 ||
      cfg->max_append_rows < 1 || cfg->max_append_rows >= (1ll << 31) || cfg->max_chunk_rows < 1 ||
      cfg->partitions * cfg->partition_rows >= (1ll << 31) ||
      (cfg->store_kind != TAURUS_RUNS_HOST && cfg->store_kind != TAURUS_RUNS_DEVICE))
    return TAURUS_ERR_INVALID_ARG;
  taurus_runs* r = new (std::nothrow) taurus_runs();
  if (!r) return TAURUS_ERR_NOMEM;
  if (cudaGetDevice(&r->device) != cudaSuccess) { cudaGetLastError(); delete r; return TAURUS_ERR_CUDA; }
  cudaDeviceGetAttribute(&r->sm_count, cudaDevAttrMultiProcessorCount, r->device);
  r->V = cfg->V; r->width = cfg->width; r->kind = cfg->store_kind; r->P = cfg->partitions; r->R = cfg->partition_rows;
  r->store_rows = cfg->store_rows; r->max_append = cfg->max_append_rows; r->max_chunk = cfg->max_chunk_rows;
  r->range_ids = (r->V + r->P - 1) / r->P;
  r->part_bits = bits_for(r->P + 1);
  r->id_bits = bits_for(r->V);
  r->fill.assign((size_t)r->P, 0);
  r->by_part.assign((size_t)r->P, std::vector<int>());
  const size_t w = (size_t)r->width;
  RALLOC(r->d_pids, (size_t)r->P * r->R);
  RALLOC(r->d_prows, (size_t)r->P * r->R * w);
  if (r->kind == TAURUS_RUNS_HOST) {
    RPINNED(r->store_host, (size_t)r->store_rows * w);
    if (cudaHostGetDevicePointer((void**)&r->store_dev, r->store_host, 0) != cudaSuccess) { cudaGetLastError(); taurus_runs_destroy(r); return TAURUS_ERR_CUDA; }
  } else {
    RALLOC(r->store_dev, (size_t)r->store_rows * w);
  }
  RPINNED(r->h_ids, (size_t)r->store_rows);
  if (cudaHostGetDevicePointer((void**)&r->d_ids, r->h_ids, 0) != cudaSuccess) { cudaGetLastError(); taurus_runs_destroy(r); return TAURUS_ERR_CUDA; }
  RALLOC(r->d_key, r->max_append); RALLOC(r->d_key_s, r->max_append); RALLOC(r->d_idx, r->max_append); RALLOC(r->d_idx_s, r->max_append);
  RALLOC(r->d_cnt, r->P + 2);
  RPINNED(r->h_cnt, (size_t)r->P + 2);
  RALLOC(r->d_segs, (size_t)SEG_RING * r->P);
  RPINNED(r->h_segs, (size_t)SEG_RING * r->P);
  r->flush_cap = std::max<long long>(r->R, std::min<long long>(r->P * r->R, 1ll << 26));
  RALLOC(r->d_fkeys, r->flush_cap); RALLOC(r->d_fvals, r->flush_cap); RALLOC(r->d_sid, r->flush_cap); RALLOC(r->d_sidx, r->flush_cap);
  size_t t1 = 0, t2 = 0;
  cub::DeviceRadixSort::SortPairs(nullptr, t1, r->d_key, r->d_key_s, r->d_idx, r->d_idx_s, (int)r->max_append, 0, r->part_bits);
  cub::DeviceRadixSort::SortPairs(nullptr, t2, r->d_fkeys, r->d_sid, r->d_fvals, r->d_sidx, (int)r->flush_cap, 0, r->id_bits);
  r->tmp_bytes = std::max(t1, t2);
  { char* t = nullptr; RALLOC(t, r->tmp_bytes); r->d_tmp = t; }
  RALLOC(r->d_stage_rows, (size_t)r->max_chunk * w);
  RALLOC(r->d_stage_ids, r->max_chunk);
  for (int i = 0; i < SEG_RING; ++i)
    if (cudaEventCreateWithFlags(&r->seg_done[i], cudaEventDisableTiming) != cudaSuccess) { taurus_runs_destroy(r); return TAURUS_ERR_CUDA; }
  if (cudaEventCreateWithFlags(&r->cnt_ready, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&r->write_done, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&r->stage_free, cudaEventDisableTiming) != cudaSuccess) { taurus_runs_destroy(r); return TAURUS_ERR_CUDA; }
  if (cudaDeviceSynchronize() != cudaSuccess) { taurus_note_cuda_error(cudaGetLastError(), "taurus_runs_create"); taurus_runs_destroy(r); return TAURUS_ERR_CUDA; }
  *out = r;
  return TAURUS_OK;
}

int runs_width(const taurus_runs* r) { return r->width; }
long long runs_max_append(const taurus_runs* r) { return r->max_append; }
long long runs_max_chunk(const taurus_runs* r) { return r->max_chunk; }
long long runs_vertices(const taurus_runs* r) { return r->V; }
bool runs_pending(const taurus_runs* r) { return r->pending; }
long long runs_launches(const taurus_runs* r) { return r->launches; }

// Phase 1 of an append, asynchronous on `st`: group the rows by id range (stable) and send the per-range
// counts to the host.  The row count is *d_count when d_count is given (clamped to n_bound), else count_host.
int runs_phase1(taurus_runs* r, const long long* ids, const float* rows, long long ld, long long n_bound, const long long* d_count,
                long long count_host, cudaStream_t st) {
  if (r->pending) return TAURUS_ERR_ORDER;
  if (n_bound < 0 || n_bound > r->max_append || ld < r->width) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaMemsetAsync(r->d_cnt, 0, (size_t)(r->P + 2) * sizeof(long long), st));
  if (n_bound > 0) {
    const int grid = (int)std::min<long long>((n_bound + 255) / 256, (long long)r->sm_count * 8);
    rs_key_kernel<<<grid, 256, (size_t)(r->P + 2) * sizeof(unsigned int), st>>>(ids, n_bound, d_count, count_host, r->V, r->range_ids,
                                                                                (int)r->P, r->d_key, r->d_idx, r->d_cnt);
    size_t tb = r->tmp_bytes;
    RCU(cub::DeviceRadixSort::SortPairs(r->d_tmp, tb, r->d_key, r->d_key_s, r->d_idx, r->d_idx_s, (int)n_bound, 0, r->part_bits, st));
    r->launches += 3;
  }
  RCU(cudaMemcpyAsync(r->h_cnt, r->d_cnt, (size_t)(r->P + 2) * sizeof(long long), cudaMemcpyDeviceToHost, st));
  RCU(cudaEventRecord(r->cnt_ready, st));
  r->p_ids = ids; r->p_rows = rows; r->p_ld = ld;
  r->pending = true;
  return TAURUS_OK;
}

// One slot of the piece-table ring, filled by the caller through *hs and uploaded by push_segs.
static int next_seg_slot(taurus_runs* r, MoveSeg** hs, MoveSeg** ds, int* slot) {
  *slot = (int)(r->seg_seq % SEG_RING);
  r->seg_seq += 1;
  if (r->seg_used[*slot]) RCU(cudaEventSynchronize(r->seg_done[*slot]));
  *hs = r->h_segs + (size_t)*slot * r->P;
  *ds = r->d_segs + (size_t)*slot * r->P;
  return TAURUS_OK;
}
static int push_segs(taurus_runs* r, int slot, int nseg, cudaStream_t st) {
  RCU(cudaMemcpyAsync(r->d_segs + (size_t)slot * r->P, r->h_segs + (size_t)slot * r->P, (size_t)nseg * sizeof(MoveSeg),
                      cudaMemcpyHostToDevice, st));
  return TAURUS_OK;
}
// Called after the kernel that reads the table has been launched: the slot (host and device copy) may be
// reused once that kernel has run, on whichever stream the next user works.
static int release_seg_slot(taurus_runs* r, int slot, cudaStream_t st) {
  RCU(cudaEventRecord(r->seg_done[slot], st));
  r->seg_used[slot] = true;
  return TAURUS_OK;
}

// Sorts the listed partition buffers (ascending range numbers) by id and writes each to the store as one run.
// Buffers are sorted together, as many per radix sort as the scratch holds: the ranges are contiguous in id,
// so one sort by id leaves them range after range, each in id order.
static int flush_many(taurus_runs* r, const std::vector<long long>& parts, cudaStream_t st) {
  long long total = 0;
  for (long long p : parts) total += r->fill[(size_t)p];
  if (r->store_top + total > r->store_rows) return TAURUS_ERR_RUN_STORE_FULL;
  size_t at = 0;
  while (at < parts.size()) {
    MoveSeg *hs, *ds;
    int slot;
    { int rc = next_seg_slot(r, &hs, &ds, &slot); if (rc) return rc; }
    int nseg = 0;
    long long m = 0, most = 0;
    const size_t first = at;
    while (at < parts.size()) {
      const long long p = parts[at], n = r->fill[(size_t)p];
      if (n == 0) { ++at; continue; }
      if (m + n > r->flush_cap) break;   // n <= R <= flush_cap, so every batch takes at least one buffer
      hs[nseg++] = MoveSeg{p * r->R, n, m};
      m += n; most = std::max(most, n);
      ++at;
    }
    if (m == 0) continue;
    { int rc = push_segs(r, slot, nseg, st); if (rc) return rc; }
    const int gx = (int)std::max<long long>(1, std::min<long long>((most + 255) / 256, std::max<long long>(1, (long long)r->sm_count * 8 / nseg)));
    rs_collect_kernel<<<dim3(gx, nseg), 256, 0, st>>>(ds, r->d_pids, r->d_fkeys, r->d_fvals);
    { int rc = release_seg_slot(r, slot, st); if (rc) return rc; }
    size_t tb = r->tmp_bytes;
    RCU(cub::DeviceRadixSort::SortPairs(r->d_tmp, tb, r->d_fkeys, r->d_sid, r->d_fvals, r->d_sidx, (int)m, 0, r->id_bits, st));
    const long long off = r->store_top;
    const int grid = (int)std::min<long long>((m * 32 + 255) / 256, (long long)r->sm_count * 8);
    rs_gather_kernel<<<grid, 256, 0, st>>>(m, r->d_sid, r->d_sidx, r->d_prows, r->width, r->d_ids + off, r->store_dev + (size_t)off * r->width);
    r->launches += 4;
    for (size_t q = first; q < at; ++q) {
      const long long p = parts[q], n = r->fill[(size_t)p];
      if (n == 0) continue;
      r->by_part[(size_t)p].push_back((int)r->dir.size());
      r->dir.push_back(RunRec{p, r->store_top, n});
      r->store_top += n;
      r->fill[(size_t)p] = 0;
    }
    r->dirty = true;
  }
  return TAURUS_OK;
}

// Phase 2: waits (host) for the counts of phase 1, then moves the grouped rows into the partition buffers on
// `st`, flushing every buffer that fills.  Errors found here leave buffers and store as they were.
int runs_phase2(taurus_runs* r, cudaStream_t st) {
  if (!r->pending) return TAURUS_OK;
  RCU(cudaEventSynchronize(r->cnt_ready));
  r->pending = false;
  const long long* cnt = r->h_cnt;
  if (cnt[r->P + 1] != 0) return TAURUS_ERR_INVALID_ARG;
  long long to_store = 0;
  for (long long p = 0; p < r->P; ++p) to_store += (r->fill[(size_t)p] + cnt[p]) / r->R * r->R;
  if (r->store_top + to_store > r->store_rows) return TAURUS_ERR_RUN_STORE_FULL;
  std::vector<long long> src((size_t)r->P), left((size_t)r->P);
  long long acc = 0, remaining = 0;
  for (long long p = 0; p < r->P; ++p) { src[(size_t)p] = acc; left[(size_t)p] = cnt[p]; acc += cnt[p]; remaining += cnt[p]; }
  std::vector<long long> full;
  while (remaining > 0) {
    MoveSeg *hs, *ds;
    int slot;
    { int rc = next_seg_slot(r, &hs, &ds, &slot); if (rc) return rc; }
    int nseg = 0;
    long long most = 0;
    for (long long p = 0; p < r->P; ++p) {
      const long long take = std::min(left[(size_t)p], r->R - r->fill[(size_t)p]);
      if (take <= 0) continue;
      hs[nseg++] = MoveSeg{src[(size_t)p], take, p * r->R + r->fill[(size_t)p]};
      r->fill[(size_t)p] += take; src[(size_t)p] += take; left[(size_t)p] -= take; remaining -= take;
      most = std::max(most, take);
    }
    { int rc = push_segs(r, slot, nseg, st); if (rc) return rc; }
    const int gx = (int)std::max<long long>(1, std::min<long long>((most * 32 + 255) / 256, std::max<long long>(1, (long long)r->sm_count * 8 / nseg)));
    rs_move_kernel<<<dim3(gx, nseg), 256, 0, st>>>(ds, r->d_idx_s, r->p_ids, r->p_rows, r->p_ld, r->width, r->d_pids, r->d_prows);
    { int rc = release_seg_slot(r, slot, st); if (rc) return rc; }
    r->launches += 1;
    full.clear();
    for (long long p = 0; p < r->P; ++p)
      if (r->fill[(size_t)p] == r->R) full.push_back(p);
    if (!full.empty()) { int rc = flush_many(r, full, st); if (rc) return rc; }
  }
  RCU(cudaGetLastError());
  RCU(cudaEventRecord(r->write_done, st));
  r->dirty = true;
  return TAURUS_OK;
}

int runs_flush_all(taurus_runs* r, cudaStream_t st) {
  if (r->pending) return TAURUS_ERR_ORDER;
  long long total = 0;
  for (long long p = 0; p < r->P; ++p) total += r->fill[(size_t)p];
  if (r->store_top + total > r->store_rows) return TAURUS_ERR_RUN_STORE_FULL;
  std::vector<long long> parts;
  for (long long p = 0; p < r->P; ++p)
    if (r->fill[(size_t)p] > 0) parts.push_back(p);
  if (!parts.empty()) { int rc = flush_many(r, parts, st); if (rc) return rc; }
  RCU(cudaGetLastError());
  RCU(cudaEventRecord(r->write_done, st));
  r->dirty = true;
  return TAURUS_OK;
}

static int wait_writes(taurus_runs* r) {
  if (r->dirty) { RCU(cudaEventSynchronize(r->write_done)); r->dirty = false; }
  return TAURUS_OK;
}

// Merge-on-read of [s, e) into out (device), asynchronous on `st`.
int runs_read_into(taurus_runs* r, long long s, long long e, float* out, long long ld, cudaStream_t st) {
  if (s < 0 || e > r->V || s >= e || e - s > r->max_chunk || !out || ld < r->width) return TAURUS_ERR_INVALID_ARG;
  if (r->pending) return TAURUS_ERR_ORDER;
  int rc = wait_writes(r);
  if (rc) return rc;
  struct Slice { long long off, n; };
  std::vector<Slice> slices;
  long long total = 0;
  for (long long p = s / r->range_ids; p <= (e - 1) / r->range_ids; ++p) {
    for (int f : r->by_part[(size_t)p]) {
      const RunRec& run = r->dir[(size_t)f];
      const int32_t* I = r->h_ids + run.offset;
      if (I[run.n - 1] < s || I[0] >= e) continue;
      const long long lo = std::lower_bound(I, I + run.n, (int32_t)s) - I;                            // first id >= s
      const long long hi = e > 0x7fffffffll ? run.n : std::lower_bound(I, I + run.n, (int32_t)e) - I;   // first id >= e
      if (hi > lo) { slices.push_back(Slice{run.offset + lo, hi - lo}); total += hi - lo; }
    }
  }
  if (total != e - s) return TAURUS_ERR_RUNS_INCOMPLETE;
  if (r->stage_used) RCU(cudaStreamWaitEvent(st, r->stage_free, 0));
  long long at = 0;
  const size_t w = (size_t)r->width;
  if (r->kind == TAURUS_RUNS_DEVICE && (long long)slices.size() <= r->P) {   // rows are read from the store in place
    MoveSeg *hs, *ds;
    int slot;
    { int rc2 = next_seg_slot(r, &hs, &ds, &slot); if (rc2) return rc2; }
    int nseg = 0;
    long long most = 0;
    for (const Slice& sl : slices) {
      RCU(cudaMemcpyAsync(r->d_stage_ids + at, r->h_ids + sl.off, (size_t)sl.n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
      hs[nseg++] = MoveSeg{sl.off, sl.n, at};
      at += sl.n; most = std::max(most, sl.n);
    }
    { int rc2 = push_segs(r, slot, nseg, st); if (rc2) return rc2; }
    const int gx = (int)std::max<long long>(1, std::min<long long>((most * 32 + 255) / 256, std::max<long long>(1, (long long)r->sm_count * 8 / nseg)));
    rs_place_slices_kernel<<<dim3(gx, nseg), 256, 0, st>>>(ds, r->d_stage_ids, r->store_dev, r->width, s, out, ld);
    { int rc2 = release_seg_slot(r, slot, st); if (rc2) return rc2; }
  } else {
    for (const Slice& sl : slices) {
      const float* src = r->kind == TAURUS_RUNS_HOST ? r->store_host + (size_t)sl.off * w : r->store_dev + (size_t)sl.off * w;
      RCU(cudaMemcpyAsync(r->d_stage_rows + (size_t)at * w, src, (size_t)sl.n * w * sizeof(float), cudaMemcpyDefault, st));
      RCU(cudaMemcpyAsync(r->d_stage_ids + at, r->h_ids + sl.off, (size_t)sl.n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
      at += sl.n;
    }
    const int grid = (int)std::min<long long>((total * 32 + 255) / 256, (long long)r->sm_count * 8);
    rs_place_kernel<<<grid, 256, 0, st>>>(total, r->d_stage_ids, r->d_stage_rows, r->width, s, out, ld);
  }
  r->launches += 1;
  RCU(cudaGetLastError());
  RCU(cudaEventRecord(r->stage_free, st));
  r->stage_used = true;
  return TAURUS_OK;
}

// Device-visible address of caller memory: device pointers as they are, pinned host memory through its
// mapping, pageable memory not at all.
template <class T>
static const T* device_view(const T* p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged) return p;
  if (at.type == cudaMemoryTypeHost) {
    void* d = nullptr;
    if (cudaHostGetDevicePointer(&d, const_cast<T*>(p), 0) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return static_cast<const T*>(d);
  }
  return nullptr;
}

extern "C" int taurus_runs_append(taurus_runs* r, const int64_t* ids, const float* rows, int64_t ld, int64_t count, void* cuda_stream) {
  if (!r || count < 0 || count > r->max_append || ld < r->width) return TAURUS_ERR_INVALID_ARG;
  if (count == 0) return TAURUS_OK;
  if (!ids || !rows) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  const long long* dids = device_view(reinterpret_cast<const long long*>(ids));
  const float* drows = device_view(rows);
  if (!dids || !drows) return TAURUS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  int rc = runs_phase1(r, dids, drows, ld, count, nullptr, count, st);
  if (rc) return rc;
  return runs_phase2(r, st);
}

extern "C" int taurus_runs_flush(taurus_runs* r, void* cuda_stream) {
  if (!r) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  return runs_flush_all(r, (cudaStream_t)cuda_stream);
}

extern "C" int taurus_runs_read_chunk(taurus_runs* r, int64_t src_begin, int64_t src_end, float* out_rows, int64_t ld, void* cuda_stream) {
  if (!r || !out_rows) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, out_rows) != cudaSuccess || (at.type != cudaMemoryTypeDevice && at.type != cudaMemoryTypeManaged)) {
    cudaGetLastError();
    return TAURUS_ERR_INVALID_ARG;
  }
  return runs_read_into(r, src_begin, src_end, out_rows, ld, (cudaStream_t)cuda_stream);
}

extern "C" int taurus_runs_info(taurus_runs* r, int64_t* out_runs, int64_t* out_stored_rows, int64_t* out_buffered_rows) {
  if (!r) return TAURUS_ERR_INVALID_ARG;
  if (out_runs) *out_runs = (int64_t)r->dir.size();
  if (out_stored_rows) *out_stored_rows = r->store_top;
  if (out_buffered_rows) {
    long long b = 0;
    for (long long f : r->fill) b += f;
    *out_buffered_rows = b;
  }
  return TAURUS_OK;
}

extern "C" int taurus_runs_directory(taurus_runs* r, int64_t* out, int64_t capacity_runs, int64_t* out_runs) {
  if (!r || !out_runs || capacity_runs < 0 || (capacity_runs > 0 && !out)) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  int rc = wait_writes(r);
  if (rc) return rc;
  const long long n = std::min<long long>(capacity_runs, (long long)r->dir.size());
  for (long long f = 0; f < n; ++f) {
    const RunRec& run = r->dir[(size_t)f];
    out[4 * f + 0] = run.partition;
    out[4 * f + 1] = run.n;
    out[4 * f + 2] = r->h_ids[run.offset];
    out[4 * f + 3] = r->h_ids[run.offset + run.n - 1];
  }
  *out_runs = n;
  return TAURUS_OK;
}

extern "C" int taurus_runs_get_run(taurus_runs* r, int64_t run, int64_t* out_ids, float* out_rows) {
  if (!r || run < 0 || run >= (int64_t)r->dir.size()) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  int rc = wait_writes(r);
  if (rc) return rc;
  const RunRec& rec = r->dir[(size_t)run];
  if (out_ids)
    for (long long i = 0; i < rec.n; ++i) out_ids[i] = r->h_ids[rec.offset + i];
  if (out_rows) {
    const size_t w = (size_t)r->width;
    const float* src = r->kind == TAURUS_RUNS_HOST ? r->store_host + (size_t)rec.offset * w : r->store_dev + (size_t)rec.offset * w;
    RCU(cudaMemcpy(out_rows, src, (size_t)rec.n * w * sizeof(float), cudaMemcpyDefault));
  }
  return TAURUS_OK;
}

extern "C" int taurus_runs_reset(taurus_runs* r) {
  if (!r) return TAURUS_ERR_INVALID_ARG;
  RCU(cudaSetDevice(r->device));
  RCU(cudaDeviceSynchronize());
  r->pending = false; r->dirty = false; r->stage_used = false;
  for (int i = 0; i < SEG_RING; ++i) r->seg_used[i] = false;
  r->store_top = 0;
  r->dir.clear();
  for (auto& v : r->by_part) v.clear();
  std::fill(r->fill.begin(), r->fill.end(), 0);
  return TAURUS_OK;
}
