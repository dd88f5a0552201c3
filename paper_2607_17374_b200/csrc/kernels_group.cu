// Destination-grouped scatter for grid-aligned chunks.
//
// The broadcast step delivers one message per propagated edge (Sect. 3.1, 3.4).  When a chunk is one cell of
// the fixed chunk grid (sources [k * chunk_sources, (k+1) * chunk_sources)), its edges are known at init, so
// they are stored a second time sorted by destination inside each chunk ("grouped order": destination, source
// and, for sampled layers, the CSR edge index).  A warp then walks a span of that list, sums the projected
// rows of consecutive edges with the same destination in registers (the rows of one chunk fit in L2), and
// issues ONE vector reduction and ONE pending-count decrement per (chunk, destination) group instead of one
// per edge.  The messages, their sum and the counts are the same as in the edge-by-edge kernel; only the
// number of read-modify-writes of accumulator rows in HBM drops (by the mean group size, 2.7 on the "mid"
// workload).  Chunks that are not grid cells use the CSR-order kernels.
#include <cub/cub.cuh>

#include "taurus_internal.h"

#define FULL 0xffffffffu
#define SPAN_TILES 4   // 32-edge tiles per warp span

static __device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

static __device__ __forceinline__ void red_add_v4(float* addr, const float4& v) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}

// ------------------------------------------------------------------------------------------------ build (init)
__global__ void group_values_kernel(long long s, long long e, const long long* row_ptr, long long e0, unsigned long long* vals) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = s + (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5); u < e; u += warps) {
    long long b = row_ptr[u], t = row_ptr[u + 1];
    for (long long k = b + lane_id(); k < t; k += 32) vals[k - e0] = ((unsigned long long)u << 32) | (unsigned long long)k;
  }
}
__global__ void group_split_kernel(long long n, const unsigned long long* vals, int32_t* g_src, uint32_t* g_eid) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    unsigned long long v = vals[i];
    g_src[i] = (int32_t)(v >> 32);
    if (g_eid) g_eid[i] = (uint32_t)v;
  }
}

// g_dst / g_src (/ g_eid): per grid chunk, the chunk's CSR edges stably sorted by destination.
int build_grouped_order(taurus_ctx* c, bool keep_edge_ids) {
  const long long V = c->V, E = c->E, cs = c->chunk_sources;
  const long long n_chunks = (V + cs - 1) / cs;
  std::vector<long long> bounds((size_t)n_chunks + 1);
  {
    std::vector<long long> idx((size_t)n_chunks + 1);
    for (long long k = 0; k <= n_chunks; ++k) idx[(size_t)k] = std::min(V, k * cs);
    // row_ptr at the chunk boundaries
    for (long long k = 0; k <= n_chunks; ++k)
      if (cudaMemcpy(&bounds[(size_t)k], c->d_row_ptr + idx[(size_t)k], sizeof(long long), cudaMemcpyDeviceToHost) != cudaSuccess)
        return TAURUS_ERR_CUDA;
  }
  long long max_edges = 1;
  for (long long k = 0; k < n_chunks; ++k) max_edges = std::max(max_edges, bounds[(size_t)k + 1] - bounds[(size_t)k]);
  if (cudaMalloc(&c->d_gdst, (size_t)(E > 0 ? E : 1) * sizeof(int32_t)) != cudaSuccess) return TAURUS_ERR_NOMEM;
  if (cudaMalloc(&c->d_gsrc, (size_t)(E > 0 ? E : 1) * sizeof(int32_t)) != cudaSuccess) return TAURUS_ERR_NOMEM;
  if (keep_edge_ids && cudaMalloc(&c->d_geid, (size_t)(E > 0 ? E : 1) * sizeof(uint32_t)) != cudaSuccess) return TAURUS_ERR_NOMEM;
  unsigned long long *vals_in = nullptr, *vals_out = nullptr;
  void* tmp = nullptr;
  size_t tmp_bytes = 0;
  int rc = TAURUS_OK;
  int end_bit = 1;
  while (end_bit < 31 && (1ll << end_bit) < V) ++end_bit;
  do {
    if (cudaMalloc(&vals_in, (size_t)max_edges * 8) != cudaSuccess || cudaMalloc(&vals_out, (size_t)max_edges * 8) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    cub::DeviceRadixSort::SortPairs(nullptr, tmp_bytes, c->d_col, c->d_gdst, vals_in, vals_out, max_edges, 0, end_bit);
    if (cudaMalloc(&tmp, tmp_bytes > 0 ? tmp_bytes : 16) != cudaSuccess) { rc = TAURUS_ERR_NOMEM; break; }
    for (long long k = 0; k < n_chunks && rc == TAURUS_OK; ++k) {
      const long long e0 = bounds[(size_t)k], ne = bounds[(size_t)k + 1] - e0;
      if (ne <= 0) continue;
      const long long s = k * cs, e = std::min(V, s + cs);
      group_values_kernel<<<c->sm_count * 4, 256>>>(s, e, c->d_row_ptr, e0, vals_in);
      size_t b = tmp_bytes;
      if (cub::DeviceRadixSort::SortPairs(tmp, b, c->d_col + e0, c->d_gdst + e0, vals_in, vals_out, ne, 0, end_bit) != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
      group_split_kernel<<<c->sm_count * 4, 256>>>(ne, vals_out, c->d_gsrc + e0, c->d_geid ? c->d_geid + e0 : nullptr);
    }
    if (rc == TAURUS_OK && cudaDeviceSynchronize() != cudaSuccess) rc = TAURUS_ERR_CUDA;
  } while (0);
  cudaFree(vals_in); cudaFree(vals_out); cudaFree(tmp);
  c->launches += 2 * n_chunks;
  return rc;
}

// Edge mask of a sampled layer in grouped order: bit i of gmask = mask bit of CSR edge g_eid[i].
__global__ void group_mask_kernel(long long E, const uint32_t* g_eid, const uint32_t* mask, uint32_t* gmask) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long words = (E + 31) >> 5;
  for (long long w = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; w < words; w += warps) {
    long long i = w * 32 + lane_id();
    bool bit = false;
    if (i < E) { uint32_t e = g_eid[i]; bit = (mask[e >> 5] >> (e & 31)) & 1u; }
    unsigned m = __ballot_sync(FULL, bit);
    if (lane_id() == 0) gmask[w] = m;
  }
}

void launch_group_mask(taurus_ctx* c, cudaStream_t st) {
  group_mask_kernel<<<c->sm_count * 8, 256, 0, st>>>(c->E, c->d_geid, c->d_mask, c->d_gmask);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ classify (S3)
// Same decisions as the CSR-order classify; adjacent duplicates of a destination are skipped before the
// epoch stamp is touched (exact layers), and the stamp is tested before the atomic.
__global__ void __launch_bounds__(256) classify_grouped_kernel(ChunkArgs a, const int32_t* __restrict__ g_dst, const uint32_t* __restrict__ gmask) {
  DevCtl* ctl = a.ctl;
  if (ctl->error) return;
  // list appends are aggregated per block: single-address atomics are the throughput limit of this kernel
  __shared__ int s_cnt[2][2][8];   // [parity][need / touched][warp]
  __shared__ int s_base[2][2];
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long ne = e1 - e0, total = ne + (a.src_end - a.src_begin);
  const long long stride = (long long)gridDim.x * blockDim.x;
  const int warp = threadIdx.x >> 5;
  int hs = 0, ns = 0, ev = 0, gs = 0, bad = 0, par = 0;
  for (long long base = (long long)blockIdx.x * blockDim.x; base < total; base += stride, par ^= 1) {
    long long i = base + threadIdx.x;
    int v = -1;
    bool sole = false;   // this item is the only one that can touch v in this chunk: no atomic needed
    if (i < ne) {
      long long e = e0 + i;
      if (gmask == nullptr) {
        v = g_dst[e];
        if (i > 0 && g_dst[e - 1] == v) v = -1;   // not the first edge of its destination group
        // only a vertex of the chunk's own range can also be touched by its self item
        sole = v < a.src_begin || v >= a.src_end;
      } else if ((gmask[e >> 5] >> (e & 31)) & 1u) {
        v = g_dst[e];
      }
    } else if (i < total) {
      v = (int)(a.src_begin + (i - ne));
    }
    bool need = false, first = false;
    if (v >= a.V) { bad = 1; v = -1; }
    if (v >= 0 && (sole || a.touch[v] != a.epoch)) {
      int old;
      if (sole) { old = 0; a.touch[v] = a.epoch; }
      else old = atomicMax(&a.touch[v], a.epoch);
      if (old != a.epoch) {
        first = true;
        int l = a.loc[v];
        int s = a.state[v];
        if (l >= a.pool_slots) {
          gs++;
          if (s == TAURUS_NOT_STARTED) a.state[v] = TAURUS_ON_GPU;
        } else if (s == TAURUS_IN_BUFFER) {
          hs++;
        } else if (s == TAURUS_NOT_STARTED) {
          ns++; need = true;
        } else if (s == TAURUS_EVICTED) {
          ev++; need = true;
        } else {
          bad = 1;
        }
      }
    }
    const unsigned mn = __ballot_sync(FULL, need), mt = __ballot_sync(FULL, first);
    if (lane_id() == 0) { s_cnt[par][0][warp] = __popc(mn); s_cnt[par][1][warp] = __popc(mt); }
    __syncthreads();
    if (threadIdx.x < 2) {
      int sum = 0;
      for (int w = 0; w < 8; ++w) { int c = s_cnt[par][threadIdx.x][w]; s_cnt[par][threadIdx.x][w] = sum; sum += c; }
      s_base[par][threadIdx.x] = sum ? atomicAdd(threadIdx.x == 0 ? &ctl->need_count : &ctl->touched_count, sum) : 0;
    }
    __syncthreads();
    if (need) {
      int idx = s_base[par][0] + s_cnt[par][0][warp] + __popc(mn & ((1u << lane_id()) - 1));
      if (idx < a.pool_slots) a.need_list[idx] = v;
    }
    if (first) {
      int idx = s_base[par][1] + s_cnt[par][1][warp] + __popc(mt & ((1u << lane_id()) - 1));
      if (idx < a.touched_capacity) a.touched_list[idx] = v; else bad = 1;
    }
  }
  for (int o = 16; o; o >>= 1) {
    hs += __shfl_xor_sync(FULL, hs, o); ns += __shfl_xor_sync(FULL, ns, o);
    ev += __shfl_xor_sync(FULL, ev, o); gs += __shfl_xor_sync(FULL, gs, o);
    bad |= __shfl_xor_sync(FULL, bad, o);
  }
  if (lane_id() == 0) {
    if (hs) atomicAdd(&ctl->hs, hs);
    if (ns) atomicAdd(&ctl->ns, ns);
    if (ev) atomicAdd(&ctl->ev, ev);
    if (gs) atomicAdd(&ctl->gs, gs);
    if (bad) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
  }
}

void launch_classify_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  classify_grouped_kernel<<<c->sm_count * 8, 256, 0, st>>>(a, c->d_gdst, c->d_mask_cur ? c->d_gmask : nullptr);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ scatter (S5, S5', S6 head)
// Lanes are grouped LPE to an edge; sub-group `sub` of a warp walks its own part of each 32-edge tile.
template <int LPE, int VPL>
__global__ void __launch_bounds__(256) scatter_grouped_kernel(ChunkArgs a, const int32_t* __restrict__ g_dst,
                                                              const int32_t* __restrict__ g_src,
                                                              const uint32_t* __restrict__ gmask) {
  DevCtl* ctl = a.ctl;
  if (ctl->error) return;
  constexpr int EPS = 32 / LPE;                 // sub-groups per warp
  const int lane = lane_id();
  const int sub = lane / LPE;
  const int c4 = lane % LPE;
  const int nvec = a.Hp >> 2;
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long n_src = a.src_end - a.src_begin;
  const long long edge_tiles = (e1 - e0 + 31) >> 5;
  const long long spans = (edge_tiles + SPAN_TILES - 1) / SPAN_TILES;
  const long long self_tiles = (n_src + 31) >> 5;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long loc_limit = a.pool_slots + a.hub_count;
  unsigned long long msgs = 0, hub_msgs = 0;
  int bad = 0;

  // state of the group this sub-group is summing; its slot is requested when the group starts so that the
  // load has landed by the time the group is flushed
  int cur = -1, cnt = 0, cur_loc = -1;
  float4 sum[VPL];
  auto flush = [&]() {
    // all LPE lanes of the sub-group call this together with the same (cur, cnt)
    if (cur < 0) return;
    const int l = cur_loc;
    if (l < 0 || l >= loc_limit) { bad = 1; cur = -1; cnt = 0; return; }
    float* dst = a.acc + (size_t)l * a.Hp;
#pragma unroll
    for (int k = 0; k < VPL; ++k)
      if (c4 + k * LPE < nvec) red_add_v4(dst + 4 * (c4 + k * LPE), sum[k]);
    if (c4 == 0) {
      atomicAdd(&a.pend[cur], -cnt);   // result unused: a reduction; completion is read after the kernel
      msgs += (unsigned)cnt;
      if (l >= a.pool_slots) hub_msgs += (unsigned)cnt;
    }
    cur = -1; cnt = 0;
  };
  auto take = [&](int dj, int lj, const float4 (&row)[VPL]) {
    if (dj != cur) {
      flush();
      cur = dj; cnt = 1; cur_loc = lj;
#pragma unroll
      for (int k = 0; k < VPL; ++k) sum[k] = row[k];
    } else {
      cnt++;
#pragma unroll
      for (int k = 0; k < VPL; ++k) { sum[k].x += row[k].x; sum[k].y += row[k].y; sum[k].z += row[k].z; sum[k].w += row[k].w; }
    }
  };
  auto fetch = [&](int sj, float4 (&row)[VPL]) {
    const float4* p = reinterpret_cast<const float4*>(a.PT + (size_t)(sj - a.src_begin) * a.ldpt);
#pragma unroll
    for (int k = 0; k < VPL; ++k)
      if (c4 + k * LPE < nvec) row[k] = p[c4 + k * LPE];
  };

  // A warp span is SPAN_TILES * 32 consecutive edges of the sorted list; sub-group g walks its own contiguous
  // stretch of SPAN_TILES * LPE edges, LPE edges per round (loaded by its LPE lanes, one edge each).
  // The rounds of all spans of this warp form one sequence that is software-pipelined: (destination, source)
  // of round i+2 and the slots of round i+1 are requested while round i is processed.
  constexpr int STRETCH = SPAN_TILES * LPE;
  const long long my_spans = warp0 < spans ? (spans - warp0 + warps - 1) / warps : 0;
  const long long rounds = my_spans * SPAN_TILES;
  auto edge_of = [&](long long i) -> long long {   // this lane's edge in round i of the warp's sequence
    const long long span = warp0 + (i / SPAN_TILES) * warps;
    return e0 + span * (SPAN_TILES * 32) + (long long)sub * STRETCH + (i % SPAN_TILES) * LPE + c4;
  };
  auto load_ds = [&](long long i, int& d, int& sx) {
    d = -1; sx = 0;
    if (i < rounds) {
      const long long e = edge_of(i);
      if (e < e1 && (gmask == nullptr || ((gmask[e >> 5] >> (e & 31)) & 1u))) { d = g_dst[e]; sx = g_src[e]; }
    }
  };
  int d0, s0, l0, d1, s1, d2, s2;
  load_ds(0, d0, s0);
  load_ds(1, d1, s1);
  l0 = d0 >= 0 ? a.loc[d0] : -1;
#pragma unroll 1
  for (long long i = 0; i < rounds; ++i) {
    const int l1 = d1 >= 0 ? a.loc[d1] : -1;   // slots of the next round
    load_ds(i + 2, d2, s2);                     // edges of the round after that
    if (__any_sync(FULL, d0 >= 0)) {
#pragma unroll 1
      for (int j = 0; j < LPE; j += 4) {
        // four edges per step: all rows are requested before any is used
        int dd[4], ss[4], ll[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          dd[q] = __shfl_sync(FULL, d0, sub * LPE + j + q);
          ss[q] = __shfl_sync(FULL, s0, sub * LPE + j + q);
          ll[q] = __shfl_sync(FULL, l0, sub * LPE + j + q);
        }
        float4 row[4][VPL];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (dd[q] >= 0) fetch(ss[q], row[q]);
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (dd[q] >= 0) take(dd[q], ll[q], row[q]);
      }
    }
    if ((i % SPAN_TILES) == SPAN_TILES - 1) flush();   // a group that continues in another warp's span is flushed by both
    d0 = d1; s0 = s1; l0 = l1; d1 = d2; s1 = s2;
  }
  flush();

  // self messages (one per chunk vertex), as in the CSR-order kernel
  for (long long t = warp0; t < self_tiles; t += warps) {
    const long long u = a.src_begin + t * 32 + lane;
    int v = u < a.src_end ? (int)u : -1;
    int l = -1;
    if (v >= 0) {
      l = a.loc[v];
      if (l < 0 || l >= loc_limit) { bad = 1; l = -1; }
      else atomicAdd(&a.pend[v], -1);
    }
    for (int step = 0; step < 32; step += EPS) {
      const int j = step + sub;
      const int lj = __shfl_sync(FULL, l, j);
      const int vj = __shfl_sync(FULL, v, j);
      if (lj < 0) continue;
      const float* p = a.PT + (size_t)(vj - a.src_begin) * a.ldpt;
      float* dst = a.acc + (size_t)lj * a.Hp;
      if (a.mode == TAURUS_SAGE_MEAN) {
        p += a.Hp;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
          if (c4 + k * LPE < nvec) red_add_v4(dst + 4 * (c4 + k * LPE), reinterpret_cast<const float4*>(p)[c4 + k * LPE]);
      } else {
        const float sc = (float)sqrt((double)a.din[vj] + 1.0);
#pragma unroll
        for (int k = 0; k < VPL; ++k)
          if (c4 + k * LPE < nvec) {
            float4 x = reinterpret_cast<const float4*>(p)[c4 + k * LPE];
            float4 b = reinterpret_cast<const float4*>(a.bias)[c4 + k * LPE];
            red_add_v4(dst + 4 * (c4 + k * LPE), make_float4(x.x + b.x * sc, x.y + b.y * sc, x.z + b.z * sc, x.w + b.w * sc));
          }
      }
    }
  }

  for (int o = 16; o; o >>= 1) {
    msgs += __shfl_xor_sync(FULL, msgs, o);
    hub_msgs += __shfl_xor_sync(FULL, hub_msgs, o);
    bad |= __shfl_xor_sync(FULL, bad, o);
  }
  if (lane == 0) {
    if (msgs) atomicAdd((unsigned long long*)&ctl->total_messages, msgs);
    if (hub_msgs) atomicAdd((unsigned long long*)&ctl->hub_messages, hub_msgs);
    if (bad) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
  }
}

void launch_scatter_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  const int blocks = c->sm_count * 8;
  const int Hp = a.Hp;
  const uint32_t* gm = c->d_mask_cur ? c->d_gmask : nullptr;
  if (Hp <= 16) scatter_grouped_kernel<4, 1><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else if (Hp <= 32) scatter_grouped_kernel<8, 1><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else if (Hp <= 64) scatter_grouped_kernel<16, 1><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else if (Hp <= 128) scatter_grouped_kernel<32, 1><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else if (Hp <= 256) scatter_grouped_kernel<32, 2><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else if (Hp <= 512) scatter_grouped_kernel<32, 4><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  else scatter_grouped_kernel<32, 8><<<blocks, 256, 0, st>>>(a, c->d_gdst, c->d_gsrc, gm);
  c->launches += 1;
}
