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

static __device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

// Projected rows are read about 18 times each while the accumulator rows stream through L2 once: the reads ask L2 to
// evict their lines last (1-2 % of the scatter on the 2.45 M-vertex workload; the same hint on the reductions, evict
// first, changes nothing).
static __device__ __forceinline__ float4 ld_v4_hint(const void* addr, unsigned long long pol) {
  float4 r;
  asm volatile("ld.global.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;" : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w) : "l"(addr), "l"(pol));
  return r;
}
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
__global__ void group_split_kernel(long long n, long long chunk_begin, const int32_t* dst_sorted, const unsigned long long* vals,
                                   int2* g_edge, uint32_t* g_eid) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    unsigned long long v = vals[i];
    g_edge[i] = make_int2(dst_sorted[i], (int32_t)((long long)(v >> 32) - chunk_begin));   // (destination, source - chunk start)
    if (g_eid) g_eid[i] = (uint32_t)v;
  }
}

// In-list sources from the grouped order.  Chunks are taken in ascending order and a chunk's edges are sorted (stably)
// by destination, so the edges of one (chunk, destination) group follow the in-list entries of every earlier chunk
// in ascending source order: entry = csc_ptr[dst] + entries of earlier chunks (cursor[dst]) + rank inside the group.
__global__ void csc_fill_kernel(long long n, const int32_t* __restrict__ dst_sorted, const unsigned long long* __restrict__ vals,
                                const long long* __restrict__ csc_ptr, const int32_t* __restrict__ cursor, int32_t* __restrict__ csc_src) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const int d = dst_sorted[i];
    long long lo = 0, hi = i;   // first edge of the group
    while (lo < hi) { const long long mid = (lo + hi) >> 1; if (dst_sorted[mid] < d) lo = mid + 1; else hi = mid; }
    csc_src[csc_ptr[d] + cursor[d] + (i - lo)] = (int32_t)(vals[i] >> 32);
  }
}
__global__ void csc_advance_kernel(long long n, const int32_t* __restrict__ dst_sorted, int32_t* __restrict__ cursor) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const int d = dst_sorted[i];
    if (i + 1 < n && dst_sorted[i + 1] == d) continue;   // only the last edge of a group advances the cursor
    long long lo = 0, hi = i;
    while (lo < hi) { const long long mid = (lo + hi) >> 1; if (dst_sorted[mid] < d) lo = mid + 1; else hi = mid; }
    cursor[d] += (int32_t)(i - lo + 1);
  }
}

// g_dst, g_edge = (destination, source - chunk start) (/ g_eid): per grid chunk, the chunk's CSR edges stably
// sorted by destination.  fill_csc_src: the in-list sources csc_src are written along the way (csc_ptr is built,
// d_vtmp serves as the per-destination cursor).
int build_grouped_order(taurus_ctx* c, bool keep_edge_ids, bool fill_csc_src) {
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
  if (cudaMalloc(&c->d_gedge, (size_t)(E > 0 ? E : 1) * sizeof(int2)) != cudaSuccess) return TAURUS_ERR_NOMEM;
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
    if (fill_csc_src) cudaMemset(c->d_vtmp, 0, (size_t)V * sizeof(int32_t));
    for (long long k = 0; k < n_chunks && rc == TAURUS_OK; ++k) {
      const long long e0 = bounds[(size_t)k], ne = bounds[(size_t)k + 1] - e0;
      if (ne <= 0) continue;
      const long long s = k * cs, e = std::min(V, s + cs);
      group_values_kernel<<<c->sm_count * 4, 256>>>(s, e, c->d_row_ptr, e0, vals_in);
      size_t b = tmp_bytes;
      if (cub::DeviceRadixSort::SortPairs(tmp, b, c->d_col + e0, c->d_gdst + e0, vals_in, vals_out, ne, 0, end_bit) != cudaSuccess) { rc = TAURUS_ERR_CUDA; break; }
      group_split_kernel<<<c->sm_count * 4, 256>>>(ne, s, c->d_gdst + e0, vals_out, c->d_gedge + e0, c->d_geid ? c->d_geid + e0 : nullptr);
      if (fill_csc_src) {
        csc_fill_kernel<<<c->sm_count * 8, 256>>>(ne, c->d_gdst + e0, vals_out, c->d_csc_ptr, c->d_vtmp, c->d_csc_src);
        csc_advance_kernel<<<c->sm_count * 8, 256>>>(ne, c->d_gdst + e0, c->d_vtmp);
      }
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
// epoch stamp is touched (exact layers), and the stamp is tested before the atomic.  Every thread handles
// CG_ITEMS items per round, stage by stage (destinations, stamps, stamp updates, slot and state), so that the
// scattered per-vertex reads of a round are in flight together and the block-wide list append (two barriers and
// one round trip to a global counter) is paid once per CG_ITEMS * 256 items: the kernel is bound by that chain
// of latencies, not by bytes.
#define CG_ITEMS 4
__global__ void __launch_bounds__(256) classify_grouped_kernel(ChunkArgs a, const int32_t* __restrict__ g_dst, const uint32_t* __restrict__ gmask) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  // list appends are aggregated per block: single-address atomics are the throughput limit of this kernel
  __shared__ int s_cnt[2][2][8];   // [parity][need / touched][warp]
  __shared__ int s_base[2][2];
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long ne = e1 - e0, total = ne + (a.src_end - a.src_begin);
  const long long stride = (long long)gridDim.x * blockDim.x * CG_ITEMS;
  const int warp = threadIdx.x >> 5;
  const unsigned lt = (1u << lane_id()) - 1;
  int hs = 0, ns = 0, ev = 0, gs = 0, bad = 0, par = 0;
  for (long long base = (long long)blockIdx.x * blockDim.x * CG_ITEMS; base < total; base += stride, par ^= 1) {
    int v[CG_ITEMS];
    bool sole[CG_ITEMS];   // this item is the only one that can touch v in this chunk: no atomic needed
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q) {
      const long long i = base + q * 256 + threadIdx.x;
      v[q] = -1;
      sole[q] = false;
      if (i < ne) {
        const long long e = e0 + i;
        if (gmask == nullptr) {
          v[q] = g_dst[e];
          if (i > 0 && g_dst[e - 1] == v[q]) v[q] = -1;   // not the first edge of its destination group
          // only a vertex of the chunk's own range can also be touched by its self item
          sole[q] = v[q] < a.src_begin || v[q] >= a.src_end;
        } else if ((gmask[e >> 5] >> (e & 31)) & 1u) {
          v[q] = g_dst[e];
        }
      } else if (i < total) {
        v[q] = (int)(a.src_begin + (i - ne));
      }
      if (v[q] >= a.V) { bad = 1; v[q] = -1; }
    }
    bool stale[CG_ITEMS];   // the stamp read before any update of this round is not this chunk's
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q) stale[q] = v[q] >= 0 && (sole[q] || a.touch[v[q]] != a.epoch);
    bool first[CG_ITEMS];
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q) {
      first[q] = false;
      if (stale[q]) {
        if (sole[q]) { a.touch[v[q]] = a.epoch; first[q] = true; }
        else first[q] = atomicMax(&a.touch[v[q]], a.epoch) != a.epoch;
      }
    }
    int l[CG_ITEMS], s[CG_ITEMS];
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q)
      if (first[q]) { l[q] = a.loc[v[q]]; s[q] = a.state[v[q]]; }
    bool need[CG_ITEMS];
    unsigned mn[CG_ITEMS], mt[CG_ITEMS];
    int wn = 0, wt = 0;
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q) {
      need[q] = false;
      if (first[q]) {
        if (l[q] >= a.pool_slots) {
          gs++;
          if (s[q] == TAURUS_NOT_STARTED) a.state[v[q]] = TAURUS_ON_GPU;
        } else if (s[q] == TAURUS_IN_BUFFER) {
          hs++;
          if (a.slot_touch) a.slot_touch[l[q]] = a.epoch;
        } else if (s[q] == TAURUS_NOT_STARTED) {
          ns++; need[q] = true;
        } else if (s[q] == TAURUS_EVICTED) {
          ev++; need[q] = true;
        } else {
          bad = 1;
        }
      }
      mn[q] = __ballot_sync(FULL, need[q]);
      mt[q] = __ballot_sync(FULL, first[q]);
      wn += __popc(mn[q]);
      wt += __popc(mt[q]);
    }
    if (lane_id() == 0) { s_cnt[par][0][warp] = wn; s_cnt[par][1][warp] = wt; }
    __syncthreads();
    if (threadIdx.x < 2) {
      int sum = 0;
      for (int w = 0; w < 8; ++w) { int c = s_cnt[par][threadIdx.x][w]; s_cnt[par][threadIdx.x][w] = sum; sum += c; }
      s_base[par][threadIdx.x] = sum ? atomicAdd(threadIdx.x == 0 ? &pc->need_count : &pc->touched_count, sum) : 0;
    }
    __syncthreads();
    int on = s_base[par][0] + s_cnt[par][0][warp], ot = s_base[par][1] + s_cnt[par][1][warp];
#pragma unroll
    for (int q = 0; q < CG_ITEMS; ++q) {
      if (need[q]) {
        const int idx = on + __popc(mn[q] & lt);
        if (idx < a.pool_slots) a.need_list[idx] = v[q];
      }
      if (first[q]) {
        const int idx = ot + __popc(mt[q] & lt);
        if (idx < a.touched_capacity) a.touched_list[idx] = v[q]; else bad = 1;
      }
      on += __popc(mn[q]);
      ot += __popc(mt[q]);
    }
  }
  for (int o = 16; o; o >>= 1) {
    hs += __shfl_xor_sync(FULL, hs, o); ns += __shfl_xor_sync(FULL, ns, o);
    ev += __shfl_xor_sync(FULL, ev, o); gs += __shfl_xor_sync(FULL, gs, o);
    bad |= __shfl_xor_sync(FULL, bad, o);
  }
  if (lane_id() == 0) {
    if (hs) atomicAdd(&pc->hs, hs);
    if (ns) atomicAdd(&pc->ns, ns);
    if (ev) atomicAdd(&pc->ev, ev);
    if (gs) atomicAdd(&pc->gs, gs);
    if (bad) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
  }
}

void launch_classify_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  classify_grouped_kernel<<<c->sm_count * 8, 256, 0, st>>>(a, c->d_gdst, c->d_mask_cur ? c->d_gmask : nullptr);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ scatter (S5, S5')
// Lanes are grouped LPE to an edge (VPL float4 of the row each); sub-group `sub` of a warp walks its own
// contiguous stretch of the sorted edge list, four edges per step: the four edge records are read with
// sub-group-uniform loads (L1 hits), the four projected rows are requested together, then the rows are
// added to the running group sum or, at a destination change, the sum is flushed with one vector reduction
// per lane and one integer reduction on the pending count.  The loop body is kept to a few tens of
// instructions per edge: an earlier version with lane-parallel edge loads and shuffles was issue-bound.
#define SPAN_EDGES 128   // edges per warp span (all sub-groups together)

// With GAT every message is weighted by exp(LeakyReLU(s_u + t_v) - max_v), recomputed from per-vertex scalars
// (the 1 / normaliser factor is applied at finalise).
// GAT: 0 no attention, 1 one head (one weight per message), 2 several heads (each lane weights its float4 columns by the
// coefficient of the head they belong to; the per-vertex scalars are [V x heads]).
template <int LPE, int VPL, bool SAMPLED, bool DIRECT, int GAT>
__global__ void __launch_bounds__(256, (VPL <= 2 ? 3 : VPL == 3 ? 2 : 1))
scatter_grouped_kernel(ChunkArgs a, const int2* __restrict__ g_edge, const uint32_t* __restrict__ gmask) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  constexpr int EPS = 32 / LPE;                 // sub-groups per warp
  constexpr int STRETCH = SPAN_EDGES / EPS;     // edges one sub-group walks per span
  const int lane = lane_id();
  const int sub = lane / LPE;
  const int c4 = lane % LPE;
  const int nvec = a.Hp >> 2;
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long n_src = a.src_end - a.src_begin;
  const long long spans = (e1 - e0 + SPAN_EDGES - 1) / SPAN_EDGES;
  const long long self_tiles = (n_src + 31) >> 5;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int loc_limit = (int)(a.pool_slots + a.hub_count);
  const int pool = (int)a.pool_slots;
  const int ld4 = a.ldpt >> 2;                  // row pitch of the projected rows in float4
  const float4* __restrict__ Pbase = reinterpret_cast<const float4*>(a.PT) + c4;
  unsigned msgs = 0, hub_msgs = 0, groups = 0;
  int bad = 0;

  int cur = -1, cnt = 0, cur_loc = -1;
  float2 cur_tm = make_float2(0.f, 0.f);
  float2 head_tm[VPL];     // several heads: (t, maximum score) of the current destination for the head of each float4 of this lane
  int hk[VPL];             //                head of each float4 of this lane
#pragma unroll
  for (int k = 0; k < VPL; ++k) { hk[k] = GAT == 2 ? (c4 + k * LPE) / a.head_vec : 0; if (hk[k] >= a.heads) hk[k] = a.heads - 1; head_tm[k] = make_float2(0.f, 0.f); }
  const float* const att_s_chunk = GAT ? a.att_s + (size_t)a.src_begin * (GAT == 2 ? a.heads : 1) : nullptr;
  float4 sum[VPL];
  // byte addressing with 32-bit x 32-bit -> 64-bit products keeps the address arithmetic to one instruction
  const char* const Pb = reinterpret_cast<const char*>(a.PT) + c4 * 16;
  char* const Ab = reinterpret_cast<char*>(a.acc) + c4 * 16;
  const unsigned p_pitch = (unsigned)a.ldpt * 4u, a_pitch = (unsigned)a.Hp * 4u;
  bool lane_on[VPL];
#pragma unroll
  for (int k = 0; k < VPL; ++k) lane_on[k] = c4 + k * LPE < nvec;

  unsigned long long pol_last;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol_last));
  auto flush = [&]() {
    const int l = DIRECT ? cur : cur_loc;
    if (!DIRECT && ((unsigned)l >= (unsigned)loc_limit)) { bad = 1; return; }
    char* dst = Ab + (unsigned long long)(unsigned)l * a_pitch;
#pragma unroll
    for (int k = 0; k < VPL; ++k)
      if (lane_on[k]) red_add_v4(reinterpret_cast<float*>(dst + k * LPE * 16), sum[k]);
    if (c4 == 0) atomicAdd(&a.pend[cur], -cnt);   // result unused: a reduction; completion is read after the kernel
    msgs += (unsigned)cnt;                          // counted by every lane; only lane c4 == 0 of each sub-group reports
    groups += 1;
    if (!DIRECT && l >= pool) hub_msgs += (unsigned)cnt;
  };
  auto weight = [&](int src_rel) {   // GAT: exp(LeakyReLU(s_u + t_v) - max_v) for the current destination
    const float e = att_s_chunk[src_rel] + cur_tm.x;
    return __expf((e > 0.f ? e : a.leaky * e) - cur_tm.y);
  };
  auto weight_of_head = [&](int src_rel, int k) {   // the same for the head of this lane's k-th float4
    const float e = att_s_chunk[(size_t)src_rel * a.heads + hk[k]] + head_tm[k].x;
    return __expf((e > 0.f ? e : a.leaky * e) - head_tm[k].y);
  };
  auto take = [&](int d, int src_rel, const float4 (&row)[VPL]) {
    if (d != cur) {
      if (cur >= 0) flush();
      cur = d; cnt = 1;
      if (!DIRECT) cur_loc = a.loc[d];
      if (GAT == 2) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          head_tm[k] = a.att_tm[(size_t)d * a.heads + hk[k]];
          const float w = weight_of_head(src_rel, k);
          sum[k] = make_float4(w * row[k].x, w * row[k].y, w * row[k].z, w * row[k].w);
        }
      } else if (GAT) {
        cur_tm = a.att_tm[d];
        const float w = weight(src_rel);
#pragma unroll
        for (int k = 0; k < VPL; ++k) sum[k] = make_float4(w * row[k].x, w * row[k].y, w * row[k].z, w * row[k].w);
      } else {
#pragma unroll
        for (int k = 0; k < VPL; ++k) sum[k] = row[k];
      }
    } else {
      cnt++;
      if (GAT == 2) {
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          const float w = weight_of_head(src_rel, k);
          sum[k].x = fmaf(w, row[k].x, sum[k].x); sum[k].y = fmaf(w, row[k].y, sum[k].y);
          sum[k].z = fmaf(w, row[k].z, sum[k].z); sum[k].w = fmaf(w, row[k].w, sum[k].w);
        }
      } else if (GAT) {
        const float w = weight(src_rel);
#pragma unroll
        for (int k = 0; k < VPL; ++k) {
          sum[k].x = fmaf(w, row[k].x, sum[k].x); sum[k].y = fmaf(w, row[k].y, sum[k].y);
          sum[k].z = fmaf(w, row[k].z, sum[k].z); sum[k].w = fmaf(w, row[k].w, sum[k].w);
        }
      } else {
#pragma unroll
        for (int k = 0; k < VPL; ++k) { sum[k].x += row[k].x; sum[k].y += row[k].y; sum[k].z += row[k].z; sum[k].w += row[k].w; }
      }
    }
  };
  auto fetch = [&](int src_rel, float4 (&row)[VPL]) {
    const char* p = Pb + (unsigned long long)(unsigned)src_rel * p_pitch;
#pragma unroll
    for (int k = 0; k < VPL; ++k)
      if (lane_on[k]) row[k] = ld_v4_hint(p + k * LPE * 16, pol_last);
  };

  // Where row transfers of the previous chunk may be running beside this kernel (bounded pool), spans are handed out
  // from a counter rather than by warp number: SMs that also host transfer warps get through fewer of them (measured on
  // "large": scatter 105 -> 34 ms per 32-chunk window).  A span is requested only when the warp is ready for it: a chunk
  // has about two spans per warp there, and a warp that asked ahead would sit on a span while it is slow.  Elsewhere the
  // spans are dealt by warp number: same-address atomics cost about 3 ns each, 75 us per launch at the 25 k spans of a
  // "mid" chunk.
  const bool dyn = a.dynamic_spans != 0;
  for (long long it = 0;; ++it) {
    long long span = warp0 + it * warps;
    if (dyn) {
      unsigned int got = 0;
      if (lane == 0) got = atomicAdd(&pc->span_next, 1u);
      span = (long long)__shfl_sync(FULL, got, 0);
    }
    if (span >= spans) break;
    long long x = e0 + span * SPAN_EDGES + (long long)sub * STRETCH;
    const long long x_end = (x + STRETCH < e1) ? x + STRETCH : e1;
    const int2* ge = g_edge + x;
    int left = x_end > x ? (int)(x_end - x) : 0;
#pragma unroll 1
    for (; left >= 4; left -= 4, ge += 4, x += 4) {   // fast path: four edges per step, all rows requested together
      int2 ed[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) ed[q] = ge[q];
      if (SAMPLED) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (!((gmask[(x + q) >> 5] >> ((x + q) & 31)) & 1u)) ed[q].x = -1;
      }
      float4 row[4][VPL];
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (!SAMPLED || ed[q].x >= 0) fetch(ed[q].y, row[q]);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        if (!SAMPLED || ed[q].x >= 0) take(ed[q].x, ed[q].y, row[q]);
    }
#pragma unroll 1
    for (; left > 0; --left, ++ge, ++x) {             // ragged end of the chunk's list
      int2 ed = ge[0];
      if (SAMPLED && !((gmask[x >> 5] >> (x & 31)) & 1u)) continue;
      float4 row[VPL];
      fetch(ed.y, row);
      take(ed.x, ed.y, row);
    }
    if (cur >= 0) flush();   // a group that continues in another stretch is flushed by both
    cur = -1;
  }
  if (c4 != 0) { msgs = 0; hub_msgs = 0; groups = 0; }

  // self messages (one per chunk vertex)
  for (long long it = 0;; ++it) {
    long long t = warp0 + it * warps;
    if (dyn) {
      unsigned int got = 0;
      if (lane == 0) got = atomicAdd(&pc->self_next, 1u);
      t = (long long)__shfl_sync(FULL, got, 0);
    }
    if (t >= self_tiles) break;
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
      if (lj < 0 || !a.self_rows) continue;   // aggregate-first SAGE: the self message is only counted here
      const float* p = a.PT + (size_t)(vj - a.src_begin) * a.ldpt;
      float* dst = a.acc + (size_t)lj * a.Hp;
      if (a.mode == TAURUS_SAGE_MEAN) {
        p += a.Hp;
#pragma unroll
        for (int k = 0; k < VPL; ++k)
          if (c4 + k * LPE < nvec) red_add_v4(dst + 4 * (c4 + k * LPE), reinterpret_cast<const float4*>(p)[c4 + k * LPE]);
      } else {
        // one shared weight: GCN  P_v + b * sqrt(din(v) + 1);  GIN  (1 + eps) * P_v + b;
        // GAT  exp(e_vv - max_v) * h'_v + b * normaliser(v)
        float ps = 1.0f, sc = 1.0f;
        if (a.mode == TAURUS_GIN_SUM) ps = a.gin_self;
        else if (a.mode == TAURUS_GCN_SYM) sc = (float)sqrt((double)a.din[vj] + 1.0);
        else if (GAT != 2) {
          const float2 tm = a.att_tm[vj];
          const float e = a.att_s[vj] + tm.x;
          ps = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
          sc = (float)a.att_z[vj];
        }
        if (!a.self_bias) sc = 0.f;             // aggregate-first: the bias is added after the transform
#pragma unroll
        for (int k = 0; k < VPL; ++k)
          if (c4 + k * LPE < nvec) {
            if (GAT == 2) {                     // the head of these columns
              const size_t at = (size_t)vj * a.heads + hk[k];
              const float2 tm = a.att_tm[at];
              const float e = a.att_s[at] + tm.x;
              ps = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
              sc = a.self_bias ? (float)a.att_z[at] : 0.f;
            }
            float4 xx = reinterpret_cast<const float4*>(p)[c4 + k * LPE];
            float4 b = reinterpret_cast<const float4*>(a.bias)[c4 + k * LPE];
            red_add_v4(dst + 4 * (c4 + k * LPE), make_float4(xx.x * ps + b.x * sc, xx.y * ps + b.y * sc, xx.z * ps + b.z * sc, xx.w * ps + b.w * sc));
          }
      }
    }
  }

  for (int o = 16; o; o >>= 1) {
    msgs += __shfl_xor_sync(FULL, msgs, o);
    hub_msgs += __shfl_xor_sync(FULL, hub_msgs, o);
    groups += __shfl_xor_sync(FULL, groups, o);
    bad |= __shfl_xor_sync(FULL, bad, o);
  }
  if (lane == 0) {
    if (groups) atomicAdd((unsigned long long*)&ctl->scatter_groups, (unsigned long long)groups);
    if (msgs) atomicAdd((unsigned long long*)&ctl->total_messages, (unsigned long long)msgs);
    if (hub_msgs) atomicAdd((unsigned long long*)&ctl->hub_messages, (unsigned long long)hub_msgs);
    if (bad) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
  }
}

template <int LPE, int VPL, bool SAMPLED, bool DIRECT, int GAT>
static void launch_sg(taurus_ctx* c, const ChunkArgs& a, const uint32_t* gm, cudaStream_t st) {
  static int blocks_per_sm = 0;
  if (blocks_per_sm == 0) {
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks_per_sm, scatter_grouped_kernel<LPE, VPL, SAMPLED, DIRECT, GAT>, 256, 0) != cudaSuccess ||
        blocks_per_sm < 1)
      blocks_per_sm = 1;
  }
  scatter_grouped_kernel<LPE, VPL, SAMPLED, DIRECT, GAT><<<c->sm_count * blocks_per_sm, 256, 0, st>>>(a, c->d_gedge, gm);
}

template <int LPE, int VPL>
static void launch_sg2(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  const uint32_t* gm = c->d_mask_cur ? c->d_gmask : nullptr;
  const bool direct = a.direct && c->hub_count == 0;
  if (a.mode == TAURUS_GAT && a.heads > 1) {   // attention-weighted, one coefficient per head
    if (gm) { if (direct) launch_sg<LPE, VPL, true, true, 2>(c, a, gm, st); else launch_sg<LPE, VPL, true, false, 2>(c, a, gm, st); }
    else    { if (direct) launch_sg<LPE, VPL, false, true, 2>(c, a, gm, st); else launch_sg<LPE, VPL, false, false, 2>(c, a, gm, st); }
    return;
  }
  if (a.mode == TAURUS_GAT) {   // attention-weighted variants
    if (gm) { if (direct) launch_sg<LPE, VPL, true, true, 1>(c, a, gm, st); else launch_sg<LPE, VPL, true, false, 1>(c, a, gm, st); }
    else    { if (direct) launch_sg<LPE, VPL, false, true, 1>(c, a, gm, st); else launch_sg<LPE, VPL, false, false, 1>(c, a, gm, st); }
    return;
  }
  if (gm) { if (direct) launch_sg<LPE, VPL, true, true, 0>(c, a, gm, st); else launch_sg<LPE, VPL, true, false, 0>(c, a, gm, st); }
  else    { if (direct) launch_sg<LPE, VPL, false, true, 0>(c, a, gm, st); else launch_sg<LPE, VPL, false, false, 0>(c, a, gm, st); }
}

void launch_scatter_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  const int Hp = a.Hp;
  if (Hp <= 16) launch_sg2<4, 1>(c, a, st);
  else if (Hp <= 32) launch_sg2<8, 1>(c, a, st);
  else if (Hp <= 48) launch_sg2<4, 3>(c, a, st);     // 12 float4: four lanes x three, no idle lanes
  else if (Hp <= 64) launch_sg2<16, 1>(c, a, st);
  else if (Hp <= 112) launch_sg2<16, 2>(c, a, st);   // up to 28 float4: sixteen lanes x two leave fewer lanes idle than thirty-two x one
  else if (Hp <= 128) launch_sg2<32, 1>(c, a, st);
  else if (Hp <= 256) launch_sg2<32, 2>(c, a, st);
  else if (Hp <= 512) launch_sg2<32, 4>(c, a, st);
  else launch_sg2<32, 8>(c, a, st);
  c->launches += 1;
}
