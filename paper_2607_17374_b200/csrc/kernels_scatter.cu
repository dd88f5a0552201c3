// Scatter step (S5, S5'): push each projected source row along the chunk's propagated CSR out-edges into
// the destination's accumulator row with vector fp32 reductions and count down the destination's pending
// messages with integer reductions (no atomic returns a value; completed destinations are compacted by the
// next kernel)
// (Sect. 3.1 broadcast; Sect. 3.4 pending counts; Sect. 3.6 graduation trigger).
//
// Work is cut by EDGES, not by sources: a warp owns a run of consecutive 32-edge tiles of the chunk's CSR
// slice, so a source with a huge out-degree is simply many tiles ("a slice of a hub") and load balance
// does not depend on the degree distribution.  Lanes are grouped LPE to an edge; each lane holds VPL
// float4 of the source's projected row and keeps them while consecutive edges share the source.
// The accumulator row is updated with red.global.add.v4.f32 (16 B per lane, 512 B contiguous per
// warp instruction).  The self message of every chunk vertex is delivered by extra tiles at the end.
#include "taurus_internal.h"

#define FULL 0xffffffffu
#define TILES_PER_RUN 8

static __device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

static __device__ __forceinline__ void red_add_v4(float* addr, const float4& v) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
               : "memory");
}

// Largest u in [lo, hi) with row_ptr[u] <= e, found by the whole warp with a 32-way search.
// Requires row_ptr[lo] <= e < row_ptr[hi].
static __device__ __forceinline__ long long warp_find_source(const long long* row_ptr, long long lo, long long hi, long long e) {
  while (hi - lo > 1) {
    long long step = (hi - lo + 31) >> 5;
    long long p = lo + lane_id() * step;
    bool ok = p < hi && row_ptr[p] <= e;
    int c = __popc(__ballot_sync(FULL, ok));   // lanes 0..c-1 hold (row_ptr is non-decreasing), c >= 1
    lo += (long long)(c - 1) * step;
    hi = (lo + step < hi) ? lo + step : hi;
  }
  return lo;
}

template <int LPE, int VPL>
__global__ void __launch_bounds__(256) scatter_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  constexpr int EPS = 32 / LPE;                 // edges handled per warp step
  const int lane = lane_id();
  const int sub = lane / LPE;                   // which edge of the step this lane works on
  const int c4 = lane % LPE;                    // first float4 column of this lane
  const int nvec = a.Hp >> 2;
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long n_src = a.src_end - a.src_begin;
  const long long edge_tiles = (e1 - e0 + 31) >> 5;
  const long long self_tiles = (n_src + 31) >> 5;
  const long long runs = (edge_tiles + TILES_PER_RUN - 1) / TILES_PER_RUN;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long loc_limit = a.pool_slots + a.hub_count;
  unsigned long long msgs = 0, hub_msgs = 0;
  int bad = 0;

  for (long long run = warp0; run < runs + self_tiles; run += warps) {
    const bool self_run = run >= runs;
    long long t_begin, t_end;
    long long u0 = 0;
    if (!self_run) {
      t_begin = run * TILES_PER_RUN;
      t_end = t_begin + TILES_PER_RUN < edge_tiles ? t_begin + TILES_PER_RUN : edge_tiles;
      u0 = warp_find_source(a.row_ptr, a.src_begin, a.src_end, e0 + t_begin * 32);
    } else {
      t_begin = run - runs;
      t_end = t_begin + 1;
    }
    for (long long t = t_begin; t < t_end; ++t) {
      int v = -1;        // destination handled by this lane (-1: nothing to do)
      long long src = 0; // source whose row this lane's item carries
      if (!self_run) {
        const long long e = e0 + t * 32 + lane;
        if (e < e1 && (a.mask == nullptr || ((a.mask[e >> 5] >> (e & 31)) & 1u))) v = a.col[e];
        // source of every edge of the tile: u0 + #{j : row_ptr[u0 + 1 + j] <= e}
        long long nxt = u0 + 1 + lane;
        long long r = a.row_ptr[nxt < a.src_end ? nxt : a.src_end];
        int cnt = 0;
#pragma unroll
        for (int s = 16; s; s >>= 1) {
          long long rj = __shfl_sync(FULL, r, cnt + s - 1);
          if (rj <= e) cnt += s;
        }
        long long r31 = __shfl_sync(FULL, r, 31);
        src = u0 + cnt;
        if (r31 <= e && e < e1) {   // more than 32 sources inside one tile (empty rows): plain binary search
          long long lo = u0 + 32, hi = a.src_end;
          while (hi - lo > 1) { long long mid = (lo + hi) >> 1; if (a.row_ptr[mid] <= e) lo = mid; else hi = mid; }
          src = lo;
        }
        long long last = __shfl_sync(FULL, src, 31);
        u0 = last < a.src_end - 1 ? last : a.src_end - 1;
        if (!__any_sync(FULL, v >= 0)) continue;
      } else {
        const long long u = a.src_begin + t * 32 + lane;
        if (u < a.src_end) { v = (int)u; src = u; }
      }
      // GAT: weight of this lane's message, exp(LeakyReLU(s_u + t_v) - max_v)
      float wgt = 1.f;
      const bool multi = a.mode == TAURUS_GAT && a.heads > 1;   // several heads: the weights are taken per float4 column below
      if (a.mode == TAURUS_GAT && !multi && v >= 0 && !self_run) {
        const float2 tm = a.att_tm[v];
        const float e = a.att_s[src] + tm.x;
        wgt = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
      }
      // pending count and slot of this lane's destination
      int l = -1;
      if (v >= 0) {
        l = a.loc[v];
        if (l < 0 || l >= loc_limit) { bad = 1; l = -1; }
        else {
          atomicAdd(&a.pend[v], -1);   // result unused: a reduction; completion is read after the kernel
          if (!self_run) { msgs++; if (l >= a.pool_slots) hub_msgs++; }
        }
      }
      const unsigned live = __ballot_sync(FULL, l >= 0);
      // accumulate: EPS items per step, LPE lanes per item
      float4 row[VPL];
      long long held = -1;   // source whose row is in `row`
#pragma unroll 1
      for (int step = 0; step < 32; step += EPS) {
        if (((live >> step) & ((EPS == 32) ? 0xffffffffu : ((1u << EPS) - 1u))) == 0u) continue;
        const int j = step + sub;
        const int lj = __shfl_sync(FULL, l, j);
        const long long sj = __shfl_sync(FULL, src, j);
        const float wj = __shfl_sync(FULL, wgt, j);
        const int vj = __shfl_sync(FULL, v, j);
        if (lj < 0) continue;
        if (self_run && !a.self_rows) continue;   // aggregate-first SAGE: the self message is only counted
        if (sj != held) {
          held = sj;
          const float* p = a.PT + (size_t)(sj - a.src_begin) * a.ldpt;
          if (self_run) {
            if (a.mode == TAURUS_SAGE_MEAN) {
              p += a.Hp;   // T columns
#pragma unroll
              for (int k = 0; k < VPL; ++k)
                if (c4 + k * LPE < nvec) row[k] = reinterpret_cast<const float4*>(p)[c4 + k * LPE];
            } else {       // one shared weight: the self message is built from the vertex's own P row
              // GCN: P_v (already scaled by c_out(v)) + b * sqrt(din(v) + 1);  GIN: (1 + eps) * P_v + b;
              // GAT: exp(e_vv - max_v) * h'_v + b * normaliser(v)
              float ps = 1.0f, s = 1.0f;
              if (a.mode == TAURUS_GIN_SUM) ps = a.gin_self;
              else if (a.mode == TAURUS_GCN_SYM) s = (float)sqrt((double)a.din[sj] + 1.0);
              else if (!multi) {
                const float2 tm = a.att_tm[sj];
                const float e = a.att_s[sj] + tm.x;
                ps = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
                s = (float)a.att_z[sj];
              }
              if (!a.self_bias) s = 0.f;          // aggregate-first: the bias is added after the transform
#pragma unroll
              for (int k = 0; k < VPL; ++k)
                if (c4 + k * LPE < nvec) {
                  if (multi) {                    // the head of these columns
                    const size_t at = (size_t)sj * a.heads + (c4 + k * LPE) / a.head_vec;
                    const float2 tm = a.att_tm[at];
                    const float e = a.att_s[at] + tm.x;
                    ps = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
                    s = a.self_bias ? (float)a.att_z[at] : 0.f;
                  }
                  float4 x = reinterpret_cast<const float4*>(p)[c4 + k * LPE];
                  float4 b = reinterpret_cast<const float4*>(a.bias)[c4 + k * LPE];
                  row[k] = make_float4(x.x * ps + b.x * s, x.y * ps + b.y * s, x.z * ps + b.z * s, x.w * ps + b.w * s);
                }
            }
          } else {
#pragma unroll
            for (int k = 0; k < VPL; ++k)
              if (c4 + k * LPE < nvec) row[k] = reinterpret_cast<const float4*>(p)[c4 + k * LPE];
          }
        }
        float* dst = a.acc + (size_t)lj * a.Hp;
        if (multi && !self_run) {
#pragma unroll
          for (int k = 0; k < VPL; ++k)
            if (c4 + k * LPE < nvec) {
              const int hd = (c4 + k * LPE) / a.head_vec;
              const float2 tm = a.att_tm[(size_t)vj * a.heads + hd];
              const float e = a.att_s[(size_t)sj * a.heads + hd] + tm.x;
              const float wk = __expf((e > 0.f ? e : a.leaky * e) - tm.y);
              red_add_v4(dst + 4 * (c4 + k * LPE), make_float4(row[k].x * wk, row[k].y * wk, row[k].z * wk, row[k].w * wk));
            }
        } else if (a.mode == TAURUS_GAT && !self_run) {
#pragma unroll
          for (int k = 0; k < VPL; ++k)
            if (c4 + k * LPE < nvec)
              red_add_v4(dst + 4 * (c4 + k * LPE), make_float4(row[k].x * wj, row[k].y * wj, row[k].z * wj, row[k].w * wj));
        } else {
#pragma unroll
          for (int k = 0; k < VPL; ++k)
            if (c4 + k * LPE < nvec) red_add_v4(dst + 4 * (c4 + k * LPE), row[k]);
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
    if (msgs) { atomicAdd((unsigned long long*)&ctl->total_messages, msgs); atomicAdd((unsigned long long*)&ctl->scatter_groups, msgs); }
    if (hub_msgs) atomicAdd((unsigned long long*)&ctl->hub_messages, hub_msgs);
    if (bad) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
  }
}

void launch_scatter(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  const int blocks = c->sm_count * 8;
  const int Hp = a.Hp;
  if (Hp <= 16) scatter_kernel<4, 1><<<blocks, 256, 0, st>>>(a);
  else if (Hp <= 32) scatter_kernel<8, 1><<<blocks, 256, 0, st>>>(a);
  else if (Hp <= 64) scatter_kernel<16, 1><<<blocks, 256, 0, st>>>(a);
  else if (Hp <= 128) scatter_kernel<32, 1><<<blocks, 256, 0, st>>>(a);
  else if (Hp <= 256) scatter_kernel<32, 2><<<blocks, 256, 0, st>>>(a);
  else if (Hp <= 512) scatter_kernel<32, 4><<<blocks, 256, 0, st>>>(a);
  else scatter_kernel<32, 8><<<blocks, 256, 0, st>>>(a);
  c->launches += 1;
}
