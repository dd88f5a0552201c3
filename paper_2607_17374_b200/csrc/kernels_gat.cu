// GATConv passes 1 and 2 (GATConv paragraph of Sect. 3.9).
//
// Pass 1 is the projection kernel with two extra weight columns, W att_src and W att_dst, so that the scalars
// s_u = att_src . h'_u and t_u = att_dst . h'_u fall out of the same GEMM; gat_split_kernel files the rows
// h' and the scalars away.  Pass 2 is topology-only: because LeakyReLU is non-decreasing, the maximum score
// of destination v is LeakyReLU(max_u s_u + t_v), so one sweep over the CSR takes a running maximum of s_u per
// destination and a second sweep sums exp(e_uv - max) into the normaliser; both use scalar atomics on
// V-sized arrays and read no feature row.  Nothing per edge is stored: pass 3 recomputes
// exp(LeakyReLU(s_u + t_v) - max_v) where it adds the message and divides by the normaliser at finalise.
#include "taurus_internal.h"

namespace {

__device__ __forceinline__ int gl() { return threadIdx.x & 31; }
__device__ __forceinline__ float lrelu(float x, float slope) { return x > 0.f ? x : slope * x; }

// Order-preserving atomic maximum for finite floats of either sign.
__device__ __forceinline__ void atomic_max_float(float* addr, float v) {
  v += 0.f;   // -0 -> +0, whose bit pattern orders correctly among the non-negative values
  if (v >= 0.f) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
  else atomicMin(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

// The per-vertex scalars are stored [V x heads]: head h of vertex v at v * heads + h.
__global__ void gat_split_kernel(const float* __restrict__ PT, int ldpt, int n, int Hp, int d_out, int heads, long long src_begin,
                                 float* __restrict__ hprime, long long ld, float* __restrict__ att_s, float* __restrict__ att_t,
                                 float* __restrict__ att_max) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    const float* src = PT + (size_t)r * ldpt;
    float* dst = hprime + (size_t)r * ld;
    for (int k = gl(); k < d_out; k += 32) dst[k] = src[k];
    if (gl() < heads) {
      const float s = src[Hp + 2 * gl()], t = src[Hp + 2 * gl() + 1];
      const size_t at = (size_t)(src_begin + r) * heads + gl();
      att_s[at] = s;
      att_t[at] = t;
      att_max[at] = s;   // the self message takes part in the maximum
    }
  }
}

// max over propagated in-edges (u -> v) of s_u, one warp per source row
template <bool ONE>   // ONE: a single head, the source's scalar is read once per row
__global__ void gat_edge_max_kernel(long long V, int heads, const long long* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                    const uint32_t* __restrict__ mask, const float* __restrict__ att_s, float* __restrict__ att_max) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    const float s1 = ONE ? att_s[u] : 0.f;
    for (long long e = row_ptr[u] + gl(); e < row_ptr[u + 1]; e += 32)
      if (!mask || ((mask[e >> 5] >> (e & 31)) & 1u)) {
        if (ONE) { atomic_max_float(&att_max[col[e]], s1); continue; }
        const size_t v = (size_t)col[e] * heads;
        for (int h = 0; h < heads; ++h) atomic_max_float(&att_max[v + h], att_s[(size_t)u * heads + h]);
      }
  }
}

// tm[v] = (t_v, LeakyReLU(max_u s_u + t_v));  z[v] starts with the self term
__global__ void gat_tm_kernel(long long V, const float* __restrict__ att_s, const float* __restrict__ att_t,
                              const float* __restrict__ att_max, float slope, float2* __restrict__ tm, double* __restrict__ z) {   // V = vertices x heads
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) {
    const float t = att_t[v];
    const float m = lrelu(att_max[v] + t, slope);
    tm[v] = make_float2(t, m);
    z[v] = (double)__expf(lrelu(att_s[v] + t, slope) - m);
  }
}

template <bool ONE>
__global__ void gat_edge_sum_kernel(long long V, int heads, const long long* __restrict__ row_ptr, const int32_t* __restrict__ col,
                                    const uint32_t* __restrict__ mask, const float* __restrict__ att_s,
                                    const float2* __restrict__ tm, float slope, double* __restrict__ z) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    const float s1 = ONE ? att_s[u] : 0.f;
    for (long long e = row_ptr[u] + gl(); e < row_ptr[u + 1]; e += 32)
      if (!mask || ((mask[e >> 5] >> (e & 31)) & 1u)) {
        if (ONE) {
          const int v1 = col[e];
          const float2 x = tm[v1];
          atomicAdd(&z[v1], (double)__expf(lrelu(s1 + x.x, slope) - x.y));
          continue;
        }
        const size_t v = (size_t)col[e] * heads;
        for (int h = 0; h < heads; ++h) {
          const float2 x = tm[v + h];
          atomicAdd(&z[v + h], (double)__expf(lrelu(att_s[(size_t)u * heads + h] + x.x, slope) - x.y));
        }
      }
  }
}

// Aggregate-first GAT layers: the scores need only s_u = h_u . (W att_src) and t_u = h_u . (W att_dst), so pass 1 is
// two dot products per row; the (zero-padded) input rows are handed back to the caller for pass 3 in place of the
// transformed rows.
__global__ void gat_scores_kernel(const float* __restrict__ X, int ldx, int n, int K, const float* __restrict__ ws,
                                  const float* __restrict__ wd, long long src_begin, float* __restrict__ rows_out, long long ld,
                                  int d_out, float* __restrict__ att_s, float* __restrict__ att_t, float* __restrict__ att_max) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    const float* x = X + (size_t)r * ldx;
    float* o = rows_out + (size_t)r * ld;
    float s = 0.f, t = 0.f;
    for (int k = gl(); k < d_out; k += 32) {
      const float v = k < K ? x[k] : 0.f;
      if (k < K) { s = fmaf(v, ws[k], s); t = fmaf(v, wd[k], t); }
      o[k] = v;
    }
    for (int off = 16; off; off >>= 1) { s += __shfl_xor_sync(0xffffffffu, s, off); t += __shfl_xor_sync(0xffffffffu, t, off); }
    if (gl() == 0) {
      att_s[src_begin + r] = s;
      att_t[src_begin + r] = t;
      att_max[src_begin + r] = s;
    }
  }
}

__global__ void gat_repack_kernel(const float* __restrict__ X, int n, int d_out, int Hp, float* __restrict__ PT) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps)
    for (int k = gl(); k < Hp; k += 32) PT[(size_t)r * Hp + k] = k < d_out ? X[(size_t)r * d_out + k] : 0.f;
}

}  // namespace

void launch_gat_split(taurus_ctx* c, int n, int Hp, int d_out, long long src_begin, float* hprime_out, long long ld, cudaStream_t st) {
  gat_split_kernel<<<c->sm_count * 8, 256, 0, st>>>(c->d_PT, taurus_proj_width(TAURUS_GAT, Hp, c->heads), n, Hp, d_out, c->heads, src_begin,
                                                    hprime_out, ld, c->d_att_s, c->d_att_t, c->d_att_max);
  c->launches += 1;
}

void launch_gat_scores(taurus_ctx* c, int layer, const float* X, int ldx, int n, long long src_begin, float* rows_out, long long ld,
                       cudaStream_t st) {
  const int K = c->dims[layer];
  gat_scores_kernel<<<c->sm_count * 8, 256, 0, st>>>(X, ldx, n, K, c->d_att_w[layer], c->d_att_w[layer] + K, src_begin, rows_out, ld,
                                                     c->dims[layer + 1], c->d_att_s, c->d_att_t, c->d_att_max);
  c->launches += 1;
}

void launch_gat_attention(taurus_ctx* c, cudaStream_t st) {
  const int grid = c->sm_count * 8;
  if (c->heads == 1) gat_edge_max_kernel<true><<<grid, 256, 0, st>>>(c->V, 1, c->d_row_ptr, c->d_col, c->d_mask_cur, c->d_att_s, c->d_att_max);
  else gat_edge_max_kernel<false><<<grid, 256, 0, st>>>(c->V, c->heads, c->d_row_ptr, c->d_col, c->d_mask_cur, c->d_att_s, c->d_att_max);
  gat_tm_kernel<<<grid, 256, 0, st>>>(c->V * c->heads, c->d_att_s, c->d_att_t, c->d_att_max, c->leaky, c->d_att_tm, c->d_att_z);
  if (c->heads == 1) gat_edge_sum_kernel<true><<<grid, 256, 0, st>>>(c->V, 1, c->d_row_ptr, c->d_col, c->d_mask_cur, c->d_att_s, c->d_att_tm, c->leaky, c->d_att_z);
  else gat_edge_sum_kernel<false><<<grid, 256, 0, st>>>(c->V, c->heads, c->d_row_ptr, c->d_col, c->d_mask_cur, c->d_att_s, c->d_att_tm, c->leaky, c->d_att_z);
  c->launches += 3;
}

void launch_gat_repack(taurus_ctx* c, const float* X, int n, int d_out, int Hp, cudaStream_t st) {
  gat_repack_kernel<<<c->sm_count * 8, 256, 0, st>>>(X, n, d_out, Hp, c->d_PT);
  c->launches += 1;
}
