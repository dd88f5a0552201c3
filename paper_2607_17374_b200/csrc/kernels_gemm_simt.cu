// Projection step (S2) as a plain fp32 FFMA GEMM: [P | T] = X . [W_neigh | W_self] with the per-row
// epilogue.  Exact fp32 arithmetic; kept as the reference shim for the tensor-core kernel and as the
// fallback for shapes that kernel does not take (TAURUS_FLAG_SIMT_GEMM selects it explicitly).
//
// Epilogue (project-then-aggregate is legal by linearity, SAGEConv paragraph of Sect. 3.9):
//   P_u = c_out(u) * (x_u W_neigh)                        message every out-neighbour receives
//   T_u = (x_u W_self + b) * max(|M(u)|, 1)     (SAGE)    self message, pre-multiplied by 1 / c_in(u) so
//                                                          that finalise is one multiply by c_in
//   (GCN has no T columns: its self message P_u + b / c_in(u) is formed by the scatter kernel.)
#include "taurus_internal.h"

#define BM 64
#define BN 64
#define BK 16

__global__ void __launch_bounds__(256) project_simt_kernel(const float* __restrict__ X, int ldx, int K, const float* __restrict__ W,
                                                           int ldw, int N, float* __restrict__ PT, long long ldo, int n, int Hp, int mode,
                                                           const float* __restrict__ bias, const long long* __restrict__ row_ptr,
                                                           const int32_t* __restrict__ din, int fanout, long long src_begin) {
  __shared__ float sA[BK][BM + 1];
  __shared__ float sB[BK][BN];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int row0 = blockIdx.y * BM, col0 = blockIdx.x * BN;
  float acc[4][4] = {{0.f}};
  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int i = threadIdx.x; i < BM * BK; i += 256) {
      int r = i / BK, k = i % BK;
      int gr = row0 + r, gk = k0 + k;
      sA[k][r] = (gr < n && gk < K) ? X[(size_t)gr * ldx + gk] : 0.f;
    }
    for (int i = threadIdx.x; i < BK * BN; i += 256) {
      int k = i / BN, cidx = i % BN;
      int gk = k0 + k, gc = col0 + cidx;
      sB[k][cidx] = (gk < K && gc < N) ? W[(size_t)gk * ldw + gc] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = sA[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = sB[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int r = row0 + ty * 4 + i;
    if (r >= n) continue;
    long long u = src_begin + r;
    float c_out = 1.f, self_mul = 1.f;
    if (mode == TAURUS_GCN_SYM) {
      c_out = (float)(1.0 / sqrt((double)(row_ptr[u + 1] - row_ptr[u]) + 1.0));
    } else if (mode == TAURUS_SAGE_MEAN) {
      int d = din[u];
      int m = (fanout > 0 && d > fanout) ? fanout : d;
      self_mul = (float)(m > 1 ? m : 1);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int cidx = col0 + tx * 4 + j;
      if (cidx >= N) continue;
      float x = acc[i][j];
      if (cidx < Hp) x *= c_out;
      else if (mode != TAURUS_GAT) x = (x + bias[cidx - Hp]) * self_mul;   // GAT: the attention scalars as they are
      PT[(size_t)r * ldo + cidx] = x;
    }
  }
}

void launch_project_simt(taurus_ctx* c, int layer, const float* X, int ldx, long long src_begin, int n, cudaStream_t st) {
  const int Hp = taurus_round_up(c->dims[layer + 1], 4);
  const int N = taurus_proj_width(c->mode, Hp, c->heads);
  dim3 grid((N + BN - 1) / BN, (n + BM - 1) / BM);
  project_simt_kernel<<<grid, 256, 0, st>>>(X, ldx, c->dims[layer], c->d_Wcat[layer], N, N, c->d_PT, N, n, Hp, c->mode,
                                            c->d_bias[layer], c->d_row_ptr, c->d_din, c->fanout[layer], src_begin);
  c->launches += 1;
}

// out[n x N] (pitch ld_out) = X[n x K] (pitch ldx) . W[:, 0..N) (row-major, pitch ldw), no epilogue.
void launch_gemm_plain_simt(taurus_ctx* c, const float* W, int ldw, int N, const float* X, int ldx, int K, int n, float* out,
                            long long ld_out, cudaStream_t st) {
  if (n <= 0) return;
  dim3 grid((N + BN - 1) / BN, (n + BM - 1) / BM);
  project_simt_kernel<<<grid, 256, 0, st>>>(X, ldx, K, W, ldw, N, out, ld_out, n, N, TAURUS_GIN_SUM, nullptr, c->d_row_ptr, c->d_din, 0, 0);
  c->launches += 1;
}
