// Aggregate-first layers.  When a layer's input rows are narrower than its output rows, the accumulators hold
// sums of (scaled) INPUT rows and the weight matrix is applied to the finished rows, as the paper's graduation
// processor does (Sect. 3.6; the split W = [W_agg  W_self] of the SAGEConv paragraph in Sect. 3.9 is what makes it
// exact): by linearity
//     c_in(v) * sum_u c_out(u) (h_u W)  =  (c_in(v) * sum_u c_out(u) h_u) W,
// and the read-modify-write traffic of the scatter, the pool and every evicted row shrink by d_in / d_out.
//   push     : S_u = c_out(u) h_u (padded to a multiple of 4 columns) is what the scatter pushes;
//              GCN / GIN / GAT add the self message in input space (c_out(v) h_v, (1 + eps) h_v, or the attention weight
//              times h_v: one shared matrix);
//              SAGE keeps every vertex's input row h_v in a per-vertex store from v's own chunk until v completes
//              (the scatter pushes the chunk's rows from that store).
//   finalise : A_i = c_in(v_i) * acc(v_i) gathered for the completed vertices (SAGE: [c_in * acc | h_v]),
//              O = A W_neigh (SAGE: A [W_neigh ; W_self]) on the tensor cores, out = act(O_i + b).
#include "taurus_internal.h"

namespace {

__device__ __forceinline__ int al() { return threadIdx.x & 31; }
__device__ __forceinline__ int af_messages(int din, int fanout) { return (fanout > 0 && din > fanout) ? fanout : din; }

// S[r][k] = c_out(u) * X[r][k] for k < K, 0 for the padding columns; u = src_begin + r.
__global__ void af_prep_kernel(const float* __restrict__ X, int ldx, int n, int K, int Kp, long long src_begin, int mode,
                               const long long* __restrict__ row_ptr, float* __restrict__ S) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < n; r += warps) {
    float scale = 1.0f;
    if (mode == TAURUS_GCN_SYM) {
      const long long u = src_begin + r;
      scale = (float)(1.0 / sqrt((double)(row_ptr[u + 1] - row_ptr[u]) + 1.0));
    }
    const float* src = X + (size_t)r * ldx;
    float* dst = S + (size_t)r * Kp;
    for (int k = al(); k < Kp; k += 32) dst[k] = k < K ? src[k] * scale : 0.f;
  }
}

// A[i] = c_in(v_i) * acc(v_i) for the completed vertices (followed by v_i's own input row when `self_store` is given:
// SAGE).  `rows` is the row count the host sized the transform for; rows behind the completed ones are left as
// they are (the tensor-core transform skips them, the FFMA one writes products nobody reads).  The slot is released
// by compact_done_kernel; its row stays intact until the next chunk.
__global__ void af_gather_kernel(ChunkArgs a, float* __restrict__ A, long long rows, const float* __restrict__ self_store) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int n = pc->done_count;
  if (n > rows) {   // the host sized the transform for fewer rows than completed: its bound was wrong
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
    return;
  }
  const int vec = a.Hp >> 2;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int pitch = self_store ? 2 * a.Hp : a.Hp;
  // Batches of up to 32 finished vertices per warp: each lane follows the dependent reads of one vertex (list entry,
  // slot, degree), then the warp walks the batch row by row.
  int per = (int)((n + warps - 1) / warps);
  per = per < 1 ? 1 : per > 32 ? 32 : per;
  for (long long i0 = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * per; i0 < n; i0 += warps * per) {
    const long long mine = i0 + al();
    int v = -1, l = 0;
    float scale = 1.0f;
    if (al() < per && mine < n) {
      v = a.done_list[mine];
      l = a.loc[v];
      if (a.mode == TAURUS_SAGE_MEAN) {
        const int m = af_messages(a.din[v], a.fanout);
        scale = 1.0f / (float)(m > 1 ? m : 1);
      } else if (a.mode == TAURUS_GCN_SYM) {
        scale = (float)(1.0 / sqrt((double)a.din[v] + 1.0));
      } else if (a.mode == TAURUS_GAT) {
        scale = (float)(1.0 / a.att_z[v]);   // softmax normaliser
      }
    }
    const int rows_here = n - i0 < per ? (int)(n - i0) : per;
    for (int j = 0; j < rows_here; ++j) {
      const int vj = __shfl_sync(0xffffffffu, v, j);
      const int lj = __shfl_sync(0xffffffffu, l, j);
      const float sj = __shfl_sync(0xffffffffu, scale, j);
      float4* dst = reinterpret_cast<float4*>(A + (size_t)(i0 + j) * pitch);
      const float4* src = reinterpret_cast<const float4*>(a.acc + (size_t)lj * a.Hp);
      for (int k = al(); k < vec; k += 32) {
        float4 x = src[k];
        x.x *= sj; x.y *= sj; x.z *= sj; x.w *= sj;
        dst[k] = x;
      }
      if (self_store) {
        const float4* own = reinterpret_cast<const float4*>(self_store + (size_t)vj * a.Hp);
        for (int k = al(); k < vec; k += 32) dst[vec + k] = own[k];
      }
    }
  }
}

// out = act(O_i + b) into the graduation buffer or straight into the caller's vertex-ordered matrix.
// O has pitch a.Hout; rows of the graduation buffer too.
__global__ void af_finish_kernel(ChunkArgs a, const float* __restrict__ O, long long rows) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int n = pc->done_count;
  if (n > rows) {   // the host sized the transform for fewer rows than completed: its bound was wrong
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
    return;
  }
  const long long base = a.dense_half >= 0 ? a.grad_off : ctl->grad_count;
  const long long limit = a.dense_half >= 0 ? a.grad_off + a.grad_cap : a.drain_rows;
  const int vec = a.Hout >> 2;
  const bool vec_ok = a.dense_direct && (a.dense_ld & 3) == 0 && (reinterpret_cast<uintptr_t>(a.dense_direct) & 15) == 0;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < n; i += warps) {
    if (!a.dense_direct && base + i >= limit) {
      if (al() == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
      continue;
    }
    const int v = a.done_list[i];
    const float4* __restrict__ o = reinterpret_cast<const float4*>(O + (size_t)i * a.Hout);
    const float4* __restrict__ b = reinterpret_cast<const float4*>(a.bias);
    float* __restrict__ drow = a.dense_direct ? a.dense_direct + (size_t)v * a.dense_ld : a.grad_rows + (size_t)(base + i) * a.Hout;
    for (int k = al(); k < vec; k += 32) {
      float4 y = o[k];
      const float4 bb = b[k];
      y.x += bb.x; y.y += bb.y; y.z += bb.z; y.w += bb.w;
      if (a.act) { y.x = fmaxf(y.x, 0.f); y.y = fmaxf(y.y, 0.f); y.z = fmaxf(y.z, 0.f); y.w = fmaxf(y.w, 0.f); }
      const int c0 = k << 2;
      if (!a.dense_direct || (vec_ok && c0 + 3 < a.d_out)) {
        reinterpret_cast<float4*>(drow)[k] = y;
      } else {
        if (c0 < a.d_out) drow[c0] = y.x;
        if (c0 + 1 < a.d_out) drow[c0 + 1] = y.y;
        if (c0 + 2 < a.d_out) drow[c0 + 2] = y.z;
        if (c0 + 3 < a.d_out) drow[c0 + 3] = y.w;
      }
    }
    if (al() == 0) {
      a.state[v] = TAURUS_COMPLETED;
      if (!a.dense_direct) a.grad_ids[base + i] = v;
    }
  }
}

}  // namespace

void launch_af_prep(taurus_ctx* c, const float* X, int ldx, int n, int K, int Kp, long long src_begin, float* out, cudaStream_t st) {
  af_prep_kernel<<<c->sm_count * 8, 256, 0, st>>>(X, ldx, n, K, Kp, src_begin, c->mode, c->d_row_ptr, out);
  c->launches += 1;
}

// S7 of an aggregate-first layer (after launch_compact_done): gather, transform, finish, commit.  `rows` is the host's
// bound on the vertices this chunk completes (the transform is sized for it; rows beyond the actual count are zero).
int launch_af_finalise(taurus_ctx* c, const ChunkArgs& a, int layer, long long rows, cudaStream_t st) {
  if (rows > 0) {
    const int grid = c->sm_count * 8;
    float* O;
    if (a.dense_direct) O = c->d_grad_rows;
    else if (a.dense_half >= 0) O = c->d_grad_rows + (size_t)a.grad_off * a.Hout;
    else {
      if (!c->d_af_O) return TAURUS_ERR_INTERNAL;   // allocated by the push before it enqueues anything
      O = c->d_af_O;   // the place in the graduation buffer is known only on the device: transform into a scratch matrix
    }
    const bool sage = c->mode == TAURUS_SAGE_MEAN;
    const int Ka = sage ? 2 * a.Hp : a.Hp;               // columns of the gathered matrix
    af_gather_kernel<<<grid, 256, 0, st>>>(a, c->d_af_A, rows, sage ? c->d_af_X : nullptr);
    c->launches += 1;
    void* image = sage ? c->tc_image_af[layer] : c->tc_image[layer];
    const bool tc = gemm_plain_tc_usable(c, image, c->d_af_A, Ka, O, a.Hout);
    // rows that go straight into the caller's matrix leave the tensor-core kernel finished (bias, activation, state)
    if (tc && a.dense_direct && a.d_out == a.Hout && (a.dense_ld & 3) == 0 && (reinterpret_cast<uintptr_t>(a.dense_direct) & 15) == 0) {
      GemmFinish fin;
      fin.done_list = a.done_list; fin.state = a.state; fin.dense = a.dense_direct; fin.dense_ld = a.dense_ld;
      fin.bias = a.bias; fin.act = a.act;
      int rc = launch_gemm_plain_tc(c, image, 0, a.Hout, c->d_af_A, Ka, Ka, (int)rows, O, a.Hout, st, &fin, &a.pc->done_count);
      if (rc) return rc;
      launch_commit(c, a, st);
      return TAURUS_OK;
    }
    if (tc) {
      int rc = launch_gemm_plain_tc(c, image, 0, a.Hout, c->d_af_A, Ka, Ka, (int)rows, O, a.Hout, st, nullptr, &a.pc->done_count);
      if (rc) return rc;
    } else if (sage) {
      launch_gemm_plain_simt(c, c->d_Waf[layer], a.Hout, a.Hout, c->d_af_A, Ka, Ka, (int)rows, O, a.Hout, st);
    } else {
      launch_gemm_plain_simt(c, c->d_Wcat[layer], taurus_proj_width(c->mode, a.Hout, c->heads), a.Hout, c->d_af_A, Ka, c->dims[layer], (int)rows, O,
                             a.Hout, st);
    }
    af_finish_kernel<<<grid, 256, 0, st>>>(a, O, rows);
    c->launches += 1;
  }
  launch_commit(c, a, st);
  return TAURUS_OK;
}
