// Projection step (S2) on the 5th-generation tensor cores: [P | T] = X . [W_neigh | W_self] with the per-row
// epilogue, for one pushed chunk (Sect. 3.6 puts the layer transform on the GPU; here it runs before the
// aggregation, which is legal by linearity, SAGEConv paragraph of Sect. 3.9).
//
// Persistent kernel: one CTA per SM walks (128-row tile of X, block of up to 256 output columns) units.  Roles (10 warps):
//   warp 0        TMA producer: cp.async.bulk.tensor loads of the raw fp32 X tile and the W operand tiles
//   warp 1        MMA issuer: tcgen05.mma, accumulators in TMEM (two buffers of up to 256 columns)
//   warps 2..5    converter: turns the raw fp32 X tile in shared memory into tensor-core operands
//                   fp32 mode : hi = x with the low 13 mantissa bits cleared (in place), lo = x - hi (exact);
//                               acc += lo.Whi + hi.Wlo + hi.Whi   (three kind::tf32 MMAs, small terms first)
//                   bf16 mode : bf16(x), one kind::f16 MMA
//   warps 6..9    epilogue: tcgen05.ld of the accumulator, per-row scaling / bias, 32 x 32 tiles staged in shared
//                 memory and written with TMA stores (full 128-byte lines)
// The output columns of a tile are processed in blocks of up to 256; (tile, block) units alternate between two
// TMEM accumulator buffers, so the epilogue of one unit overlaps the main loop of the next, also across tiles.
//
// Every wait on an mbarrier is bounded: after WAIT_LIMIT polls the kernel raises a CTA-wide abort flag,
// records TAURUS_ERR_INTERNAL in the control block, waits (bounded) for its TMA copies in flight, frees its
// TMEM and returns.  Every TMA load is a plain load of the issuing CTA alone.
#include <cuda.h>
#include <cuda_bf16.h>

#include <vector>

#include "taurus_internal.h"

namespace {

constexpr int BM = 128;            // rows per CTA tile (UMMA M)
constexpr int BN_MAX = 256;        // output columns per block (UMMA N)
constexpr int STAGES = 2;            // stages of 128-byte operand rows with full-width (256-column) weight tiles: sizes the shared memory
constexpr int MAX_STAGES = 8;        // shorter operand rows and narrower weight tiles leave room for more stages in the same memory
constexpr int TILE_A_BYTES = BM * 128;           // 128 rows x 128 B
constexpr int TILE_B_BYTES = BN_MAX * 128;       // 256 rows x 128 B
// fp32 mode: K columns per stage, 32 (128-byte operand rows, 128-byte swizzle) or 16 (64-byte rows and swizzle: stages half
// as large, twice as many in flight).  Both are exact and measure the same (projection of the "mid" workload 6.1 against
// 6.3 ms per step): the three TF32 MMAs of a K step read their operands from shared memory without reuse between them
// (12 KB per 128 x 256 x 8 MMA, one MMA per 134 cycles at the pipe's rate = 92 B per cycle), and with the TMA fill and the
// operand split on top the SM's 128 B per cycle of shared memory are the limit, not the depth of the pipeline.
constexpr int KS32 = 32;
constexpr int ROW32 = KS32 * 4;                  // operand row bytes in fp32 mode
constexpr int A32_BYTES = BM * ROW32;            // one fp32-mode feature tile (raw / hi, or lo)
constexpr unsigned WAIT_LIMIT = 1u << 24;
constexpr int NUM_THREADS = 320;
constexpr int OUT_TILE_BYTES = 32 * 128;        // epilogue staging tile: 32 rows x 32 fp32, 128B-swizzled
constexpr int OUT_STAGING_BYTES = 4 * 2 * OUT_TILE_BYTES;   // 4 epilogue warps x 2 tiles

struct __align__(8) Barriers {
  unsigned long long full[MAX_STAGES], conv[MAX_STAGES], empty[MAX_STAGES], acc_full[2], acc_empty[2];
  unsigned int tmem_base;
  int abort_flag;
};

// shared memory per stage: fp32 mode  A_hi(raw) 16K | A_lo 16K | B_hi 32K | B_lo 32K       = 96 KB (32 K-columns)
//                          bf16 mode  A_raw0 16K | A_raw1 16K | A_bf16 16K | B_bf16 32K     = 80 KB (64 K-columns)
// with weight tiles of 256 columns; the memory is sized for two such stages, and a launch whose weight tiles are
// narrower runs as many stages as fit (GemmArgs::stages, stage_bytes).
constexpr int STAGE_BYTES_FP32 = 2 * TILE_A_BYTES + 2 * TILE_B_BYTES;
constexpr int STAGE_BYTES_BF16 = 3 * TILE_A_BYTES + TILE_B_BYTES;

__device__ __forceinline__ unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
               : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the CTA is aborting (this wait or another one ran out).
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag) {
  for (unsigned i = 0; i < WAIT_LIMIT; ++i) {
    if (mbar_try(bar, parity)) return true;
    if ((i & 63u) == 63u && *abort_flag) return false;
  }
  *abort_flag = 1;
  return false;
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

// K-major operand tile with ROW-byte rows (128: 128-byte swizzle; 64: 64-byte swizzle), 8-row groups 8 * ROW bytes apart.
template <int ROW>
__device__ __forceinline__ unsigned long long umma_desc(unsigned smem_addr) {
  static_assert(ROW == 128 || ROW == 64, "operand rows of 128 or 64 bytes");
  unsigned long long d = 0;
  d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);   // start address
  d |= 1ull << 16;                                           // leading byte offset (unused for swizzled K-major)
  d |= (unsigned long long)((8 * ROW) >> 4) << 32;           // stride byte offset: next 8-row group
  d |= 1ull << 46;                                           // descriptor version of this architecture
  d |= (ROW == 128 ? 2ull : 4ull) << 61;                     // SWIZZLE_128B / SWIZZLE_64B
  return d;
}

__device__ __forceinline__ void umma(unsigned tmem_d, unsigned long long a, unsigned long long b, unsigned idesc,
                                     unsigned accumulate, bool tf32) {
  if (tf32)
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n}"
                 ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
  else
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
                 ::"r"(tmem_d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

struct GemmArgs {
  float* PT;            // [n x N]
  int n, N, Np;         // rows, output columns, columns padded to a multiple of 16
  int k_stages;         // K padded / (KS32 fp32 mode, 64 bf16 mode)
  int b_box_bytes;      // bytes one W-operand TMA box delivers (box rows x operand row bytes)
  int stages;           // operand stages in flight (2 .. MAX_STAGES)
  int stage_bytes;      // fp32 mode 2 * A32_BYTES + 2 * b_box_bytes, bf16 mode 3 * TILE_A_BYTES + b_box_bytes
  int Hp, mode, fanout;
  const float* bias;
  const long long* row_ptr;
  const int32_t* din;
  long long src_begin;
  DevCtl* ctl;
  const int32_t* done_count;   // non-null: the rows that matter are the first *done_count ones (read on the device): row tiles behind them are skipped
  int finish;           // epilogue of finished rows: act(row + fin.bias) into fin.dense[fin.done_list[row]], no store to PT
  GemmFinish fin;
};

template <bool BF16>
__global__ void __launch_bounds__(NUM_THREADS, 1)
project_tc_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_b0,
                  const __grid_constant__ CUtensorMap map_b1, const __grid_constant__ CUtensorMap map_out, GemmArgs g) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  constexpr int STAGE_BYTES_MAX = BF16 ? STAGE_BYTES_BF16 : STAGE_BYTES_FP32;
  const int STAGE_BYTES = g.stage_bytes;
  const int n_stages = g.stages;
  unsigned char* out_staging = smem + STAGES * STAGE_BYTES_MAX;
  Barriers* bars = reinterpret_cast<Barriers*>(out_staging + OUT_STAGING_BYTES);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int n_rows = g.n;
  if (g.done_count) { const int nd = *g.done_count; n_rows = nd < g.n ? nd : g.n; }   // same value in every thread
  const int n_tiles = (n_rows + BM - 1) / BM;
  const int n_blocks = (g.Np + BN_MAX - 1) / BN_MAX;
  const int tmem_cols = 512;   // two accumulator buffers of 256 columns; one CTA per SM

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->conv[s], 128); mbar_init(&bars->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&bars->acc_full[b], 1); mbar_init(&bars->acc_empty[b], 128); }
    bars->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation by one full warp
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = bars->tmem_base;

  auto stage_ptr = [&](int s) { return smem + s * STAGE_BYTES; };

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int it = 0;
      for (int w = blockIdx.x; w < n_tiles * n_blocks && !*abort_flag; w += gridDim.x) {
        const int tile = w / n_blocks, nb = w % n_blocks;
        const int row0 = tile * BM;
        const int col0 = nb * BN_MAX;
        for (int ks = 0; ks < g.k_stages; ++ks, ++it) {
          const int s = it % n_stages;
          const unsigned ph = (it / n_stages) & 1;
          if (it >= n_stages && !mbar_wait(&bars->empty[s], ph ^ 1, abort_flag)) break;
          unsigned char* st = stage_ptr(s);
          if (BF16) {
            mbar_expect_tx(&bars->full[s], 2 * TILE_A_BYTES + g.b_box_bytes);
            tma_load_2d(st, &map_x, ks * 64, row0, &bars->full[s]);
            tma_load_2d(st + TILE_A_BYTES, &map_x, ks * 64 + 32, row0, &bars->full[s]);
            tma_load_2d(st + 3 * TILE_A_BYTES, &map_b0, ks * 64, col0, &bars->full[s]);
          } else {
            mbar_expect_tx(&bars->full[s], A32_BYTES + 2 * g.b_box_bytes);
            tma_load_2d(st, &map_x, ks * KS32, row0, &bars->full[s]);
            tma_load_2d(st + 2 * A32_BYTES, &map_b0, ks * KS32, col0, &bars->full[s]);
            tma_load_2d(st + 2 * A32_BYTES + g.b_box_bytes, &map_b1, ks * KS32, col0, &bars->full[s]);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      int it = 0, unit = 0;
      for (int w = blockIdx.x; w < n_tiles * n_blocks && !*abort_flag; w += gridDim.x, ++unit) {
        const int nb = w % n_blocks;
        const int bw = (g.Np - nb * BN_MAX) < BN_MAX ? (g.Np - nb * BN_MAX) : BN_MAX;
        const int buf = unit & 1;
        if (unit >= 2 && !mbar_wait(&bars->acc_empty[buf], ((unit >> 1) & 1) ^ 1, abort_flag)) break;
        tc_fence_after();
        const unsigned tmem_d = tmem_base + (unsigned)(buf * BN_MAX);
        const unsigned idesc = (1u << 4) | ((BF16 ? 1u : 2u) << 7) | ((BF16 ? 1u : 2u) << 10) |
                               ((unsigned)(bw >> 3) << 17) | ((unsigned)(BM >> 4) << 24);
        bool ok = true;
        for (int ks = 0; ks < g.k_stages; ++ks, ++it) {
          const int s = it % n_stages;
          const unsigned ph = (it / n_stages) & 1;
          if (!mbar_wait(&bars->conv[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const unsigned base = smem_u32(stage_ptr(s));
          if (BF16) {
            const unsigned long long da = umma_desc<128>(base + 2 * TILE_A_BYTES), db = umma_desc<128>(base + 3 * TILE_A_BYTES);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) umma(tmem_d, da + 2 * kk, db + 2 * kk, idesc, (ks | kk) != 0, false);
          } else {
            const unsigned long long a_hi = umma_desc<ROW32>(base), a_lo = umma_desc<ROW32>(base + A32_BYTES);
            const unsigned long long b_hi = umma_desc<ROW32>(base + 2 * A32_BYTES), b_lo = umma_desc<ROW32>(base + 2 * A32_BYTES + g.b_box_bytes);
#pragma unroll
            for (int kk = 0; kk < KS32 / 8; ++kk) {
              umma(tmem_d, a_lo + 2 * kk, b_hi + 2 * kk, idesc, (ks | kk) != 0, true);
              umma(tmem_d, a_hi + 2 * kk, b_lo + 2 * kk, idesc, 1u, true);
              umma(tmem_d, a_hi + 2 * kk, b_hi + 2 * kk, idesc, 1u, true);
            }
          }
          umma_commit(&bars->empty[s]);    // stage reusable once these MMAs have read it
        }
        if (!ok) break;
        umma_commit(&bars->acc_full[buf]);  // accumulator of this block complete
      }
    }
  } else if (warp < 6) {
    // ---------------------------------------------------------------- converter (128 threads)
    const int t = threadIdx.x - 64;
    int it = 0;
    for (int w = blockIdx.x; w < n_tiles * n_blocks && !*abort_flag; w += gridDim.x) {
      bool ok = true;
      for (int ks = 0; ks < g.k_stages; ++ks, ++it) {
        const int s = it % n_stages;
        const unsigned ph = (it / n_stages) & 1;
        if (!mbar_wait(&bars->full[s], ph, abort_flag)) { ok = false; break; }
        unsigned char* st = stage_ptr(s);
        if (BF16) {
          // raw sub-tile h holds columns 32h..32h+31; its physical 16-byte chunk p of row r is logical chunk p ^ (r & 7).
          // bf16 tile: 128-byte rows, logical 16-byte chunk q of row r sits at physical chunk q ^ (r & 7).
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int idx = t + i * 128;        // 0..1023: (h, r, pair m of logical chunks 2m, 2m+1)
            const int m = idx & 3, r = (idx >> 2) & 127, h = idx >> 9;
            const unsigned char* rawrow = st + h * TILE_A_BYTES + r * 128;
            const float4 v0 = *reinterpret_cast<const float4*>(rawrow + (((2 * m) ^ (r & 7)) << 4));
            const float4 v1 = *reinterpret_cast<const float4*>(rawrow + (((2 * m + 1) ^ (r & 7)) << 4));
            __nv_bfloat162 b0 = __floats2bfloat162_rn(v0.x, v0.y), b1 = __floats2bfloat162_rn(v0.z, v0.w);
            __nv_bfloat162 b2 = __floats2bfloat162_rn(v1.x, v1.y), b3 = __floats2bfloat162_rn(v1.z, v1.w);
            uint4 o;
            o.x = *reinterpret_cast<unsigned*>(&b0); o.y = *reinterpret_cast<unsigned*>(&b1);
            o.z = *reinterpret_cast<unsigned*>(&b2); o.w = *reinterpret_cast<unsigned*>(&b3);
            const int q = 4 * h + m;
            *reinterpret_cast<uint4*>(st + 2 * TILE_A_BYTES + r * 128 + ((q ^ (r & 7)) << 4)) = o;
          }
        } else {
          // element-wise and layout-preserving: the swizzle does not matter
          float4* hi = reinterpret_cast<float4*>(st);
          float4* lo = reinterpret_cast<float4*>(st + A32_BYTES);
#pragma unroll
          for (int i = 0; i < A32_BYTES / 16 / 128; ++i) {
            const int idx = t + i * 128;
            float4 x = hi[idx], h4, l4;
            h4.x = __uint_as_float(__float_as_uint(x.x) & 0xFFFFE000u); l4.x = x.x - h4.x;
            h4.y = __uint_as_float(__float_as_uint(x.y) & 0xFFFFE000u); l4.y = x.y - h4.y;
            h4.z = __uint_as_float(__float_as_uint(x.z) & 0xFFFFE000u); l4.z = x.z - h4.z;
            h4.w = __uint_as_float(__float_as_uint(x.w) & 0xFFFFE000u); l4.w = x.w - h4.w;
            hi[idx] = h4; lo[idx] = l4;
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the tensor core
        mbar_arrive(&bars->conv[s]);
      }
      if (!ok) break;
    }
  } else {
    // ---------------------------------------------------------------- epilogue (warps 6..9, TMEM lanes 32 * (warp % 4))
    const int q = warp & 3;
    int unit = 0, out_it = 0;
    for (int w = blockIdx.x; w < n_tiles * n_blocks && !*abort_flag; w += gridDim.x, ++unit) {
    const int tile = w / n_blocks, nb = w % n_blocks;
    const int r = tile * BM + q * 32 + lane;
    float c_out = 1.f, self_mul = 1.f;
    int vrow = -1;        // finish mode: the vertex this lane's row belongs to
    if (g.finish) {
      if (r < g.n && r < *g.done_count && !g.ctl->error) {
        vrow = g.fin.done_list[r];
        if (nb == 0) g.fin.state[vrow] = TAURUS_COMPLETED;
      }
    } else if (r < g.n) {
      const long long u = g.src_begin + r;
      if (g.mode == TAURUS_GCN_SYM) {
        c_out = (float)(1.0 / sqrt((double)(g.row_ptr[u + 1] - g.row_ptr[u]) + 1.0));
      } else if (g.mode == TAURUS_SAGE_MEAN) {
        const int d = g.din[u];
        const int m = (g.fanout > 0 && d > g.fanout) ? g.fanout : d;
        self_mul = (float)(m > 1 ? m : 1);
      }
    }
    {
      const int bw = (g.Np - nb * BN_MAX) < BN_MAX ? (g.Np - nb * BN_MAX) : BN_MAX;
      const int buf = unit & 1;
      if (!mbar_wait(&bars->acc_full[buf], (unit >> 1) & 1, abort_flag)) break;
      tc_fence_after();
      for (int c0 = 0; c0 < bw; c0 += 32) {
        unsigned v[32];
        const unsigned taddr = tmem_base + ((unsigned)(q * 32) << 16) + (unsigned)(buf * BN_MAX + c0);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
              "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
              "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr) : "memory");
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        const int cbase = nb * BN_MAX + c0;
        if (cbase >= g.N) continue;           // padding columns of the last block
        // this warp's staging tile: 32 rows (lane = row) x 32 columns, 16-byte chunk c of row r at chunk c ^ (r & 7)
        unsigned char* tile_smem = out_staging + (q * 2 + (out_it & 1)) * OUT_TILE_BYTES;
        if (g.finish) {
          // transpose through the staging tile, then the warp writes four rows per step, each as one 128-byte piece of
          // the row's place in the vertex-ordered matrix
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const int c = cbase + j;
            const float4 b = c < g.N ? *reinterpret_cast<const float4*>(g.fin.bias + c) : make_float4(0.f, 0.f, 0.f, 0.f);
            float4 o = make_float4(__uint_as_float(v[j]) + b.x, __uint_as_float(v[j + 1]) + b.y, __uint_as_float(v[j + 2]) + b.z,
                                   __uint_as_float(v[j + 3]) + b.w);
            if (g.fin.act) { o.x = fmaxf(o.x, 0.f); o.y = fmaxf(o.y, 0.f); o.z = fmaxf(o.z, 0.f); o.w = fmaxf(o.w, 0.f); }
            *reinterpret_cast<float4*>(tile_smem + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)) = o;
          }
          __syncwarp();
#pragma unroll
          for (int it = 0; it < 8; ++it) {
            const int rr = it * 4 + (lane >> 3), ch = lane & 7;
            const int vv = __shfl_sync(0xffffffffu, vrow, rr);
            const float4 y = *reinterpret_cast<const float4*>(tile_smem + rr * 128 + ((ch ^ (rr & 7)) << 4));
            if (vv >= 0 && cbase + ch * 4 < g.N)
              *reinterpret_cast<float4*>(g.fin.dense + (size_t)vv * g.fin.dense_ld + cbase + ch * 4) = y;
          }
          __syncwarp();   // the tile is rewritten in the next round
          continue;
        }
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the store that last used this tile has read it
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          float4 o;
          float* po = &o.x;
          const int c = cbase + j;
          if (c >= g.Hp && c < g.N) {         // T columns: (x W_self + b) * max(|M(u)|, 1); GAT: the two attention scalars as they are
            const float4 b = g.mode == TAURUS_GAT ? make_float4(0.f, 0.f, 0.f, 0.f) : *reinterpret_cast<const float4*>(g.bias + (c - g.Hp));
            po[0] = (__uint_as_float(v[j]) + b.x) * self_mul; po[1] = (__uint_as_float(v[j + 1]) + b.y) * self_mul;
            po[2] = (__uint_as_float(v[j + 2]) + b.z) * self_mul; po[3] = (__uint_as_float(v[j + 3]) + b.w) * self_mul;
          } else {                            // P columns: c_out(u) * (x W_neigh)
            po[0] = __uint_as_float(v[j]) * c_out; po[1] = __uint_as_float(v[j + 1]) * c_out;
            po[2] = __uint_as_float(v[j + 2]) * c_out; po[3] = __uint_as_float(v[j + 3]) * c_out;
          }
          *reinterpret_cast<float4*>(tile_smem + lane * 128 + (((j >> 2) ^ (lane & 7)) << 4)) = o;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {                      // rows beyond n and columns beyond N are clipped by the tensor map
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                       ::"l"(&map_out), "r"(cbase), "r"(tile * BM + q * 32), "r"(smem_u32(tile_smem)) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
        ++out_it;
      }
      tc_fence_before();
      mbar_arrive(&bars->acc_empty[buf]);
    }
    }
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // all stores of this warp are complete
  }

  // ---------------------------------------------------------------- teardown
  __syncthreads();
  if (*abort_flag) {
    if (threadIdx.x == 0) {
      atomicCAS(&g.ctl->error, 0, TAURUS_ERR_INTERNAL);
      // give copies that may still be in flight a bounded time to land before the shared memory is released
      for (int s = 0; s < n_stages; ++s)
        for (unsigned i = 0; i < (1u << 16); ++i)
          if (mbar_try(&bars->full[s], 0) || mbar_try(&bars->full[s], 1)) break;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  }
  return fn;
}

// 2-D row-major tensor [rows x cols] of `elem` bytes, box [box_rows x box_cols], 128-byte swizzle, zero fill
// on loads, clipping on stores.
bool make_map(CUtensorMap* m, const void* base, CUtensorMapDataType dt, int elem, long long rows, long long cols,
              long long ld_elems, int box_rows, int box_cols) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld_elems * elem};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle swz = box_cols * elem == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B;   // box rows of 64 or 128 bytes
  return fn(m, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Stages that fit the shared memory sized for STAGES full-width stages.
void set_stages(GemmArgs& g, bool bf16) {
  const int budget = STAGES * (bf16 ? STAGE_BYTES_BF16 : STAGE_BYTES_FP32);
  g.stage_bytes = bf16 ? 3 * TILE_A_BYTES + g.b_box_bytes : 2 * A32_BYTES + 2 * g.b_box_bytes;
  int n = budget / g.stage_bytes;
  g.stages = n < STAGES ? STAGES : n > MAX_STAGES ? MAX_STAGES : n;
}

// Per-layer tensor-core images of Wcat, K-major: [Np x Kp].
struct WImage {
  void* hi = nullptr;   // fp32 mode: tf32-exact high part; bf16 mode: bf16 weights
  void* lo = nullptr;   // fp32 mode: residual
  int Np = 0, Kp = 0;
  CUtensorMap map_hi, map_lo;
};

}  // namespace

int prepare_tc_weights(taurus_ctx* c, void** slot, const std::vector<float>& cat, int K, int N) {
  const bool bf16 = c->gemm_mode == TAURUS_GEMM_BF16;
  WImage* w = new WImage();
  *slot = w;
  w->Np = taurus_round_up(N, 16);
  w->Kp = taurus_round_up(K, bf16 ? 64 : KS32);
  const size_t cnt = (size_t)w->Np * w->Kp;
  const int bw = w->Np < BN_MAX ? w->Np : BN_MAX;
  if (bf16) {
    std::vector<__nv_bfloat16> img(cnt, __float2bfloat16(0.f));
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < N; ++j) img[(size_t)j * w->Kp + k] = __float2bfloat16(cat[(size_t)k * N + j]);
    if (cudaMalloc(&w->hi, cnt * 2) != cudaSuccess) return TAURUS_ERR_NOMEM;
    if (cudaMemcpy(w->hi, img.data(), cnt * 2, cudaMemcpyHostToDevice) != cudaSuccess) return TAURUS_ERR_CUDA;
    if (!make_map(&w->map_hi, w->hi, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, w->Np, w->Kp, w->Kp, bw, 64)) return TAURUS_ERR_CUDA;
    w->map_lo = w->map_hi;
  } else {
    std::vector<float> hi(cnt, 0.f), lo(cnt, 0.f);
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < N; ++j) {
        float x = cat[(size_t)k * N + j];
        uint32_t b; memcpy(&b, &x, 4); b &= 0xFFFFE000u;
        float h; memcpy(&h, &b, 4);
        float l = x - h;
        uint32_t lb; memcpy(&lb, &l, 4); lb &= 0xFFFFE000u; memcpy(&l, &lb, 4);
        hi[(size_t)j * w->Kp + k] = h;
        lo[(size_t)j * w->Kp + k] = l;
      }
    if (cudaMalloc(&w->hi, cnt * 4) != cudaSuccess || cudaMalloc(&w->lo, cnt * 4) != cudaSuccess) return TAURUS_ERR_NOMEM;
    if (cudaMemcpy(w->hi, hi.data(), cnt * 4, cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(w->lo, lo.data(), cnt * 4, cudaMemcpyHostToDevice) != cudaSuccess) return TAURUS_ERR_CUDA;
    if (!make_map(&w->map_hi, w->hi, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, w->Np, w->Kp, w->Kp, bw, KS32) ||
        !make_map(&w->map_lo, w->lo, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, w->Np, w->Kp, w->Kp, bw, KS32)) return TAURUS_ERR_CUDA;
  }
  return TAURUS_OK;
}

void free_tc_weights(taurus_ctx* c) {
  for (int l = 0; l < 2 * TAURUS_MAX_LAYERS; ++l) {
    void** slot = l < TAURUS_MAX_LAYERS ? &c->tc_image[l] : &c->tc_image_af[l - TAURUS_MAX_LAYERS];
    WImage* w = static_cast<WImage*>(*slot);
    if (!w) continue;
    cudaFree(w->hi); cudaFree(w->lo);
    delete w;
    *slot = nullptr;
  }
}

// Shapes the tensor-core kernel takes: feature rows that TMA can address (16-byte aligned base and pitch).
bool project_tc_usable(const taurus_ctx* c, int layer, const float* X, int ldx) {
  if (c->flags & TAURUS_FLAG_SIMT_GEMM) return false;
  if (!c->tc_image[layer] || !encode_fn()) return false;
  if ((ldx & 3) != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0) return false;
  return true;
}

int launch_project_tc(taurus_ctx* c, int layer, const float* X, int ldx, long long src_begin, int n, cudaStream_t st) {
  const bool bf16 = c->gemm_mode == TAURUS_GEMM_BF16;
  WImage* w = static_cast<WImage*>(c->tc_image[layer]);
  const int K = c->dims[layer], Hp = taurus_round_up(c->dims[layer + 1], 4);
  const int N = taurus_proj_width(c->mode, Hp, c->heads);
  CUtensorMap map_x;
  if (!make_map(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, n, K, ldx, BM, bf16 ? 32 : KS32)) return TAURUS_ERR_CUDA;
  CUtensorMap map_out;
  if (!make_map(&map_out, c->d_PT, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, n, N, N, 32, 32)) return TAURUS_ERR_CUDA;
  GemmArgs g;
  g.PT = c->d_PT; g.n = n; g.N = N; g.Np = w->Np; g.k_stages = w->Kp / (bf16 ? 64 : KS32);
  g.b_box_bytes = (w->Np < BN_MAX ? w->Np : BN_MAX) * (bf16 ? 128 : ROW32);
  set_stages(g, bf16);
  g.Hp = Hp; g.mode = c->mode; g.fanout = c->fanout[layer]; g.bias = c->d_bias[layer];
  g.row_ptr = c->d_row_ptr; g.din = c->d_din; g.src_begin = src_begin; g.ctl = c->d_ctl;
  g.finish = 0; g.fin = GemmFinish(); g.done_count = nullptr;
  const int smem = STAGES * (bf16 ? STAGE_BYTES_BF16 : STAGE_BYTES_FP32) + OUT_STAGING_BYTES + (int)sizeof(Barriers) + 1024;
  const int n_tiles = (n + BM - 1) / BM;
  const int n_units = n_tiles * ((w->Np + BN_MAX - 1) / BN_MAX);
  const int grid = n_units < c->sm_count ? n_units : c->sm_count;
  if (!c->tc_smem_set) {   // once per context (the attribute belongs to the context's device)
    cudaError_t e = bf16 ? cudaFuncSetAttribute(project_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                         : cudaFuncSetAttribute(project_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) { cudaGetLastError(); return TAURUS_ERR_CUDA; }
    c->tc_smem_set = true;
  }
  if (bf16) project_tc_kernel<true><<<grid, NUM_THREADS, smem, st>>>(map_x, w->map_hi, w->map_lo, map_out, g);
  else project_tc_kernel<false><<<grid, NUM_THREADS, smem, st>>>(map_x, w->map_hi, w->map_lo, map_out, g);
  c->launches += 1;
  return TAURUS_OK;
}

// Plain product on the tensor cores: out[n x N] (pitch ld_out floats) = X[n x K] (pitch ldx) . columns
// [col0, col0 + N) of the layer's weight image, no epilogue scaling (used when a layer aggregates raw rows
// first and transforms the finished rows afterwards).  col0 and N are multiples of 4.
bool gemm_plain_tc_usable(const taurus_ctx* c, const void* image, const float* X, int ldx, const float* out, long long ld_out) {
  if (c->flags & TAURUS_FLAG_SIMT_GEMM) return false;
  if (!image || !encode_fn()) return false;
  if ((ldx & 3) != 0 || (reinterpret_cast<uintptr_t>(X) & 15) != 0) return false;
  if ((ld_out & 3) != 0 || (reinterpret_cast<uintptr_t>(out) & 15) != 0) return false;
  return true;
}

int launch_gemm_plain_tc(taurus_ctx* c, void* image, int col0, int N, const float* X, int ldx, int K, int n, float* out, long long ld_out,
                         cudaStream_t st, const GemmFinish* finish, const int32_t* done_count) {
  if (n <= 0) return TAURUS_OK;
  if (finish && ((N & 3) != 0 || (finish->dense_ld & 3) != 0 || (reinterpret_cast<uintptr_t>(finish->dense) & 15) != 0)) return TAURUS_ERR_INTERNAL;
  const bool bf16 = c->gemm_mode == TAURUS_GEMM_BF16;
  WImage* w = static_cast<WImage*>(image);
  const int rows_left = w->Np - col0;                       // image rows (= output columns) from col0 on
  const int Np = std::min(taurus_round_up(N, 16), rows_left);
  const int bw = Np < BN_MAX ? Np : BN_MAX;
  const int elem = bf16 ? 2 : 4;
  CUtensorMap map_x, map_out, map_hi, map_lo;
  if (!make_map(&map_x, X, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, n, K, ldx, BM, bf16 ? 32 : KS32)) return TAURUS_ERR_CUDA;
  if (!make_map(&map_out, out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, n, N, ld_out, 32, 32)) return TAURUS_ERR_CUDA;
  const char* hi = static_cast<const char*>(w->hi) + (size_t)col0 * w->Kp * elem;
  if (!make_map(&map_hi, hi, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, elem, rows_left, w->Kp, w->Kp, bw,
                bf16 ? 64 : KS32))
    return TAURUS_ERR_CUDA;
  map_lo = map_hi;
  if (!bf16) {
    const char* lo = static_cast<const char*>(w->lo) + (size_t)col0 * w->Kp * elem;
    if (!make_map(&map_lo, lo, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, rows_left, w->Kp, w->Kp, bw, KS32)) return TAURUS_ERR_CUDA;
  }
  GemmArgs g;
  g.PT = out; g.n = n; g.N = N; g.Np = Np; g.k_stages = w->Kp / (bf16 ? 64 : KS32);
  g.b_box_bytes = bw * (bf16 ? 128 : ROW32);
  set_stages(g, bf16);
  g.Hp = N; g.mode = TAURUS_GIN_SUM; g.fanout = 0; g.bias = nullptr;
  g.row_ptr = c->d_row_ptr; g.din = c->d_din; g.src_begin = 0; g.ctl = c->d_ctl;
  g.finish = finish ? 1 : 0; g.fin = finish ? *finish : GemmFinish();
  g.done_count = done_count;
  const int smem = STAGES * (bf16 ? STAGE_BYTES_BF16 : STAGE_BYTES_FP32) + OUT_STAGING_BYTES + (int)sizeof(Barriers) + 1024;
  const int n_tiles = (n + BM - 1) / BM;
  const int n_units = n_tiles * ((Np + BN_MAX - 1) / BN_MAX);
  const int grid = n_units < c->sm_count ? n_units : c->sm_count;
  if (!c->tc_smem_set) {
    cudaError_t e = bf16 ? cudaFuncSetAttribute(project_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem)
                         : cudaFuncSetAttribute(project_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) { cudaGetLastError(); return TAURUS_ERR_CUDA; }
    c->tc_smem_set = true;
  }
  if (bf16) project_tc_kernel<true><<<grid, NUM_THREADS, smem, st>>>(map_x, map_hi, map_lo, map_out, g);
  else project_tc_kernel<false><<<grid, NUM_THREADS, smem, st>>>(map_x, map_hi, map_lo, map_out, g);
  c->launches += 1;
  return TAURUS_OK;
}
