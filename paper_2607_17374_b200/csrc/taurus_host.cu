// Host side of libtaurus: the C ABI of include/taurus.h.  Validation, allocation, per-layer set-up and the
// launch sequence of a push.  No arithmetic of the method happens on the host: a push enqueues kernels
// and returns.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "taurus_internal.h"

static thread_local char g_cuda_err[256] = "";

static bool cuda_ok(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return true;
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
  cudaGetLastError();
  return false;
}
void taurus_note_cuda_error(cudaError_t e, const char* what) { cuda_ok(e, what); }
#define CU(call) do { if (!cuda_ok((call), #call)) return TAURUS_ERR_CUDA; } while (0)

template <class T>
static int dev_alloc(T** p, size_t count) {
  *p = nullptr;
  cudaError_t e = cudaMalloc((void**)p, (count > 0 ? count : 1) * sizeof(T));
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); snprintf(g_cuda_err, sizeof(g_cuda_err), "cudaMalloc of %zu bytes failed", count * sizeof(T)); return TAURUS_ERR_NOMEM; }
  return cuda_ok(e, "cudaMalloc") ? TAURUS_OK : TAURUS_ERR_CUDA;
}
#define ALLOC(p, n) do { int rc_ = dev_alloc(&(p), (size_t)(n)); if (rc_) return rc_; } while (0)

enum { PK_HOST_PAGEABLE = 0, PK_HOST_PINNED = 1, PK_DEVICE = 2 };
static int pointer_kind(const void* p) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, p) != cudaSuccess) { cudaGetLastError(); return PK_HOST_PAGEABLE; }
  if (at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged) return PK_DEVICE;
  if (at.type == cudaMemoryTypeHost) return PK_HOST_PINNED;
  return PK_HOST_PAGEABLE;
}

extern "C" const char* taurus_last_cuda_error(void) { return g_cuda_err; }

extern "C" const char* taurus_strerror(int code) {
  switch (code) {
    case TAURUS_OK: return "ok";
    case TAURUS_ERR_INVALID_ARG: return "invalid argument";
    case TAURUS_ERR_ORDER: return "call out of order (chunk order, layer not begun, or layer incomplete)";
    case TAURUS_ERR_POOL_TOO_SMALL: return "accumulator pool too small for one chunk";
    case TAURUS_ERR_HOST_STORE_FULL: return "pinned host store for evicted rows is full";
    case TAURUS_ERR_DRAIN_FULL: return "graduation buffer could overflow: drain first";
    case TAURUS_ERR_CUDA: return "CUDA runtime error";
    case TAURUS_ERR_INTERNAL: return "device-side consistency check failed";
    case TAURUS_ERR_NOMEM: return "out of memory";
    case TAURUS_ERR_UNSUPPORTED: return "unsupported shape or size";
    case TAURUS_ERR_RUN_STORE_FULL: return "run store is full";
    case TAURUS_ERR_RUNS_INCOMPLETE: return "the runs do not hold every vertex of the chunk exactly once";
    default: return "unknown error";
  }
}

extern "C" void taurus_destroy(taurus_ctx* c) {
  if (!c) return;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(c->device);
  cudaDeviceSynchronize();
  cudaFree(c->d_row_ptr); cudaFree(c->d_col); cudaFree(c->d_din);
  for (int l = 0; l < TAURUS_MAX_LAYERS; ++l) { cudaFree(c->d_Wcat[l]); cudaFree(c->d_bias[l]); }
  free_tc_weights(c);
  cudaFree(c->d_pend); cudaFree(c->d_state); cudaFree(c->d_loc); cudaFree(c->d_touch); cudaFree(c->d_reload);
  cudaFree(c->d_hub); cudaFree(c->d_hub_ids); cudaFree(c->d_acc); cudaFree(c->d_owner); cudaFree(c->d_free_stack);
  cudaFree(c->d_touched_list); cudaFree(c->d_need_list); cudaFree(c->d_slot_epoch); cudaFree(c->d_slot_touch); cudaFree(c->d_slot_pend); cudaFree(c->d_victims); cudaFree(c->d_keys);
  cudaFree(c->d_cand[0]); cudaFree(c->d_cand[1]); cudaFree(c->d_ext_free); cudaFree(c->d_ext_live); cudaFree(c->d_bk_tail_ext);
  cudaFree(c->d_bk_tail_fill); cudaFree(c->d_bk_new); cudaFree(c->d_bk_off); cudaFree(c->d_bk_base); cudaFree(c->d_new_ext);
  cudaFree(c->d_vic_place); cudaFree(c->d_csc_src); cudaFree(c->d_ext_ret[0]); cudaFree(c->d_ext_ret[1]); cudaFree(c->d_xfer_list);
  cudaFree(c->d_stage_out);
  if (c->moves_ready) cudaEventDestroy(c->moves_ready);
  if (c->xfer_done) cudaEventDestroy(c->xfer_done);
  if (c->xfer_stream) cudaStreamDestroy(c->xfer_stream);
  delete c->pend_chunk;
  if (c->h_store) cudaFreeHost(c->h_store);
  cudaFree(c->d_grad_ids); cudaFree(c->d_grad_rows); cudaFree(c->d_done_list); cudaFree(c->d_X[0]); cudaFree(c->d_X[1]); cudaFree(c->d_PT);
  cudaFree(c->d_af_A); cudaFree(c->d_af_O); cudaFree(c->d_af_X);
  for (int l = 0; l < TAURUS_MAX_LAYERS; ++l) { cudaFree(c->d_Waf[l]); cudaFree(c->d_att_w[l]); }
  cudaFree(c->d_att_s); cudaFree(c->d_att_t); cudaFree(c->d_att_max); cudaFree(c->d_att_tm); cudaFree(c->d_att_z);
  cudaFree(c->d_csc_ptr); cudaFree(c->d_csc_eid); cudaFree(c->d_mask); cudaFree(c->d_vtmp); cudaFree(c->d_rank_hist);
  cudaFree(c->d_gdst); cudaFree(c->d_gedge); cudaFree(c->d_geid); cudaFree(c->d_gmask);
  cudaFree(c->d_ctl); cudaFree(c->d_chunk_log); cudaFree(c->d_reload_hist);
  if (c->h_ctl) cudaFreeHost(c->h_ctl);
  if (c->order_event) cudaEventDestroy(c->order_event);
  for (int i = 0; i < 2; ++i) {
    if (c->x_ready[i]) cudaEventDestroy(c->x_ready[i]);
    if (c->x_free[i]) cudaEventDestroy(c->x_free[i]);
    if (c->fin_done[i]) cudaEventDestroy(c->fin_done[i]);
    if (c->out_done[i]) cudaEventDestroy(c->out_done[i]);
  }
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->out_stream) cudaStreamDestroy(c->out_stream);
  for (auto& e : c->phase_ev) if (e) cudaEventDestroy(e);
  cudaGetLastError();
  cudaSetDevice(prev);
  delete c;
}

static int init_impl(taurus_ctx* c, const taurus_graph* g, const taurus_model* m, const taurus_run* r) {
  cudaDeviceProp prop;
  CU(cudaGetDevice(&c->device));
  CU(cudaGetDeviceProperties(&prop, c->device));
  c->sm_count = prop.multiProcessorCount;
  c->V = g->V; c->E = g->E; c->L = m->L; c->mode = m->mode; c->gemm_mode = m->gemm_mode; c->flags = r->flags;
  c->seed = r->seed;
  c->gin_eps = m->gin_eps;
  c->leaky = m->leaky_slope;
  c->heads = (m->mode == TAURUS_GAT && m->gat_heads > 1) ? m->gat_heads : 1;
  c->chunk_sources = r->chunk_sources; c->pool_slots = r->pool_slots; c->hub_count = r->hub_count;
  c->host_rows = r->host_evict_rows; c->drain_rows = r->drain_rows; c->evict_policy = r->evict_policy;
  bool any_sampled = false;
  for (int l = 0; l <= m->L; ++l) c->dims[l] = m->dims[l];
  for (int l = 0; l < m->L; ++l) {
    c->act[l] = m->act ? m->act[l] : 0;
    c->fanout[l] = r->fanout ? r->fanout[l] : 0;
    any_sampled |= c->fanout[l] > 0;
    c->Hmax = std::max(c->Hmax, taurus_round_up(c->dims[l + 1], 4));
    c->Kmax = std::max(c->Kmax, taurus_round_up(c->dims[l], 4));
    if (c->mode == TAURUS_GAT) c->Kmax = std::max(c->Kmax, taurus_round_up(c->dims[l + 1], 4));   // pass 3 streams h' rows
  }
  const long long V = c->V, E = c->E;

  // graph
  ALLOC(c->d_row_ptr, V + 1); ALLOC(c->d_col, E); ALLOC(c->d_din, V); ALLOC(c->d_vtmp, V);
  CU(cudaMemcpy(c->d_row_ptr, g->row_ptr, (size_t)(V + 1) * sizeof(long long), cudaMemcpyDefault));
  if (E > 0) CU(cudaMemcpy(c->d_col, g->col_idx, (size_t)E * sizeof(int32_t), cudaMemcpyDefault));
  CU(cudaMemcpy(c->d_din, g->in_degree, (size_t)V * sizeof(int32_t), cudaMemcpyDefault));
  long long ends[2] = {-1, -1};
  CU(cudaMemcpy(&ends[0], c->d_row_ptr, sizeof(long long), cudaMemcpyDeviceToHost));
  CU(cudaMemcpy(&ends[1], c->d_row_ptr + V, sizeof(long long), cudaMemcpyDeviceToHost));
  if (ends[0] != 0 || ends[1] != E) return TAURUS_ERR_INVALID_ARG;
  int bad = check_in_degrees(c, nullptr);
  if (bad < 0) return TAURUS_ERR_NOMEM;
  if (bad) return TAURUS_ERR_INVALID_ARG;
  CU(cudaGetLastError());

  // hub set: the hub_count largest by (in_degree descending, id ascending)
  ALLOC(c->d_hub, V); ALLOC(c->d_hub_ids, c->hub_count);
  CU(cudaMemset(c->d_hub, 0, (size_t)V));
  if (c->hub_count > 0) {
    std::vector<int32_t> din((size_t)V);
    CU(cudaMemcpy(din.data(), c->d_din, (size_t)V * sizeof(int32_t), cudaMemcpyDeviceToHost));
    std::vector<unsigned long long> key((size_t)V);
    for (long long v = 0; v < V; ++v)
      key[(size_t)v] = ((unsigned long long)(0x7fffffffu - (unsigned)din[(size_t)v]) << 32) | (unsigned long long)v;
    std::nth_element(key.begin(), key.begin() + (c->hub_count - 1), key.end());
    std::sort(key.begin(), key.begin() + c->hub_count);
    std::vector<int32_t> ids((size_t)c->hub_count);
    std::vector<uint8_t> flag((size_t)V, 0);
    for (long long i = 0; i < c->hub_count; ++i) { ids[(size_t)i] = (int32_t)(key[(size_t)i] & 0xffffffffu); flag[(size_t)ids[(size_t)i]] = 1; }
    CU(cudaMemcpy(c->d_hub_ids, ids.data(), ids.size() * sizeof(int32_t), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(c->d_hub, flag.data(), flag.size(), cudaMemcpyHostToDevice));
  }

  // aggregate-first layers: input rows at most 3/4 as wide as output rows.  SAGE keeps every vertex's input row until
  // the vertex completes (its self term goes through W_self with the transform): only while that store stays small.
  int af_kmax = 0;
  size_t free_b = 0, total_b = 0;
  CU(cudaMemGetInfo(&free_b, &total_b));
  // what the context still allocates besides that store, roughly: pool and hub rows, the grouped edge order (12 B per
  // edge, 20 B while it is sorted), in-lists where rows can be evicted or layers are sampled, per-vertex words
  const double other = (double)(c->pool_slots + c->hub_count) * c->Hmax * 4.0 + (double)E * 28.0 + (double)V * 64.0 +
                       (double)c->pool_slots * 40.0 + (double)c->drain_rows * c->Hmax * 8.0;
  for (int l = 0; l < c->L; ++l) {
    const int Kp = taurus_round_up(c->dims[l], 4), Hp = taurus_round_up(c->dims[l + 1], 4);
    bool af = !(c->flags & TAURUS_FLAG_PROJECT_FIRST) && 4 * Kp <= 3 * Hp;
    if (c->heads > 1) af = false;   // every head weights the messages differently: the sums cannot be shared in input space
    // SAGE keeps V input rows on the device for such a layer: only while they fit beside everything else
    if (af && c->mode == TAURUS_SAGE_MEAN && (double)V * Kp * sizeof(float) + other > 0.92 * (double)free_b) af = false;
    c->agg_first[l] = af;
    if (af) af_kmax = std::max(af_kmax, Kp);
  }

  // weights: Wcat = [W_neigh | W_self] with both halves padded to Hp columns
  for (int l = 0; l < c->L; ++l) {
    const int K = c->dims[l], d_out = c->dims[l + 1], Hp = taurus_round_up(d_out, 4);
    const int N = taurus_proj_width(c->mode, Hp, c->heads);
    std::vector<float> wn((size_t)K * d_out), ws, b((size_t)Hp, 0.f), cat((size_t)K * N, 0.f);
    CU(cudaMemcpy(wn.data(), m->W_neigh[l], wn.size() * sizeof(float), cudaMemcpyDefault));
    if (c->mode == TAURUS_SAGE_MEAN) {
      ws.resize((size_t)K * d_out);
      CU(cudaMemcpy(ws.data(), m->W_self[l], ws.size() * sizeof(float), cudaMemcpyDefault));
    }
    if (m->bias && m->bias[l]) CU(cudaMemcpy(b.data(), m->bias[l], (size_t)d_out * sizeof(float), cudaMemcpyDefault));
    for (int k = 0; k < K; ++k)
      for (int j = 0; j < d_out; ++j) {
        cat[(size_t)k * N + j] = wn[(size_t)k * d_out + j];
        if (c->mode == TAURUS_SAGE_MEAN) cat[(size_t)k * N + Hp + j] = ws[(size_t)k * d_out + j];
      }
    if (c->mode == TAURUS_GAT) {   // two more columns per head, W att_src and W att_dst over the head's block: the attention scalars come out of the same GEMM
      std::vector<float> as((size_t)d_out), ad((size_t)d_out);
      CU(cudaMemcpy(as.data(), m->att_src[l], as.size() * sizeof(float), cudaMemcpyDefault));
      CU(cudaMemcpy(ad.data(), m->att_dst[l], ad.size() * sizeof(float), cudaMemcpyDefault));
      const int dh = d_out / c->heads;
      for (int k = 0; k < K; ++k)
        for (int hd = 0; hd < c->heads; ++hd) {
          double ss = 0.0, sd = 0.0;
          for (int j = hd * dh; j < (hd + 1) * dh; ++j) { ss += (double)wn[(size_t)k * d_out + j] * as[(size_t)j]; sd += (double)wn[(size_t)k * d_out + j] * ad[(size_t)j]; }
          cat[(size_t)k * N + Hp + 2 * hd] = (float)ss;
          cat[(size_t)k * N + Hp + 2 * hd + 1] = (float)sd;
        }
      std::vector<float> wv((size_t)2 * K);   // the same two vectors on their own, for layers that never form the transformed rows
      for (int k = 0; k < K; ++k) { wv[(size_t)k] = cat[(size_t)k * N + Hp]; wv[(size_t)K + k] = cat[(size_t)k * N + Hp + 1]; }
      ALLOC(c->d_att_w[l], wv.size());
      CU(cudaMemcpy(c->d_att_w[l], wv.data(), wv.size() * sizeof(float), cudaMemcpyHostToDevice));
    }
    ALLOC(c->d_Wcat[l], cat.size()); ALLOC(c->d_bias[l], b.size());
    CU(cudaMemcpy(c->d_Wcat[l], cat.data(), cat.size() * sizeof(float), cudaMemcpyHostToDevice));
    CU(cudaMemcpy(c->d_bias[l], b.data(), b.size() * sizeof(float), cudaMemcpyHostToDevice));
    if (!(c->flags & TAURUS_FLAG_SIMT_GEMM)) {
      int rc = prepare_tc_weights(c, &c->tc_image[l], cat, K, N);
      if (rc == TAURUS_ERR_NOMEM) return rc;
      if (rc != TAURUS_OK) { cudaGetLastError(); free_tc_weights(c); }   // no tensor-map support: the FFMA kernel is used
    }
    if (c->agg_first[l] && c->mode == TAURUS_SAGE_MEAN) {
      // [W_neigh ; W_self] stacked along K (each padded to Kp rows): one product transforms [c_in * agg | h_v]
      const int Kp = taurus_round_up(K, 4);
      std::vector<float> st2((size_t)2 * Kp * Hp, 0.f);
      for (int k = 0; k < K; ++k)
        for (int j = 0; j < d_out; ++j) {
          st2[(size_t)k * Hp + j] = wn[(size_t)k * d_out + j];
          st2[(size_t)(Kp + k) * Hp + j] = ws[(size_t)k * d_out + j];
        }
      ALLOC(c->d_Waf[l], st2.size());
      CU(cudaMemcpy(c->d_Waf[l], st2.data(), st2.size() * sizeof(float), cudaMemcpyHostToDevice));
      if (!(c->flags & TAURUS_FLAG_SIMT_GEMM) && c->tc_image[l]) {
        int rc = prepare_tc_weights(c, &c->tc_image_af[l], st2, 2 * Kp, Hp);
        if (rc == TAURUS_ERR_NOMEM) return rc;
        if (rc != TAURUS_OK) { cudaGetLastError(); free_tc_weights(c); }
      }
    }
  }

  // per-vertex state
  ALLOC(c->d_pend, V); ALLOC(c->d_state, V); ALLOC(c->d_loc, V); ALLOC(c->d_touch, V); ALLOC(c->d_reload, V);
  ALLOC(c->d_rank_hist, (V + 63) / 64);
  // pool, hub store
  ALLOC(c->d_acc, (size_t)(c->pool_slots + c->hub_count) * c->Hmax);
  {
    // a push of at most chunk_sources sources touches at most its edges plus its own vertices
    long long max_edges = max_window_edges(c);
    if (max_edges < 0) return TAURUS_ERR_CUDA;
    c->touched_capacity = std::min<long long>(V, max_edges + c->chunk_sources);
    ALLOC(c->d_touched_list, c->touched_capacity);
  }
  ALLOC(c->d_owner, c->pool_slots); ALLOC(c->d_free_stack, c->pool_slots); ALLOC(c->d_need_list, c->pool_slots);
  ALLOC(c->d_slot_epoch, c->pool_slots);   // written at every slot hand-out, also when no eviction can happen
  const bool can_evict = c->pool_slots < V - c->hub_count;
  if (can_evict) {   // a chunk evicts at most what it needs, and it needs at most what it touches
    c->victim_capacity = std::min<long long>(c->pool_slots, c->touched_capacity);
    ALLOC(c->d_victims, c->victim_capacity); ALLOC(c->d_keys, c->pool_slots);
    ALLOC(c->d_cand[0], c->pool_slots); ALLOC(c->d_cand[1], c->pool_slots);
    ALLOC(c->d_slot_touch, c->pool_slots); ALLOC(c->d_slot_pend, c->pool_slots);
    ALLOC(c->d_vic_place, c->victim_capacity);
  }
  if (can_evict && c->host_rows > 0) {
    // Host store of evicted rows: extents of 2^ext_shift rows.  Evicted rows are filed by the grid cell of their
    // vertex's next sender (one open extent per cell), so the store holds up to one partly filled extent per cell on
    // top of the rows themselves; twice that many spare extents cover pushes that are not whole grid cells.
    c->n_buckets = (V + c->chunk_sources - 1) / c->chunk_sources;
    long long per = c->host_rows / (4 * c->n_buckets);
    c->ext_shift = 3;
    while (c->ext_shift < 10 && (2ll << c->ext_shift) <= per) c->ext_shift += 1;
    const long long ext_rows = 1ll << c->ext_shift;
    // ... and the extents emptied by one chunk's reloads wait for two chunks before they return to the free stack
    c->n_ext = (c->host_rows + ext_rows - 1) / ext_rows + 2 * c->n_buckets + 8 + 2 * ((c->victim_capacity >> c->ext_shift) + 1);
    if (c->n_ext * ext_rows >= (1ll << 31) - 2) return TAURUS_ERR_INVALID_ARG;
    ALLOC(c->d_ext_free, c->n_ext); ALLOC(c->d_ext_live, c->n_ext);
    ALLOC(c->d_bk_tail_ext, c->n_buckets); ALLOC(c->d_bk_tail_fill, c->n_buckets); ALLOC(c->d_bk_new, c->n_buckets);
    ALLOC(c->d_bk_off, c->n_buckets); ALLOC(c->d_bk_base, c->n_buckets);
    ALLOC(c->d_new_ext, (c->victim_capacity >> c->ext_shift) + c->n_buckets + 1);
    ALLOC(c->d_ext_ret[0], c->n_ext); ALLOC(c->d_ext_ret[1], c->n_ext);
    ALLOC(c->d_xfer_list, std::min<long long>(c->pool_slots, c->touched_capacity));   // one entry per need-list entry: a chunk needs at most what it touches
    ALLOC(c->d_stage_out, (size_t)c->victim_capacity * c->Hmax);
    CU(cudaStreamCreateWithFlags(&c->xfer_stream, cudaStreamNonBlocking));
    CU(cudaEventCreateWithFlags(&c->moves_ready, cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&c->xfer_done, cudaEventDisableTiming));
    c->pipelined = true;
    cudaError_t e = cudaHostAlloc((void**)&c->h_store, (size_t)c->n_ext * ext_rows * c->Hmax * sizeof(float), cudaHostAllocMapped);
    if (e != cudaSuccess) { cuda_ok(e, "cudaHostAlloc(evicted-row store)"); c->h_store = nullptr; return TAURUS_ERR_NOMEM; }
    CU(cudaHostGetDevicePointer((void**)&c->d_store_alias, c->h_store, 0));
  }
  // graduation buffer, chunk buffers
  ALLOC(c->d_grad_ids, c->drain_rows); ALLOC(c->d_grad_rows, (size_t)c->drain_rows * c->Hmax); ALLOC(c->d_done_list, c->drain_rows);
  ALLOC(c->d_X[0], (size_t)c->chunk_sources * c->Kmax);
  ALLOC(c->d_X[1], (size_t)c->chunk_sources * c->Kmax);
  CU(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  CU(cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking));
  for (int i = 0; i < 2; ++i) {
    CU(cudaEventCreateWithFlags(&c->x_ready[i], cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&c->x_free[i], cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&c->fin_done[i], cudaEventDisableTiming));
    CU(cudaEventCreateWithFlags(&c->out_done[i], cudaEventDisableTiming));
  }
  ALLOC(c->d_PT, (size_t)c->chunk_sources * 2 * c->Hmax);
  if (c->mode == TAURUS_GAT) {
    const size_t nh = (size_t)V * c->heads;
    ALLOC(c->d_att_s, nh); ALLOC(c->d_att_t, nh); ALLOC(c->d_att_max, nh); ALLOC(c->d_att_tm, nh); ALLOC(c->d_att_z, nh);
  }
  if (af_kmax > 0) {
    const bool sage = c->mode == TAURUS_SAGE_MEAN;
    ALLOC(c->d_af_A, (size_t)c->drain_rows * af_kmax * (sage ? 2 : 1));
    // rows behind a chunk's finished ones are read (and their products dropped) by the last row tile: keep them finite
    CU(cudaMemset(c->d_af_A, 0, (size_t)c->drain_rows * af_kmax * (sage ? 2 : 1) * sizeof(float)));
    if (sage) ALLOC(c->d_af_X, (size_t)V * af_kmax);
  }
  // In-lists (ascending source id).  Sampled layers pick in-list positions; the host store files an evicted row by the
  // next sender of its vertex, read from the vertex's in-list.
  const bool grouping = !(c->flags & TAURUS_FLAG_NO_GROUPING);
  const bool need_src = c->n_ext > 0;
  if (any_sampled || (need_src && !grouping)) {
    int rc = build_in_edge_order(c);
    if (rc) { cuda_ok(cudaGetLastError(), "build_in_edge_order"); return rc; }
    if (any_sampled) ALLOC(c->d_mask, (E + 31) / 32);
  }
  bool src_from_groups = false;
  if (need_src) {
    ALLOC(c->d_csc_src, E);
    if (c->d_csc_eid) {
      int rc = build_csc_src_from_eid(c);
      if (rc) { cuda_ok(cudaGetLastError(), "build_csc_src_from_eid"); return rc; }
      if (!any_sampled) { cudaFree(c->d_csc_eid); c->d_csc_eid = nullptr; }
    } else {
      int rc = build_csc_ptr(c);
      if (rc) { cuda_ok(cudaGetLastError(), "build_csc_ptr"); return rc; }
      src_from_groups = true;
    }
  }
  // destination-grouped edge order of the chunk grid
  if (grouping) {
    int rc = build_grouped_order(c, any_sampled, src_from_groups);
    if (rc) { cuda_ok(cudaGetLastError(), "build_grouped_order"); return rc; }
    if (any_sampled) ALLOC(c->d_gmask, (E + 31) / 32);
  }
  // control
  ALLOC(c->d_ctl, 1);
  ALLOC(c->d_reload_hist, 18);
  CU(cudaMemset(c->d_ctl, 0, sizeof(DevCtl)));
  CU(cudaHostAlloc((void**)&c->h_ctl, sizeof(DevCtl), cudaHostAllocDefault));
  memset(c->h_ctl, 0, sizeof(DevCtl));
  c->log_capacity = std::max<long long>(1024, 4 * ((V + c->chunk_sources - 1) / c->chunk_sources));
  ALLOC(c->d_chunk_log, (size_t)c->log_capacity * TAURUS_CK_COLUMNS);
  CU(cudaEventCreateWithFlags(&c->order_event, cudaEventDisableTiming));
  c->rank_cum_cache.assign((size_t)c->L, std::vector<long long>());
  CU(cudaDeviceSynchronize());
  return TAURUS_OK;
}

extern "C" int taurus_graph_init(taurus_ctx** out, const taurus_graph* g, const taurus_model* m, const taurus_run* r) {
  if (!out) return TAURUS_ERR_INVALID_ARG;
  *out = nullptr;
  if (!g || !m || !r || !g->row_ptr || !g->in_degree || (g->E > 0 && !g->col_idx)) return TAURUS_ERR_INVALID_ARG;
  if (g->V < 1 || g->V >= (1ll << 31) || g->E < 0 || g->E >= (1ll << 32)) return TAURUS_ERR_INVALID_ARG;
  if (m->L < 1 || m->L > TAURUS_MAX_LAYERS || !m->dims || !m->W_neigh) return TAURUS_ERR_INVALID_ARG;
  if (m->mode != TAURUS_SAGE_MEAN && m->mode != TAURUS_GCN_SYM && m->mode != TAURUS_GIN_SUM && m->mode != TAURUS_GAT) return TAURUS_ERR_INVALID_ARG;
  if (m->mode == TAURUS_GAT) {
    if (!m->att_src || !m->att_dst || !(m->leaky_slope >= 0.f && m->leaky_slope <= 1.f)) return TAURUS_ERR_INVALID_ARG;
    if (m->gemm_mode != TAURUS_GEMM_FP32) return TAURUS_ERR_UNSUPPORTED;   // the scores need the fp32-accurate projection
    if (m->gat_heads < 0 || m->gat_heads > 16) return TAURUS_ERR_INVALID_ARG;
    if (m->gat_heads > 1)
      for (int l = 0; l < m->L; ++l)
        if (m->dims[l + 1] % (4 * m->gat_heads) != 0) return TAURUS_ERR_INVALID_ARG;   // a head is a whole number of float4
    for (int l = 0; l < m->L; ++l)
      if (!m->att_src[l] || !m->att_dst[l]) return TAURUS_ERR_INVALID_ARG;
  }
  if (m->gemm_mode != TAURUS_GEMM_FP32 && m->gemm_mode != TAURUS_GEMM_BF16) return TAURUS_ERR_INVALID_ARG;
  if (m->mode == TAURUS_SAGE_MEAN && !m->W_self) return TAURUS_ERR_INVALID_ARG;
  for (int l = 0; l <= m->L; ++l)
    if (m->dims[l] < 1 || m->dims[l] > TAURUS_MAX_DIM) return TAURUS_ERR_INVALID_ARG;
  for (int l = 0; l < m->L; ++l) {
    if (!m->W_neigh[l] || (m->mode == TAURUS_SAGE_MEAN && !m->W_self[l])) return TAURUS_ERR_INVALID_ARG;
    if (r->fanout && (r->fanout[l] < 0 || r->fanout[l] > TAURUS_MAX_FANOUT)) return TAURUS_ERR_INVALID_ARG;
  }
  if (r->chunk_sources < 1 || r->chunk_sources > (1 << 24) || r->pool_slots < 1 || r->pool_slots >= (1ll << 31)) return TAURUS_ERR_INVALID_ARG;
  if (r->hub_count < 0 || r->hub_count > g->V || r->host_evict_rows < 0 || r->host_evict_rows >= (1ll << 31)) return TAURUS_ERR_INVALID_ARG;
  if (r->drain_rows < 1 || r->drain_rows >= (1ll << 31)) return TAURUS_ERR_INVALID_ARG;
  if (r->evict_policy < TAURUS_EVICT_FEWEST_PENDING || r->evict_policy > TAURUS_EVICT_RANDOM) return TAURUS_ERR_INVALID_ARG;
  if (r->pool_slots + r->hub_count >= (1ll << 31)) return TAURUS_ERR_INVALID_ARG;
  taurus_ctx* c = new (std::nothrow) taurus_ctx();
  if (!c) return TAURUS_ERR_NOMEM;
  c->pend_chunk = new (std::nothrow) PendingChunk();
  if (!c->pend_chunk) { delete c; return TAURUS_ERR_NOMEM; }
  int rc;
  try { rc = init_impl(c, g, m, r); } catch (const std::bad_alloc&) { rc = TAURUS_ERR_NOMEM; }
  if (rc != TAURUS_OK) { taurus_destroy(c); return rc; }
  *out = c;
  return TAURUS_OK;
}

// Reads the device control block (after synchronising `st`) and returns its sticky error.
static int finish_chunk(taurus_ctx* c, cudaStream_t st);
static int read_ctl(taurus_ctx* c, cudaStream_t st) {
  { int rc = finish_chunk(c, st); if (rc) return rc; }   // the last chunk's finalise may still be waiting for a successor
  CU(cudaStreamSynchronize(st));
  CU(cudaStreamSynchronize(c->out_stream));
  CU(cudaMemcpy(c->h_ctl, c->d_ctl, sizeof(DevCtl), cudaMemcpyDeviceToHost));
  return c->h_ctl->error;
}

extern "C" int taurus_layer_begin(taurus_ctx* c, int32_t layer, void* cuda_stream) {
  if (!c || layer < 0 || layer >= c->L) return TAURUS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CU(cudaSetDevice(c->device));
  if (c->last_stream != st) CU(cudaStreamSynchronize(c->last_stream));
  CU(cudaStreamSynchronize(c->copy_stream));
  CU(cudaStreamSynchronize(c->out_stream));
  if (c->xfer_stream) CU(cudaStreamSynchronize(c->xfer_stream));
  c->pending = false;   // an abandoned layer's last chunk is dropped with it
  c->layer = layer;
  c->dense_out = nullptr; c->dense_ld = 0;
  c->run_out = nullptr; c->run_pending_half = -1;
  c->gat_next_src = 0; c->gat_ready = false;
  c->half_used[0] = c->half_used[1] = false;
  c->x_used[0] = c->x_used[1] = false;
  memset(c->h_ctl, 0, sizeof(DevCtl));
  c->next_src = 0; c->chunk_seq = 0; c->ub_since_drain = 0; c->last_stream = st;
  launch_layer_reset(c, layer, st);
  c->d_mask_cur = nullptr;
  if (c->fanout[layer] > 0) {
    launch_sample_mask(c, layer, st);
    c->d_mask_cur = c->d_mask;
    if (c->d_gdst) launch_group_mask(c, st);
  }
  if (c->rank_cum_cache[(size_t)layer].empty()) {
    // completion ranks depend only on the topology and the layer's edge mask: computed once per layer
    launch_completion_ranks(c, st);
    CU(cudaGetLastError());
    const long long nb = (c->V + 63) / 64;
    std::vector<int32_t> hist((size_t)nb);
    CU(cudaMemcpyAsync(hist.data(), c->d_rank_hist, (size_t)nb * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    std::vector<long long>& cum = c->rank_cum_cache[(size_t)layer];
    cum.assign((size_t)nb + 1, 0);
    for (long long i = 0; i < nb; ++i) cum[(size_t)i + 1] = cum[(size_t)i] + hist[(size_t)i];
  }
  c->rank_cum = &c->rank_cum_cache[(size_t)layer];
  CU(cudaGetLastError());
  CU(cudaStreamSynchronize(st));
  return TAURUS_OK;
}

static long long completion_bound(const taurus_ctx* c, long long s, long long e) {
  const std::vector<long long>& cum = *c->rank_cum;
  const long long nb = (long long)cum.size() - 1;
  long long b0 = s / 64, b1 = std::min(nb, (e + 63) / 64);
  return cum[(size_t)b1] - cum[(size_t)b0];
}

extern "C" int taurus_completion_bound(taurus_ctx* c, int64_t src_begin, int64_t src_end, int64_t* out_bound) {
  if (!c || !out_bound || src_begin < 0 || src_end > c->V || src_begin > src_end) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  *out_bound = completion_bound(c, src_begin, src_end);
  return TAURUS_OK;
}

static ChunkArgs make_args(taurus_ctx* c, long long s, long long e) {
  ChunkArgs a;
  const int l = c->layer;
  a.row_ptr = c->d_row_ptr; a.col = c->d_col; a.din = c->d_din; a.mask = c->d_mask_cur;
  a.pend = c->d_pend; a.state = c->d_state; a.loc = c->d_loc; a.touch = c->d_touch; a.reload_count = c->d_reload;
  a.acc = c->d_acc; a.owner = c->d_owner; a.free_stack = c->d_free_stack; a.need_list = c->d_need_list; a.slot_epoch = c->d_slot_epoch;
  a.slot_touch = c->d_slot_touch; a.slot_pend = c->d_slot_pend;
  a.touched_list = c->d_touched_list; a.touched_capacity = c->touched_capacity;
  a.victims = c->d_victims; a.victim_capacity = c->victim_capacity; a.keys = c->d_keys; a.host_store = c->d_store_alias;
  a.cand[0] = c->d_cand[0]; a.cand[1] = c->d_cand[1];
  a.ext_free = c->d_ext_free; a.ext_live = c->d_ext_live; a.bk_tail_ext = c->d_bk_tail_ext; a.bk_tail_fill = c->d_bk_tail_fill;
  a.bk_new = c->d_bk_new; a.bk_off = c->d_bk_off; a.bk_base = c->d_bk_base; a.new_ext = c->d_new_ext; a.vic_place = c->d_vic_place;
  a.csc_ptr = c->d_csc_ptr; a.csc_src = c->d_csc_src; a.csc_eid = c->d_csc_eid;
  a.ext_ret[0] = c->d_ext_ret[0]; a.ext_ret[1] = c->d_ext_ret[1]; a.xfer_list = c->d_xfer_list; a.stage_out = c->d_stage_out;
  a.chunk_sources = c->chunk_sources; a.n_ext = c->n_ext; a.n_buckets = c->n_buckets; a.ext_shift = c->ext_shift;
  a.grad_ids = c->d_grad_ids; a.grad_rows = c->d_grad_rows; a.done_list = c->d_done_list;
  a.Hp = taurus_round_up(c->dims[l + 1], 4);
  a.PT = c->d_PT; a.ldpt = c->mode == TAURUS_SAGE_MEAN ? 2 * a.Hp : a.Hp;   // GAT pass 3 scatters h' rows repacked to pitch Hp
  a.att_s = c->d_att_s; a.att_tm = c->d_att_tm; a.att_z = c->d_att_z; a.leaky = c->leaky;
  a.heads = c->heads; a.head_vec = (taurus_round_up(c->dims[l + 1], 4) / c->heads) >> 2;
  a.bias = c->d_bias[l];
  a.ctl = c->d_ctl; a.pc = &c->d_ctl->pc[c->chunk_seq & 1]; a.chunk_log = c->d_chunk_log; a.log_capacity = c->log_capacity;
  a.V = c->V; a.pool_slots = c->pool_slots; a.hub_count = c->hub_count; a.host_rows = c->host_rows; a.drain_rows = c->drain_rows;
  a.src_begin = s; a.src_end = e;
  a.epoch = (int32_t)(c->chunk_seq + 1);
  a.mode = c->mode; a.act = c->act[l]; a.fanout = c->fanout[l]; a.evict_policy = c->evict_policy; a.seed = c->seed;
  a.gin_self = 1.0f + c->gin_eps;
  a.direct = c->pool_slots >= c->V ? 1 : 0;
  a.dynamic_spans = c->pipelined ? 1 : 0;
  const bool direct_dense = c->dense_out && c->dense_is_device;
  const bool halves = (c->dense_out && !direct_dense) || c->run_out;   // the graduation buffer alternates between two halves
  a.dense_direct = direct_dense ? c->dense_out : nullptr;
  a.dense_ld = c->dense_ld;
  a.d_out = c->dims[l + 1];
  a.Hout = a.Hp; a.self_rows = 1; a.self_bias = 1;
  a.dense_half = halves ? (int)(c->chunk_seq & 1) : -1;
  a.grad_cap = halves ? c->drain_rows / 2 : c->drain_rows;
  a.grad_off = halves ? (long long)a.dense_half * (c->drain_rows / 2) : 0;
  return a;
}

// Run-output mode: phase 2 of the append that is still open (rows of half run_pending_half), on the output stream.
static int finish_run_append(taurus_ctx* c) {
  if (!c->run_out || c->run_pending_half < 0) return TAURUS_OK;
  const int h = c->run_pending_half;
  c->run_pending_half = -1;
  int rc = runs_phase2(c->run_out, c->out_stream);
  if (rc) return rc;
  CU(cudaEventRecord(c->out_done[h], c->out_stream));
  c->half_used[h] = true;
  return TAURUS_OK;
}

static int finish_chunk(taurus_ctx* c, cudaStream_t st) {
  if (!c->pending) return TAURUS_OK;
  c->pending = false;
  const PendingChunk& p = *c->pend_chunk;
  const ChunkArgs& a = p.a;
  const int l = p.layer;
  cudaEvent_t* pev = p.timed_index >= 0 && c->timing != 2 ? &c->phase_ev[(size_t)p.timed_index * TAURUS_PUSH_EVENTS] : nullptr;
  if (c->pipelined) {
    CU(cudaStreamWaitEvent(st, c->xfer_done, 0));   // reloaded partial sums have been added to the chunk's rows
    if (pev) cudaEventRecord(pev[8], st);           // (without transfers the finalise follows event 7 directly)
  }
  if (a.dense_half >= 0 && c->half_used[a.dense_half]) CU(cudaStreamWaitEvent(st, c->out_done[a.dense_half], 0));
  if (p.af) {
    int rc = launch_af_finalise(c, a, l, std::min<long long>(p.bound, a.grad_cap), st);
    if (rc) { c->h_ctl->error = rc; return rc; }   // the chunk is half applied: the layer has to be begun again
  } else {
    launch_finalise(c, a, st);
  }
  int run_rc = TAURUS_OK;
  if (a.dense_half >= 0 && c->dense_out) {   // hand this chunk's rows to the output stream (matrix in pinned host memory)
    const int h = a.dense_half, d_out = c->dims[l + 1];
    CU(cudaEventRecord(c->fin_done[h], st));
    CU(cudaStreamWaitEvent(c->out_stream, c->fin_done[h], 0));
    launch_place_half(c, h, d_out, a.Hout, c->out_stream);
    CU(cudaEventRecord(c->out_done[h], c->out_stream));
    c->half_used[h] = true;
  } else if (a.dense_half >= 0) {
    // Run-output mode.  The previous chunk's rows are already grouped by id range and its per-range counts are
    // on their way to the host: now that this chunk's kernels are queued behind it, wait for them (the device
    // stays busy), move those rows into the partition buffers and flush the full ones; then group this chunk's
    // rows once its finalise has run.
    const int h = a.dense_half;
    CU(cudaEventRecord(c->fin_done[h], st));
    run_rc = finish_run_append(c);
    if (!run_rc) {
      CU(cudaStreamWaitEvent(c->out_stream, c->fin_done[h], 0));
      const long long off = a.grad_off;
      run_rc = runs_phase1(c->run_out, c->d_grad_ids + off, c->d_grad_rows + (size_t)off * a.Hout, a.Hout, std::min(p.bound, a.grad_cap),
                           &c->d_ctl->out_count[h], 0, c->out_stream);
      if (!run_rc) c->run_pending_half = h;
    }
  }
  if (pev) cudaEventRecord(pev[9], st);
  CU(cudaGetLastError());
  return run_rc;
}

// S1: features of sources [s, e) ([n x K], rows contiguous) to the device.  Host chunks are copied on the library's
// copy stream into one of two staging buffers, so that the copy of chunk k+1 overlaps the kernels of chunk k; a
// chunk read from sorted runs is merged into the same buffers; a device pointer is used in place (*xbuf = -1).
static int stage_chunk(taurus_ctx* c, const float* features, taurus_runs* src_runs, long long s, long long e, int K, cudaStream_t st,
                       const float** X, int* xbuf) {
  *X = features;
  *xbuf = -1;
  if (!src_runs && pointer_kind(features) == PK_DEVICE) return TAURUS_OK;
  const int b = (int)(c->host_pushes & 1);
  if (c->x_used[b]) CU(cudaStreamWaitEvent(c->copy_stream, c->x_free[b], 0));
  if (src_runs) {   // merge-on-read; fails before anything is enqueued when the runs do not cover the chunk
    int rc = runs_read_into(src_runs, s, e, c->d_X[b], K, c->copy_stream);
    if (rc) return rc;
  } else {
    CU(cudaMemcpyAsync(c->d_X[b], features, (size_t)(e - s) * K * sizeof(float), cudaMemcpyHostToDevice, c->copy_stream));
  }
  c->host_pushes += 1;
  CU(cudaEventRecord(c->x_ready[b], c->copy_stream));
  CU(cudaStreamWaitEvent(st, c->x_ready[b], 0));
  *X = c->d_X[b];
  *xbuf = b;
  return TAURUS_OK;
}

// One chunk through S1..S7.  The features come from `features` (host or device memory) or, when `src_runs` is
// given, from the sorted runs of the previous layer by merge-on-read.
static int push_core(taurus_ctx* c, int64_t src_begin, int64_t src_end, const float* features, taurus_runs* src_runs, void* cuda_stream) {
  if (!c || (!features && !src_runs)) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  if (src_begin != c->next_src) return TAURUS_ERR_ORDER;
  if (src_end <= src_begin || src_end > c->V || src_end - src_begin > c->chunk_sources) return TAURUS_ERR_INVALID_ARG;
  if (features && (reinterpret_cast<uintptr_t>(features) & 3) != 0) return TAURUS_ERR_INVALID_ARG;
  const bool gat = c->mode == TAURUS_GAT;   // pass 3: the features are the transformed rows h'
  if (gat && !c->gat_ready) return TAURUS_ERR_ORDER;
  if (src_runs && (runs_width(src_runs) != c->dims[c->layer + (gat ? 1 : 0)] || runs_vertices(src_runs) != c->V ||
                   runs_max_chunk(src_runs) < src_end - src_begin || src_runs == c->run_out))
    return TAURUS_ERR_INVALID_ARG;
  if (c->h_ctl->error) return c->h_ctl->error;
  const long long bound = completion_bound(c, src_begin, src_end);
  const bool direct_dense = c->dense_out && c->dense_is_device;   // rows are finalised straight into the caller's matrix
  const bool halves = (c->dense_out && !direct_dense) || c->run_out;
  if (halves ? bound > c->drain_rows / 2 : (direct_dense ? bound : c->ub_since_drain + bound) > c->drain_rows) return TAURUS_ERR_DRAIN_FULL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CU(cudaSetDevice(c->device));
  const int l = c->layer;
  if (c->agg_first[l] && !direct_dense && !halves && !c->d_af_O) {
    // rows drained by the caller: their place in the graduation buffer is a device-side count, so the transform of
    // the finished rows writes a scratch matrix first.  Allocated here, before anything of the chunk is enqueued, so
    // that a failure leaves the layer untouched.
    ALLOC(c->d_af_O, (size_t)c->drain_rows * c->Hmax);
  }
  if (st != c->last_stream) {   // keep chunk order across streams
    CU(cudaEventRecord(c->order_event, c->last_stream));
    CU(cudaStreamWaitEvent(st, c->order_event, 0));
    c->last_stream = st;
  }
  const int K = gat ? c->dims[l + 1] : c->dims[l];
  const int n = (int)(src_end - src_begin);
  cudaEvent_t* pev = nullptr;
  if (c->timing && c->timed_pushes < TAURUS_MAX_TIMED_PUSHES) {
    const size_t need = (size_t)(c->timed_pushes + 1) * TAURUS_PUSH_EVENTS;
    while (c->phase_ev.size() < need) { cudaEvent_t e; CU(cudaEventCreate(&e)); c->phase_ev.push_back(e); }
    pev = &c->phase_ev[(size_t)c->timed_pushes * TAURUS_PUSH_EVENTS];
    c->timed_pushes += 1;
  }
  const bool scatter_timing = pev != nullptr;           // level 2 records the two events around the scatter only
  const bool timing = pev != nullptr && c->timing != 2;
  if (timing) cudaEventRecord(pev[0], st);
  // S1: features to the device
  const float* X = nullptr;
  int ldx = K;
  int xbuf = -1;
  { int rc = stage_chunk(c, features, src_runs, src_begin, src_end, K, st, &X, &xbuf); if (rc) return rc; }
  if (timing) cudaEventRecord(pev[1], st);
  ChunkArgs a = make_args(c, src_begin, src_end);
  // S2: projection (GAT: already done in pass 1; rows narrower than their padded width are repacked).
  // Aggregate-first layers push the (scaled, padded) input rows instead and transform the finished rows in S7.
  bool x_in_use = false;
  const bool af = c->agg_first[l];
  if (af && gat) {
    // pass 3 of an aggregate-first GAT layer: the rows handed back by pass 1 are the zero-padded INPUT rows (pitch
    // dims[l+1]); their first pad4(dims[l]) columns are what the attention-weighted scatter pushes
    const int Kp = taurus_round_up(c->dims[l], 4);
    a.Hout = a.Hp; a.Hp = Kp; a.self_rows = 1; a.self_bias = 0;
    if ((K & 3) == 0 && (reinterpret_cast<uintptr_t>(X) & 15) == 0) { a.PT = X; a.ldpt = K; x_in_use = true; }
    else { launch_gat_repack(c, X, n, K, Kp, st); a.ldpt = Kp; }
  } else if (af) {
    const int Kp = taurus_round_up(K, 4);
    a.Hout = a.Hp; a.Hp = Kp; a.ldpt = Kp;
    a.self_rows = c->mode == TAURUS_SAGE_MEAN ? 0 : 1;
    a.self_bias = 0;
    if (c->mode == TAURUS_SAGE_MEAN) {
      // the chunk's (padded) input rows go to the per-vertex store: the scatter pushes them from there, and the
      // transform of a finished vertex reads its own row back for the W_self term
      float* rows = c->d_af_X + (size_t)src_begin * Kp;
      launch_af_prep(c, X, ldx, n, K, Kp, src_begin, rows, st);
      a.PT = rows;
    } else if (c->mode != TAURUS_GCN_SYM && K == Kp && (reinterpret_cast<uintptr_t>(X) & 15) == 0) {
      a.PT = X; x_in_use = true;
    } else {
      launch_af_prep(c, X, ldx, n, K, Kp, src_begin, c->d_PT, st);
    }
  } else if (gat) {
    if (K == a.Hp && (reinterpret_cast<uintptr_t>(X) & 15) == 0) { a.PT = X; x_in_use = true; }
    else launch_gat_repack(c, X, n, K, a.Hp, st);
  } else if (project_tc_usable(c, l, X, ldx)) {
    int rc = launch_project_tc(c, l, X, ldx, src_begin, n, st);
    if (rc) return rc;
  } else {
    launch_project_simt(c, l, X, ldx, src_begin, n, st);
  }
  if (xbuf >= 0 && !x_in_use) { CU(cudaEventRecord(c->x_free[xbuf], st)); c->x_used[xbuf] = true; }
  if (timing) cudaEventRecord(pev[2], st);
  // S3, S4
  const bool grouped = c->d_gdst != nullptr && src_begin % c->chunk_sources == 0 &&
                       src_end == std::min<long long>(c->V, src_begin + c->chunk_sources);
  if (grouped) launch_classify_grouped(c, a, st); else launch_classify(c, a, st);
  launch_make_room(c, a, st, timing ? pev[3] : nullptr);   // pev[3]: victims chosen and placed, rows not yet moved
  // The chunk before this one: its rows have been crossing the host link since its slots were handed out.  Its
  // finalise runs now, before this chunk takes over the slots it released.
  int run_rc = finish_chunk(c, st);
  if (timing && c->pipelined) cudaEventRecord(pev[4], st);
  launch_alloc(c, a, st);
  if (scatter_timing) cudaEventRecord(pev[5], st);
  if (c->pipelined) {
    CU(cudaEventRecord(c->moves_ready, st));
    CU(cudaStreamWaitEvent(c->xfer_stream, c->moves_ready, 0));
    if (timing) cudaEventRecord(pev[10], c->xfer_stream);
    launch_transfer(c, a, c->xfer_stream);
    if (timing) cudaEventRecord(pev[11], c->xfer_stream);
    CU(cudaEventRecord(c->xfer_done, c->xfer_stream));
  }
  // S5, S5', S6
  if (grouped) launch_scatter_grouped(c, a, st); else launch_scatter(c, a, st);
  if (xbuf >= 0 && x_in_use) { CU(cudaEventRecord(c->x_free[xbuf], st)); c->x_used[xbuf] = true; }   // the scatter read the staged rows in place
  if (scatter_timing) cudaEventRecord(pev[6], st);
  launch_compact_done(c, a, st, c->pipelined);   // with transfers in flight the chunk record is written now, else by the commit after finalise
  if (timing) cudaEventRecord(pev[7], st);
  // S7: deferred behind the next chunk's select when rows cross the host link, else at once
  c->pend_chunk->a = a; c->pend_chunk->layer = l; c->pend_chunk->af = af; c->pend_chunk->bound = bound;
  c->pend_chunk->timed_index = scatter_timing ? c->timed_pushes - 1 : -1;
  c->pending = true;
  if (!c->pipelined) { int rc = finish_chunk(c, st); if (!run_rc) run_rc = rc; }
  CU(cudaGetLastError());
  c->next_src = src_end;
  c->chunk_seq += 1;
  if (!halves && !direct_dense) c->ub_since_drain += bound;
  return run_rc;
}

static int gat_project_core(taurus_ctx* c, int64_t src_begin, int64_t src_end, const float* features, taurus_runs* src_runs,
                            float* hprime_out, int64_t ld, void* cuda_stream) {
  if (!c || (!features && !src_runs) || !hprime_out) return TAURUS_ERR_INVALID_ARG;
  if (c->mode != TAURUS_GAT) return TAURUS_ERR_UNSUPPORTED;
  if (c->layer < 0 || c->gat_ready || c->chunk_seq != 0 || src_begin != c->gat_next_src) return TAURUS_ERR_ORDER;
  if (src_end <= src_begin || src_end > c->V || src_end - src_begin > c->chunk_sources) return TAURUS_ERR_INVALID_ARG;
  const int l = c->layer, K = c->dims[l], d_out = c->dims[l + 1], Hp = taurus_round_up(d_out, 4);
  if (ld < d_out || (features && (reinterpret_cast<uintptr_t>(features) & 3) != 0) || pointer_kind(hprime_out) != PK_DEVICE) return TAURUS_ERR_INVALID_ARG;
  if (src_runs && (runs_width(src_runs) != K || runs_vertices(src_runs) != c->V || runs_max_chunk(src_runs) < src_end - src_begin))
    return TAURUS_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CU(cudaSetDevice(c->device));
  if (st != c->last_stream) {
    CU(cudaEventRecord(c->order_event, c->last_stream));
    CU(cudaStreamWaitEvent(st, c->order_event, 0));
    c->last_stream = st;
  }
  const int n = (int)(src_end - src_begin);
  const float* X = nullptr;
  int xbuf = -1;
  { int rc = stage_chunk(c, features, src_runs, src_begin, src_end, K, st, &X, &xbuf); if (rc) return rc; }
  if (c->agg_first[l]) {   // scores from two dot products per row; the input rows go back to the caller for pass 3
    launch_gat_scores(c, l, X, K, n, src_begin, hprime_out, ld, st);
    if (xbuf >= 0) { CU(cudaEventRecord(c->x_free[xbuf], st)); c->x_used[xbuf] = true; }
    CU(cudaGetLastError());
    c->gat_next_src = src_end;
    return TAURUS_OK;
  }
  if (project_tc_usable(c, l, X, K)) {
    int rc = launch_project_tc(c, l, X, K, src_begin, n, st);
    if (rc) return rc;
  } else {
    launch_project_simt(c, l, X, K, src_begin, n, st);
  }
  if (xbuf >= 0) { CU(cudaEventRecord(c->x_free[xbuf], st)); c->x_used[xbuf] = true; }
  launch_gat_split(c, n, Hp, d_out, src_begin, hprime_out, ld, st);
  CU(cudaGetLastError());
  c->gat_next_src = src_end;
  return TAURUS_OK;
}

extern "C" int taurus_gat_project_chunk(taurus_ctx* c, int64_t src_begin, int64_t src_end, const float* features, float* hprime_out,
                                        int64_t ld, void* cuda_stream) {
  if (!features) return TAURUS_ERR_INVALID_ARG;
  return gat_project_core(c, src_begin, src_end, features, nullptr, hprime_out, ld, cuda_stream);
}

extern "C" int taurus_gat_project_chunk_from_runs(taurus_ctx* c, int64_t src_begin, int64_t src_end, taurus_runs* runs, float* hprime_out,
                                                  int64_t ld, void* cuda_stream) {
  if (!runs) return TAURUS_ERR_INVALID_ARG;
  return gat_project_core(c, src_begin, src_end, nullptr, runs, hprime_out, ld, cuda_stream);
}

extern "C" int taurus_gat_attention(taurus_ctx* c, void* cuda_stream) {
  if (!c) return TAURUS_ERR_INVALID_ARG;
  if (c->mode != TAURUS_GAT) return TAURUS_ERR_UNSUPPORTED;
  if (c->layer < 0 || c->gat_ready || c->gat_next_src != c->V) return TAURUS_ERR_ORDER;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  CU(cudaSetDevice(c->device));
  if (st != c->last_stream) {
    CU(cudaEventRecord(c->order_event, c->last_stream));
    CU(cudaStreamWaitEvent(st, c->order_event, 0));
    c->last_stream = st;
  }
  launch_gat_attention(c, st);
  CU(cudaGetLastError());
  c->gat_ready = true;
  return TAURUS_OK;
}

extern "C" int taurus_push_chunk(taurus_ctx* c, int64_t src_begin, int64_t src_end, const float* features, void* cuda_stream) {
  if (!features) return TAURUS_ERR_INVALID_ARG;
  return push_core(c, src_begin, src_end, features, nullptr, cuda_stream);
}

extern "C" int taurus_push_chunk_from_runs(taurus_ctx* c, int64_t src_begin, int64_t src_end, taurus_runs* runs, void* cuda_stream) {
  if (!runs) return TAURUS_ERR_INVALID_ARG;
  return push_core(c, src_begin, src_end, nullptr, runs, cuda_stream);
}

extern "C" int taurus_layer_set_run_output(taurus_ctx* c, taurus_runs* runs) {
  if (!c || !runs) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0 || c->chunk_seq != 0 || c->dense_out) return TAURUS_ERR_ORDER;
  if (runs_width(runs) != c->dims[c->layer + 1] || runs_vertices(runs) != c->V || runs_max_append(runs) < c->drain_rows / 2 ||
      runs_pending(runs))
    return TAURUS_ERR_INVALID_ARG;
  c->run_out = runs;
  c->run_pending_half = -1;
  return TAURUS_OK;
}

static int drain_common(taurus_ctx* c, long long capacity, long long* out_count, long long* count) {
  if (!c || !out_count || capacity < 0) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  int err = read_ctl(c, c->last_stream);
  if (err) return err;
  *count = c->h_ctl->grad_count;
  *out_count = *count;
  if (*count > capacity) return TAURUS_ERR_INVALID_ARG;
  return TAURUS_OK;
}

static int drain_reset(taurus_ctx* c) {
  CU(cudaMemsetAsync(reinterpret_cast<char*>(c->d_ctl) + offsetof(DevCtl, grad_count), 0, sizeof(long long), c->last_stream));
  CU(cudaStreamSynchronize(c->last_stream));
  c->ub_since_drain = 0;
  return TAURUS_OK;
}

extern "C" int taurus_drain_completed(taurus_ctx* c, int64_t* out_ids, float* out_rows, int64_t capacity_rows, int64_t* out_count) {
  long long count = 0, oc = 0;
  int rc = drain_common(c, capacity_rows, &oc, &count);
  if (out_count) *out_count = oc;
  if (rc) return rc;
  if (count > 0) {
    if (!out_ids || !out_rows) return TAURUS_ERR_INVALID_ARG;
    const int d_out = c->dims[c->layer + 1], Hp = taurus_round_up(d_out, 4);
    cudaStream_t st = c->last_stream;
    CU(cudaMemcpyAsync(out_ids, c->d_grad_ids, (size_t)count * sizeof(long long), cudaMemcpyDefault, st));
    CU(cudaMemcpy2DAsync(out_rows, (size_t)d_out * sizeof(float), c->d_grad_rows, (size_t)Hp * sizeof(float),
                         (size_t)d_out * sizeof(float), (size_t)count, cudaMemcpyDefault, st));
  }
  return drain_reset(c);
}

extern "C" int taurus_drain_dense(taurus_ctx* c, float* dense_rows, int64_t ld, int64_t* out_ids, int64_t capacity_rows,
                                  int64_t* out_count) {
  if (!c || !dense_rows) return TAURUS_ERR_INVALID_ARG;
  if (c->layer >= 0 && ld < c->dims[c->layer + 1]) return TAURUS_ERR_INVALID_ARG;
  float* dense_dev = dense_rows;
  int kind = pointer_kind(dense_rows);
  if (kind == PK_HOST_PAGEABLE) return TAURUS_ERR_INVALID_ARG;
  if (kind == PK_HOST_PINNED) {
    if (!cuda_ok(cudaHostGetDevicePointer((void**)&dense_dev, dense_rows, 0), "cudaHostGetDevicePointer")) return TAURUS_ERR_INVALID_ARG;
  }
  long long count = 0, oc = 0;
  int rc = drain_common(c, capacity_rows, &oc, &count);
  if (out_count) *out_count = oc;
  if (rc) return rc;
  if (count > 0) {
    const int d_out = c->dims[c->layer + 1], Hp = taurus_round_up(d_out, 4);
    cudaStream_t st = c->last_stream;
    launch_place_rows(c, dense_dev, ld, d_out, Hp, count, st);
    if (out_ids) CU(cudaMemcpyAsync(out_ids, c->d_grad_ids, (size_t)count * sizeof(long long), cudaMemcpyDefault, st));
    CU(cudaGetLastError());
  }
  return drain_reset(c);
}

extern "C" int taurus_layer_set_dense_output(taurus_ctx* c, float* dense_rows, int64_t ld) {
  if (!c || !dense_rows) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0 || c->chunk_seq != 0 || c->run_out) return TAURUS_ERR_ORDER;
  if (ld < c->dims[c->layer + 1]) return TAURUS_ERR_INVALID_ARG;
  float* dev = dense_rows;
  int kind = pointer_kind(dense_rows);
  if (kind == PK_HOST_PAGEABLE) return TAURUS_ERR_INVALID_ARG;
  if (kind == PK_HOST_PINNED && !cuda_ok(cudaHostGetDevicePointer((void**)&dev, dense_rows, 0), "cudaHostGetDevicePointer"))
    return TAURUS_ERR_INVALID_ARG;
  c->dense_out = dev;
  c->dense_ld = ld;
  c->dense_is_device = kind == PK_DEVICE;
  return TAURUS_OK;
}

static int fill_stats(taurus_ctx* c, taurus_stats* s) {
  const DevCtl* h = c->h_ctl;
  memset(s, 0, sizeof(*s));
  launch_reload_histogram(c, c->d_reload_hist, c->last_stream);
  long long hist[18];
  CU(cudaMemcpyAsync(hist, c->d_reload_hist, sizeof(hist), cudaMemcpyDeviceToHost, c->last_stream));
  CU(cudaStreamSynchronize(c->last_stream));
  long long nonzero = 0;
  for (int i = 1; i < 17; ++i) { s->reload_histogram[i] = hist[i]; nonzero += hist[i]; }
  s->reload_histogram[0] = c->V - nonzero;
  s->max_reload_count = hist[17];
  s->evictions = h->evictions; s->reloads = h->reloads; s->peak_occupancy = h->peak_occupancy;
  s->hub_messages = h->hub_messages; s->total_messages = h->total_messages; s->hub_vertices = c->hub_count;
  s->completed = h->completed; s->sum_hs = h->sum_hs; s->sum_ns = h->sum_ns; s->sum_ev = h->sum_ev; s->sum_gs = h->sum_gs;
  s->free_slots = h->free_top; s->chunks = h->chunks; s->scatter_groups = h->scatter_groups;
  return TAURUS_OK;
}

extern "C" int taurus_get_stats(taurus_ctx* c, taurus_stats* stats) {
  if (!c || !stats) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  int err = read_ctl(c, c->last_stream);
  if (err) return err;
  return fill_stats(c, stats);
}

extern "C" int taurus_layer_end(taurus_ctx* c, taurus_stats* stats) {
  if (!c) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  { int rc = finish_chunk(c, c->last_stream); if (rc) return rc; }
  if (c->run_out) {   // last chunk's rows, then every partition buffer leaves as a run
    int rc = finish_run_append(c);
    if (!rc) rc = runs_flush_all(c->run_out, c->out_stream);
    if (rc) return rc;
  }
  int err = read_ctl(c, c->last_stream);
  if (err) return err;
  if (stats) { int rc = fill_stats(c, stats); if (rc) return rc; }
  if (c->next_src != c->V || c->h_ctl->completed != c->V || c->h_ctl->free_top != c->pool_slots) return TAURUS_ERR_ORDER;
  return TAURUS_OK;
}

extern "C" int taurus_get_chunk_log(taurus_ctx* c, int64_t* out, int64_t capacity_chunks, int64_t* out_chunks) {
  if (!c || !out || !out_chunks || capacity_chunks < 0) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  int err = read_ctl(c, c->last_stream);
  if (err) return err;
  long long n = std::min<long long>(std::min<long long>(c->h_ctl->chunks, c->log_capacity), capacity_chunks);
  if (n > 0) CU(cudaMemcpy(out, c->d_chunk_log, (size_t)n * TAURUS_CK_COLUMNS * sizeof(long long), cudaMemcpyDeviceToHost));
  *out_chunks = n;
  return TAURUS_OK;
}

extern "C" int taurus_get_vertex_array(taurus_ctx* c, int32_t which, void* out_host) {
  if (!c || !out_host || which < 0 || which > 3) return TAURUS_ERR_INVALID_ARG;
  CU(cudaSetDevice(c->device));
  { int rc = finish_chunk(c, c->last_stream); if (rc) return rc; }
  CU(cudaStreamSynchronize(c->last_stream));
  const void* src = which == 0 ? (const void*)c->d_state : which == 1 ? (const void*)c->d_pend
                    : which == 2 ? (const void*)c->d_reload : (const void*)c->d_hub;
  size_t bytes = (size_t)c->V * ((which == 0 || which == 3) ? 1 : 4);
  CU(cudaMemcpy(out_host, src, bytes, cudaMemcpyDeviceToHost));
  return TAURUS_OK;
}

extern "C" int taurus_get_sampled_edges(taurus_ctx* c, int32_t layer, int64_t dst, int64_t* out_edge_ids, int32_t* out_sources,
                                        int32_t capacity, int32_t* n) {
  if (!c || !n || layer < 0 || layer >= c->L || dst < 0 || dst >= c->V || capacity < 0) return TAURUS_ERR_INVALID_ARG;
  if (capacity > 0 && (!out_edge_ids || !out_sources)) return TAURUS_ERR_INVALID_ARG;
  if (!c->d_csc_eid) return TAURUS_ERR_ORDER;   // built only when some layer is sampled
  CU(cudaSetDevice(c->device));
  CU(cudaStreamSynchronize(c->last_stream));
  int rc = sampled_edges_of(c, layer, dst, (long long*)out_edge_ids, out_sources, capacity, n);
  if (rc == TAURUS_ERR_CUDA) cuda_ok(cudaGetLastError(), "sampled_edges_of");
  return rc;
}

extern "C" int taurus_get_edge_mask(taurus_ctx* c, uint32_t* out_words) {
  if (!c || !out_words) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  CU(cudaStreamSynchronize(c->last_stream));
  size_t words = (size_t)((c->E + 31) / 32);
  if (c->d_mask_cur) CU(cudaMemcpy(out_words, c->d_mask_cur, words * sizeof(uint32_t), cudaMemcpyDeviceToHost));
  else {
    memset(out_words, 0xff, words * sizeof(uint32_t));
    if (c->E & 31) out_words[words - 1] = (1u << (c->E & 31)) - 1u;
  }
  return TAURUS_OK;
}

extern "C" int taurus_get_sample_digest(taurus_ctx* c, uint64_t* out_digest) {
  if (!c || !out_digest) return TAURUS_ERR_INVALID_ARG;
  if (c->layer < 0) return TAURUS_ERR_ORDER;
  CU(cudaSetDevice(c->device));
  CU(cudaStreamSynchronize(c->last_stream));
  unsigned long long* d = nullptr;
  ALLOC(d, (size_t)2 * c->V);
  cudaError_t e = cudaMemset(d, 0, (size_t)2 * c->V * sizeof(unsigned long long));
  if (e == cudaSuccess) { launch_sample_digest(c, d, nullptr); e = cudaGetLastError(); }
  if (e == cudaSuccess) e = cudaMemcpy(out_digest, d, (size_t)2 * c->V * sizeof(unsigned long long), cudaMemcpyDefault);
  cudaFree(d);
  CU(e);
  return TAURUS_OK;
}

extern "C" int64_t taurus_launch_count(const taurus_ctx* c) { return c ? c->launches : 0; }

extern "C" int taurus_get_layer_plan(const taurus_ctx* c, int32_t layer, int32_t* out_aggregate_first, int32_t* out_row_floats) {
  if (!c || layer < 0 || layer >= c->L) return TAURUS_ERR_INVALID_ARG;
  const bool af = c->agg_first[layer];
  if (out_aggregate_first) *out_aggregate_first = af ? 1 : 0;
  if (out_row_floats) *out_row_floats = taurus_round_up(af ? c->dims[layer] : c->dims[layer + 1], 4);
  return TAURUS_OK;
}

extern "C" int taurus_set_timing(taurus_ctx* c, int32_t on) {
  if (!c) return TAURUS_ERR_INVALID_ARG;
  if (on < 0 || on > 2) return TAURUS_ERR_INVALID_ARG;
  CU(cudaSetDevice(c->device));
  { int rc = finish_chunk(c, c->last_stream); if (rc) return rc; }   // a deferred finalise belongs to the level it was pushed under
  c->timing = on;
  if (on) { c->timed_pushes = 0; c->timed_level = on; }
  return TAURUS_OK;
}

extern "C" int taurus_get_phase_ms(taurus_ctx* c, float* out, int64_t capacity_pushes, int64_t* out_pushes) {
  if (!c || !out || !out_pushes || capacity_pushes < 0) return TAURUS_ERR_INVALID_ARG;
  CU(cudaSetDevice(c->device));
  { int rc = finish_chunk(c, c->last_stream); if (rc) return rc; }
  CU(cudaStreamSynchronize(c->last_stream));
  if (c->xfer_stream) CU(cudaStreamSynchronize(c->xfer_stream));
  long long n = std::min<long long>(c->timed_pushes, capacity_pushes);
  // event pairs of the nine durations; without row transfers events 4, 8, 10 and 11 are not recorded: no wait, the
  // slot hand-out runs from event 3, the finalise from event 7
  static const int from_x[TAURUS_PHASES] = {0, 1, 2, 3, 4, 5, 6, 8, 10}, to_x[TAURUS_PHASES] = {1, 2, 3, 4, 5, 6, 7, 9, 11};
  static const int from_d[TAURUS_PHASES] = {0, 1, 2, -1, 3, 5, 6, 7, -1}, to_d[TAURUS_PHASES] = {1, 2, 3, -1, 5, 6, 7, 9, -1};
  const int* from = c->pipelined ? from_x : from_d;
  const int* to = c->pipelined ? to_x : to_d;
  for (long long p = 0; p < n; ++p)
    for (int i = 0; i < TAURUS_PHASES; ++i) {
      out[p * TAURUS_PHASES + i] = 0.f;
      if (from[i] >= 0 && (c->timed_level == 1 || i == 5))
        CU(cudaEventElapsedTime(&out[p * TAURUS_PHASES + i], c->phase_ev[(size_t)p * TAURUS_PUSH_EVENTS + from[i]],
                                c->phase_ev[(size_t)p * TAURUS_PUSH_EVENTS + to[i]]));
    }
  *out_pushes = n;
  return TAURUS_OK;
}
