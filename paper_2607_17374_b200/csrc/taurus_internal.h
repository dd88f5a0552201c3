// Internal declarations shared by the translation units of libtaurus.
// Host control lives in taurus_host.cu; each kernels_*.cu file holds kernels and their launchers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "taurus.h"

#define TAURUS_MAX_LAYERS 16
#define TAURUS_MAX_DIM 1024
#define TAURUS_MAX_FANOUT 64
#define TAURUS_MAX_TIMED_PUSHES 16384
#define TAURUS_PUSH_EVENTS 12                   // CUDA events per timed push
#define TAURUS_PHASES 9                         // durations reported per timed push
#define TAURUS_SEL_BITS 11                      // radix-select digit width
#define TAURUS_SEL_BINS (1 << TAURUS_SEL_BITS)
#define TAURUS_SEL_LEVELS 6                     // 6 x 11 = 66 bits >= the 62-bit (score, id) key

// Counters of ONE chunk that its kernels hand to one another.  Two of them alternate (chunk sequence number & 1): with a
// bounded pool the finalise step of chunk k runs after the classify / select steps of chunk k + 1 (while chunk k's rows
// are still crossing the host link), so the two chunks' counters are alive together.
struct ChunkCtl {
  int32_t need_count;     // touched vertices that need a slot (NOT_STARTED or EVICTED)
  int32_t done_count;     // vertices whose pending count reached zero
  int32_t touched_count;  // vertices touched by this chunk (first touches)
  int32_t deficit;        // slots to free by eviction
  int32_t victim_count;   // victims listed so far
  int32_t hs, ns, ev, gs; // touched vertices by state at chunk start
  int32_t reloaded;       // reloads
  unsigned int span_next; // scatter: next span of the chunk's edge list to hand to a warp
  unsigned int self_next; // scatter: next tile of 32 self messages to hand to a warp
  unsigned int tile_next[4];  // pool passes of the victim select: next tile of slots to hand to a block
  long long alloc_base;   // need-list entry i takes free_stack[alloc_base - 1 - i]
  // Victim select, level by level (level 0 scans the pool, deeper levels the candidates the level above left):
  long long sel_k[TAURUS_SEL_LEVELS + 1];               // rank still to resolve among the keys entering the level
  unsigned long long sel_min[TAURUS_SEL_LEVELS + 1];    // smallest / largest key entering the level: the digit of a level
  unsigned long long sel_max[TAURUS_SEL_LEVELS + 1];    //   starts at the highest bit in which they differ
  int32_t sel_count[TAURUS_SEL_LEVELS + 1];             // keys entering the level
  int32_t sel_final_level;                              // level that listed the last victims; kernels of deeper levels return
  unsigned int hist[2][TAURUS_SEL_BINS];                // digit histogram, alternating between levels
};

// Device-resident control block: counters the kernels hand to one another, so that no step of a push needs
// the host.  One per context.
struct DevCtl {
  int32_t error;            // sticky TAURUS_ERR_* found on the device
  int32_t ext_ret_count[2]; // extents emptied by the row transfers of the chunks of each parity, waiting to go back on the free stack
  long long free_top;       // entries on the free-slot stack
  long long ext_free_top;   // entries on the free-extent stack of the host store
  long long host_live;      // rows currently held by the host store
  long long grad_count;     // rows waiting in the graduation buffer
  long long out_count[2];   // dense-output mode: rows finalise left in each half of the graduation buffer
  // layer totals
  long long evictions, reloads, peak_occupancy, hub_messages, total_messages, completed;
  long long sum_hs, sum_ns, sum_ev, sum_gs, chunks;
  long long scatter_groups; // accumulator-row reductions issued by the scatter (self messages not counted)
  ChunkCtl pc[2];
};

// Everything the per-chunk kernels need, passed by value.
struct ChunkArgs {
  // graph
  const long long* row_ptr;
  const int32_t* col;
  const int32_t* din;
  const uint32_t* mask;     // NULL = every edge propagated
  // per-vertex state
  int32_t* pend;
  uint8_t* state;
  int32_t* loc;             // pool slot / hub row (>= pool_slots) / host row while EVICTED; -1 = none
  int32_t* touch;           // chunk epoch of the last touch
  int32_t* reload_count;
  // pool
  float* acc;               // [(pool_slots + hub_count) x Hp]
  int32_t* owner;           // [pool_slots] vertex in the slot, -1 = free
  int32_t* slot_epoch;      // [pool_slots] chunk epoch at which the slot's vertex entered the pool (FIFO policy)
  // Per-slot copies of the owner's epoch stamp and pending count, kept so that the victim select reads the pool
  // front to back instead of three scattered per-vertex words per slot; null when nothing can be evicted.
  // slot_touch[s] is written whenever the owner is touched (hit: classify, hand-out: alloc); slot_pend[s] after
  // every chunk that touched the owner (compact_done), and the pending count only changes in such chunks.
  int32_t* slot_touch;
  int32_t* slot_pend;
  int32_t* free_stack;      // [pool_slots]
  int32_t* need_list;       // [pool_slots]
  int32_t* touched_list;    // [touched_capacity] every vertex the chunk touches, listed at its first touch
  long long touched_capacity;
  int2* victims;            // [victim_capacity] (slot, pinned host row) of this chunk's victims
  long long victim_capacity;
  unsigned long long* keys; // [pool_slots]
  int32_t* cand[2];         // [pool_slots] each: slots still in the running for the last victims, alternating between levels
  // Host store of evicted rows (pinned, mapped): extents of (1 << ext_shift) rows handed out from a free stack.  A
  // victim's row is filed under the grid cell of the source that sends its vertex the next message ("bucket"), so
  // the rows a chunk reloads sit together and the rows it evicts are appended to a few hundred open extents.
  float* host_store;        // device alias of the pinned host rows [(n_ext << ext_shift) x Hp]
  int32_t* ext_free;        // [n_ext] stack of free extents
  int32_t* ext_live;        // [n_ext] rows of the extent not yet reloaded, plus its rows not yet handed out
  int32_t* bk_tail_ext;     // [buckets] extent the bucket appends to, -1 none
  int32_t* bk_tail_fill;    // [buckets] rows handed out of that extent
  int32_t* bk_new;          // [buckets] this chunk: victims filed under the bucket
  int32_t* bk_off;          // [buckets] this chunk: first of the bucket's new extents in new_ext
  int2* bk_base;            // [buckets] this chunk: (tail extent, tail fill) before the chunk's victims
  int32_t* new_ext;         // [victim_capacity >> ext_shift + buckets] this chunk: extents taken from the stack
  int2* vic_place;          // [victim_capacity] this chunk: (bucket, rank among the chunk's victims of that bucket)
  int32_t* ext_ret[2];      // [n_ext] each: extents emptied by the transfers of the chunks of each parity
  // Row transfers of the chunk: entry i = (slot, host row to add into it or -1, host row that takes stage_out[i] or -1)
  int4* xfer_list;          // [need capacity]
  float* stage_out;         // [victim_capacity x Hp] victims' rows on their way to the host store
  const long long* csc_ptr; // [V + 1] in-lists (ascending source id): offsets,
  const int32_t* csc_src;   // [E]       sources,
  const uint32_t* csc_eid;  // [E]       CSR edge indices (sampled layers: the mask is looked up through them), else NULL
  long long chunk_sources;  // width of a grid cell in sources
  long long n_ext, n_buckets;
  int32_t ext_shift;
  // graduation buffer
  long long* grad_ids;
  float* grad_rows;         // [drain_rows x Hp]
  int32_t* done_list;       // [drain_rows]
  // projected rows of this chunk: P at column 0, T at column Hp (SAGE only)
  const float* PT;
  int32_t ldpt;
  const float* bias;        // [Hp]
  DevCtl* ctl;
  ChunkCtl* pc;             // this chunk's counters: &ctl->pc[chunk sequence number & 1]
  long long* chunk_log;     // [log_capacity x TAURUS_CK_COLUMNS]
  long long log_capacity;
  long long V, pool_slots, hub_count, host_rows, drain_rows;
  long long src_begin, src_end;
  int32_t epoch;            // chunk sequence number + 1 within the layer
  int32_t Hp;               // padded accumulator width (multiple of 4)
  int32_t mode, act, fanout;
  int32_t evict_policy;
  float gin_self;           // GIN: 1 + eps, the weight of the self message
  // GAT: per-vertex scalars from which every attention coefficient is recomputed
  const float* att_s;       // [V] att_src . h'_u
  const float2* att_tm;     // [V] (att_dst . h'_v, maximum score of v's neighbourhood)
  const double* att_z;      // [V x heads] softmax normaliser (summed in double: a hub's sum has thousands of terms of very different size)
  float leaky;              // LeakyReLU slope
  int32_t heads;            // GAT: attention heads (the per-vertex scalars are [V x heads])
  int32_t head_vec;         // GAT: float4 per head (d_head / 4)
  unsigned long long seed;
  long long grad_off;       // dense-output mode: first row of this chunk's half of the graduation buffer
  long long grad_cap;       // rows the chunk may write (drain_rows, or half of it in dense-output mode)
  int32_t dense_half;       // -1: graduation buffer drained by the caller; 0 / 1: half used by this chunk
  int32_t direct;           // pool_slots >= V: vertex v owns slot v, no free stack, no eviction
  int32_t dynamic_spans;    // the scatter hands its spans out from a counter (row transfers may run beside it)
  float* dense_direct;      // dense-output mode with the matrix in device memory: finalise writes row v at dense_direct + v * dense_ld
  long long dense_ld;
  int32_t d_out;            // unpadded output width
  // aggregate-first layers (input rows narrower than output rows): the accumulators hold sums of input rows, Hp is
  // the padded INPUT width, and the transform runs on the finished rows
  int32_t Hout;             // padded output width (= Hp for project-first layers)
  int32_t self_rows;        // 1: the scatter adds a self row; 0: it only counts the self message (the self term is added after the transform)
  int32_t self_bias;        // 1: the self row carries the bias (project-first); 0: the bias is added after the transform
};

// What is still to be enqueued for the chunk pushed last: S7 (finalise) and the hand-off of its rows.  With a bounded
// pool this waits until the next chunk has chosen its victims, so that the chunk's rows cross the host link in the
// meantime (Sect. 3.6 runs graduation beside aggregation in the same way); otherwise it follows the push at once.
struct PendingChunk {
  ChunkArgs a;
  int layer = 0;
  bool af = false;
  long long bound = 0;
  long long timed_index = -1;   // index of the push among the timed ones (its events live in a vector that may grow), -1 = not timed
};

struct taurus_ctx {
  int device = 0;
  long long V = 0, E = 0;
  int L = 0, mode = 0, gemm_mode = 0, flags = 0;
  int dims[TAURUS_MAX_LAYERS + 1] = {0};
  int act[TAURUS_MAX_LAYERS] = {0};
  int fanout[TAURUS_MAX_LAYERS] = {0};
  int Hmax = 0, Kmax = 0;   // padded maxima over layers
  unsigned long long seed = 0;
  long long chunk_sources = 0, pool_slots = 0, hub_count = 0, host_rows = 0, drain_rows = 0;
  // device graph
  long long* d_row_ptr = nullptr;
  int32_t* d_col = nullptr;
  int32_t* d_din = nullptr;
  // weights per layer: Wcat is [Kp x Ncat] row-major fp32 (P columns then T columns), bias [Hp]
  float* d_Wcat[TAURUS_MAX_LAYERS] = {nullptr};
  float* d_bias[TAURUS_MAX_LAYERS] = {nullptr};
  bool tc_smem_set = false;                        // dynamic shared memory limit of the projection kernel raised
  void* tc_image[TAURUS_MAX_LAYERS] = {nullptr};   // tensor-core operand images of Wcat (owned by kernels_gemm_tc.cu)
  void* tc_image_af[TAURUS_MAX_LAYERS] = {nullptr};   // SAGE aggregate-first layers: image of [W_neigh ; W_self] stacked along K
  float* d_Waf[TAURUS_MAX_LAYERS] = {nullptr};       //   the same matrix row-major [2 Kp x Hp] for the FFMA kernel
  // state
  int32_t* d_pend = nullptr;
  uint8_t* d_state = nullptr;
  int32_t* d_loc = nullptr;
  int32_t* d_touch = nullptr;
  int32_t* d_reload = nullptr;
  uint8_t* d_hub = nullptr;
  int32_t* d_hub_ids = nullptr;
  float* d_acc = nullptr;
  int32_t* d_owner = nullptr;
  int32_t* d_slot_epoch = nullptr;
  int32_t* d_slot_touch = nullptr;
  int32_t* d_slot_pend = nullptr;
  int evict_policy = 0;
  float gin_eps = 0.f;
  // GAT mode
  float leaky = 0.2f;
  int heads = 1;                // GAT: attention heads
  float* d_att_s = nullptr;     // [V] att_src . h'
  float* d_att_t = nullptr;     // [V] att_dst . h'
  float* d_att_max = nullptr;   // [V] running maximum of att_src . h'_u over the neighbourhood
  float2* d_att_tm = nullptr;   // [V] (t, maximum score)
  float* d_att_w[TAURUS_MAX_LAYERS] = {nullptr};   // per layer: W att_src then W att_dst, dims[l] floats each (scores without the transformed rows)
  double* d_att_z = nullptr;    // [V x heads] normaliser
  long long gat_next_src = 0;   // next source taurus_gat_project_chunk expects
  bool gat_ready = false;       // taurus_gat_attention has run for this layer
  // aggregate-first layers
  bool agg_first[TAURUS_MAX_LAYERS] = {false};
  float* d_af_A = nullptr;      // [drain_rows x max padded input width of such layers] finished rows gathered for the transform
  float* d_af_O = nullptr;      // [drain_rows x Hmax] transform output when its place in the graduation buffer is known only on the device
  float* d_af_X = nullptr;      // [V x Kp] SAGE: the (padded) input row of every vertex, kept from its chunk until it completes;
                                //   the scatter reads the chunk's rows from here and the transform multiplies them by W_self
  int32_t* d_free_stack = nullptr;
  int32_t* d_need_list = nullptr;
  int32_t* d_touched_list = nullptr;
  long long touched_capacity = 0;
  int2* d_victims = nullptr;
  long long victim_capacity = 0;
  unsigned long long* d_keys = nullptr;
  int32_t* d_cand[2] = {nullptr, nullptr};
  float* h_store = nullptr;      // pinned, mapped
  float* d_store_alias = nullptr;
  int32_t* d_ext_free = nullptr;
  int32_t* d_ext_live = nullptr;
  int32_t* d_bk_tail_ext = nullptr;
  int32_t* d_bk_tail_fill = nullptr;
  int32_t* d_bk_new = nullptr;
  int32_t* d_bk_off = nullptr;
  int2* d_bk_base = nullptr;
  int32_t* d_new_ext = nullptr;
  int2* d_vic_place = nullptr;
  int32_t* d_ext_ret[2] = {nullptr, nullptr};
  int4* d_xfer_list = nullptr;
  float* d_stage_out = nullptr;
  cudaStream_t xfer_stream = nullptr;   // rows cross the host link here while the compute stream goes on
  cudaEvent_t moves_ready = nullptr, xfer_done = nullptr;
  bool pipelined = false;               // bounded pool with a host store: finalise of chunk k is deferred behind chunk k + 1's select
  bool pending = false;                 // a chunk's finalise (and what follows it) is still to be enqueued
  struct PendingChunk* pend_chunk = nullptr;
  int32_t* d_csc_src = nullptr;   // in-list sources, built when rows can be evicted
  long long n_ext = 0, n_buckets = 0;
  int ext_shift = 0;
  long long* d_grad_ids = nullptr;
  float* d_grad_rows = nullptr;
  int32_t* d_done_list = nullptr;
  float* d_X[2] = {nullptr, nullptr};   // staged feature chunks [chunk_sources x Kmax], double-buffered
  cudaStream_t copy_stream = nullptr;   // host -> device feature copies run here, ahead of the compute stream
  cudaEvent_t x_ready[2] = {nullptr, nullptr}, x_free[2] = {nullptr, nullptr};
  bool x_used[2] = {false, false};
  long long host_pushes = 0;
  // dense-output mode (taurus_layer_set_dense_output)
  float* dense_out = nullptr;           // device-visible address of the caller's matrix, NULL = mode off
  long long dense_ld = 0;
  bool dense_is_device = false;         // the matrix is device memory: rows are finalised straight into it (no graduation halves)
  struct taurus_runs* run_out = nullptr;  // run-output mode (taurus_layer_set_run_output), NULL = mode off
  int run_pending_half = -1;            // half whose rows are grouped but not yet moved to the partition buffers
  cudaStream_t out_stream = nullptr;    // rows leave the graduation buffer here while the next chunk computes
  cudaEvent_t fin_done[2] = {nullptr, nullptr}, out_done[2] = {nullptr, nullptr};
  bool half_used[2] = {false, false};
  float* d_PT = nullptr;         // projected chunk [chunk_sources x 2 Hmax]
  long long* d_csc_ptr = nullptr;
  uint32_t* d_csc_eid = nullptr;
  uint32_t* d_mask = nullptr;
  int32_t* d_gdst = nullptr;      // grouped order (per grid chunk, edges sorted by destination): destinations
  int2* d_gedge = nullptr;        //   (destination, source - chunk start) pairs
  uint32_t* d_geid = nullptr;     //   CSR edge indices (kept only when some layer is sampled)
  uint32_t* d_gmask = nullptr;    // current layer's edge mask in grouped order
  uint32_t* d_mask_cur = nullptr; // d_mask when the current layer is sampled, else NULL (every edge propagated)
  int32_t* d_vtmp = nullptr;     // [V] scratch for layer_begin
  int32_t* d_rank_hist = nullptr;
  DevCtl* d_ctl = nullptr;
  long long* d_reload_hist = nullptr;   // 18 words for the reload histogram of taurus_get_stats
  DevCtl* h_ctl = nullptr;       // pinned
  long long* d_chunk_log = nullptr;
  long long log_capacity = 0;
  // host bookkeeping
  int layer = -1;
  long long next_src = 0;
  long long chunk_seq = 0;
  const std::vector<long long>* rank_cum = nullptr;   // current layer: completions by block of 64 completion ranks, prefix sums
  long long ub_since_drain = 0;      // upper bound on rows in the graduation buffer
  cudaStream_t last_stream = nullptr;
  cudaEvent_t order_event = nullptr;
  long long launches = 0;
  int timing = 0;                      // 0 off, 1 every phase, 2 the scatter only
  int timed_level = 1;                 // level of the recorded pushes
  std::vector<cudaEvent_t> phase_ev;   // TAURUS_PUSH_EVENTS events per timed push, created on demand
  long long timed_pushes = 0;          // pushes recorded since timing was switched on
  std::vector<std::vector<long long>> rank_cum_cache;   // per layer: rank_cum computed at the first layer_begin
  int sm_count = 148;
};

static inline int taurus_round_up(int x, int m) { return (x + m - 1) / m * m; }
// Columns of the projection output: [P | T] for SAGE, [h' | (att_src.h', att_dst.h') per head, padded to 4] for GAT, P otherwise.
static inline int taurus_proj_width(int mode, int Hp, int heads = 1) {
  return mode == TAURUS_SAGE_MEAN ? 2 * Hp : mode == TAURUS_GAT ? Hp + taurus_round_up(2 * heads, 4) : Hp;
}

// ---- kernels_state.cu
void launch_layer_reset(taurus_ctx* c, int layer, cudaStream_t st);
void launch_classify(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);
void launch_make_room(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st, cudaEvent_t before_moves = nullptr);   // plan, select, placement, [event]
void launch_alloc(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);       // slots handed out, victims' rows staged, new rows cleared
void launch_transfer(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);    // staged rows to the host store, reloaded rows added into their slots
void launch_finalise(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);    // finalise + commit (after launch_compact_done)
void launch_compact_done(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st, bool write_record);   // completions listed (and the chunk record written)
void launch_commit(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);
void launch_place_rows(taurus_ctx* c, float* dense, long long ld, int d_out, int Hp, long long count, cudaStream_t st);
void launch_place_half(taurus_ctx* c, int half, int d_out, int Hp, cudaStream_t st);   // dense-output mode
void launch_reload_histogram(taurus_ctx* c, long long* d_hist18, cudaStream_t st);
void launch_completion_ranks(taurus_ctx* c, cudaStream_t st);                // fills d_rank_hist
long long max_window_edges(taurus_ctx* c);                                  // most edges of any chunk_sources consecutive sources
int check_in_degrees(taurus_ctx* c, cudaStream_t st);                        // 0 ok, 1 mismatch
// ---- run_store.cu (sorted runs and merge-on-read)
struct taurus_runs;
int runs_width(const taurus_runs* r);
long long runs_max_append(const taurus_runs* r);
long long runs_max_chunk(const taurus_runs* r);
long long runs_vertices(const taurus_runs* r);
bool runs_pending(const taurus_runs* r);
long long runs_launches(const taurus_runs* r);
int runs_phase1(taurus_runs* r, const long long* ids, const float* rows, long long ld, long long n_bound, const long long* d_count,
                long long count_host, cudaStream_t st);
int runs_phase2(taurus_runs* r, cudaStream_t st);
int runs_flush_all(taurus_runs* r, cudaStream_t st);
int runs_read_into(taurus_runs* r, long long s, long long e, float* out, long long ld, cudaStream_t st);
// ---- taurus_host.cu
void taurus_note_cuda_error(cudaError_t e, const char* what);   // keeps the text for taurus_last_cuda_error
// ---- kernels_aggfirst.cu
void launch_af_prep(taurus_ctx* c, const float* X, int ldx, int n, int K, int Kp, long long src_begin, float* out, cudaStream_t st);   // out [n x Kp]
int launch_af_finalise(taurus_ctx* c, const ChunkArgs& a, int layer, long long bound, cudaStream_t st);
// ---- kernels_gat.cu
void launch_gat_scores(taurus_ctx* c, int layer, const float* X, int ldx, int n, long long src_begin, float* rows_out, long long ld, cudaStream_t st);
void launch_gat_split(taurus_ctx* c, int n, int Hp, int d_out, long long src_begin, float* hprime_out, long long ld, cudaStream_t st);   // c->heads heads
void launch_gat_attention(taurus_ctx* c, cudaStream_t st);
void launch_gat_repack(taurus_ctx* c, const float* X, int n, int d_out, int Hp, cudaStream_t st);   // X [n x d_out] -> d_PT [n x Hp]
// ---- kernels_scatter.cu
void launch_scatter(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);
// ---- kernels_gemm_simt.cu
void launch_project_simt(taurus_ctx* c, int layer, const float* X, int ldx, long long src_begin, int n, cudaStream_t st);
void launch_gemm_plain_simt(taurus_ctx* c, const float* W, int ldw, int N, const float* X, int ldx, int K, int n, float* out, long long ld_out,
                            cudaStream_t st);   // out = X . W[:, 0..N), W row-major with pitch ldw
// ---- kernels_gemm_tc.cu
bool gemm_plain_tc_usable(const taurus_ctx* c, const void* image, const float* X, int ldx, const float* out, long long ld_out);
// Optional epilogue of the plain product for finished rows: row i of the product belongs to vertex done_list[i]
// (i < ctl->done_count); act(row + bias) goes to dense[vertex * dense_ld ...] and the vertex becomes COMPLETED.
// Needs N % 4 == 0, dense_ld % 4 == 0 and a 16-byte aligned dense base.
struct GemmFinish {
  const int32_t* done_list;
  uint8_t* state;
  float* dense;
  long long dense_ld;
  const float* bias;
  int act;
};
int launch_gemm_plain_tc(taurus_ctx* c, void* image, int col0, int N, const float* X, int ldx, int K, int n, float* out, long long ld_out,
                         cudaStream_t st, const GemmFinish* finish = nullptr, const int32_t* done_count = nullptr);
// done_count (device pointer): n is only the host's bound; the kernel works on the first *done_count rows (read on the
// device at launch) and leaves the others untouched.
int prepare_tc_weights(taurus_ctx* c, void** slot, const std::vector<float>& cat, int K, int N);   // image of cat [K x N] into *slot
void free_tc_weights(taurus_ctx* c);
bool project_tc_usable(const taurus_ctx* c, int layer, const float* X, int ldx);
int launch_project_tc(taurus_ctx* c, int layer, const float* X, int ldx, long long src_begin, int n, cudaStream_t st);
// ---- kernels_group.cu
int build_grouped_order(taurus_ctx* c, bool keep_edge_ids, bool fill_csc_src);   // fill_csc_src: also writes csc_src (needs csc_ptr)
void launch_group_mask(taurus_ctx* c, cudaStream_t st);
void launch_classify_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);
void launch_scatter_grouped(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st);
// ---- kernels_sample.cu
int build_in_edge_order(taurus_ctx* c);                                      // csc_ptr, csc_eid
int build_csc_ptr(taurus_ctx* c);                                            // csc_ptr alone
int build_csc_src_from_eid(taurus_ctx* c);                                   // csc_src from csc_eid (both in in-list order)
void launch_sample_mask(taurus_ctx* c, int layer, cudaStream_t st);
int sampled_edges_of(taurus_ctx* c, int layer, long long dst, long long* out_eids, int32_t* out_src, int cap, int* n);
void launch_sample_digest(taurus_ctx* c, unsigned long long* d_digest, cudaStream_t st);   // d_digest [2V], zeroed by the caller
