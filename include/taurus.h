/*
 * libtaurus: source-centric, layer-wise broadcast step of out-of-core GNN
 * inference on one NVIDIA B200 (sm_100a).  C ABI, no C++ or framework types.
 *
 * One layer pass streams the vertices once in id order (Sect. 3.1): the caller
 * pushes chunks of contiguous source vertices with their feature rows
 * (Sect. 3.3, "chunk"); the library projects the rows through the layer's
 * weights, pushes each projected row along the chunk's CSR out-edges
 * (Sect. 3.2) into per-destination accumulators, counts down each
 * destination's pending messages (Sect. 3.4), and finalises destinations whose
 * count reached zero into a graduation buffer (Sect. 3.6) that the caller
 * drains.  (Where a layer's input rows are the narrower ones the same sums are
 * formed from the input rows and the weights are applied to the finished rows:
 * see TAURUS_FLAG_PROJECT_FIRST.  Results and accounting do not depend on it.)  Accumulators of the highest in-degree vertices are pinned in a
 * GPU-resident hub store (Sect. 3.5.1); all others live in a bounded slot pool
 * (Sect. 3.5.2) whose fewest-pending rows are evicted to pinned host memory
 * when the pool is full (Sect. 3.5.3-3.5.4) and reloaded before they receive
 * further messages.  Per-layer fanout sampling suppresses all but `fanout`
 * hashed in-edges per destination (Sect. 3.9, sampling paragraph).
 *
 * Layer formula (Eq. 1-2 with the SAGEConv split of Sect. 3.9):
 *   out_v = act( c_in(v) * sum_{u in M(v)} c_out(u) * (h_u W_neigh)
 *                + c_self(v) * (h_v W_self) + b )
 *   SAGE-mean: c_out = 1, c_in = 1 / max(|M(v)|, 1), c_self = 1
 *   GCN-sym  : c_out(u) = (dout(u)+1)^-1/2, c_in(v) = (din(v)+1)^-1/2,
 *              c_self = c_out * c_in, W_self = W_neigh
 *   GIN-sum  : c_out = 1, c_in = 1, c_self = 1 + gin_eps, W_self = W_neigh ("GCN/GIN-style aggregation", Sect. 3.9)
 *   GAT      : attention coefficients in place of c_in * c_out, see taurus_gat_project_chunk
 * M(v) is the multiset of propagated in-edges of v (all of them, or the
 * sampled ones); every CSR entry is one message, duplicates and self-loops
 * included.
 *
 * General rules.  Every function returns TAURUS_OK (0) or a negative
 * TAURUS_ERR_* code; nothing throws, aborts or traps.  Unless stated
 * otherwise a pointer argument may point to host or device memory (the
 * library asks the CUDA runtime which).  The caller owns every buffer it
 * passes and may free it as soon as the call that took it has returned, with
 * the exceptions stated at taurus_push_chunk.  The library owns all state
 * behind taurus_ctx.  A context is bound to the device current at
 * taurus_graph_init and is not thread-safe.  Errors found on the device
 * (pool too small, host store full, a slot / vertex index or pending count out of range)
 * are sticky: the chunk that hit one is not applied and every later call
 * on the context returns the code.
 */
#ifndef TAURUS_H
#define TAURUS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  TAURUS_OK = 0,
  TAURUS_ERR_INVALID_ARG = -1,     /* null / misaligned pointer, size out of range, inconsistent graph        */
  TAURUS_ERR_ORDER = -2,           /* chunk not contiguous / ascending, or no layer begun, or layer not drained */
  TAURUS_ERR_POOL_TOO_SMALL = -3,  /* one chunk needs more slots than pool_slots, or too few eligible victims  */
  TAURUS_ERR_HOST_STORE_FULL = -4, /* more rows evicted at once than host_evict_rows                            */
  TAURUS_ERR_DRAIN_FULL = -5,      /* the chunk could overflow the graduation buffer: drain, then push again    */
  TAURUS_ERR_CUDA = -6,            /* a CUDA runtime call failed (see taurus_last_cuda_error)                   */
  TAURUS_ERR_INTERNAL = -7,        /* a device-side consistency check failed                                    */
  TAURUS_ERR_NOMEM = -8,           /* host or device allocation failed                                          */
  TAURUS_ERR_UNSUPPORTED = -9,     /* shape or size outside what the kernels were built for                     */
  TAURUS_ERR_RUN_STORE_FULL = -10, /* a flush would exceed store_rows of the run store                          */
  TAURUS_ERR_RUNS_INCOMPLETE = -11 /* a chunk read found fewer (or more) rows than vertices in its id range      */
};

enum { TAURUS_SAGE_MEAN = 0, TAURUS_GCN_SYM = 1, TAURUS_GIN_SUM = 2, TAURUS_GAT = 3 };
enum { TAURUS_GEMM_FP32 = 0, TAURUS_GEMM_BF16 = 1 };
/* vertex states of Sect. 3.4 */
enum { TAURUS_NOT_STARTED = 0, TAURUS_IN_BUFFER = 1, TAURUS_EVICTED = 2, TAURUS_ON_GPU = 3, TAURUS_COMPLETED = 4 };

typedef struct taurus_ctx taurus_ctx;
typedef struct taurus_runs taurus_runs;   /* sorted runs of (vertex id, row) records: the output side, declared below */

/* CSR out-edge topology (Sect. 3.2).  Copied at init. */
typedef struct {
  int64_t V, E;              /* V < 2^31, E < 2^32                                             */
  const int64_t* row_ptr;    /* [V+1] offsets, row_ptr[0] = 0, row_ptr[V] = E, non-decreasing  */
  const int32_t* col_idx;    /* [E] destinations in [0, V); multi-edges and self-loops allowed */
  const int32_t* in_degree;  /* [V] with multiplicity; must equal the histogram of col_idx     */
} taurus_graph;

/* Layer weights.  Copied at init.  dims[l] -> dims[l+1]; matrices are row-major dims[l] x dims[l+1] fp32. */
typedef struct {
  int32_t mode;                /* TAURUS_SAGE_MEAN, TAURUS_GCN_SYM, TAURUS_GIN_SUM or TAURUS_GAT */
  int32_t L;                   /* number of layers, 1..16                                     */
  const int32_t* dims;         /* [L+1], each in 1..1024 (host pointer)                       */
  const float* const* W_neigh; /* [L] (host array of pointers)                                */
  const float* const* W_self;  /* [L]; used by SAGE only (GCN and GIN apply W_neigh to the self term) */
  const float* const* bias;    /* [L] each dims[l+1]; an entry may be NULL for zero bias      */
  const int32_t* act;          /* [L] 0 = identity, 1 = ReLU (host pointer)                   */
  int32_t gemm_mode;           /* TAURUS_GEMM_FP32: fp32-accurate projection; TAURUS_GEMM_BF16: bf16 operands, fp32 accumulate */
  float gin_eps;               /* TAURUS_GIN_SUM only: the self message is weighted 1 + gin_eps */
  const float* const* att_src; /* TAURUS_GAT only: [L] each dims[l+1], the half of the attention vector applied to the source */
  const float* const* att_dst; /* TAURUS_GAT only: [L] each dims[l+1], the half applied to the destination      */
  float leaky_slope;           /* TAURUS_GAT only: negative slope of the LeakyReLU on the scores, in [0, 1]     */
  int32_t gat_heads;           /* TAURUS_GAT only: attention heads, 0 or 1 = one.  Head i owns columns [i d, (i+1) d) of
                                  W_neigh[l], att_src[l], att_dst[l], bias[l] and of the layer's output, d = dims[l+1] / heads
                                  (every dims[l+1] must be a multiple of 4 * heads); the heads' outputs are concatenated */
} taurus_model;

typedef struct {
  int64_t chunk_sources;    /* largest number of sources one push may carry (Sect. 3.3)                    */
  int64_t pool_slots;       /* capacity of the accumulator slot pool (hot store, Sect. 3.5.2)              */
  int64_t hub_count;        /* vertices pinned in the hub store: the largest by (in_degree desc, id asc)   */
  const int32_t* fanout;    /* [L] per-layer fanout, 0 = exact; NULL = all exact; at most 64 (host pointer) */
  uint64_t seed;            /* seed of the neighbour-sampling hash                                         */
  int64_t host_evict_rows;  /* capacity (rows) of the pinned host store for evicted accumulators; 0 = none.
                               Must cover the rows evicted at once plus one chunk's victims (a chunk's victims
                               leave before its reloads hand their host rows back); V - hub_count always suffices.
                               The store is handed out in extents of up to 1 024 rows, one open extent per grid cell
                               of chunk_sources sources (evicted rows are filed by the cell that will next need
                               them): the library pins a few extents per cell more than this many rows */
  int64_t drain_rows;       /* capacity (rows) of the graduation buffer; must hold the completions of any one
                               pushed range as bounded by taurus_completion_bound (64-source granularity)  */
  int32_t flags;            /* TAURUS_FLAG_*                                                               */
  int32_t evict_policy;     /* TAURUS_EVICT_*: which IN_BUFFER vertices leave first when the pool is full     */
} taurus_run;

/* Eviction policies: the paper's (Sect. 3.5.3) and the alternatives of its ablation (Sect. 4.5).  Victims are
 * always the `deficit` smallest (score, vertex id) among IN_BUFFER vertices the chunk does not touch. */
enum {
  TAURUS_EVICT_FEWEST_PENDING = 0,  /* score = pending messages: closest to completion first          */
  TAURUS_EVICT_FIFO = 1,            /* score = chunk in which the vertex (last) entered the pool       */
  TAURUS_EVICT_LRU = 2,             /* score = chunk that last touched the vertex                      */
  TAURUS_EVICT_RANDOM = 3           /* score = 31-bit hash of (seed, vertex, chunk index)              */
};

enum {
  TAURUS_FLAG_SIMT_GEMM = 2,    /* use the plain fp32 FFMA projection kernel instead of the tensor-core one         */
  TAURUS_FLAG_NO_GROUPING = 4,  /* do not build the destination-grouped edge order: every chunk takes the CSR-order kernels */
  TAURUS_FLAG_PROJECT_FIRST = 8 /* always project a chunk before scattering it.  Without this flag a layer whose
                                   input rows are at most 3/4 as wide as its output rows aggregates the (scaled) input rows and
                                   applies the weights to the finished rows instead (exact by linearity, Sect. 3.6 / 3.9): the
                                   accumulators, the scatter traffic and every evicted row shrink by d_in / d_out.  SAGE layers
                                   keep every vertex's input row on the device until the vertex completes (its self term goes
                                   through W_self with the transform): V x d_in floats of device memory that stay allocated
                                   for the life of the context.  They take this order only while that store fits in the
                                   device memory free at taurus_graph_init beside an estimate of everything else the context
                                   allocates; taurus_get_layer_plan tells which order a layer got */
};

/* Integer accounting of one layer pass (Sect. 4.4-4.7 report these quantities). */
typedef struct {
  int64_t evictions;           /* IN_BUFFER -> EVICTED transitions                               */
  int64_t reloads;             /* EVICTED -> IN_BUFFER transitions                               */
  int64_t max_reload_count;    /* most reloads of one vertex                                     */
  int64_t reload_histogram[17];/* vertices by reload count 0..15, last bin = 16 or more          */
  int64_t peak_occupancy;      /* most pool slots in use at once                                 */
  int64_t hub_messages;        /* propagated messages delivered to hub-store vertices            */
  int64_t total_messages;      /* propagated messages, self messages not counted                 */
  int64_t hub_vertices;
  int64_t completed;           /* vertices finalised                                             */
  int64_t sum_hs, sum_ns, sum_ev, sum_gs; /* per-chunk touched vertices by state at the start of the chunk, summed over chunks:
                                  IN_BUFFER, NOT_STARTED, EVICTED (non-hub) and hub vertices    */
  int64_t free_slots;          /* free pool slots now                                            */
  int64_t chunks;              /* chunks pushed                                                  */
  int64_t scatter_groups;      /* accumulator-row reductions the scatter issued for propagated messages: one per
                                  message in CSR order, one per (chunk, destination) group in grouped order    */
} taurus_stats;

/* Columns of one per-chunk record returned by taurus_get_chunk_log. */
enum {
  TAURUS_CK_HS = 0, TAURUS_CK_NS, TAURUS_CK_EV, TAURUS_CK_GS, TAURUS_CK_NEED, TAURUS_CK_EVICTED,
  TAURUS_CK_RELOADED, TAURUS_CK_COMPLETED, TAURUS_CK_OCCUPANCY, TAURUS_CK_COLUMNS
};

/*
 * Creates a context on the current device: copies topology, degrees and weights, selects the hub set,
 * allocates the slot pool, the hub store, the pinned host store and the graduation buffer.  When any
 * fanout is non-zero it also builds the in-edge order (ascending source id, equal sources in CSR order)
 * that the sampler indexes (Sect. 3.9).  Blocking.  On failure *out is NULL.
 */
int taurus_graph_init(taurus_ctx** out, const taurus_graph* graph, const taurus_model* model, const taurus_run* run);

/*
 * Starts layer `layer` (0-based): every vertex NOT_STARTED, pending count |M(v)| + 1 (the +1 is the
 * vertex's own self message, delivered with its chunk), pool empty; builds the layer's edge mask when
 * fanout[layer] > 0 (Sect. 3.9).  Blocking (synchronises `cuda_stream`).  A layer may be begun again.
 */
int taurus_layer_begin(taurus_ctx* ctx, int32_t layer, void* cuda_stream);

/*
 * Pushes sources [src_begin, src_end): Sect. 3.1 broadcast of one chunk.  `features` is
 * [src_end - src_begin] x dims[layer] fp32 row-major, rows contiguous, in device memory or in host
 * memory (pinned host memory makes the copy asynchronous).  Chunks must arrive in ascending, contiguous
 * order starting at 0, at most chunk_sources per push.  All work is enqueued on `cuda_stream`
 * (a cudaStream_t, NULL = default stream) and the call returns without waiting; `features` must stay
 * valid and unchanged until that work has run (synchronise the stream, or drain).  Returns
 * TAURUS_ERR_DRAIN_FULL, before changing any state, when the vertices this chunk completes might not
 * fit the graduation buffer: drain and push the same chunk again.
 * Where rows can be evicted (pool_slots < V - hub_count) the chunk's evicted and reloaded rows cross the host link on
 * a stream of the library's own, beside the chunk's scatter and the next chunk's classification and victim
 * selection; the chunk's finished rows are then finalised by the NEXT call on the context that needs them (the next
 * push, a drain, taurus_layer_end, taurus_get_*): synchronising `cuda_stream` after a push does not by itself make that
 * chunk's rows appear, a drain does.
 */
int taurus_push_chunk(taurus_ctx* ctx, int64_t src_begin, int64_t src_end, const float* features, void* cuda_stream);

/*
 * GATConv in three sequential passes (GATConv paragraph of Sect. 3.9); contexts created with TAURUS_GAT, fp32
 * projection only.  One head or several (taurus_model.gat_heads: Sect. 3.9 runs the three passes once per head; here one pass over
 * the topology serves all heads, each head weighting its own block of columns).  Per head, with h' = h W,
 *     e_uv = LeakyReLU(att_src . h'_u + att_dst . h'_v),  alpha_uv = softmax over u in N(v) of e_uv,
 *     out_v = act(sum_{u in N(v)} alpha_uv h'_u + b),
 * where N(v) is the propagated in-multiset of v (all in-edges, or the layer's sampled ones) plus v itself:
 * every vertex aggregates its own self message.  After taurus_layer_begin:
 *   pass 1  taurus_gat_project_chunk for every chunk in ascending, contiguous order: writes the rows pass 3 will
 *           stream for sources [src_begin, src_end) to hprime_out (DEVICE memory, row i at hprime_out + i * ld,
 *           ld >= dims[layer+1] floats, dims[layer+1] floats per row) and keeps the two scalars att_src . h'_u and
 *           att_dst . h'_u of every vertex (per head).  The rows are the transformed rows h'; in a layer that aggregates input
 *           rows first (see TAURUS_FLAG_PROJECT_FIRST) they are the input rows, zero-padded, and h' is never formed:
 *           the caller treats them as opaque.  `features` as in taurus_push_chunk.  Asynchronous on the stream.
 *   pass 2  taurus_gat_attention, once all vertices are projected: a topology-only sweep over the CSR that
 *           computes, per destination, the maximum score and the softmax normaliser (no per-edge state is
 *           stored; the coefficients are recomputed from four per-vertex scalars where they are used).
 *   pass 3  taurus_push_chunk / taurus_push_chunk_from_runs for every chunk with the rows of pass 1 as
 *           `features` ([n] x dims[layer+1], rows contiguous): the broadcast of Sect. 3.1 with each message
 *           weighted by its attention coefficient; draining and taurus_layer_end as for the other modes.
 * Calls out of this order return TAURUS_ERR_ORDER.
 */
int taurus_gat_project_chunk(taurus_ctx* ctx, int64_t src_begin, int64_t src_end, const float* features, float* hprime_out,
                             int64_t ld, void* cuda_stream);
int taurus_gat_attention(taurus_ctx* ctx, void* cuda_stream);
/* Pass 1 with the chunk's features read from sorted runs (see taurus_runs below; width dims[layer]) by
 * merge-on-read, as taurus_push_chunk_from_runs does for the other modes. */
int taurus_gat_project_chunk_from_runs(taurus_ctx* ctx, int64_t src_begin, int64_t src_end, taurus_runs* runs,
                                       float* hprime_out, int64_t ld, void* cuda_stream);

/*
 * Copies out the vertices finalised since the last drain (Sect. 3.6): out_ids[i] and the dims[layer+1]
 * floats out_rows[i * dims[layer+1] ...], in no particular order, and empties the graduation buffer.
 * Blocking (synchronises the stream of the last push).  Fails with TAURUS_ERR_INVALID_ARG and drains
 * nothing when more than capacity_rows rows are waiting (*out_count then holds that number).
 */
int taurus_drain_completed(taurus_ctx* ctx, int64_t* out_ids, float* out_rows, int64_t capacity_rows, int64_t* out_count);

/*
 * Same as taurus_drain_completed, but row i is written to dense_rows[out_id * ld ...] (ld in floats,
 * ld >= dims[layer+1]): the vertex-ordered matrix the next layer streams (Sect. 3.7 keeps outputs
 * sorted by vertex id for this reason).  dense_rows may be device memory or pinned host memory.
 * out_ids may be NULL.
 */
int taurus_drain_dense(taurus_ctx* ctx, float* dense_rows, int64_t ld, int64_t* out_ids, int64_t capacity_rows,
                       int64_t* out_count);

/*
 * Dense-output mode for the current layer (Sect. 3.6 double-buffers graduation so that collecting and
 * off-loading overlap; Sect. 3.7 keeps outputs in vertex order for the next layer).  Call after
 * taurus_layer_begin and before the first push.  Every finalised row is then written to
 * dense_rows[id * ld ...] (ld in floats, >= dims[layer+1]; device memory or pinned host memory) by the
 * library itself and the caller never drains (taurus_drain_* report zero rows).  Device memory: the
 * finalise kernel writes each row straight to its place; a chunk whose completion bound exceeds drain_rows
 * is refused with TAURUS_ERR_DRAIN_FULL.  Pinned host memory: the graduation buffer is split in two halves,
 * the rows of chunk k leave one half on an internal stream while chunk k+1 computes into the other, and the
 * refusal threshold is drain_rows / 2 (create the context with a larger drain_rows).  taurus_layer_end waits
 * until every row has arrived.  The mode ends with the layer.
 */
int taurus_layer_set_dense_output(taurus_ctx* ctx, float* dense_rows, int64_t ld);

/* Ends the layer: blocking; checks that every vertex completed and every slot is free (else
 * TAURUS_ERR_ORDER), and fills *stats (may be NULL). */
int taurus_layer_end(taurus_ctx* ctx, taurus_stats* stats);

/* Accounting so far in the current layer (blocking). */
int taurus_get_stats(taurus_ctx* ctx, taurus_stats* stats);

/* Per-chunk records of the current layer: out[c * TAURUS_CK_COLUMNS + k], host memory, at most
 * capacity_chunks records; *out_chunks = records written. */
int taurus_get_chunk_log(taurus_ctx* ctx, int64_t* out, int64_t capacity_chunks, int64_t* out_chunks);

/* Per-vertex arrays of the current layer copied to host memory (blocking): which = 0 state (uint8 [V]),
 * 1 pending count (int32 [V]), 2 reload count (int32 [V]), 3 hub flag (uint8 [V]). */
int taurus_get_vertex_array(taurus_ctx* ctx, int32_t which, void* out_host);

/*
 * Sampled in-edges of one destination in layer `layer` (Sect. 3.9): the CSR edge indices kept, ascending,
 * and their sources; n = min(in_degree, fanout) (all in-edges when fanout is 0).  Host outputs.
 */
int taurus_get_sampled_edges(taurus_ctx* ctx, int32_t layer, int64_t dst, int64_t* out_edge_ids, int32_t* out_sources,
                             int32_t capacity, int32_t* n);

/* The propagated-edge mask of the current layer as one bit per CSR edge (bit e & 31 of word e >> 5),
 * host output of ceil(E / 32) words; all ones in exact mode. */
int taurus_get_edge_mask(taurus_ctx* ctx, uint32_t* out_words);

/* Per-destination digest of the current layer's propagated in-edges, for checking sampled neighbour sets of all
 * V vertices at once (Sect. 3.9 sampling paragraph): with h(u, e) = mix64(((u << 32) | e) + 0x9E3779B97F4A7C15)
 * for a propagated edge number e (its CSR index) from source u, where mix64(x) is x ^= x >> 30;
 * x *= 0xBF58476D1CE4E5B9; x ^= x >> 27; x *= 0x94D049BB133111EB; x ^= x >> 31 on 64-bit words,
 * out_digest[2 v] = sum of h over the propagated in-edges of v (mod 2^64) and out_digest[2 v + 1] = their
 * xor; both 0 for a vertex without propagated in-edges.  out_digest: [2 V] words, host or device memory.
 * Blocking. */
int taurus_get_sample_digest(taurus_ctx* ctx, uint64_t* out_digest);

/* Upper bound on the vertices that sources [src_begin, src_end) complete in the current layer
 * (exact when both ends are multiples of 64 or the ends of the graph). */
int taurus_completion_bound(taurus_ctx* ctx, int64_t src_begin, int64_t src_end, int64_t* out_bound);

/*
 * (No counterpart in the paper: an addition of this library.)
 *
 * Completion counts without any allocation.  Some callers cannot let a library allocate device memory
 * while they run: a serving process whose framework allocator already owns the whole GPU (cudaMalloc
 * would fail or fragment it), a real-time loop in which cudaMalloc / cudaFree would stall every stream of
 * the device, or an embedder whose memory is accounted per request.  For them this entry point computes
 * what taurus_layer_begin computes for taurus_completion_bound, but with its scratch (one int32 per
 * vertex) in a static device array inside the library image instead of memory obtained at run time.
 * It calls no cudaMalloc, cudaFree, cudaHostAlloc or other allocating routine.
 *
 * out_counts[b], b in [0, ceil(V / 64)), receives the number of vertices whose completion rank
 * max(v, largest source among the propagated in-edges of v) lies in [64 b, 64 b + 64): the vertices a
 * push of those 64 sources completes (Sect. 3.8, c(v)).  edge_mask is the layer's propagated-edge mask in
 * the format of taurus_get_edge_mask, or NULL when every edge is propagated.  *out_bad_index is set to 1
 * if a destination outside [0, V) was met (such edges are skipped) or if a row of row_ptr does not lie
 * inside [0, E] in ascending order (the row is cut to the part inside [0, E], so col_idx and edge_mask are
 * never read beyond their E entries, and the counts are then not meaningful), else 0.
 *
 * Arguments: row_ptr [V+1], col_idx [E], edge_mask [ceil(E/32)] or NULL, out_counts [ceil(V/64)] and
 * out_bad_index [1] are DEVICE pointers owned by the caller; the work is enqueued on cuda_stream
 * (a cudaStream_t, NULL = default stream) on the current device and the call does not wait for it.
 *
 * Limits and sharing: V may not exceed TAURUS_NOALLOC_MAX_VERTICES (else TAURUS_ERR_UNSUPPORTED, nothing
 * is enqueued).  The scratch array (16 MiB) is part of the library image: every GPU on which the library
 * is loaded keeps it until the process exits.  All calls on a device share it and it keeps the previous
 * call's contents; each call rewrites the entries it reads, so calls issued one after another on one
 * stream are independent, but two calls whose kernels overlap on the GPU (different streams, or different
 * host threads) race on it and must be serialised by the caller.  The first call on each device looks up
 * the array's device address (cudaGetSymbolAddress, with that device current); make that first call
 * before starting any stream capture.
 */
#define TAURUS_NOALLOC_MAX_VERTICES (4 * 1024 * 1024)
int taurus_completion_counts_noalloc(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx,
                                     const uint32_t* edge_mask, int32_t* out_counts, int32_t* out_bad_index,
                                     void* cuda_stream);

/*
 * Topology-aware reordering, Alg. 1 of Sect. 3.8 (pre-processing; needs no context).  Starting from the
 * positions r(v) = initial_rank[v] (identity when NULL) it repeats `iterations` times
 *     mu(v) = (r(v) + sum_{u -> v} r(u)) / d(v)                                     d(v) = in-degree + 1
 *     r(w)  = (mu(w)/d(w) + sum_{w -> v} mu(v)/d(v)) / (1/d(w) + sum_{w -> v} 1/d(v))
 * (every vertex also aggregates its own self message, so d >= 1 and each vertex belongs to its own
 * neighbourhoods) and returns pi = ArgSort(r), ties by vertex id, as out_rank[v] = new processing rank of v.
 * The real-valued positions are carried from one iteration to the next as Alg. 1 states them.
 * out_positions ([V] doubles, may be NULL) receives the final r.  out_J and out_span ([iterations + 1], HOST
 * memory, may be NULL) receive, for the initial order and after every iteration, the dispersion J and the
 * total span C(pi) = sum_v (max - min) of the ranks of v's in-neighbours and v, both evaluated on the ordering
 * itself (positions = ranks, centres = their optimum).  row_ptr, col_idx, initial_rank, out_rank and
 * out_positions may be host or device memory.  Blocking; all arithmetic in fp64.
 */
int taurus_reorder(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx, const int32_t* initial_rank,
                   int32_t iterations, int32_t* out_rank, double* out_positions, double* out_J, int64_t* out_span,
                   void* cuda_stream);

/* ------------------------------------------------------------------------------------------------------------
 * Output side of a layer: sorted runs (embedding writer, Sect. 3.7) and merge-on-read (graph reader, Sect. 3.3).
 *
 * Finished rows leave the graduation buffer in completion order, not vertex order.  A taurus_runs object
 * cuts the id space [0, V) into `partitions` fixed ranges of ceil(V / partitions) ids and keeps one
 * partition buffer of `partition_rows` rows per range in device memory.  An appended row goes to the buffer
 * of its range, in arrival order; a buffer that reaches partition_rows rows is sorted by vertex id on the
 * GPU and written sequentially to the run store as one sorted run (ids I_f, rows X_f); runs are never
 * merged.  taurus_runs_read_chunk rebuilds the matrix of a chunk [s, e) in vertex order: for every run that
 * overlaps it, two binary searches (first id >= s, first id >= e) delimit a contiguous slice, the slice is
 * copied to the device in one transfer, and the slices are merged by vertex id.  The run store stands for the
 * paper's run files on SSD: pinned host memory (TAURUS_RUNS_HOST) or device memory (TAURUS_RUNS_DEVICE); the
 * ids of all runs are always kept in pinned host memory, where the searches run.
 *
 * Run k of a range holds that range's arrivals k * partition_rows .. (k + 1) * partition_rows - 1 (arrival
 * order = order of the rows within each append, appends in call order), so the set of runs is a function of
 * the arrival sequence alone.  One object is used from one host thread at a time; calls on it are ordered on
 * the streams given (the library inserts the dependencies between streams itself).
 */
enum { TAURUS_RUNS_HOST = 0, TAURUS_RUNS_DEVICE = 1 };
typedef struct {
  int64_t V;                /* vertex ids are in [0, V), V < 2^31                                              */
  int32_t width;            /* floats per row, 1..1024                                                          */
  int32_t store_kind;       /* TAURUS_RUNS_HOST | TAURUS_RUNS_DEVICE                                            */
  int64_t partitions;       /* number of id ranges, 1..1024                                                     */
  int64_t partition_rows;   /* rows a partition buffer holds before it is sorted and flushed                   */
  int64_t store_rows;       /* capacity of the run store in rows (V holds one layer's output)                  */
  int64_t max_append_rows;  /* most rows one taurus_runs_append call (or one chunk of a layer) may bring        */
  int64_t max_chunk_rows;   /* most ids one taurus_runs_read_chunk call may span                                */
} taurus_runs_config;

/* Allocates the partition buffers, the run store and the scratch (all sizes fixed here).  TAURUS_ERR_NOMEM /
 * TAURUS_ERR_INVALID_ARG on failure, *out untouched. */
int taurus_runs_create(taurus_runs** out, const taurus_runs_config* config);
/* Appends `count` rows: ids[i] is the vertex of rows[i * ld .. i * ld + width).  ids and rows are device
 * memory or pinned host memory and must stay valid until the stream has passed this call.  Flushes every
 * partition buffer that fills on the way.  Blocks the host once for the per-range counts.  An id outside
 * [0, V) gives TAURUS_ERR_INVALID_ARG and appends nothing; a flush that does not fit the store gives
 * TAURUS_ERR_RUN_STORE_FULL before anything is changed. */
int taurus_runs_append(taurus_runs* runs, const int64_t* ids, const float* rows, int64_t ld, int64_t count, void* cuda_stream);
/* End of the layer: every non-empty partition buffer is sorted and written as a (short) run. */
int taurus_runs_flush(taurus_runs* runs, void* cuda_stream);
/* Merge-on-read.  Writes rows of vertices [src_begin, src_end) in vertex order to out_rows (device memory,
 * row v - src_begin at out_rows + (v - src_begin) * ld), asynchronously on the stream.  Every vertex of the
 * range must be present in exactly one run: otherwise TAURUS_ERR_RUNS_INCOMPLETE (rows still held in a
 * partition buffer do not count: flush first) and out_rows is untouched. */
int taurus_runs_read_chunk(taurus_runs* runs, int64_t src_begin, int64_t src_end, float* out_rows, int64_t ld, void* cuda_stream);
/* Counters (any pointer may be NULL): runs written, rows in the store, rows still in partition buffers. */
int taurus_runs_info(taurus_runs* runs, int64_t* out_runs, int64_t* out_stored_rows, int64_t* out_buffered_rows);
/* Directory in writing order: out[4 r + 0..3] = range, rows, first id, last id of run r (HOST memory).
 * Blocking. */
int taurus_runs_directory(taurus_runs* runs, int64_t* out, int64_t capacity_runs, int64_t* out_runs);
/* Copies run `run` to HOST memory: out_ids [rows] and out_rows [rows x width] (either may be NULL).  Blocking. */
int taurus_runs_get_run(taurus_runs* runs, int64_t run, int64_t* out_ids, float* out_rows);
/* Forgets every run and every buffered row (the object is reused for the next layer's output).  Blocking. */
int taurus_runs_reset(taurus_runs* runs);
void taurus_runs_destroy(taurus_runs* runs);

/* Run-output mode for the layer just begun (call after taurus_layer_begin, before the first push; exclusive
 * with taurus_layer_set_dense_output).  Each chunk's finished rows are appended to `runs` (width must be
 * dims[layer + 1]) on the library's output stream while the next chunk computes; the graduation buffer is
 * split in halves as in dense-output mode (same drain_rows rule), runs->max_append_rows must be at least
 * drain_rows / 2, and taurus_drain_* are not needed.  taurus_layer_end appends the last chunk's rows, flushes
 * all partition buffers and waits, so that the runs can be read afterwards.  Which rows share a run depends
 * on the order in which vertices of one chunk complete, which is not fixed; the rows themselves are. */
int taurus_layer_set_run_output(taurus_ctx* ctx, taurus_runs* runs);
/* taurus_push_chunk with the chunk's features read from `runs` (merge-on-read into the library's staging
 * buffer on its copy stream, overlapping the previous chunk's kernels).  runs' width must be dims[layer]. */
int taurus_push_chunk_from_runs(taurus_ctx* ctx, int64_t src_begin, int64_t src_end, taurus_runs* runs, void* cuda_stream);

/*
 * Applying an ordering (Sect. 3.8: topology relabelling and feature relabelling).  rank is a permutation of
 * [0, V), e.g. out_rank of taurus_reorder: vertex v becomes vertex rank[v].
 * taurus_relabel_csr: row rank[u] of the output holds the out-edges of u in their original order with every
 * destination v renamed rank[v]; out_in_degree (may be NULL) receives the in-degrees of the relabelled graph.
 * All pointers host or device memory; blocking; TAURUS_ERR_INVALID_ARG when rank is not a permutation or a
 * destination lies outside [0, V) (outputs then undefined).
 * taurus_permute_rows: out_rows[rank[v]] = in_rows[v] for a [V x width] matrix (ld_in, ld_out in floats);
 * DEVICE memory only, in_rows != out_rows, asynchronous on the stream; rank is not checked here.
 */
int taurus_relabel_csr(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col_idx, const int32_t* rank,
                       int64_t* out_row_ptr, int32_t* out_col_idx, int32_t* out_in_degree, void* cuda_stream);
int taurus_permute_rows(int64_t V, int32_t width, const float* in_rows, int64_t ld_in, const int32_t* rank, float* out_rows,
                        int64_t ld_out, void* cuda_stream);

/* Which order layer `layer` runs in: *out_aggregate_first = 1 when it aggregates (scaled) input rows and applies the
 * weights to the finished rows (see TAURUS_FLAG_PROJECT_FIRST), 0 when it projects every chunk first;
 * *out_row_floats = floats per accumulator row (and per evicted row) of that layer.  Either pointer may be NULL.
 * Decided at taurus_graph_init; no device work. */
int taurus_get_layer_plan(const taurus_ctx* ctx, int32_t layer, int32_t* out_aggregate_first, int32_t* out_row_floats);

/* Kernels launched by this context since init (for launch accounting in benchmarks). */
int64_t taurus_launch_count(const taurus_ctx* ctx);

/* Per-push device times.  taurus_set_timing(ctx, 1) starts a recording window: every later push (up to
 * 16384) brackets its phases with CUDA events.  taurus_get_phase_ms (blocking) returns, for each recorded push p,
 * out[p * 9 + k] in milliseconds: k = 0 copy-in, 1 projection, 2 classify and victim selection, 3 the wait for the
 * previous chunk's row transfers plus that chunk's finalise (bounded pools; else about zero), 4 slot hand-out (victims'
 * rows staged, new rows cleared), 5 scatter, 6 completion list, 7 the chunk's own finalise, 8 the chunk's row
 * transfers over the host link (evicted rows out, reloaded rows in; on the library's transfer stream, beside
 * k = 5, 6 of this chunk and k = 0..2 of the next); *out_pushes = pushes written (at most capacity_pushes).
 * An event between two kernels costs about 2 us of the stream (twelve per push: 4-5 % of a pass whose pushes take half a
 * millisecond); taurus_set_timing(ctx, 2) records only the two events around the scatter, and taurus_get_phase_ms then
 * fills k = 5 and leaves the other columns 0.  on = 0 ends the window; another value is TAURUS_ERR_INVALID_ARG.  The
 * call first enqueues the finalise of a chunk whose finalise was deferred (bounded pools), as the blocking calls do. */
int taurus_set_timing(taurus_ctx* ctx, int32_t on);
int taurus_get_phase_ms(taurus_ctx* ctx, float* out, int64_t capacity_pushes, int64_t* out_pushes);

void taurus_destroy(taurus_ctx* ctx);
const char* taurus_strerror(int code);
/* Text of the last CUDA runtime error seen by this library on this thread ("" if none). */
const char* taurus_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TAURUS_H */
