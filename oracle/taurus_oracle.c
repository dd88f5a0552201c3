/*
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain, slow CPU oracle for the layer-wise GNN step: the destination-centric
 * (pull, "gather") form of Eq. 1-2, evaluated in fp64, plus an integer-only
 * simulator of the per-vertex state machine at chunk granularity.  It shares no
 * code with the CUDA library and only tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it.
 *
 * Everything here is written for checking by eye against the paper, not for
 * speed: no blocking, no fusion, no atomics.
 *
 * Parity pins (tests marked "not gpu"): dense-adjacency matrix products on tiny
 * graphs, ring/star/complete closed forms, constant-feature and linearity
 * invariants, split-vs-concatenated weights, sampler set properties and a
 * chi-square uniformity check, completion-chunk closed form vs simulator, the
 * active-set identity, and a second independent pure-Python simulator.
 * No function in this file is "parity unpinned".
 */
#include <stdint.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ in-lists
 * Sect. 2.2 (gather model): destination v pulls from its in-neighbours N^-(v).
 * The in-list of v holds one entry per CSR edge (u -> v) (multigraph: duplicates
 * kept), ordered by ascending source id, equal sources in CSR order.  A single
 * pass over the CSR in storage order yields exactly that order.
 */
int to_build_in_lists(int64_t V, int64_t E, const int64_t* row_ptr, const int32_t* col,
                      int64_t* in_ptr /*[V+1]*/, int32_t* in_src /*[E]*/, int64_t* in_eid /*[E]*/) {
  int64_t* cur = (int64_t*)calloc((size_t)V + 1, sizeof(int64_t));
  if (!cur) return -1;
  for (int64_t e = 0; e < E; ++e) cur[col[e]] += 1;
  in_ptr[0] = 0;
  for (int64_t v = 0; v < V; ++v) in_ptr[v + 1] = in_ptr[v] + cur[v];
  for (int64_t v = 0; v < V; ++v) cur[v] = in_ptr[v];
  for (int64_t u = 0; u < V; ++u)
    for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) {
      int64_t p = cur[col[e]]++;
      in_src[p] = (int32_t)u;
      in_eid[p] = e;
    }
  free(cur);
  return 0;
}

/* In-edges of a marked subset of destinations: every CSR edge (u -> v) with wanted[v] != 0, in ascending edge index
 * (= ascending source, CSR order among equal sources).  Rows are cut into one contiguous block per thread; the blocks
 * are counted, then filled at their offsets, so the output order does not depend on the thread count.
 * out_eid / out_src may be NULL (count only).  Returns the number of such edges, or -1 if it exceeds `capacity`
 * when filling. */
int64_t to_scan_in_edges(int64_t V, const int64_t* row_ptr, const int32_t* col, const uint8_t* wanted,
                         int64_t* out_eid, int64_t* out_src, int64_t capacity) {
  int T = 1;
#ifdef _OPENMP
  T = omp_get_max_threads();
#endif
  int64_t* cnt = (int64_t*)calloc((size_t)T + 1, sizeof(int64_t));
  if (!cnt) return -1;
#pragma omp parallel for schedule(static, 1)
  for (int t = 0; t < T; ++t) {
    const int64_t u0 = V * t / T, u1 = V * (t + 1) / T;
    int64_t n = 0;
    for (int64_t e = row_ptr[u0]; e < row_ptr[u1]; ++e) n += wanted[col[e]] != 0;
    cnt[t + 1] = n;
  }
  for (int t = 0; t < T; ++t) cnt[t + 1] += cnt[t];
  const int64_t total = cnt[T];
  if (out_eid && out_src) {
    if (total > capacity) { free(cnt); return -1; }
#pragma omp parallel for schedule(static, 1)
    for (int t = 0; t < T; ++t) {
      const int64_t u0 = V * t / T, u1 = V * (t + 1) / T;
      int64_t p = cnt[t];
      for (int64_t u = u0; u < u1; ++u)
        for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e)
          if (wanted[col[e]]) { out_eid[p] = e; out_src[p] = u; ++p; }
    }
  }
  free(cnt);
  return total;
}

/* Completion rank of every vertex for an exact layer: max(v, largest in-neighbour of v) (Sect. 3.8, c(v) with the self
 * message).  One pass over the CSR; the maximum is taken with a compare-and-swap so that the rows can be split among
 * threads. */
void to_completion_rank_exact(int64_t V, const int64_t* row_ptr, const int32_t* col, int32_t* rank /*[V]*/) {
#pragma omp parallel for schedule(static)
  for (int64_t v = 0; v < V; ++v) rank[v] = (int32_t)v;
#pragma omp parallel for schedule(static, 4096)
  for (int64_t u = 0; u < V; ++u)
    for (int64_t e = row_ptr[u]; e < row_ptr[u + 1]; ++e) {
      int32_t* p = &rank[col[e]];
      int32_t old = __atomic_load_n(p, __ATOMIC_RELAXED);
      while (old < (int32_t)u && !__atomic_compare_exchange_n(p, &old, (int32_t)u, 1, __ATOMIC_RELAXED, __ATOMIC_RELAXED)) {}
    }
}

/* ------------------------------------------------------------------ sampling
 * Sect. 3.9, "Sampling-based Inference": up to k incoming edges per vertex are
 * kept for a layer, the rest suppressed.  The choice is a deterministic function
 * of (seed, layer, dst): a partial Fisher-Yates shuffle of the in-list positions
 * 0..din-1 driven by a counter hash; the first k entries after k swaps are kept.
 */
static uint64_t to_mix(uint64_t x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27; x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}
static uint64_t to_absorb(uint64_t h, uint64_t x) { return to_mix(h ^ (0x9E3779B97F4A7C15ull * (x + 1ull))); }

uint64_t to_sample_hash(uint64_t seed, uint64_t layer, uint64_t dst, uint64_t k) {
  uint64_t h = 0x243F6A8885A308D3ull;
  h = to_absorb(h, seed);
  h = to_absorb(h, layer);
  h = to_absorb(h, dst);
  h = to_absorb(h, k);
  return h;
}

/* Writes the kept positions (count = min(din, fanout)) in draw order. */
int to_sample_positions(uint64_t seed, int32_t layer, int64_t dst, int64_t din, int32_t fanout, int64_t* out_pos) {
  if (fanout <= 0 || din <= fanout) {
    for (int64_t i = 0; i < din; ++i) out_pos[i] = i;
    return 0;
  }
  int64_t* perm = (int64_t*)malloc(sizeof(int64_t) * (size_t)din);
  if (!perm) return -1;
  for (int64_t i = 0; i < din; ++i) perm[i] = i;
  for (int64_t k = 0; k < fanout; ++k) {
    uint64_t h = to_sample_hash(seed, (uint64_t)layer, (uint64_t)dst, (uint64_t)k);
    /* j uniform on [k, din): k + floor(h * (din - k) / 2^64) */
    int64_t j = k + (int64_t)(((unsigned __int128)h * (unsigned __int128)(uint64_t)(din - k)) >> 64);
    int64_t t = perm[k]; perm[k] = perm[j]; perm[j] = t;
  }
  for (int64_t k = 0; k < fanout; ++k) out_pos[k] = perm[k];
  free(perm);
  return 0;
}

static int cmp_i64(const void* a, const void* b) {
  int64_t x = *(const int64_t*)a, y = *(const int64_t*)b;
  return (x > y) - (x < y);
}

/*
 * Message sets M(v) for one layer: all in-edges when fanout == 0 or din <= fanout,
 * else the sampled ones.  msg_ptr[V+1] must already hold the prefix sums of
 * min(din, fanout) (or din).  Entries of M(v) are stored in ascending in-list
 * position.  prop[E] (may be NULL) gets 1 for every propagated CSR edge.
 */
int to_message_sets(int64_t V, const int64_t* in_ptr, const int32_t* in_src, const int64_t* in_eid,
                    int32_t fanout, uint64_t seed, int32_t layer,
                    const int64_t* msg_ptr, int32_t* msg_src, int64_t* msg_eid, uint8_t* prop) {
  int rc = 0;
#pragma omp parallel for schedule(dynamic, 1024)
  for (int64_t v = 0; v < V; ++v) {
    int64_t din = in_ptr[v + 1] - in_ptr[v];
    int64_t m = msg_ptr[v + 1] - msg_ptr[v];
    int64_t* pos = (int64_t*)malloc(sizeof(int64_t) * (size_t)(m > 0 ? m : 1));
    if (!pos || to_sample_positions(seed, layer, v, din, fanout, pos) != 0) { rc = -1; free(pos); continue; }
    qsort(pos, (size_t)m, sizeof(int64_t), cmp_i64);
    for (int64_t i = 0; i < m; ++i) {
      int64_t p = in_ptr[v] + pos[i];
      msg_src[msg_ptr[v] + i] = in_src[p];
      msg_eid[msg_ptr[v] + i] = in_eid[p];
      if (prop) prop[in_eid[p]] = 1;
    }
    free(pos);
  }
  return rc;
}

/* ------------------------------------------------------------------ aggregate
 * Eq. 1: x_v = AGGREGATE({h_u : u in M(v)}) as the weighted sum
 *   agg[i] = sum_{u in M(dst[i])} c_out[u] * h[u]      (fp64)
 * c_out may be NULL (all ones).  h is [*, d] row-major, indexed by the values
 * stored in msg_src.
 */
int to_aggregate(int64_t n_dst, const int64_t* dst, const int64_t* msg_ptr, const int32_t* msg_src,
                 const double* c_out, const double* h, int32_t d, double* agg /*[n_dst, d]*/) {
#pragma omp parallel for schedule(dynamic, 256)
  for (int64_t i = 0; i < n_dst; ++i) {
    int64_t v = dst[i];
    double* a = agg + i * (int64_t)d;
    for (int32_t c = 0; c < d; ++c) a[c] = 0.0;
    for (int64_t p = msg_ptr[v]; p < msg_ptr[v + 1]; ++p) {
      int64_t u = msg_src[p];
      double w = c_out ? c_out[u] : 1.0;
      const double* hu = h + u * (int64_t)d;
      for (int32_t c = 0; c < d; ++c) a[c] += w * hu[c];
    }
  }
  return 0;
}

/* ------------------------------------------------------------------ state machine
 * Sect. 3.4 (states and transitions), 3.5.1-3.5.3 (GPU store, hot store, fewest-
 * pending eviction), 3.6 (graduation at pending == 0), at chunk granularity.
 *
 * Per layer: state NOT_STARTED, pend[v] = |M(v)| + 1 (the +1 is v's own self
 * message, delivered in v's chunk), free = pool_slots.  Per chunk [s, e):
 *   1. T = non-hub vertices that receive >= 1 propagated message from [s, e),
 *      together with the non-hub vertices of [s, e) themselves.
 *   2. record the split of T by state, and the hub vertices touched.
 *   3. need = #{v in T : NOT_STARTED or EVICTED};  need > pool_slots -> error.
 *   4. deficit = need - free; if > 0 evict the `deficit` smallest (score, id)
 *      among IN_BUFFER vertices outside T (too few -> error).  The score is the
 *      pending count (the paper's policy, Sect. 3.5.3) or, for the ablation of
 *      Sect. 4.5: the chunk in which the vertex entered the pool (FIFO), the
 *      chunk that last touched it (LRU), or a hash of (seed, vertex, chunk)
 *      (random).
 *   5. EVICTED in T -> IN_BUFFER (a reload); NOT_STARTED in T -> IN_BUFFER.
 *   6. deliver: pend[v] -= messages from [s, e) into v, and -1 for v in [s, e).
 *   7. vertices whose pend reached 0 complete; non-hub ones free their slot.
 */
enum { ST_NS = 0, ST_IB = 1, ST_EV = 2, ST_OG = 3, ST_CP = 4 };
enum {
  SK_EVICTIONS = 0, SK_RELOADS, SK_MAX_RELOAD, SK_PEAK_OCC, SK_HUB_MSGS, SK_TOTAL_MSGS, SK_HUB_VERTS,
  SK_COMPLETED, SK_SUM_HS, SK_SUM_NS, SK_SUM_EV, SK_SUM_GS, SK_FREE_END, SK_BAD_TRANSITIONS, SK_COUNT
};
/* per-chunk record columns */
enum { CK_HS = 0, CK_NS, CK_EV, CK_GS, CK_NEED, CK_EVICTED, CK_RELOADED, CK_COMPLETED, CK_OCC, CK_COUNT };

enum { EV_FEWEST_PENDING = 0, EV_FIFO = 1, EV_LRU = 2, EV_RANDOM = 3 };

/* 31-bit score of the random policy */
uint32_t to_evict_hash(uint64_t seed, uint64_t vertex, uint64_t chunk) {
  uint64_t h = 0x452821E638D01377ull;
  h = to_absorb(h, seed);
  h = to_absorb(h, vertex);
  h = to_absorb(h, chunk);
  return (uint32_t)(h >> 33);
}

typedef struct { int32_t pend; int32_t id; } to_key;   /* pend holds the policy's score */
static int cmp_key(const void* a, const void* b) {
  const to_key* x = (const to_key*)a; const to_key* y = (const to_key*)b;
  if (x->pend != y->pend) return (x->pend > y->pend) - (x->pend < y->pend);
  return (x->id > y->id) - (x->id < y->id);
}

/* allowed transitions: NS->IB, NS->OG, IB->EV, EV->IB, IB->CP, OG->CP */
static int to_allowed(int a, int b) {
  return (a == ST_NS && (b == ST_IB || b == ST_OG)) || (a == ST_IB && (b == ST_EV || b == ST_CP)) ||
         (a == ST_EV && b == ST_IB) || (a == ST_OG && b == ST_CP);
}

/* returns 0, -1 (out of memory), -2 (pool too small: need > pool), -3 (pool too small: too few victims) */
int to_simulate(int64_t V, const int64_t* row_ptr, const int32_t* col, const uint8_t* prop /*NULL = all*/,
                const int32_t* m /*[V] = |M(v)|*/, const uint8_t* is_hub /*[V]*/,
                int64_t chunk_sources, int64_t pool_slots, int32_t policy, uint64_t seed,
                int64_t* stats /*[SK_COUNT]*/, int32_t* complete_chunk /*[V]*/, int32_t* reload_count /*[V]*/,
                int64_t* per_chunk /*[n_chunks, CK_COUNT]*/, int32_t* evict_chunk_log /*[V] last chunk evicted, -1*/) {
  int64_t n_chunks = (V + chunk_sources - 1) / chunk_sources;
  uint8_t* state = (uint8_t*)calloc((size_t)V, 1);
  int32_t* pend = (int32_t*)malloc(sizeof(int32_t) * (size_t)V);
  int32_t* stamp = (int32_t*)malloc(sizeof(int32_t) * (size_t)V);
  int32_t* T = (int32_t*)malloc(sizeof(int32_t) * (size_t)V);
  int32_t* hubT = (int32_t*)malloc(sizeof(int32_t) * (size_t)V);
  to_key* cand = (to_key*)malloc(sizeof(to_key) * (size_t)V);
  int32_t* entered = (int32_t*)calloc((size_t)V, sizeof(int32_t));   /* chunk of the latest NS/EV -> IB */
  int32_t* touched_at = (int32_t*)calloc((size_t)V, sizeof(int32_t)); /* chunk of the latest touch */
  if (!state || !pend || !stamp || !T || !hubT || !cand || !entered || !touched_at) return -1;
  memset(stats, 0, sizeof(int64_t) * SK_COUNT);
  int64_t free_slots = pool_slots, occupied = 0;
  int rc = 0;
  for (int64_t v = 0; v < V; ++v) {
    pend[v] = m[v] + 1; stamp[v] = -1; complete_chunk[v] = -1; reload_count[v] = 0;
    if (evict_chunk_log) evict_chunk_log[v] = -1;
    if (is_hub[v]) stats[SK_HUB_VERTS] += 1;
  }
#define TRANSITION(v, to) do { if (!to_allowed(state[v], (to))) stats[SK_BAD_TRANSITIONS] += 1; state[v] = (to); } while (0)
  for (int64_t c = 0; c < n_chunks && rc == 0; ++c) {
    int64_t s = c * chunk_sources, e = s + chunk_sources < V ? s + chunk_sources : V;
    int64_t* rec = per_chunk + c * CK_COUNT;
    memset(rec, 0, sizeof(int64_t) * CK_COUNT);
    /* step 1 */
    int64_t nT = 0, nHub = 0;
    for (int64_t u = s; u < e; ++u) {
      if (stamp[u] != c) { stamp[u] = (int32_t)c; if (is_hub[u]) hubT[nHub++] = (int32_t)u; else T[nT++] = (int32_t)u; }
      for (int64_t ed = row_ptr[u]; ed < row_ptr[u + 1]; ++ed) {
        if (prop && !prop[ed]) continue;
        int32_t v = col[ed];
        if (stamp[v] != c) { stamp[v] = (int32_t)c; if (is_hub[v]) hubT[nHub++] = v; else T[nT++] = v; }
      }
    }
    /* step 2, 3 */
    int64_t need = 0;
    for (int64_t i = 0; i < nT; ++i) {
      int st = state[T[i]];
      if (st == ST_IB) rec[CK_HS] += 1;
      else if (st == ST_NS) { rec[CK_NS] += 1; need += 1; }
      else if (st == ST_EV) { rec[CK_EV] += 1; need += 1; }
    }
    rec[CK_GS] = nHub;
    rec[CK_NEED] = need;
    if (need > pool_slots) { rc = -2; break; }
    /* step 4 */
    int64_t deficit = need - free_slots;
    if (deficit > 0) {
      int64_t nc = 0;
      for (int64_t v = 0; v < V; ++v)
        if (state[v] == ST_IB && stamp[v] != c) {
          int32_t score = pend[v];
          if (policy == EV_FIFO) score = entered[v];
          else if (policy == EV_LRU) score = touched_at[v];
          else if (policy == EV_RANDOM) score = (int32_t)to_evict_hash(seed, (uint64_t)v, (uint64_t)c);
          cand[nc].pend = score; cand[nc].id = (int32_t)v; nc++;
        }
      if (nc < deficit) { rc = -3; break; }
      qsort(cand, (size_t)nc, sizeof(to_key), cmp_key);
      for (int64_t i = 0; i < deficit; ++i) {
        int32_t v = cand[i].id;
        TRANSITION(v, ST_EV);
        if (evict_chunk_log) evict_chunk_log[v] = (int32_t)c;
        stats[SK_EVICTIONS] += 1;
      }
      rec[CK_EVICTED] = deficit;
      free_slots += deficit; occupied -= deficit;
    }
    /* step 5 */
    for (int64_t i = 0; i < nT; ++i) {
      int32_t v = T[i];
      touched_at[v] = (int32_t)c;
      if (state[v] != ST_IB) entered[v] = (int32_t)c;
      if (state[v] == ST_EV) {
        TRANSITION(v, ST_IB); stats[SK_RELOADS] += 1; rec[CK_RELOADED] += 1; reload_count[v] += 1;
        if (reload_count[v] > stats[SK_MAX_RELOAD]) stats[SK_MAX_RELOAD] = reload_count[v];
      } else if (state[v] == ST_NS) TRANSITION(v, ST_IB);
    }
    for (int64_t i = 0; i < nHub; ++i) if (state[hubT[i]] == ST_NS) TRANSITION(hubT[i], ST_OG);
    free_slots -= need; occupied += need;
    if (occupied > stats[SK_PEAK_OCC]) stats[SK_PEAK_OCC] = occupied;
    /* step 6 */
    for (int64_t u = s; u < e; ++u) {
      pend[u] -= 1;
      for (int64_t ed = row_ptr[u]; ed < row_ptr[u + 1]; ++ed) {
        if (prop && !prop[ed]) continue;
        int32_t v = col[ed];
        pend[v] -= 1;
        stats[SK_TOTAL_MSGS] += 1;
        if (is_hub[v]) stats[SK_HUB_MSGS] += 1;
      }
    }
    /* step 7 */
    for (int64_t i = 0; i < nT; ++i) {
      int32_t v = T[i];
      if (pend[v] == 0) { TRANSITION(v, ST_CP); complete_chunk[v] = (int32_t)c; free_slots += 1; occupied -= 1; rec[CK_COMPLETED] += 1; }
      else if (pend[v] < 0) stats[SK_BAD_TRANSITIONS] += 1;
    }
    for (int64_t i = 0; i < nHub; ++i) {
      int32_t v = hubT[i];
      if (pend[v] == 0) { TRANSITION(v, ST_CP); complete_chunk[v] = (int32_t)c; rec[CK_COMPLETED] += 1; }
      else if (pend[v] < 0) stats[SK_BAD_TRANSITIONS] += 1;
    }
    stats[SK_COMPLETED] += rec[CK_COMPLETED];
    stats[SK_SUM_HS] += rec[CK_HS]; stats[SK_SUM_NS] += rec[CK_NS];
    stats[SK_SUM_EV] += rec[CK_EV]; stats[SK_SUM_GS] += rec[CK_GS];
    rec[CK_OCC] = occupied;
  }
#undef TRANSITION
  stats[SK_FREE_END] = free_slots;
  free(state); free(pend); free(stamp); free(T); free(hubT); free(cand); free(entered); free(touched_at);
  return rc;
}
