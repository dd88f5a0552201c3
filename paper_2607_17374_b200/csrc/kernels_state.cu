// Per-vertex state machine on the device (Sect. 3.4-3.6): classify the destinations a chunk touches,
// make room in the slot pool (fewest-pending eviction, Sect. 3.5.3), allocate / reload slots,
// finalise completed vertices into the graduation buffer.  All decisions are taken from integer state
// at chunk granularity, so the accounting is deterministic although the scatter is not ordered.
//
// Every kernel reads the counts it depends on from the device control block and is launched with a
// fixed grid, so a push never waits for the host.  A kernel that finds ctl->error set returns at once.
#include "taurus_internal.h"

#define FULL 0xffffffffu

static __device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

static __device__ __forceinline__ bool edge_propagated(const uint32_t* mask, long long e) {
  return mask == nullptr || ((mask[e >> 5] >> (e & 31)) & 1u);
}

static __device__ __forceinline__ int messages_of(int din, int fanout) {
  return (fanout > 0 && din > fanout) ? fanout : din;
}

// ------------------------------------------------------------------------------------------------ layer reset
__global__ void reset_vertices_kernel(long long V, const int32_t* din, int fanout, int32_t* pend, uint8_t* state,
                                      int32_t* loc, int32_t* touch, int32_t* reload, int direct) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) {
    pend[v] = messages_of(din[v], fanout) + 1;
    state[v] = TAURUS_NOT_STARTED;
    loc[v] = direct ? (int32_t)v : -1;
    touch[v] = 0;
    reload[v] = 0;
  }
}

__global__ void reset_pool_kernel(long long pool_slots, long long n_ext, long long n_buckets, long long hub_count, const int32_t* hub_ids,
                                  int32_t* loc, int32_t* owner, int32_t* free_stack, int32_t* ext_free, int32_t* ext_live,
                                  int32_t* bk_tail_ext, int32_t* bk_tail_fill, int32_t* bk_new, DevCtl* ctl) {
  long long stride = (long long)gridDim.x * blockDim.x;
  long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long i = tid; i < pool_slots; i += stride) {
    owner[i] = -1;
    free_stack[i] = (int32_t)(pool_slots - 1 - i);   // slot 0 is handed out first
  }
  for (long long i = tid; i < n_ext; i += stride) { ext_free[i] = (int32_t)(n_ext - 1 - i); ext_live[i] = 0; }
  for (long long i = tid; i < n_buckets; i += stride) { bk_tail_ext[i] = -1; bk_tail_fill[i] = 0; bk_new[i] = 0; }
  for (long long i = tid; i < hub_count; i += stride) loc[hub_ids[i]] = (int32_t)(pool_slots + i);
  if (tid == 0) {
    ctl->free_top = pool_slots;
    ctl->ext_free_top = n_ext;
    ctl->host_live = 0;
  }
}

void launch_layer_reset(taurus_ctx* c, int layer, cudaStream_t st) {
  int blocks = c->sm_count * 8;
  cudaMemsetAsync(c->d_ctl, 0, sizeof(DevCtl), st);
  reset_vertices_kernel<<<blocks, 256, 0, st>>>(c->V, c->d_din, c->fanout[layer], c->d_pend, c->d_state, c->d_loc,
                                                c->d_touch, c->d_reload, c->pool_slots >= c->V ? 1 : 0);
  reset_pool_kernel<<<blocks, 256, 0, st>>>(c->pool_slots, c->n_ext, c->n_ext > 0 ? c->n_buckets : 0, c->hub_count, c->d_hub_ids, c->d_loc,
                                            c->d_owner, c->d_free_stack, c->d_ext_free, c->d_ext_live, c->d_bk_tail_ext,
                                            c->d_bk_tail_fill, c->d_bk_new, c->d_ctl);
  // accumulator rows are as wide as what the scatter pushes: input rows in aggregate-first layers, output rows otherwise
  int Hp = taurus_round_up(c->agg_first[layer] ? c->dims[layer] : c->dims[layer + 1], 4);
  if (c->hub_count > 0)
    cudaMemsetAsync(c->d_acc + (size_t)c->pool_slots * Hp, 0, (size_t)c->hub_count * Hp * sizeof(float), st);
  c->launches += 2;
}

// ------------------------------------------------------------------------------------------------ classify (S3)
// One item per CSR edge of the chunk and one per chunk vertex (its self message).  The first item that
// touches a vertex in this chunk (atomicMax on the epoch stamp) classifies it by its state at chunk start.
// loc encoding: -1 none, [0, pool_slots) pool slot, >= pool_slots hub row, <= -2 host row (-2 - loc).
__global__ void __launch_bounds__(256) classify_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  // list appends are aggregated per block: single-address atomics are the throughput limit of this kernel
  __shared__ int s_cnt[2][2][8];   // [parity][need / touched][warp]
  __shared__ int s_base[2][2];
  const long long e0 = a.row_ptr[a.src_begin], e1 = a.row_ptr[a.src_end];
  const long long ne = e1 - e0, total = ne + (a.src_end - a.src_begin);
  const long long stride = (long long)gridDim.x * blockDim.x;
  const int warp = threadIdx.x >> 5;
  int hs = 0, ns = 0, ev = 0, gs = 0, bad = 0, par = 0;
  for (long long base = (long long)blockIdx.x * blockDim.x; base < total; base += stride, par ^= 1) {
    long long i = base + threadIdx.x;
    int v = -1;
    if (i < ne) {
      long long e = e0 + i;
      if (edge_propagated(a.mask, e)) v = a.col[e];
    } else if (i < total) {
      v = (int)(a.src_begin + (i - ne));
    }
    bool need = false, first = false;
    if (v >= a.V) { bad = 1; v = -1; }
    if (v >= 0 && a.touch[v] != a.epoch) {
      int old = atomicMax(&a.touch[v], a.epoch);
      if (old != a.epoch) {   // first touch in this chunk
        first = true;
        int l = a.loc[v];
        int s = a.state[v];
        if (l >= a.pool_slots) {          // hub store: pinned, never takes a pool slot
          gs++;
          if (s == TAURUS_NOT_STARTED) a.state[v] = TAURUS_ON_GPU;
        } else if (s == TAURUS_IN_BUFFER) {
          hs++;
          if (a.slot_touch) a.slot_touch[l] = a.epoch;
        } else if (s == TAURUS_NOT_STARTED) {
          ns++; need = true;
        } else if (s == TAURUS_EVICTED) {
          ev++; need = true;
        } else {
          bad = 1;                        // a completed vertex cannot receive a message
        }
      }
    }
    const unsigned mn = __ballot_sync(FULL, need), mt = __ballot_sync(FULL, first);
    if (lane_id() == 0) { s_cnt[par][0][warp] = __popc(mn); s_cnt[par][1][warp] = __popc(mt); }
    __syncthreads();
    if (threadIdx.x < 2) {
      int sum = 0;
      for (int w = 0; w < 8; ++w) { int c = s_cnt[par][threadIdx.x][w]; s_cnt[par][threadIdx.x][w] = sum; sum += c; }
      s_base[par][threadIdx.x] = sum ? atomicAdd(threadIdx.x == 0 ? &pc->need_count : &pc->touched_count, sum) : 0;
    }
    __syncthreads();
    if (need) {
      int idx = s_base[par][0] + s_cnt[par][0][warp] + __popc(mn & ((1u << lane_id()) - 1));
      if (idx < a.pool_slots) a.need_list[idx] = v;
    }
    if (first) {
      int idx = s_base[par][1] + s_cnt[par][1][warp] + __popc(mt & ((1u << lane_id()) - 1));
      if (idx < a.touched_capacity) a.touched_list[idx] = v; else bad = 1;
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

void launch_classify(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  classify_kernel<<<c->sm_count * 8, 256, 0, st>>>(a);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ make room (S4)
// plan: need, deficit, capacity checks, peak occupancy.
static __device__ void plan_chunk(const ChunkArgs& a, DevCtl* ctl, ChunkCtl* pc) {   // one thread
  long long need = pc->need_count;
  if (need > a.pool_slots) { ctl->error = TAURUS_ERR_POOL_TOO_SMALL; return; }
  long long deficit = need - ctl->free_top;
  if (deficit < 0) deficit = 0;
  // this chunk's victims leave before its reloads hand their host rows back
  if (ctl->host_live + deficit > a.host_rows) { ctl->error = TAURUS_ERR_HOST_STORE_FULL; return; }
  ctl->host_live += deficit - pc->ev;
  pc->deficit = (int32_t)deficit;
  pc->victim_count = 0;
  for (int l = 0; l <= TAURUS_SEL_LEVELS; ++l) { pc->sel_k[l] = 0; pc->sel_min[l] = ~0ull; pc->sel_max[l] = 0ull; pc->sel_count[l] = 0; }
  pc->sel_k[0] = deficit;
  pc->sel_final_level = deficit > 0 ? TAURUS_SEL_LEVELS + 1 : -1;
  // Slots are handed out by list index, not by per-item atomics: need-list entry i < deficit takes over the slot
  // of victim deficit - 1 - i, entry i >= deficit pops free_stack[F + deficit - 1 - i].  The counter is brought to
  // its end-of-chunk value here.
  const long long F = ctl->free_top;
  pc->alloc_base = F + deficit;
  ctl->free_top = F + deficit - need;
  long long occ = a.pool_slots - ctl->free_top;
  if (occ > ctl->peak_occupancy) ctl->peak_occupancy = occ;
}
__global__ void plan_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  for (int i = threadIdx.x; i < 2 * TAURUS_SEL_BINS; i += blockDim.x) (&pc->hist[0][0])[i] = 0;
  if (threadIdx.x == 0) plan_chunk(a, ctl, pc);
}

// Victims are the `deficit` smallest keys (score << 31 | id) among IN_BUFFER vertices the chunk does not
// touch (Sect. 3.5.3: fewest pending messages first).  Keys are unique, so an MSB-first radix select finds
// them exactly.  Level 0 scans the pool; every level lists the keys below the digit that holds rank k as
// victims and hands the keys inside that digit to the next level, so deeper levels see a small candidate list.
// The digit of a level starts at the highest bit in which the keys entering it differ (from their minimum and
// maximum): pending counts are small numbers, and a fixed digit grid would spend its first passes on bits that
// are zero in every key.
// 31-bit score of the random policy: a hash of (seed, vertex, chunk index); constants are part of its definition.
static __device__ __forceinline__ unsigned long long ev_mix(unsigned long long x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27; x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}
static __device__ __forceinline__ unsigned evict_hash(unsigned long long seed, unsigned long long vertex, unsigned long long chunk) {
  unsigned long long h = 0x452821E638D01377ull;
  h = ev_mix(h ^ (0x9E3779B97F4A7C15ull * (seed + 1ull)));
  h = ev_mix(h ^ (0x9E3779B97F4A7C15ull * (vertex + 1ull)));
  h = ev_mix(h ^ (0x9E3779B97F4A7C15ull * (chunk + 1ull)));
  return (unsigned)(h >> 33);
}

static __device__ __forceinline__ int sel_shift_of(unsigned long long lo, unsigned long long hi) {
  const unsigned long long diff = lo ^ hi;
  if (diff == 0ull) return 0;
  const int top = 63 - __clzll((long long)diff);
  return top >= TAURUS_SEL_BITS ? top - (TAURUS_SEL_BITS - 1) : 0;
}

// Block-wide minimum / maximum / count of the eligible keys a thread saw, folded into level `lvl` of the control block.
static __device__ __forceinline__ void sel_fold(ChunkCtl* pc, int lvl, unsigned long long kmin, unsigned long long kmax, int cnt) {
  for (int o = 16; o; o >>= 1) {
    const unsigned long long m = __shfl_xor_sync(FULL, kmin, o), M = __shfl_xor_sync(FULL, kmax, o);
    if (m < kmin) kmin = m;
    if (M > kmax) kmax = M;
    cnt += __shfl_xor_sync(FULL, cnt, o);
  }
  if (lane_id() == 0 && cnt) {
    atomicMin(&pc->sel_min[lvl], kmin);
    atomicMax(&pc->sel_max[lvl], kmax);
    atomicAdd(&pc->sel_count[lvl], cnt);
  }
}

// The passes over the pool work on tiles of SEL_TILE slots.  A block takes the tiles of its own number, or, where row
// transfers may run beside the kernel (dynamic_spans), the next tile of a counter: blocks on SMs that also host transfer
// warps are several times slower, and with a fixed deal the pass would wait for them.
#define SEL_ITEMS 8
#define SEL_TILE (256 * SEL_ITEMS)
static __device__ __forceinline__ long long next_tile(bool dyn, unsigned int* counter, long long it, long long* s_tile) {
  if (!dyn) return (long long)blockIdx.x + it * gridDim.x;
  __syncthreads();   // every thread has read the previous value
  if (threadIdx.x == 0) *s_tile = (long long)atomicAdd(counter, 1u);
  __syncthreads();
  return *s_tile;
}

__global__ void __launch_bounds__(256) select_keys_kernel(ChunkArgs a) {   // key of every slot; range of the eligible keys
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error || pc->sel_final_level < 0) return;
  unsigned long long kmin = ~0ull, kmax = 0ull;
  int cnt = 0;
  __shared__ long long s_tile;
  for (long long it = 0;; ++it) {
    const long long base = next_tile(a.dynamic_spans != 0, &pc->tile_next[0], it, &s_tile) * SEL_TILE;
    if (base >= a.pool_slots) break;
#pragma unroll
  for (int j = 0; j < SEL_ITEMS; ++j) {
    const long long s = base + j * 256 + threadIdx.x;
    if (s >= a.pool_slots) break;
    const int v = a.owner[s];
    unsigned long long key = ~0ull;
    if (v >= 0) {
      const int t = a.slot_touch[s];   // = touch[v]
      if (t != a.epoch) {
        unsigned score;
        if (a.evict_policy == TAURUS_EVICT_FIFO) score = (unsigned)a.slot_epoch[s];
        else if (a.evict_policy == TAURUS_EVICT_LRU) score = (unsigned)t;
        else if (a.evict_policy == TAURUS_EVICT_RANDOM) score = evict_hash(a.seed, (unsigned long long)v, (unsigned long long)(a.epoch - 1));
        else score = (unsigned)a.slot_pend[s];   // = pend[v]: v was not touched since the copy was taken
        key = ((unsigned long long)score << 31) | (unsigned long long)v;
        if (key < kmin) kmin = key;
        if (key > kmax) kmax = key;
        cnt++;
      }
    }
    a.keys[s] = key;
  }
  }
  sel_fold(pc, 0, kmin, kmax, cnt);
}

// Histogram of the level's digit over the keys entering the level.  Threads of a warp that hit the same bin add
// once (most keys of a level often share a bin).
__global__ void __launch_bounds__(256) select_hist_kernel(ChunkArgs a, int level) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error || pc->sel_final_level < level) return;
  const long long k = pc->sel_k[level];
  const long long n = level == 0 ? a.pool_slots : (long long)pc->sel_count[level];
  if (pc->sel_count[level] < k) {   // fewer eligible victims than needed
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(&ctl->error, 0, level == 0 ? TAURUS_ERR_POOL_TOO_SMALL : TAURUS_ERR_INTERNAL);
    return;
  }
  __shared__ unsigned int sh[TAURUS_SEL_BINS];
  for (int i = threadIdx.x; i < TAURUS_SEL_BINS; i += blockDim.x) sh[i] = 0;
  __syncthreads();
  const int shift = sel_shift_of(pc->sel_min[level], pc->sel_max[level]);
  const int32_t* __restrict__ cand = level == 0 ? nullptr : a.cand[level & 1];
  __shared__ long long s_tile;
  const bool dyn = level == 0 && a.dynamic_spans != 0;   // deeper levels see short candidate lists
  for (long long it = 0;; ++it) {
    const long long base = next_tile(dyn, &pc->tile_next[1], it, &s_tile) * SEL_TILE;
    if (base >= n) break;
#pragma unroll
    for (int j = 0; j < SEL_ITEMS; ++j) {
      const long long i = base + j * 256 + threadIdx.x;
      unsigned long long key = ~0ull;
      if (i < n) key = a.keys[level == 0 ? i : (long long)cand[i]];
      const bool on = key != ~0ull;
      const unsigned digit = on ? (unsigned)(key >> shift) & (TAURUS_SEL_BINS - 1) : 0xffffffffu;
      const unsigned peers = __match_any_sync(FULL, digit);
      if (on && lane_id() == __ffs(peers) - 1) atomicAdd(&sh[digit], (unsigned)__popc(peers));
    }
  }
  __syncthreads();
  unsigned int* hist = pc->hist[level & 1];
  for (int b = threadIdx.x; b < TAURUS_SEL_BINS; b += blockDim.x)
    if (sh[b]) atomicAdd(&hist[b], sh[b]);
}

// Every block finds the digit that holds rank k from the level's histogram; keys below it are victims, keys inside
// it go to the next level (or are victims too when the digit holds exactly the ranks still missing).
__global__ void __launch_bounds__(256) select_split_kernel(ChunkArgs a, int level) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error || pc->sel_final_level < level) return;
  __shared__ unsigned int sh[TAURUS_SEL_BINS];
  __shared__ unsigned int part[256];
  __shared__ int s_digit;
  __shared__ long long s_rest;
  const unsigned int* hist = pc->hist[level & 1];
  const long long k = pc->sel_k[level];
  // bins per thread: TAURUS_SEL_BINS / 256 consecutive ones
  constexpr int PER = TAURUS_SEL_BINS / 256;
  unsigned int mine[PER], sum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) { mine[j] = hist[threadIdx.x * PER + j]; sh[threadIdx.x * PER + j] = mine[j]; sum += mine[j]; }
  part[threadIdx.x] = sum;
  if (threadIdx.x == 0) s_digit = -1;
  __syncthreads();
  if (threadIdx.x == 0) {
    long long cum = 0;
    int t = 0;
    for (; t < 256; ++t) { if (cum + part[t] >= k) break; cum += part[t]; }
    if (t < 256) {
      int b = t * PER;
      for (; b < t * PER + PER; ++b) { if (cum + sh[b] >= k) break; cum += sh[b]; }
      s_digit = b;
      s_rest = k - cum;
    }
  }
  __syncthreads();
  const int digit_k = s_digit;
  if (digit_k < 0) {   // the histogram holds fewer keys than k: cannot happen after the count check
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
    return;
  }
  const long long rest = s_rest;
  const bool final = rest == (long long)sh[digit_k];   // the whole digit is victims: nothing left to resolve
  const int shift = sel_shift_of(pc->sel_min[level], pc->sel_max[level]);
  const long long n = level == 0 ? a.pool_slots : (long long)pc->sel_count[level];
  const int32_t* __restrict__ cand = level == 0 ? nullptr : a.cand[level & 1];
  int32_t* __restrict__ next = a.cand[(level + 1) & 1];
  if (blockIdx.x == 0) {
    unsigned int* other = pc->hist[(level + 1) & 1];   // the next level's histogram (read last by the level above this one)
    for (int b = threadIdx.x; b < TAURUS_SEL_BINS; b += blockDim.x) other[b] = 0;
    if (threadIdx.x == 0) {
      if (final) pc->sel_final_level = level;
      else if (level == TAURUS_SEL_LEVELS - 1 || shift == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);   // unique keys always end in a final level
      else pc->sel_k[level + 1] = rest;
    }
  }
  unsigned long long kmin = ~0ull, kmax = 0ull;
  int cnt = 0;
  const unsigned lt = (1u << lane_id()) - 1;
  __shared__ long long s_tile;
  const bool dyn = level == 0 && a.dynamic_spans != 0;
  for (long long it = 0;; ++it) {
    const long long base = next_tile(dyn, &pc->tile_next[2], it, &s_tile) * SEL_TILE;
    if (base >= n) break;
#pragma unroll 2
  for (int j = 0; j < SEL_ITEMS; ++j) {
    const long long i = base + j * 256 + threadIdx.x;
    unsigned long long key = ~0ull;
    int slot = -1;
    if (i < n) { slot = level == 0 ? (int)i : cand[i]; key = a.keys[slot]; }
    const bool on = key != ~0ull;
    const int digit = on ? (int)((unsigned)(key >> shift) & (TAURUS_SEL_BINS - 1)) : TAURUS_SEL_BINS;
    const bool victim = digit < digit_k || (final && digit == digit_k);
    const bool keep = !final && digit == digit_k;
    const unsigned mv = __ballot_sync(FULL, victim), mk = __ballot_sync(FULL, keep);
    if (mv) {
      int idx = 0;
      const int leader = __ffs(mv) - 1;
      if (lane_id() == leader) idx = atomicAdd(&pc->victim_count, __popc(mv));
      idx = __shfl_sync(FULL, idx, leader) + __popc(mv & lt);
      if (victim && idx < a.victim_capacity) a.victims[idx].x = slot;
    }
    if (mk) {
      int idx = 0;
      const int leader = __ffs(mk) - 1;
      if (lane_id() == leader) idx = atomicAdd(&pc->sel_count[level + 1], __popc(mk));
      idx = __shfl_sync(FULL, idx, leader) + __popc(mk & lt);
      if (keep) {
        next[idx] = slot;   // at most pool_slots keys enter any level
        if (key < kmin) kmin = key;
        if (key > kmax) kmax = key;
        cnt++;
      }
    }
  }
  }
  // sel_count of the next level is already counted by the appends: fold only the key range
  for (int o = 16; o; o >>= 1) {
    const unsigned long long m = __shfl_xor_sync(FULL, kmin, o), M = __shfl_xor_sync(FULL, kmax, o);
    if (m < kmin) kmin = m;
    if (M > kmax) kmax = M;
    cnt += __shfl_xor_sync(FULL, cnt, o);
  }
  if (lane_id() == 0 && cnt) {
    atomicMin(&pc->sel_min[level + 1], kmin);
    atomicMax(&pc->sel_max[level + 1], kmax);
  }
}

// ---- host store: where a victim's row goes
// Largest in-list position of v whose source is below `src_end` ... the first message still to come decides the
// bucket: the source of the first propagated in-edge of v at or behind src_end, or v itself while its own chunk (which
// delivers its self message) has not been pushed.
static __device__ __forceinline__ long long next_sender(const ChunkArgs& a, int v) {
  long long lo = a.csc_ptr[v];
  const long long end = a.csc_ptr[v + 1];
  long long hi = end;
  while (lo < hi) {   // first in-list entry with source >= src_end (the in-list is sorted by source)
    const long long mid = (lo + hi) >> 1;
    if ((long long)a.csc_src[mid] < a.src_end) lo = mid + 1; else hi = mid;
  }
  if (a.mask && a.csc_eid) {
    while (lo < end) {
      const uint32_t e = a.csc_eid[lo];
      if ((a.mask[e >> 5] >> (e & 31)) & 1u) break;
      ++lo;
    }
  }
  long long ns = lo < end ? (long long)a.csc_src[lo] : a.V;
  if (v >= a.src_end && v < ns) ns = v;
  return ns;
}

__global__ void __launch_bounds__(256) victim_bucket_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error || pc->deficit == 0) return;
  const int n = pc->deficit;
  if (pc->victim_count != n) {   // the select must have produced exactly `deficit` victims
    if (threadIdx.x == 0 && blockIdx.x == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
    return;
  }
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const int slot = a.victims[i].x;
    const int v = a.owner[slot];
    long long ns = next_sender(a, v);
    if (ns >= a.V) { atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL); ns = a.V - 1; }   // a victim has a message to come
    const int b = (int)(ns / a.chunk_sources);
    a.vic_place[i] = make_int2(b, atomicAdd(&a.bk_new[b], 1));
  }
}

// One block.  First the tails of the buckets whose grid cell ends inside this push are closed (no victim can be
// filed there any more: its next sender would lie behind the push); then every bucket that received victims gets
// the extents it lacks from the free stack.
__global__ void __launch_bounds__(1024) extent_plan_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int E = 1 << a.ext_shift;
  __shared__ int warp_sum[32];
  __shared__ long long s_running;
  __shared__ int s_fail;
  if (threadIdx.x == 0) { s_running = 0; s_fail = 0; }
  // phase 0: the extents emptied by the transfers of the last chunk of this parity go back on the free stack.  Those
  // transfers are complete (the chunk in between waited for them before it moved its own rows); the transfers of the
  // chunk in between may still be running and append to the other list.
  {
    const int par = a.epoch & 1;
    const int n_ret = ctl->ext_ret_count[par];
    const long long top = ctl->ext_free_top;
    for (int i = threadIdx.x; i < n_ret; i += blockDim.x) a.ext_free[top + i] = a.ext_ret[par][i];
    __syncthreads();
    if (threadIdx.x == 0) { ctl->ext_free_top = top + n_ret; ctl->ext_ret_count[par] = 0; }
    __syncthreads();
  }
  // phase 1: close tails
  {
    const long long first = a.src_begin / a.chunk_sources;
    const long long b = first + threadIdx.x;
    if (threadIdx.x < 2 && b < a.n_buckets) {
      long long cell_end = (b + 1) * a.chunk_sources;
      if (cell_end > a.V) cell_end = a.V;
      const int t = a.bk_tail_ext[b];
      if (cell_end <= a.src_end && t >= 0) {
        const int unused = E - a.bk_tail_fill[b];
        if (unused > 0 && atomicSub(&a.ext_live[t], unused) == unused) {   // every row it held is already back in the pool
          const long long top = (long long)atomicAdd((unsigned long long*)&ctl->ext_free_top, 1ull);
          a.ext_free[top] = t;
        }
        a.bk_tail_ext[b] = -1;
        a.bk_tail_fill[b] = 0;
      }
    }
  }
  __syncthreads();
  if (pc->deficit == 0) return;
  // phase 2: extents needed per bucket, exclusive prefix over the buckets
  for (long long base = 0; base < a.n_buckets; base += blockDim.x) {
    const long long b = base + threadIdx.x;
    int want = 0;
    if (b < a.n_buckets) {
      const int nw = a.bk_new[b];
      if (nw > 0) {
        const int t = a.bk_tail_ext[b], f = a.bk_tail_fill[b];
        a.bk_base[b] = make_int2(t, f);
        const int room = t >= 0 ? E - f : 0;
        const int extra = nw > room ? nw - room : 0;
        want = (extra + E - 1) >> a.ext_shift;
      }
    }
    int x = want;
    for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(FULL, x, o); if (lane_id() >= o) x += y; }
    if (lane_id() == 31) warp_sum[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x < 32) {
      int w = warp_sum[threadIdx.x];
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(FULL, w, o); if (lane_id() >= o) w += y; }
      warp_sum[threadIdx.x] = w;   // inclusive over warps
    }
    __syncthreads();
    const long long before = s_running + ((threadIdx.x >> 5) ? warp_sum[(threadIdx.x >> 5) - 1] : 0) + (x - want);
    if (b < a.n_buckets && a.bk_new[b] > 0) a.bk_off[b] = (int32_t)before;
    __syncthreads();
    if (threadIdx.x == 0) s_running += warp_sum[31];
    __syncthreads();
  }
  const long long total = s_running;
  if (total > ctl->ext_free_top) {
    if (threadIdx.x == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_HOST_STORE_FULL);
    return;
  }
  const long long stack_base = ctl->ext_free_top - total;
  __syncthreads();
  if (threadIdx.x == 0) ctl->ext_free_top = stack_base;
  // phase 3: hand the extents out and move the tails
  for (long long b = threadIdx.x; b < a.n_buckets; b += blockDim.x) {
    const int nw = a.bk_new[b];
    if (nw <= 0) continue;
    const int2 base = a.bk_base[b];
    const int room = base.x >= 0 ? E - base.y : 0;
    const int extra = nw > room ? nw - room : 0;
    const int want = (extra + E - 1) >> a.ext_shift;
    const int off = a.bk_off[b];
    for (int j = 0; j < want; ++j) {
      const int e = a.ext_free[stack_base + off + j];
      a.new_ext[off + j] = e;
      a.ext_live[e] = E;
    }
    if (want > 0) { a.bk_tail_ext[b] = a.new_ext[off + want - 1]; a.bk_tail_fill[b] = extra - ((want - 1) << a.ext_shift); }
    else a.bk_tail_fill[b] = base.y + nw;
  }
}

__global__ void __launch_bounds__(256) victim_place_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error || pc->deficit == 0) return;
  const int n = pc->deficit;
  const int E = 1 << a.ext_shift;
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const int2 pl = a.vic_place[i];
    const int2 base = a.bk_base[pl.x];
    const int room = base.x >= 0 ? E - base.y : 0;
    int ext, idx;
    if (pl.y < room) { ext = base.x; idx = base.y + pl.y; }
    else { const int q = pl.y - room; ext = a.new_ext[a.bk_off[pl.x] + (q >> a.ext_shift)]; idx = q & (E - 1); }
    a.victims[i].y = (ext << a.ext_shift) + idx;
    a.bk_new[pl.x] = 0;   // same value from every victim of the bucket; nothing reads the count after the plan
  }
}

// One warp per vertex that needs a slot.  Need-list entry i < deficit takes over the slot of victim
// deficit - 1 - i: the warp reads the victim's accumulator row and, if its own vertex was EVICTED, the vertex's
// host row, then writes the victim's row to its pinned host row (IN_BUFFER -> EVICTED) and the reloaded row (or
// zeros for a NOT_STARTED vertex) into the slot, so that evictions (device -> host) and reloads (host -> device)
// use both directions of the link at the same time.  Entries i >= deficit pop the free stack.  Either way
// the vertex is IN_BUFFER afterwards.
__global__ void alloc_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int n = pc->need_count;
  const int deficit = pc->deficit;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int vec = a.Hp >> 2;
  if (a.direct) {
    // Every vertex owns the slot of its own number and nothing is ever evicted: each entry is a NOT_STARTED vertex
    // whose row is cleared.  Batches of up to 32 entries per warp, one lane per entry for the list and state
    // accesses, then the warp clears the rows one after the other.
    // No other thread of this kernel reads what the plan writes (there is no deficit and no stack to pop), so one
    // thread does the chunk's bookkeeping here and the separate plan launch is left out.
    if (blockIdx.x == 0 && threadIdx.x == 0) plan_chunk(a, ctl, pc);
    int per = (int)((n + warps - 1) / warps);
    per = per < 1 ? 1 : per > 32 ? 32 : per;
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
    for (long long i0 = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * per; i0 < n; i0 += warps * per) {
      const long long mine = i0 + lane_id();
      int v = -1;
      if (lane_id() < per && mine < n) {
        v = a.need_list[mine];
        if (a.state[v] != TAURUS_NOT_STARTED) { atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL); v = -1; }
        else a.state[v] = TAURUS_IN_BUFFER;
      }
      const int rows = n - i0 < per ? (int)(n - i0) : per;
      for (int j = 0; j < rows; ++j) {
        const int vj = __shfl_sync(FULL, v, j);
        if (vj < 0) continue;
        float4* __restrict__ row = reinterpret_cast<float4*>(a.acc + (size_t)vj * a.Hp);
        for (int k = lane_id(); k < vec; k += 32) row[k] = zero;
      }
    }
    return;
  }
  // Bounded pool.  Need-list entry i < deficit takes over the slot of victim deficit - 1 - i: the victim's row is
  // copied to the staging buffer (it leaves for its pinned host row in transfer_kernel) and the victim becomes
  // EVICTED; entry i >= deficit pops the free stack.  Either way the slot is cleared and handed to the vertex, which
  // is IN_BUFFER afterwards; the partial sum of a vertex that was EVICTED is ADDED into the slot by transfer_kernel
  // (sums commute: the scatter may already be adding this chunk's messages to the same row).
  // Batches of up to 32 entries per warp: each lane follows the chain of dependent reads of one entry (vertex, victim,
  // slot, state) and writes its metadata, then the warp walks the batch row by row.
  int reloaded = 0;
  const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
  int per = (int)((n + warps - 1) / warps);
  per = per < 1 ? 1 : per > 32 ? 32 : per;
  for (long long i0 = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * per; i0 < n; i0 += warps * per) {
    const long long i = i0 + lane_id();
    int slot = -1, out_hrow = -1;
    if (lane_id() < per && i < n) {
      const int v = a.need_list[i];
      int victim = -1;
      if (i < deficit) {
        const int2 vic = a.victims[deficit - 1 - i];
        slot = vic.x; out_hrow = vic.y; victim = a.owner[slot];
      } else { const long long f = pc->alloc_base - 1 - i; slot = f >= 0 ? a.free_stack[f] : -1; }
      if (slot < 0) {
        atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
      } else {
        const int in_hrow = a.state[v] == TAURUS_EVICTED ? -2 - a.loc[v] : -1;
        if (a.xfer_list) a.xfer_list[i] = make_int4(slot, in_hrow, out_hrow, 0);
        if (out_hrow >= 0) {
          a.loc[victim] = -2 - out_hrow;
          a.state[victim] = TAURUS_EVICTED;
        }
        if (in_hrow >= 0) {
          a.reload_count[v] += 1;
          reloaded++;
        }
        a.loc[v] = slot; a.owner[slot] = v; a.slot_epoch[slot] = a.epoch;
        if (a.slot_touch) a.slot_touch[slot] = a.epoch;   // slot_pend follows in compact_done: v is on the touched list
        a.state[v] = TAURUS_IN_BUFFER;
      }
    }
    const int rows = n - i0 < per ? (int)(n - i0) : per;
    for (int j = 0; j < rows; ++j) {
      const int sj = __shfl_sync(FULL, slot, j);
      const int oj = __shfl_sync(FULL, out_hrow, j);
      if (sj < 0) continue;
      float4* __restrict__ row = reinterpret_cast<float4*>(a.acc + (size_t)sj * a.Hp);
      if (oj >= 0) {
        float4* __restrict__ keep = reinterpret_cast<float4*>(a.stage_out + (size_t)(i0 + j) * a.Hp);
        for (int k = lane_id(); k < vec; k += 32) { keep[k] = row[k]; row[k] = zero; }
      } else {
        for (int k = lane_id(); k < vec; k += 32) row[k] = zero;
      }
    }
  }
  for (int o = 16; o; o >>= 1) reloaded += __shfl_xor_sync(FULL, reloaded, o);
  if (lane_id() == 0 && reloaded) atomicAdd(&pc->reloaded, reloaded);
}

// The rows of one chunk across the host link: the staged row of the victim whose slot a need-list entry took over
// goes to its pinned host row (device -> host), and the host row of a vertex that was EVICTED is added into its new
// slot (host -> device), so both directions of the link are busy at once.  A warp takes R entries per round, R chosen so
// that it has four float4 per lane and direction in flight whatever the row width (R = 4 for rows of up to 32 float4,
// 2 up to 64, else 1): the link is fed by bytes in flight, and narrow rows otherwise leave it short.  An extent whose
// last row has come back is listed for the free stack (taken back two chunks later by extent_plan_kernel).
template <int R>
__global__ void __launch_bounds__(256) transfer_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  constexpr int QPR = 4 / R;   // float4 steps of one row per round
  const int n = pc->need_count;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int vec = a.Hp >> 2;
  const int par = a.epoch & 1;
  for (long long i0 = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * R; i0 < n; i0 += warps * R) {
    int4 x[R];
#pragma unroll
    for (int r = 0; r < R; ++r) x[r] = i0 + r < n ? a.xfer_list[i0 + r] : make_int4(0, -1, -1, 0);   // same address for the whole warp
    for (int k0 = 0; k0 < vec; k0 += 32 * QPR) {
      float4 keep[4], in[4];
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        const int r = s4 / QPR, k = k0 + (s4 % QPR) * 32 + lane_id();
        if (k < vec) {
          if (x[r].z >= 0) keep[s4] = reinterpret_cast<const float4*>(a.stage_out + (size_t)(i0 + r) * a.Hp)[k];
          if (x[r].y >= 0) in[s4] = reinterpret_cast<const float4*>(a.host_store + (size_t)x[r].y * a.Hp)[k];
        }
      }
#pragma unroll
      for (int s4 = 0; s4 < 4; ++s4) {
        const int r = s4 / QPR, k = k0 + (s4 % QPR) * 32 + lane_id();
        if (k < vec) {
          if (x[r].z >= 0) reinterpret_cast<float4*>(a.host_store + (size_t)x[r].z * a.Hp)[k] = keep[s4];
          if (x[r].y >= 0) {
            float* row = a.acc + (size_t)x[r].x * a.Hp + 4 * k;
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(row), "f"(in[s4].x), "f"(in[s4].y), "f"(in[s4].z), "f"(in[s4].w) : "memory");
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
      if (lane_id() == r && x[r].y >= 0) {
        const int e = x[r].y >> a.ext_shift;
        if (atomicSub(&a.ext_live[e], 1) == 1) a.ext_ret[par][atomicAdd(&ctl->ext_ret_count[par], 1)] = e;   // last row of the extent
      }
  }
}

void launch_make_room(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st, cudaEvent_t before_moves) {
  const int blocks = c->sm_count * 8;
  if (!a.direct) {   // direct-mapped pools plan inside alloc_kernel
    plan_kernel<<<1, 256, 0, st>>>(a);
    c->launches += 1;
  }
  if (c->pool_slots < c->V - c->hub_count) {   // eviction is impossible when every non-hub vertex has a slot
    select_keys_kernel<<<blocks, 256, 0, st>>>(a);
    for (int l = 0; l < TAURUS_SEL_LEVELS; ++l) {
      // deeper levels work on what is left of one digit of the level above: a handful of blocks is enough
      const int b = l == 0 ? blocks : l == 1 ? c->sm_count * 2 : c->sm_count;
      select_hist_kernel<<<b, 256, 0, st>>>(a, l);
      select_split_kernel<<<b, 256, 0, st>>>(a, l);
    }
    victim_bucket_kernel<<<c->sm_count * 8, 256, 0, st>>>(a);
    extent_plan_kernel<<<1, 1024, 0, st>>>(a);
    victim_place_kernel<<<c->sm_count * 2, 256, 0, st>>>(a);
    c->launches += 2 * TAURUS_SEL_LEVELS + 4;
  }
  if (before_moves) cudaEventRecord(before_moves, st);
}

// Slots handed out, victims' rows staged, new rows cleared (S4, device side).
void launch_alloc(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  alloc_kernel<<<c->sm_count * 8, 256, 0, st>>>(a);
  c->launches += 1;
}
// Rows across the host link (bounded pools only).
void launch_transfer(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  // One block per SM.  The warps spend their time waiting for the host link; measured on the "large" workload, fewer
  // blocks leave the link short of requests (64 blocks: 36 + 33 GB/s, 148: 38 + 34, 1 184: 39 + 35), more blocks only
  // take thread slots from the scatter and select kernels that run beside the transfers on the compute stream.
  const int vec = a.Hp >> 2;
  if (vec <= 32) transfer_kernel<4><<<c->sm_count, 256, 0, st>>>(a);
  else if (vec <= 64) transfer_kernel<2><<<c->sm_count, 256, 0, st>>>(a);
  else transfer_kernel<1><<<c->sm_count, 256, 0, st>>>(a);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ finalise (S6 tail, S7)
// S6: compact the touched vertices whose pending count reached zero (warp ballot + prefix) into done_list.
// The scatter only decrements the counts with fire-and-forget reductions; completion is read here, after
// the kernel boundary, when every reduction of the chunk has landed.
// Each lane takes CD_ITEMS entries per round so that their scattered reads (pending count, slot) are in flight
// together and one pair of counter round trips serves CD_ITEMS * 32 entries.
#define CD_ITEMS 4
__global__ void compact_done_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int n = pc->touched_count;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long warp0 = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const unsigned lt = (1u << lane_id()) - 1;
  int bad = 0;
  for (long long base = warp0 * (32 * CD_ITEMS); base < n; base += warps * (32 * CD_ITEMS)) {
    int v[CD_ITEMS], l[CD_ITEMS];
    bool done[CD_ITEMS], rel[CD_ITEMS];
#pragma unroll
    for (int q = 0; q < CD_ITEMS; ++q) {
      const long long i = base + q * 32 + lane_id();
      v[q] = i < n ? a.touched_list[i] : -1;
    }
    int pq[CD_ITEMS];
#pragma unroll
    for (int q = 0; q < CD_ITEMS; ++q) {
      pq[q] = v[q] >= 0 ? a.pend[v[q]] : 1;
      done[q] = pq[q] == 0;
      if (pq[q] < 0) bad = 1;
    }
    // the slots of the completed non-hub vertices go back on the free stack (finalise still reads the rows:
    // nothing allocates before the next chunk); the slots of the others take a copy of the new pending count
    const bool mirror = a.slot_pend != nullptr;
#pragma unroll
    for (int q = 0; q < CD_ITEMS; ++q) l[q] = (done[q] || (mirror && v[q] >= 0)) ? a.loc[v[q]] : 0x7fffffff;
    if (mirror) {
#pragma unroll
      for (int q = 0; q < CD_ITEMS; ++q)
        if (!done[q] && v[q] >= 0 && l[q] >= 0 && l[q] < a.pool_slots) a.slot_pend[l[q]] = pq[q];
    }
    unsigned md[CD_ITEMS], mr[CD_ITEMS];
    int cd = 0, cr = 0;
#pragma unroll
    for (int q = 0; q < CD_ITEMS; ++q) {
      rel[q] = done[q] && l[q] < a.pool_slots;
      md[q] = __ballot_sync(FULL, done[q]);
      mr[q] = __ballot_sync(FULL, rel[q]);
      cd += __popc(md[q]);
      cr += __popc(mr[q]);
    }
    int idx = 0;
    long long f = 0;
    if (lane_id() == 0) {
      if (cd) idx = atomicAdd(&pc->done_count, cd);
      if (cr) f = (long long)atomicAdd((unsigned long long*)&ctl->free_top, (unsigned long long)cr);
    }
    idx = __shfl_sync(FULL, idx, 0);
    f = __shfl_sync(FULL, f, 0);
#pragma unroll
    for (int q = 0; q < CD_ITEMS; ++q) {
      if (done[q]) {
        const int at = idx + __popc(md[q] & lt);
        if (at < a.grad_cap) a.done_list[at] = v[q]; else bad = 1;
      }
      if (rel[q] && !a.direct) {
        const long long at = f + __popc(mr[q] & lt);
        a.free_stack[at] = l[q];
        a.owner[l[q]] = -1;
      }
      idx += __popc(md[q]);
      f += __popc(mr[q]);
    }
  }
  if (__any_sync(FULL, bad) && lane_id() == 0) atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
}

// Completed vertices (listed by compact_done_kernel) in batches of 32 per warp: each lane first fetches the
// vertex, its slot and its normalisation of one row of the batch (one dependent chain for 32 rows), then the
// warp walks the batch row by row: out = act(c_in(v) * acc) into the graduation buffer, or straight into the
// caller's vertex-ordered matrix (Sect. 3.6); the slot is released by compact_done_kernel.
__global__ void finalise_kernel(ChunkArgs a) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (ctl->error) return;
  const int n = pc->done_count;
  const long long base = a.dense_half >= 0 ? a.grad_off : ctl->grad_count;
  const long long limit = a.dense_half >= 0 ? a.grad_off + a.grad_cap : a.drain_rows;
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int vec = a.Hp >> 2;
  const bool vec_ok = a.dense_direct && (a.dense_ld & 3) == 0 && (reinterpret_cast<uintptr_t>(a.dense_direct) & 15) == 0;
  // rows per warp batch: as many as keep every warp busy, at most one per lane
  int per = (int)((n + warps - 1) / warps);
  per = per < 1 ? 1 : per > 32 ? 32 : per;
  for (long long i0 = (((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * per; i0 < n; i0 += warps * per) {
    const long long mine = i0 + lane_id();
    int v = -1, l = 0;
    float scale = 1.0f;
    if (lane_id() < per && mine < n) {
      if (!a.dense_direct && base + mine >= limit) {
        atomicCAS(&ctl->error, 0, TAURUS_ERR_INTERNAL);
      } else {
        v = a.done_list[mine];
        l = a.loc[v];
        if (a.mode == TAURUS_SAGE_MEAN) {
          int m = messages_of(a.din[v], a.fanout);
          scale = 1.0f / (float)(m > 1 ? m : 1);
        } else if (a.mode == TAURUS_GCN_SYM) {
          scale = (float)(1.0 / sqrt((double)a.din[v] + 1.0));
        } else if (a.mode == TAURUS_GAT) {
          scale = (float)(1.0 / a.att_z[v]);   // softmax normaliser
        }                              // GIN: plain sum
        a.state[v] = TAURUS_COMPLETED;
        if (!a.dense_direct) a.grad_ids[base + mine] = v;
      }
    }
    const int rows = n - i0 < per ? (int)(n - i0) : per;
    for (int j = 0; j < rows; ++j) {
      const int vj = __shfl_sync(FULL, v, j);
      if (vj < 0) continue;
      const int lj = __shfl_sync(FULL, l, j);
      const float sj = __shfl_sync(FULL, scale, j);
      const float4* __restrict__ src = reinterpret_cast<const float4*>(a.acc + (size_t)lj * a.Hp);
      float* __restrict__ drow = a.dense_direct ? a.dense_direct + (size_t)vj * a.dense_ld : a.grad_rows + (size_t)(base + i0 + j) * a.Hp;
      for (int k0 = 0; k0 < vec; k0 += 128) {   // up to four float4 per lane in flight before the first store
        float4 x[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int k = k0 + q * 32 + lane_id();
          if (k < vec) x[q] = src[k];
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int k = k0 + q * 32 + lane_id();
          if (k >= vec) continue;
          float4 y = x[q];
          float sk = sj;
          if (a.mode == TAURUS_GAT && a.heads > 1) sk = (float)(1.0 / a.att_z[(size_t)vj * a.heads + k / a.head_vec]);   // normaliser of the column's head
          y.x *= sk; y.y *= sk; y.z *= sk; y.w *= sk;
          if (a.act) { y.x = fmaxf(y.x, 0.f); y.y = fmaxf(y.y, 0.f); y.z = fmaxf(y.z, 0.f); y.w = fmaxf(y.w, 0.f); }
          const int c0 = k << 2;
          if (!a.dense_direct || (vec_ok && c0 + 3 < a.d_out)) {
            reinterpret_cast<float4*>(drow)[k] = y;
          } else {   // ragged last columns, or a matrix whose rows are not 16-byte aligned
            if (c0 < a.d_out) drow[c0] = y.x;
            if (c0 + 1 < a.d_out) drow[c0 + 1] = y.y;
            if (c0 + 2 < a.d_out) drow[c0 + 2] = y.z;
            if (c0 + 3 < a.d_out) drow[c0 + 3] = y.w;
          }
        }
      }
    }
  }
}

// After the chunk's completions are listed: fold the chunk's counters into the layer totals, write the chunk record.
static __device__ void commit_counts(const ChunkArgs& a, DevCtl* ctl, ChunkCtl* pc) {   // one thread
  long long c = ctl->chunks;
  if (c < a.log_capacity) {
    long long* r = a.chunk_log + c * TAURUS_CK_COLUMNS;
    r[TAURUS_CK_HS] = pc->hs; r[TAURUS_CK_NS] = pc->ns; r[TAURUS_CK_EV] = pc->ev; r[TAURUS_CK_GS] = pc->gs;
    r[TAURUS_CK_NEED] = pc->need_count; r[TAURUS_CK_EVICTED] = pc->deficit; r[TAURUS_CK_RELOADED] = pc->reloaded;
    r[TAURUS_CK_COMPLETED] = pc->done_count; r[TAURUS_CK_OCCUPANCY] = a.pool_slots - ctl->free_top;
  }
  ctl->sum_hs += pc->hs; ctl->sum_ns += pc->ns; ctl->sum_ev += pc->ev; ctl->sum_gs += pc->gs;
  ctl->evictions += pc->deficit;
  ctl->reloads += pc->reloaded;
  ctl->completed += pc->done_count;
  ctl->chunks = c + 1;
}
__global__ void commit_counts_kernel(ChunkArgs a) {
  if (threadIdx.x != 0 || a.ctl->error) return;
  commit_counts(a, a.ctl, a.pc);
}
// One thread, after the chunk's rows are finalised: the graduation buffer's row count, and the chunk's counters are
// cleared for the chunk after next.  with_counts: the chunk record has not been written yet (no transfers in flight:
// finalise followed the completion list directly).
__global__ void commit_kernel(ChunkArgs a, int with_counts) {
  DevCtl* ctl = a.ctl;
  ChunkCtl* pc = a.pc;
  if (threadIdx.x != 0 || ctl->error) return;
  if (with_counts) commit_counts(a, ctl, pc);
  if (a.dense_direct) { /* rows already sit in the caller's matrix */ }
  else if (a.dense_half >= 0) ctl->out_count[a.dense_half] = pc->done_count;
  else ctl->grad_count += pc->done_count;
  pc->hs = pc->ns = pc->ev = pc->gs = 0;
  pc->need_count = 0; pc->done_count = 0; pc->touched_count = 0; pc->deficit = 0; pc->victim_count = 0; pc->reloaded = 0;
  pc->span_next = 0; pc->self_next = 0;
  pc->tile_next[0] = pc->tile_next[1] = pc->tile_next[2] = pc->tile_next[3] = 0;
}

// S6: completions listed, slots released, chunk record written.
void launch_compact_done(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st, bool write_record) {
  compact_done_kernel<<<c->sm_count * 8, 256, 0, st>>>(a);
  if (write_record) commit_counts_kernel<<<1, 32, 0, st>>>(a);
  c->launches += write_record ? 2 : 1;
}
void launch_commit(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  commit_kernel<<<1, 32, 0, st>>>(a, c->pipelined ? 0 : 1);
  c->launches += 1;
}

// S7 of a project-first layer (after launch_compact_done): rows finalised, graduation bookkeeping.
void launch_finalise(taurus_ctx* c, const ChunkArgs& a, cudaStream_t st) {
  finalise_kernel<<<c->sm_count * 8, 256, 0, st>>>(a);
  commit_kernel<<<1, 32, 0, st>>>(a, c->pipelined ? 0 : 1);
  c->launches += 2;
}

// ------------------------------------------------------------------------------------------------ drain helpers
// Row i of the graduation buffer goes to dense[id * ld ...]: the vertex-ordered matrix the next layer streams.
__global__ void place_rows_kernel(const long long* ids, const float* rows, int Hp, int d_out, float* dense, long long ld,
                                  long long count) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const bool vec_ok = (ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(dense) & 15) == 0);
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < count; i += warps) {
    long long id = ids[i];
    const float* src = rows + (size_t)i * Hp;
    float* dst = dense + (size_t)id * ld;
    if (vec_ok) {
      int full = d_out >> 2;
      for (int k = lane_id(); k < full; k += 32)
        reinterpret_cast<float4*>(dst)[k] = reinterpret_cast<const float4*>(src)[k];
      for (int k = (full << 2) + lane_id(); k < d_out; k += 32) dst[k] = src[k];
    } else {
      for (int k = lane_id(); k < d_out; k += 32) dst[k] = src[k];
    }
  }
}

void launch_place_rows(taurus_ctx* c, float* dense, long long ld, int d_out, int Hp, long long count, cudaStream_t st) {
  if (count <= 0) return;
  long long blocks = (count + 7) / 8;
  if (blocks > c->sm_count * 16) blocks = c->sm_count * 16;
  place_rows_kernel<<<(int)blocks, 256, 0, st>>>(c->d_grad_ids, c->d_grad_rows, Hp, d_out, dense, ld, count);
  c->launches += 1;
}

__global__ void reload_histogram_kernel(long long V, const int32_t* reload, long long* hist18) {
  __shared__ unsigned int sh[17];
  __shared__ int shmax;
  if (threadIdx.x < 17) sh[threadIdx.x] = 0;
  if (threadIdx.x == 0) shmax = 0;
  __syncthreads();
  long long stride = (long long)gridDim.x * blockDim.x;
  int mx = 0;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) {
    int r = reload[v];
    if (r > mx) mx = r;
    if (r > 0) atomicAdd(&sh[r < 16 ? r : 16], 1u);   // bin 0 is derived on the host from V
  }
  if (mx) atomicMax(&shmax, mx);
  __syncthreads();
  if (threadIdx.x < 17 && sh[threadIdx.x]) atomicAdd((unsigned long long*)&hist18[threadIdx.x], (unsigned long long)sh[threadIdx.x]);
  if (threadIdx.x == 0 && shmax) atomicMax(&hist18[17], (long long)shmax);
}

// Dense-output mode: the rows of one half of the graduation buffer go to dense[id * ld ...]; the row count is
// read from the control block, so the launch needs no host round trip.
__global__ void place_half_kernel(const DevCtl* ctl, int half, const long long* ids, const float* rows, int Hp, int d_out,
                                  float* dense, long long ld) {
  const long long count = ctl->out_count[half];
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const bool vec_ok = (ld % 4 == 0) && ((reinterpret_cast<uintptr_t>(dense) & 15) == 0);
  for (long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < count; i += warps) {
    long long id = ids[i];
    const float* src = rows + (size_t)i * Hp;
    float* dst = dense + (size_t)id * ld;
    if (vec_ok) {
      int full = d_out >> 2;
      for (int k = lane_id(); k < full; k += 32)
        reinterpret_cast<float4*>(dst)[k] = reinterpret_cast<const float4*>(src)[k];
      for (int k = (full << 2) + lane_id(); k < d_out; k += 32) dst[k] = src[k];
    } else {
      for (int k = lane_id(); k < d_out; k += 32) dst[k] = src[k];
    }
  }
}

void launch_place_half(taurus_ctx* c, int half, int d_out, int Hp, cudaStream_t st) {
  const long long off = (long long)half * (c->drain_rows / 2);
  place_half_kernel<<<c->sm_count * 4, 256, 0, st>>>(c->d_ctl, half, c->d_grad_ids + off, c->d_grad_rows + (size_t)off * Hp, Hp, d_out,
                                                     c->dense_out, c->dense_ld);
  c->launches += 1;
}

void launch_reload_histogram(taurus_ctx* c, long long* d_hist18, cudaStream_t st) {
  cudaMemsetAsync(d_hist18, 0, 18 * sizeof(long long), st);
  reload_histogram_kernel<<<c->sm_count * 4, 256, 0, st>>>(c->V, c->d_reload, d_hist18);
  c->launches += 1;
}

// ------------------------------------------------------------------------------------------------ completion ranks
// Completion rank of v = max(v, largest source among its propagated in-edges): the chunk holding that
// rank is the one in which v completes (Sect. 3.8, c(v)).  A histogram over blocks of 64 ranks lets the
// host bound, without a device round trip, how many rows a pushed range can add to the graduation buffer.
__global__ void rank_init_kernel(long long V, int32_t* last) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) last[v] = (int32_t)v;
}
__global__ void rank_max_kernel(long long V, const long long* row_ptr, const int32_t* col, const uint32_t* mask, int32_t* last) {
  const long long warps = ((long long)gridDim.x * blockDim.x) >> 5;
  for (long long u = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < V; u += warps) {
    long long b = row_ptr[u], e = row_ptr[u + 1];
    for (long long k = b + lane_id(); k < e; k += 32)
      if (edge_propagated(mask, k)) atomicMax(&last[col[k]], (int32_t)u);
  }
}
__global__ void rank_hist_kernel(long long V, const int32_t* last, int32_t* hist) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride) atomicAdd(&hist[last[v] >> 6], 1);
}

void launch_completion_ranks(taurus_ctx* c, cudaStream_t st) {
  int blocks = c->sm_count * 8;
  long long nb = (c->V + 63) / 64;
  cudaMemsetAsync(c->d_rank_hist, 0, (size_t)nb * sizeof(int32_t), st);
  rank_init_kernel<<<blocks, 256, 0, st>>>(c->V, c->d_vtmp);
  rank_max_kernel<<<blocks, 256, 0, st>>>(c->V, c->d_row_ptr, c->d_col, c->d_mask_cur, c->d_vtmp);
  rank_hist_kernel<<<blocks, 256, 0, st>>>(c->V, c->d_vtmp, c->d_rank_hist);
  c->launches += 3;
}

// ------------------------------------------------------------------------------------------------ init check
__global__ void degree_hist_kernel(long long E, const int32_t* col, long long V, int32_t* hist, int* flag) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < E; e += stride) {
    int v = col[e];
    if (v < 0 || v >= V) *flag = 1; else atomicAdd(&hist[v], 1);
  }
}
__global__ void degree_compare_kernel(long long V, const int32_t* hist, const int32_t* din, const long long* row_ptr, int* flag) {
  long long stride = (long long)gridDim.x * blockDim.x;
  for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < V; v += stride)
    if (hist[v] != din[v] || row_ptr[v + 1] < row_ptr[v]) *flag = 1;
}

int check_in_degrees(taurus_ctx* c, cudaStream_t st) {
  int* d_flag = nullptr;
  if (cudaMalloc(&d_flag, sizeof(int)) != cudaSuccess) return -1;
  cudaMemsetAsync(d_flag, 0, sizeof(int), st);
  cudaMemsetAsync(c->d_vtmp, 0, (size_t)c->V * sizeof(int32_t), st);
  int blocks = c->sm_count * 8;
  degree_hist_kernel<<<blocks, 256, 0, st>>>(c->E, c->d_col, c->V, c->d_vtmp, d_flag);
  degree_compare_kernel<<<blocks, 256, 0, st>>>(c->V, c->d_vtmp, c->d_din, c->d_row_ptr, d_flag);
  int flag = 0;
  cudaMemcpyAsync(&flag, d_flag, sizeof(int), cudaMemcpyDeviceToHost, st);
  cudaStreamSynchronize(st);
  cudaFree(d_flag);
  c->launches += 2;
  return flag;
}

// ------------------------------------------------------------------------------------------------ sizing
__global__ void window_edges_kernel(long long V, long long window, const long long* row_ptr, unsigned long long* out_max) {
  long long stride = (long long)gridDim.x * blockDim.x;
  unsigned long long mx = 0;
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < V; u += stride) {
    long long e = u + window < V ? u + window : V;
    unsigned long long n = (unsigned long long)(row_ptr[e] - row_ptr[u]);
    if (n > mx) mx = n;
  }
  for (int o = 16; o; o >>= 1) { unsigned long long t = __shfl_xor_sync(FULL, mx, o); if (t > mx) mx = t; }
  if (lane_id() == 0 && mx) atomicMax(out_max, mx);
}

long long max_window_edges(taurus_ctx* c) {
  unsigned long long* d = nullptr;
  if (cudaMalloc(&d, sizeof(unsigned long long)) != cudaSuccess) return -1;
  cudaMemset(d, 0, sizeof(unsigned long long));
  window_edges_kernel<<<c->sm_count * 8, 256>>>(c->V, c->chunk_sources, c->d_row_ptr, d);
  unsigned long long h = 0;
  cudaError_t e = cudaMemcpy(&h, d, sizeof(h), cudaMemcpyDeviceToHost);
  cudaFree(d);
  c->launches += 1;
  return e == cudaSuccess ? (long long)h : -1;
}
