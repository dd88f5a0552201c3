/*
 * Seeded synthetic problem generator: graphs (CSR out-edges), feature rows and
 * layer weights.  Everything is a pure function of (seed, stream tag, i, j)
 * through one counter hash, so any row can be regenerated on demand and no
 * state is kept.
 *
 * This module defines the PROBLEM only.  It holds none of the method's
 * arithmetic (no aggregation, no sampling of neighbours, no state machine)
 * and is the one piece of code both the CPU oracle's tests and the CUDA
 * library's tests may call.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define TG_GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t tg_mix(uint64_t x) {
  x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
  x ^= x >> 27; x *= 0x94D049BB133111EBull;
  x ^= x >> 31;
  return x;
}
static inline uint64_t tg_absorb(uint64_t h, uint64_t x) { return tg_mix((h ^ x) + TG_GOLDEN); }

uint64_t tg_hash64(uint64_t seed, uint64_t tag, uint64_t i, uint64_t j) {
  uint64_t h = tg_absorb(0x7461757275735F67ull, seed);
  h = tg_absorb(h, tag);
  h = tg_absorb(h, i);
  h = tg_absorb(h, j);
  return h;
}

/* uniform in [0,1) with 53 bits */
static inline double tg_u01(uint64_t h) { return (double)(h >> 11) * (1.0 / 9007199254740992.0); }

/* stream tags */
enum { TAG_DEG = 1, TAG_DST_KIND = 2, TAG_DST_A = 3, TAG_DST_B = 4, TAG_FEAT = 5, TAG_WEIGHT = 6 };

typedef struct {
  uint64_t seed;
  int64_t V;
  double alpha;      /* out-degree power-law exponent */
  double kappa;      /* degree scale (found by tg_calibrate_kappa) */
  int64_t d_max;     /* cap on the raw weight */
  int32_t dst_mode;  /* 0: uniform destinations; 1: local + hub-Zipf mixture */
  double lambda;     /* probability of a local destination (mode 1) */
  double local_B;    /* mean of the exponential local offset (mode 1) */
  double beta;       /* Zipf exponent of the hub ranks (mode 1) */
  double r0;         /* Zipf shift (mode 1) */
  int64_t perm_a;    /* dst = (perm_a * rank + perm_b) mod V, gcd(perm_a, V) = 1 */
  int64_t perm_b;
} tg_graph_params;

static inline double tg_weight(const tg_graph_params* p, int64_t u) {
  double x = tg_u01(tg_hash64(p->seed, TAG_DEG, (uint64_t)u, 0));
  double w = pow(1.0 - x, -1.0 / (p->alpha - 1.0));
  if (w > (double)p->d_max) w = (double)p->d_max;
  return w;
}

static inline int32_t tg_degree_of(const tg_graph_params* p, double kappa, int64_t u) {
  double d = floor(kappa * tg_weight(p, u));
  if (d < 1.0) d = 1.0;
  if (d > 2.0e9) d = 2.0e9;
  return (int32_t)d;
}

/* Bisection on kappa so that the sum of out-degrees lands within 0.1 % of target_E. */
double tg_calibrate_kappa(const tg_graph_params* p, int64_t target_E) {
  int64_t V = p->V;
  double* w = (double*)malloc(sizeof(double) * (size_t)V);
  if (!w) return -1.0;
#pragma omp parallel for schedule(static)
  for (int64_t u = 0; u < V; ++u) w[u] = tg_weight(p, u);
  double lo = 0.0, hi = 1.0;
  for (;;) { /* grow hi until the sum exceeds the target */
    double s = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : s)
    for (int64_t u = 0; u < V; ++u) { double d = floor(hi * w[u]); s += d < 1.0 ? 1.0 : d; }
    if (s >= (double)target_E || hi > 1e12) break;
    hi *= 2.0;
  }
  for (int it = 0; it < 60; ++it) {
    double mid = 0.5 * (lo + hi), s = 0.0;
#pragma omp parallel for schedule(static) reduction(+ : s)
    for (int64_t u = 0; u < V; ++u) { double d = floor(mid * w[u]); s += d < 1.0 ? 1.0 : d; }
    if (s < (double)target_E) lo = mid; else hi = mid;
    if (fabs(s - (double)target_E) <= 0.0005 * (double)target_E) { lo = hi = mid; break; }
  }
  free(w);
  return 0.5 * (lo + hi);
}

/* out-degrees and their exclusive prefix sum (row_ptr has V+1 entries) */
int tg_out_degrees(const tg_graph_params* p, int64_t* row_ptr) {
  int64_t V = p->V;
  row_ptr[0] = 0;
#pragma omp parallel for schedule(static)
  for (int64_t u = 0; u < V; ++u) row_ptr[u + 1] = tg_degree_of(p, p->kappa, u);
  for (int64_t u = 0; u < V; ++u) row_ptr[u + 1] += row_ptr[u];
  return 0;
}

/* destination of the j-th generated out-edge of u */
static inline int64_t tg_dst(const tg_graph_params* p, int64_t u, int64_t j) {
  int64_t V = p->V;
  if (p->dst_mode == 0) {
    uint64_t h = tg_hash64(p->seed, TAG_DST_A, (uint64_t)u, (uint64_t)j);
    return (int64_t)(((unsigned __int128)h * (unsigned __int128)(uint64_t)V) >> 64);
  }
  uint64_t hk = tg_hash64(p->seed, TAG_DST_KIND, (uint64_t)u, (uint64_t)j);
  double x = tg_u01(tg_hash64(p->seed, TAG_DST_A, (uint64_t)u, (uint64_t)j));
  if (tg_u01(hk) < p->lambda) { /* local: u +- floor(-B ln(1-x)) */
    double off = floor(-p->local_B * log(1.0 - x));
    if (off > (double)(V - 1)) off = (double)(V - 1);
    int64_t o = (int64_t)off;
    int64_t v = (hk & 1ull) ? u + o : u - o;
    v %= V; if (v < 0) v += V;
    return v;
  }
  /* hub-Zipf: P(r) ~ (r + r0)^-beta on [0, V), closed-form inverse CDF */
  double r;
  double r0 = p->r0, Vd = (double)V;
  if (fabs(p->beta - 1.0) < 1e-12) {
    r = r0 * exp(x * log((Vd + r0) / r0)) - r0;
  } else {
    double e = 1.0 - p->beta;
    double a = pow(r0, e), b = pow(Vd + r0, e);
    r = pow(a + x * (b - a), 1.0 / e) - r0;
  }
  int64_t ri = (int64_t)floor(r);
  if (ri < 0) ri = 0;
  if (ri >= V) ri = V - 1;
  unsigned __int128 t = (unsigned __int128)(uint64_t)p->perm_a * (uint64_t)ri + (uint64_t)p->perm_b;
  return (int64_t)(t % (unsigned __int128)(uint64_t)V);
}

/* directed graph: fill col[row_ptr[u] + j] for every u, j */
int tg_fill_directed(const tg_graph_params* p, const int64_t* row_ptr, int32_t* col) {
  int64_t V = p->V;
#pragma omp parallel for schedule(dynamic, 4096)
  for (int64_t u = 0; u < V; ++u) {
    int64_t b = row_ptr[u], d = row_ptr[u + 1] - b;
    for (int64_t j = 0; j < d; ++j) col[b + j] = (int32_t)tg_dst(p, u, j);
  }
  return 0;
}

/*
 * Symmetric multigraph: every generated edge (u -> v) is kept and its reverse
 * (v -> u) is added.  gen_ptr is the directed generator's row_ptr.  Row u of
 * the result holds u's generated edges in j order, then the reverse edges in
 * order of their generating (u', j).  sym_ptr [V+1] and sym_col [2 * gen E]
 * are outputs.
 */
int tg_fill_symmetric(const tg_graph_params* p, const int64_t* gen_ptr, int64_t* sym_ptr, int32_t* sym_col) {
  int64_t V = p->V, Eg = gen_ptr[V];
  int32_t* fwd = (int32_t*)malloc(sizeof(int32_t) * (size_t)(Eg > 0 ? Eg : 1));
  int64_t* cur = (int64_t*)calloc((size_t)V + 1, sizeof(int64_t));
  if (!fwd || !cur) { free(fwd); free(cur); return -1; }
  tg_fill_directed(p, gen_ptr, fwd);
  for (int64_t u = 0; u < V; ++u) cur[u] = gen_ptr[u + 1] - gen_ptr[u];
  for (int64_t e = 0; e < Eg; ++e) cur[fwd[e]] += 1;
  sym_ptr[0] = 0;
  for (int64_t u = 0; u < V; ++u) sym_ptr[u + 1] = sym_ptr[u] + cur[u];
  for (int64_t u = 0; u < V; ++u) { /* forward part, and cursor for the reverse part */
    int64_t d = gen_ptr[u + 1] - gen_ptr[u];
    memcpy(sym_col + sym_ptr[u], fwd + gen_ptr[u], sizeof(int32_t) * (size_t)d);
    cur[u] = sym_ptr[u] + d;
  }
  for (int64_t u = 0; u < V; ++u)
    for (int64_t e = gen_ptr[u]; e < gen_ptr[u + 1]; ++e) sym_col[cur[fwd[e]]++] = (int32_t)u;
  free(fwd); free(cur);
  return 0;
}

/* histogram of destinations (in-degree with multiplicity) */
int tg_in_degrees(int64_t V, int64_t E, const int32_t* col, int32_t* din) {
  memset(din, 0, sizeof(int32_t) * (size_t)V);
  for (int64_t e = 0; e < E; ++e) din[col[e]] += 1;
  return 0;
}

/*
 * Feature rows v_begin..v_end-1, F columns, fp32 N(0,1): Box-Muller in fp64 on
 * two hash-derived uniforms, one pair of normals per pair of columns, keyed
 * (seed, layer_tag, v, column pair).  out is row-major with leading dimension ld.
 */
int tg_features(uint64_t seed, uint64_t layer_tag, int64_t v_begin, int64_t v_end, int32_t F, int64_t ld, float* out) {
  const double two_pi = 6.283185307179586476925286766559;
#pragma omp parallel for schedule(static)
  for (int64_t v = v_begin; v < v_end; ++v) {
    float* row = out + (v - v_begin) * ld;
    uint64_t hv = tg_hash64(seed, TAG_FEAT, layer_tag, (uint64_t)v);
    for (int32_t d = 0; d < F; d += 2) {
      uint64_t h1 = tg_absorb(hv, (uint64_t)d);
      uint64_t h2 = tg_absorb(h1, 0x5bd1e995ull);
      double u1 = 1.0 - tg_u01(h1); /* (0, 1] */
      double u2 = tg_u01(h2);
      double r = sqrt(-2.0 * log(u1));
      row[d] = (float)(r * cos(two_pi * u2));
      if (d + 1 < F) row[d + 1] = (float)(r * sin(two_pi * u2));
    }
  }
  return 0;
}

/* The same rows for an arbitrary list of vertex ids (row i of out = features of ids[i]). */
int tg_features_rows(uint64_t seed, uint64_t layer_tag, const int64_t* ids, int64_t n, int32_t F, int64_t ld, float* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) tg_features(seed, layer_tag, ids[i], ids[i] + 1, F, ld, out + i * ld);
  return 0;
}

/* Xavier-uniform rows x cols matrix, U(-a, a), a = sqrt(6 / (rows + cols)), row-major fp32 */
int tg_weights(uint64_t seed, uint64_t layer, uint64_t which, int32_t rows, int32_t cols, float* out) {
  double a = sqrt(6.0 / ((double)rows + (double)cols));
  uint64_t hl = tg_hash64(seed, TAG_WEIGHT, layer, which);
  for (int32_t i = 0; i < rows; ++i)
    for (int32_t j = 0; j < cols; ++j) {
      double x = tg_u01(tg_absorb(tg_absorb(hl, (uint64_t)i), (uint64_t)j));
      out[(int64_t)i * cols + j] = (float)((2.0 * x - 1.0) * a);
    }
  return 0;
}

/* Expected in-degree of Zipf rank 0 per generated hub edge: CDF(1) of the rank law. */
double tg_zipf_top_mass(double beta, double r0, double V) {
  if (fabs(beta - 1.0) < 1e-12) return log((1.0 + r0) / r0) / log((V + r0) / r0);
  double e = 1.0 - beta;
  return (pow(1.0 + r0, e) - pow(r0, e)) / (pow(V + r0, e) - pow(r0, e));
}
