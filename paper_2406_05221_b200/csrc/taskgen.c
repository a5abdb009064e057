/*
 * taskgen.c -- seeded synthetic taskset generator (CPU only).
 *
 * Produces the inputs of the response-time analysis in the CSR structure-of-arrays layout of
 * gcaps_rta.h.  It follows the generation procedure of the paper's Sec. 7.1 / Table 3 (tasks per
 * CPU, UUniFast utilisations per CPU, period, number of GPU segments, segment parameters,
 * rate-monotonic priorities, optional worst-fit-decreasing re-allocation) with the ranges left
 * as parameters.  It holds none of the analysis arithmetic: it only draws numbers.
 *
 * Determinism: taskset number g (global index) of a stream is a pure function of
 * (seed, stream, g); any taskset can be regenerated alone and the result does not depend on
 * the number of threads.  The random source is SplitMix64 (Steele, Lea, Flood 2014) run as a
 * counter-based generator: the k-th draw of a taskset is mix(key + k * GOLDEN).
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define TG_MAX_TASKS 256
#define TG_MAX_CORES 64
#define TG_MAX_SEGS 16

typedef struct {
  uint64_t seed;
  uint64_t stream;       /* sweep point / sub-stream id                                        */
  int32_t cores_lo, cores_hi;
  int32_t tpc_lo, tpc_hi; /* tasks per core                                                    */
  double util_lo, util_hi; /* utilisation per core, uniform                                    */
  double period_lo, period_hi; /* us, log-uniform                                              */
  double harmonic_frac;  /* fraction of tasksets whose periods are P0 * 2^k                    */
  int32_t gpu_mode;      /* 0: exactly round(gpu_frac*n) GPU-using tasks, eta^g in [seg_lo,seg_hi]
                            1: every task draws eta^g uniformly in [seg_lo,seg_hi] (0 allowed) */
  double gpu_frac;
  int32_t seg_lo, seg_hi;
  double ratio_lo, ratio_hi; /* G_i / (task WCET), uniform                                     */
  int32_t wfd;           /* 1: re-allocate tasks to cores by worst-fit decreasing              */
  int32_t pad_;
} tg_params_t;

typedef struct {
  uint64_t key;
  uint64_t ctr;
} tg_rng_t;

static inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
static inline void rng_init(tg_rng_t *r, uint64_t seed, uint64_t stream, uint64_t index) {
  uint64_t k = mix64(seed + 0x9E3779B97F4A7C15ULL);
  k = mix64(k ^ (stream * 0xD1B54A32D192ED03ULL + 0x632BE59BD9B4E019ULL));
  k = mix64(k ^ (index * 0x9E3779B97F4A7C15ULL + 0x2545F4914F6CDD1DULL));
  r->key = k;
  r->ctr = 0;
}
static inline uint64_t rng_u64(tg_rng_t *r) {
  r->ctr += 1;
  return mix64(r->key + r->ctr * 0x9E3779B97F4A7C15ULL);
}
/* uniform double in (0,1): 53 random bits, never 0 */
static inline double rng_unit(tg_rng_t *r) {
  return ((double)(rng_u64(r) >> 11) + 0.5) * (1.0 / 9007199254740992.0);
}
static inline double rng_range(tg_rng_t *r, double lo, double hi) {
  return lo + (hi - lo) * rng_unit(r);
}
/* uniform integer in [lo, hi] */
static inline int32_t rng_int(tg_rng_t *r, int32_t lo, int32_t hi) {
  if (hi <= lo) return lo;
  uint64_t span = (uint64_t)(hi - lo) + 1;
  return lo + (int32_t)(rng_u64(r) % span);
}

typedef struct {
  int n;
  int64_t T[TG_MAX_TASKS];
  int64_t prio[TG_MAX_TASKS];
  int32_t core[TG_MAX_TASKS];
  int32_t n_c[TG_MAX_TASKS], n_g[TG_MAX_TASKS];
  int64_t cseg[TG_MAX_TASKS][TG_MAX_SEGS + 1];
  int64_t gm[TG_MAX_TASKS][TG_MAX_SEGS];
  int64_t ge[TG_MAX_TASKS][TG_MAX_SEGS];
  double util[TG_MAX_TASKS];
} tg_one_t;

/* Splits `total` into `parts` integers >= 1 (needs total >= parts) in proportion to random
 * weights in [1,2); the last part takes the rounding remainder. */
static void split_weighted(tg_rng_t *r, int64_t total, int parts, int64_t *out) {
  double w[TG_MAX_SEGS + 1], ws = 0.0;
  for (int j = 0; j < parts; ++j) {
    w[j] = 1.0 + rng_unit(r);
    ws += w[j];
  }
  int64_t spare = total - parts, used = 0;
  for (int j = 0; j < parts; ++j) {
    int64_t x;
    if (j == parts - 1) {
      x = spare - used;
    } else {
      x = (int64_t)floor((double)spare * w[j] / ws);
      if (x > spare - used) x = spare - used;
    }
    used += x;
    out[j] = 1 + x;
  }
}

static int cmp_desc_util(const void *a, const void *b, void *ctx) {
  const tg_one_t *o = (const tg_one_t *)ctx;
  int ia = *(const int *)a, ib = *(const int *)b;
  if (o->util[ia] > o->util[ib]) return -1;
  if (o->util[ia] < o->util[ib]) return 1;
  return ia - ib;
}

static void gen_one(const tg_params_t *p, uint64_t index, tg_one_t *o) {
  tg_rng_t rng;
  rng_init(&rng, p->seed, p->stream, index);
  int cores = rng_int(&rng, p->cores_lo, p->cores_hi);
  if (cores > TG_MAX_CORES) cores = TG_MAX_CORES;
  int harmonic = rng_unit(&rng) < p->harmonic_frac;
  double ln_lo = log(p->period_lo), ln_hi = log(p->period_hi);
  int n = 0;
  for (int c = 0; c < cores; ++c) {
    int m = rng_int(&rng, p->tpc_lo, p->tpc_hi);
    if (n + m > TG_MAX_TASKS) m = TG_MAX_TASKS - n;
    double U = rng_range(&rng, p->util_lo, p->util_hi);
    /* UUniFast (Bini & Buttazzo): m utilisations summing to U */
    double sum = U;
    for (int k = 0; k < m; ++k) {
      double u;
      if (k == m - 1) {
        u = sum;
      } else {
        double next = sum * pow(rng_unit(&rng), 1.0 / (double)(m - 1 - k));
        u = sum - next;
        sum = next;
      }
      o->util[n + k] = u;
      o->core[n + k] = c;
    }
    n += m;
  }
  o->n = n;
  /* periods */
  for (int i = 0; i < n; ++i) {
    double t;
    if (harmonic) {
      double hi0 = p->period_lo * 100.0 < p->period_hi ? p->period_lo * 100.0 : p->period_hi;
      double p0 = floor(exp(rng_range(&rng, ln_lo, log(hi0))) + 0.5);
      int k = rng_int(&rng, 0, 10);
      t = p0 * (double)(1 << k);
    } else {
      t = floor(exp(rng_range(&rng, ln_lo, ln_hi)) + 0.5);
    }
    if (t < p->period_lo) t = p->period_lo;
    if (t > p->period_hi) t = p->period_hi;
    o->T[i] = (int64_t)t;
  }
  /* which tasks use the GPU */
  int want[TG_MAX_TASKS];
  if (p->gpu_mode == 0) {
    int idx[TG_MAX_TASKS];
    for (int i = 0; i < n; ++i) idx[i] = i, want[i] = 0;
    int ng = (int)floor(p->gpu_frac * (double)n + 0.5);
    if (ng > n) ng = n;
    for (int k = 0; k < ng; ++k) { /* partial Fisher-Yates */
      int j = k + (int)(rng_u64(&rng) % (uint64_t)(n - k));
      int tmp = idx[k];
      idx[k] = idx[j];
      idx[j] = tmp;
      want[idx[k]] = rng_int(&rng, p->seg_lo < 1 ? 1 : p->seg_lo, p->seg_hi);
    }
  } else {
    for (int i = 0; i < n; ++i) want[i] = rng_int(&rng, p->seg_lo, p->seg_hi);
  }
  /* execution demand and its split into segments */
  for (int i = 0; i < n; ++i) {
    int64_t E = (int64_t)floor(o->util[i] * (double)o->T[i] + 0.5);
    if (E < 1) E = 1;
    if (E > o->T[i]) E = o->T[i];
    double rho = rng_range(&rng, p->ratio_lo, p->ratio_hi);
    int eta = want[i] > TG_MAX_SEGS ? TG_MAX_SEGS : want[i];
    int64_t G = (int64_t)floor(rho * (double)E + 0.5);
    /* every GPU segment and every CPU segment gets >= 1 us: drop segments until E can hold
     * eta GPU segments and eta+1 CPU segments, then clamp G into the feasible range */
    while (eta > 0 && E < 2 * (int64_t)eta + 1) eta -= 1;
    if (eta == 0) {
      G = 0;
    } else {
      if (G < eta) G = eta;
      if (G > E - eta - 1) G = E - eta - 1;
    }
    o->n_g[i] = eta;
    o->n_c[i] = eta + 1;
    if (eta > 0) {
      int64_t g[TG_MAX_SEGS];
      split_weighted(&rng, G, eta, g);
      for (int j = 0; j < eta; ++j) {
        o->gm[i][j] = g[j] / 5; /* 20 % miscellaneous CPU work, 80 % pure GPU work */
        o->ge[i][j] = g[j] - o->gm[i][j];
      }
    }
    split_weighted(&rng, E - G, eta + 1, o->cseg[i]);
    o->util[i] = (double)E / (double)o->T[i];
  }
  /* rate-monotonic priorities, unique: shorter period = higher, ties by position */
  for (int i = 0; i < n; ++i) {
    int higher = 0;
    for (int k = 0; k < n; ++k)
      if (o->T[k] < o->T[i] || (o->T[k] == o->T[i] && k < i)) higher += 1;
    o->prio[i] = (int64_t)(n - higher);
  }
  if (p->wfd) {
    int order[TG_MAX_TASKS];
    double load[TG_MAX_CORES];
    for (int i = 0; i < n; ++i) order[i] = i;
    for (int c = 0; c < cores; ++c) load[c] = 0.0;
    qsort_r(order, (size_t)n, sizeof(int), cmp_desc_util, o);
    for (int k = 0; k < n; ++k) {
      int best = 0;
      for (int c = 1; c < cores; ++c)
        if (load[c] < load[best]) best = c;
      o->core[order[k]] = best;
      load[best] += o->util[order[k]];
    }
  }
}

/* Pass 1: per-taskset sizes.  counts[3*t+0..2] = tasks, CPU segments, GPU segments of taskset
 * first+t. */
void tg_sizes(const tg_params_t *p, int64_t first, int64_t count, int64_t *counts) {
#pragma omp parallel
  {
    tg_one_t *o = (tg_one_t *)malloc(sizeof(tg_one_t));
#pragma omp for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
      gen_one(p, (uint64_t)(first + t), o);
      int64_t nc = 0, ng = 0;
      for (int i = 0; i < o->n; ++i) nc += o->n_c[i], ng += o->n_g[i];
      counts[3 * t + 0] = o->n;
      counts[3 * t + 1] = nc;
      counts[3 * t + 2] = ng;
    }
    free(o);
  }
}

/* Pass 2: fill.  task_off [count+1], cseg_off/gseg_off [n_tasks+1] are written here from the
 * exclusive prefix sums starts[3*t+0..2] of tg_sizes' counts. */
void tg_fill(const tg_params_t *p, int64_t first, int64_t count, const int64_t *starts,
             int64_t *task_off, int64_t *period, int64_t *deadline, int64_t *priority,
             int64_t *core, int64_t *cseg_off, int64_t *cseg_wcet, int64_t *gseg_off,
             int64_t *gseg_misc, int64_t *gseg_exec) {
#pragma omp parallel
  {
    tg_one_t *o = (tg_one_t *)malloc(sizeof(tg_one_t));
#pragma omp for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
      gen_one(p, (uint64_t)(first + t), o);
      int64_t k0 = starts[3 * t + 0], c0 = starts[3 * t + 1], g0 = starts[3 * t + 2];
      task_off[t] = k0;
      for (int i = 0; i < o->n; ++i) {
        period[k0 + i] = o->T[i];
        deadline[k0 + i] = o->T[i];
        priority[k0 + i] = o->prio[i];
        core[k0 + i] = o->core[i];
        cseg_off[k0 + i] = c0;
        gseg_off[k0 + i] = g0;
        for (int j = 0; j < o->n_c[i]; ++j) cseg_wcet[c0 + j] = o->cseg[i][j];
        for (int j = 0; j < o->n_g[i]; ++j) {
          gseg_misc[g0 + j] = o->gm[i][j];
          gseg_exec[g0 + j] = o->ge[i][j];
        }
        c0 += o->n_c[i];
        g0 += o->n_g[i];
      }
      if (t == count - 1) {
        task_off[count] = k0 + o->n;
        cseg_off[k0 + o->n] = c0;
        gseg_off[k0 + o->n] = g0;
      }
    }
    free(o);
  }
}

int tg_max_tasks(void) { return TG_MAX_TASKS; }
size_t tg_params_size(void) { return sizeof(tg_params_t); }

/* ---------------------------------------------------------------------------------------------
 * The integer-only generator (igen.h) on the host: the same two passes as above.  Its output is
 * bit-identical to what the CUDA library's on-device generator writes for the same parameters.
 * ------------------------------------------------------------------------------------------- */
#include "igen.h"

void ig_sizes(const igen_params_t *p, int64_t first, int64_t count, int64_t *counts) {
#pragma omp parallel
  {
    igen_state_t *s = (igen_state_t *)malloc(sizeof(igen_state_t));
#pragma omp for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
      igen_begin(p, (uint64_t)(first + t), s);
      counts[3 * t + 0] = s->n;
      counts[3 * t + 1] = s->n_csegs;
      counts[3 * t + 2] = s->n_gsegs;
    }
    free(s);
  }
}

void ig_fill(const igen_params_t *p, int64_t first, int64_t count, const int64_t *starts,
             int64_t *task_off, int64_t *period, int64_t *deadline, int64_t *priority,
             int64_t *core, int64_t *cseg_off, int64_t *cseg_wcet, int64_t *gseg_off,
             int64_t *gseg_misc, int64_t *gseg_exec) {
#pragma omp parallel
  {
    igen_state_t *s = (igen_state_t *)malloc(sizeof(igen_state_t));
#pragma omp for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
      igen_begin(p, (uint64_t)(first + t), s);
      int64_t k0 = starts[3 * t + 0], c0 = starts[3 * t + 1], g0 = starts[3 * t + 2];
      task_off[t] = k0;
      for (int i = 0; i < s->n; ++i) {
        int64_t cs[IGEN_MAX_SEGS + 1], gm[IGEN_MAX_SEGS], ge[IGEN_MAX_SEGS];
        igen_segments(s, i, cs, gm, ge);
        period[k0 + i] = s->T[i];
        deadline[k0 + i] = s->T[i];
        priority[k0 + i] = s->prio[i];
        core[k0 + i] = s->core[i];
        cseg_off[k0 + i] = c0;
        gseg_off[k0 + i] = g0;
        for (int j = 0; j <= s->eta[i]; ++j) cseg_wcet[c0 + j] = cs[j];
        for (int j = 0; j < s->eta[i]; ++j) {
          gseg_misc[g0 + j] = gm[j];
          gseg_exec[g0 + j] = ge[j];
        }
        c0 += s->eta[i] + 1;
        g0 += s->eta[i];
      }
      if (t == count - 1) {
        task_off[count] = k0 + s->n;
        cseg_off[k0 + s->n] = c0;
        gseg_off[k0 + s->n] = g0;
      }
    }
    free(s);
  }
}

size_t ig_params_size(void) { return sizeof(igen_params_t); }
uint64_t ig_exp2(uint64_t y) { return igen_exp2(y); }
