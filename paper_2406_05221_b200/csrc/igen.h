/*
 * igen.h -- the integer-only taskset generator, as one definition that compiles both as C (the
 * host generator, gcc) and as CUDA device code (the on-device generator, nvcc).
 *
 * It follows the generation procedure of the paper's Sec. 7.1 / Table 3 like the floating-point
 * host generator (taskgen.c) does -- tasks per CPU, utilisation per CPU split over its tasks,
 * period, number of GPU segments, segment parameters, rate-monotonic priorities, optional
 * worst-fit-decreasing re-allocation -- but every step is integer arithmetic, so a taskset is
 * the same bit pattern wherever it is generated:
 *   - real-valued ranges are fixed point with 32 fractional bits (Q32);
 *   - the utilisation of a CPU is split by uniform spacings (m-1 sorted uniform cut points of
 *     [0,1)), which has the distribution of UUniFast (uniform on the simplex) without pow();
 *   - a log-uniform period is 2^y for y uniform in [log2 lo, log2 hi] (Q32, passed in as
 *     parameters); 2^frac is a product of the constants 2^(2^-i), i = 1..24, held in Q62;
 *   - random numbers are SplitMix64 (Steele, Lea, Flood 2014) run as a counter-based generator
 *     keyed by (seed, stream, taskset index), as in taskgen.c.
 * It holds none of the analysis arithmetic: it only draws numbers.
 *
 * Use: igen_begin() draws everything per task except the segment split and leaves the per-task
 * scalars (and the segment counts) in the state; igen_segments() must then be called for tasks
 * 0, 1, ... in order and yields the task's segment values.
 */
#ifndef GCAPS_IGEN_H_
#define GCAPS_IGEN_H_

#include <stdint.h>

#ifdef __CUDACC__
#define IGEN_FN __host__ __device__ static inline
#else
#define IGEN_FN static inline
#endif

#define IGEN_MAX_TASKS 256
#define IGEN_MAX_CORES 64
#define IGEN_MAX_SEGS 16
#define IGEN_FRAC_BITS 24 /* bits of the fraction of y that 2^y looks at */

typedef struct {
  uint64_t seed;
  uint64_t stream;             /* sweep point / sub-stream id                                  */
  int32_t cores_lo, cores_hi;
  int32_t tpc_lo, tpc_hi;      /* tasks per core                                               */
  uint64_t util_lo, util_hi;   /* utilisation per core, Q32, uniform                            */
  uint64_t log2_lo, log2_hi;   /* log2 of the period range in us, Q32: y uniform in between     */
  uint64_t log2_hi0;           /* harmonic tasksets: upper end of log2 of the base period, Q32  */
  int64_t period_lo, period_hi; /* us; every period is clamped into this range                  */
  uint64_t harmonic;           /* Q32 probability that a taskset's periods are P0 * 2^k         */
  uint64_t gpu_frac;           /* Q32 share of GPU-using tasks (gpu_mode 0)                     */
  uint64_t ratio_lo, ratio_hi; /* G_i / (task WCET), Q32, uniform                               */
  int32_t gpu_mode;            /* 0: exactly round(gpu_frac*n) GPU-using tasks, eta^g in
                                  [seg_lo,seg_hi]; 1: every task draws eta^g in [seg_lo,seg_hi] */
  int32_t seg_lo, seg_hi;
  int32_t wfd;                 /* 1: re-allocate tasks to cores by worst-fit decreasing         */
} igen_params_t;

typedef struct {
  uint64_t key, ctr;
} igen_rng_t;

typedef struct {
  igen_rng_t rng;
  int32_t n, n_csegs, n_gsegs;  /* tasks, CPU segments, GPU segments of the taskset              */
  uint64_t ratio_lo, ratio_hi;
  uint32_t T[IGEN_MAX_TASKS];   /* period = deadline, us                                         */
  uint32_t E[IGEN_MAX_TASKS];   /* execution demand C_i + G_i, us                                */
  uint16_t prio[IGEN_MAX_TASKS];
  uint8_t core[IGEN_MAX_TASKS];
  uint8_t eta[IGEN_MAX_TASKS];  /* GPU segments; the task has eta + 1 CPU segments               */
} igen_state_t;

/* 2^(2^-i) in Q62, i = 1 .. 24: c[1] = floor(sqrt(2 * 2^124)), c[i+1] = floor(sqrt(c[i] * 2^62)) */
IGEN_FN uint64_t igen_root(int i) {
  switch (i) {
    case 1: return 6521908912666391106ULL;
    case 2: return 5484249825272419511ULL;
    case 3: return 5029079263719320435ULL;
    case 4: return 4815862801830788490ULL;
    case 5: return 4712668792719003883ULL;
    case 6: return 4661903986662671289ULL;
    case 7: return 4636727017470743989ULL;
    case 8: return 4624189567668517719ULL;
    case 9: return 4617933561212708775ULL;
    case 10: return 4614808732577250067ULL;
    case 11: return 4613247111281068007ULL;
    case 12: return 4612466498810092973ULL;
    case 13: return 4612076242109103706ULL;
    case 14: return 4611881126141011235ULL;
    case 15: return 4611783571252412753ULL;
    case 16: return 4611734794581956352ULL;
    case 17: return 4611710406440186475ULL;
    case 18: return 4611698212417665818ULL;
    case 19: return 4611692115418496523ULL;
    case 20: return 4611689066921934629ULL;
    case 21: return 4611687542674409370ULL;
    case 22: return 4611686780550835663ULL;
    case 23: return 4611686399489096040ULL;
    default: return 4611686208958238036ULL;
  }
}

IGEN_FN uint64_t igen_mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
IGEN_FN void igen_rng_init(igen_rng_t *r, uint64_t seed, uint64_t stream, uint64_t index) {
  uint64_t k = igen_mix64(seed + 0x9E3779B97F4A7C15ULL);
  k = igen_mix64(k ^ (stream * 0xD1B54A32D192ED03ULL + 0x632BE59BD9B4E019ULL));
  k = igen_mix64(k ^ (index * 0x9E3779B97F4A7C15ULL + 0x2545F4914F6CDD1DULL));
  r->key = k;
  r->ctr = 0;
}
IGEN_FN uint64_t igen_u64(igen_rng_t *r) {
  r->ctr += 1;
  return igen_mix64(r->key + r->ctr * 0x9E3779B97F4A7C15ULL);
}
/* uniform fraction of [0,1) in Q32 */
IGEN_FN uint64_t igen_unit(igen_rng_t *r) { return igen_u64(r) >> 32; }
/* (a * b) >> 32 for a * b < 2^96 */
IGEN_FN uint64_t igen_mul_shr32(uint64_t a, uint64_t b) {
#ifdef __CUDA_ARCH__
  return (__umul64hi(a, b) << 32) | ((a * b) >> 32);
#else
  return (uint64_t)(((unsigned __int128)a * b) >> 32);
#endif
}
/* uniform Q32 value in [lo, hi) (lo for hi <= lo) */
IGEN_FN uint64_t igen_range(igen_rng_t *r, uint64_t lo, uint64_t hi) {
  const uint64_t u = igen_unit(r);
  if (hi <= lo) return lo;
  return lo + igen_mul_shr32(hi - lo, u);
}
/* uniform integer in [lo, hi] */
IGEN_FN int32_t igen_int(igen_rng_t *r, int32_t lo, int32_t hi) {
  const uint64_t x = igen_u64(r);
  if (hi <= lo) return lo;
  return lo + (int32_t)(x % ((uint64_t)(hi - lo) + 1));
}

/* (a * b) >> 62 for a, b < 2^63 */
IGEN_FN uint64_t igen_mul_q62(uint64_t a, uint64_t b) {
#ifdef __CUDA_ARCH__
  return (__umul64hi(a, b) << 2) | ((a * b) >> 62);
#else
  return (uint64_t)(((unsigned __int128)a * b) >> 62);
#endif
}

/* round(2^y) for y in Q32, 0 <= y < 40 */
IGEN_FN uint64_t igen_exp2(uint64_t y) {
  const int k = (int)(y >> 32);
  const uint32_t f = (uint32_t)y >> (32 - IGEN_FRAC_BITS);
  uint64_t r = 1ULL << 62;
  for (int i = 1; i <= IGEN_FRAC_BITS; ++i)
    if ((f >> (IGEN_FRAC_BITS - i)) & 1u) r = igen_mul_q62(r, igen_root(i));
  /* r = 2^frac in Q62, in [1, 2); scale by 2^k and round to nearest */
  return ((r >> (61 - k)) + 1) >> 1;
}

/* floor(a / d) for 0 < d < 2^40 and a < 2^63 */
IGEN_FN uint64_t igen_div(uint64_t a, uint64_t d) {
#ifdef __CUDA_ARCH__
  /* no 64-bit division: two single-precision estimates, the second of what the first left over,
   * then the remainder settles the quotient exactly (differences are taken modulo 2^64 and read
   * as signed: the true ones are far below 2^63) */
  const float inv = 1.0f / (float)d;
  uint64_t q = (uint64_t)((float)a * inv);
  int64_t rem = (int64_t)(a - q * d);
  const int64_t q2 = (int64_t)((float)rem * inv);
  q += (uint64_t)q2;
  rem -= q2 * (int64_t)d;
  while (rem < 0) {
    rem += (int64_t)d;
    q -= 1;
  }
  while (rem >= (int64_t)d) {
    rem -= (int64_t)d;
    q += 1;
  }
  return q;
#else
  return a / d;
#endif
}

/* Splits `total` into `parts` integers >= 1 (needs total >= parts) in proportion to random
 * weights in [1,2); the last part takes the rounding remainder.  With `fifth` given, a fifth of
 * every part (rounded down) goes there and the rest to `out`.  The weights are drawn twice (once
 * for their sum, once to use them: the random source is counter-based) instead of being kept. */
IGEN_FN void igen_split(igen_rng_t *r, int64_t total, int parts, int64_t *out, int64_t *fifth) {
  const uint64_t first_draw = r->ctr;
  uint64_t ws = 0;
  for (int j = 0; j < parts; ++j) ws += (1ULL << 32) + igen_unit(r);
  r->ctr = first_draw;
  const uint64_t spare = (uint64_t)(total - parts); /* < 2^30: spare * w stays inside 63 bits */
  uint64_t used = 0;
  for (int j = 0; j < parts; ++j) {
    const uint64_t w = (1ULL << 32) + igen_unit(r);
    uint64_t x;
    if (j == parts - 1) {
      x = spare - used;
    } else {
      x = igen_div(spare * w, ws);
      if (x > spare - used) x = spare - used;
    }
    used += x;
    const int64_t part = 1 + (int64_t)x;
    if (fifth) {
      fifth[j] = part / 5;
      out[j] = part - part / 5;
    } else {
      out[j] = part;
    }
  }
}

/* Everything of taskset `index` except the segment split. */
IGEN_FN void igen_begin(const igen_params_t *p, uint64_t index, igen_state_t *s) {
  igen_rng_t *rng = &s->rng;
  igen_rng_init(rng, p->seed, p->stream, index);
  s->ratio_lo = p->ratio_lo, s->ratio_hi = p->ratio_hi;
  int cores = igen_int(rng, p->cores_lo, p->cores_hi);
  if (cores > IGEN_MAX_CORES) cores = IGEN_MAX_CORES;
  const int harmonic = igen_unit(rng) < p->harmonic;
  uint64_t util[IGEN_MAX_TASKS]; /* Q32; after the demand is known: E / T */
  int n = 0;
  for (int c = 0; c < cores; ++c) {
    int m = igen_int(rng, p->tpc_lo, p->tpc_hi);
    if (n + m > IGEN_MAX_TASKS) m = IGEN_MAX_TASKS - n;
    const uint64_t U = igen_range(rng, p->util_lo, p->util_hi);
    /* uniform spacings: m - 1 cut points of [0,1), sorted; task k gets U * (cut_k - cut_{k-1}) */
    uint64_t cut[IGEN_MAX_TASKS];
    for (int k = 0; k + 1 < m; ++k) {
      const uint64_t x = igen_unit(rng);
      int j = k;
      while (j > 0 && cut[j - 1] > x) {
        cut[j] = cut[j - 1];
        j -= 1;
      }
      cut[j] = x;
    }
    uint64_t before = 0, given = 0;
    for (int k = 0; k < m; ++k) {
      uint64_t u;
      if (k == m - 1) {
        u = U - given;
      } else {
        u = (U * (cut[k] - before)) >> 32; /* U < 2^32, spacing <= 2^32 */
        before = cut[k];
      }
      given += u;
      util[n + k] = u;
      s->core[n + k] = (uint8_t)c;
    }
    n += m;
  }
  s->n = n;
  /* periods */
  for (int i = 0; i < n; ++i) {
    int64_t t;
    if (harmonic) {
      const int64_t p0 = (int64_t)igen_exp2(igen_range(rng, p->log2_lo, p->log2_hi0));
      const int k = igen_int(rng, 0, 10);
      t = p0 << k;
    } else {
      t = (int64_t)igen_exp2(igen_range(rng, p->log2_lo, p->log2_hi));
    }
    if (t < p->period_lo) t = p->period_lo;
    if (t > p->period_hi) t = p->period_hi;
    s->T[i] = (uint32_t)t;
  }
  /* which tasks use the GPU, and how many segments they ask for */
  for (int i = 0; i < n; ++i) s->eta[i] = 0;
  if (p->gpu_mode == 0) {
    uint8_t idx[IGEN_MAX_TASKS];
    for (int i = 0; i < n; ++i) idx[i] = (uint8_t)i;
    int ng = (int)((p->gpu_frac * (uint64_t)n + (1ULL << 31)) >> 32);
    if (ng > n) ng = n;
    for (int k = 0; k < ng; ++k) { /* partial Fisher-Yates */
      const int j = k + (int)(igen_u64(rng) % (uint64_t)(n - k));
      const uint8_t tmp = idx[k];
      idx[k] = idx[j];
      idx[j] = tmp;
      s->eta[idx[k]] = (uint8_t)igen_int(rng, p->seg_lo < 1 ? 1 : p->seg_lo, p->seg_hi);
    }
  } else {
    for (int i = 0; i < n; ++i) s->eta[i] = (uint8_t)igen_int(rng, p->seg_lo, p->seg_hi);
  }
  /* execution demand; every GPU segment and every CPU segment gets >= 1 us: drop segments
   * until E can hold eta GPU segments and eta + 1 CPU segments */
  int nc = 0, ngs = 0;
  for (int i = 0; i < n; ++i) {
    const uint64_t T = s->T[i];
    uint64_t E = (util[i] * T + (1ULL << 31)) >> 32; /* util < 2^32, T < 2^24 */
    if (E < 1) E = 1;
    if (E > T) E = T;
    int eta = s->eta[i] > IGEN_MAX_SEGS ? IGEN_MAX_SEGS : s->eta[i];
    while (eta > 0 && E < 2 * (uint64_t)eta + 1) eta -= 1;
    s->E[i] = (uint32_t)E;
    s->eta[i] = (uint8_t)eta;
    util[i] = (E << 32) / T;
    nc += eta + 1;
    ngs += eta;
  }
  s->n_csegs = nc, s->n_gsegs = ngs;
  /* rate-monotonic priorities, unique: shorter period = higher, ties by position */
  for (int i = 0; i < n; ++i) {
    int higher = 0;
    for (int k = 0; k < n; ++k)
      if (s->T[k] < s->T[i] || (s->T[k] == s->T[i] && k < i)) higher += 1;
    s->prio[i] = (uint16_t)(n - higher);
  }
  if (p->wfd) { /* worst-fit decreasing by utilisation (ties: lower index first) */
    uint64_t load[IGEN_MAX_CORES];
    uint8_t done[IGEN_MAX_TASKS];
    for (int c = 0; c < cores; ++c) load[c] = 0;
    for (int i = 0; i < n; ++i) done[i] = 0;
    for (int k = 0; k < n; ++k) {
      int pick = -1;
      for (int i = 0; i < n; ++i)
        if (!done[i] && (pick < 0 || util[i] > util[pick])) pick = i;
      int best = 0;
      for (int c = 1; c < cores; ++c)
        if (load[c] < load[best]) best = c;
      done[pick] = 1;
      s->core[pick] = (uint8_t)best;
      load[best] += util[pick];
    }
  }
}

/* Random draws igen_task_segments() takes for a task with eta GPU segments: the ratio, eta
 * weights of the GPU split (none for a CPU-only task), eta + 1 weights of the CPU split. */
IGEN_FN uint32_t igen_task_draws(int eta) { return 2u * (uint32_t)eta + 2u; }

/* The segments of a task with execution demand E and eta GPU segments, drawn from `rng`:
 * cseg[0 .. eta], gm / ge[0 .. eta-1]. */
IGEN_FN void igen_task_segments(igen_rng_t *rng, int64_t E, int eta, uint64_t ratio_lo,
                                uint64_t ratio_hi, int64_t *cseg, int64_t *gm, int64_t *ge) {
  const uint64_t rho = igen_range(rng, ratio_lo, ratio_hi);
  int64_t G = (int64_t)((rho * (uint64_t)E + (1ULL << 31)) >> 32); /* rho < 2^32, E < 2^31 */
  if (eta == 0) {
    G = 0;
  } else {
    if (G < eta) G = eta;
    if (G > E - eta - 1) G = E - eta - 1;
    igen_split(rng, G, eta, ge, gm); /* 20 % miscellaneous CPU work, 80 % pure GPU work */
  }
  igen_split(rng, E - G, eta + 1, cseg, 0);
}

/* The segments of task i of the state (call for i = 0, 1, ... in order). */
IGEN_FN void igen_segments(igen_state_t *s, int i, int64_t *cseg, int64_t *gm, int64_t *ge) {
  igen_task_segments(&s->rng, s->E[i], s->eta[i], s->ratio_lo, s->ratio_hi, cseg, gm, ge);
}

#endif /* GCAPS_IGEN_H_ */
