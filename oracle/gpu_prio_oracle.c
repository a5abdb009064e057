/*
 * gpu_prio_oracle.c -- CPU oracle of the GCAPS analysis with separate GPU-segment priorities
 * (GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 5.3 and Sec. 6.4).
 *
 * THIS IS TEST INFRASTRUCTURE (see rta_oracle.c): plain, single-threaded, 128-bit integers, no
 * code shared with the CUDA path.
 *
 * Sec. 6.4 changes the analysis of Sec. 6.3 in two places: hp(tau_i) becomes the set of tasks
 * with a higher GPU-segment priority (hpp(tau_i), the same-core tasks of higher CPU priority,
 * stays), and every release jitter uses D_h where Sec. 6.3 uses R_h.  Tasks then no longer
 * depend on each other's response times, so every task is analysed on its own.
 *
 * Sec. 5.3 assigns the GPU priorities after Audsley: priority levels are filled from the lowest
 * upwards; at each level the unassigned tasks are tried from the lowest CPU priority upwards and
 * the first one whose bound meets its deadline, with all other unassigned tasks above it, takes
 * the level.  The order of GPU priorities of tasks on one core must equal their CPU order, so a
 * task is only a candidate while no task of lower CPU priority on its core is unassigned.
 *
 * Readings taken where the paper is silent (parity unpinned beyond the paper's Table 2 verdicts): tasks without GPU
 * segments take part in the assignment like any other; every task gets its own outcome (bound,
 * MISS or ITER_LIMIT; nothing is SKIPPED because nothing depends on an earlier task); when the
 * assignment fails at some level the tasks still unassigned get MISS and GPU priority 0; given
 * GPU priorities that break the same-core rule make the taskset INVALID; a jitter D_h - (C_h +
 * G^m_h) or D_h - G^e_h that would be negative (a task that cannot meet its own deadline) is 0.
 */
#include <stdint.h>

typedef __int128 wide;

#define MAX_TASKS 256
#define MAX_SEGMENTS 65536
#define MAX_TIME (1LL << 40)
#define MAX_CORE ((1LL << 31) - 1)
#define FLAG_BUSY 0x100
#define FLAG_LITERAL 0x200
#define FLAG_ASSIGN 0x400
#define SCHED_NO 0
#define SCHED_YES 1
#define SCHED_INVALID 2
#define WCRT_MISS (-1)
#define WCRT_ITER_LIMIT (-3)
#define WCRT_INVALID (-4)

typedef struct {
  int64_t n_tasks, n_csegs, n_gsegs;
  const int64_t *task_off, *period, *deadline, *priority, *core;
  const int64_t *cseg_off, *cseg_wcet, *gseg_off, *gseg_misc, *gseg_exec;
} oracle_tasksets_t;

static wide ceil_div(wide a, wide b) { return (a + b - 1) / b; }

static int taskset_is_valid(const oracle_tasksets_t *ts, int64_t t, int *range_ok) {
  int64_t a = ts->task_off[t], b = ts->task_off[t + 1];
  *range_ok = !(a < 0 || b < a || b > ts->n_tasks || b - a > MAX_TASKS);
  if (!*range_ok) return 0;
  int ok = 1;
  for (int64_t k = a; k < b; ++k) {
    int64_t c0 = ts->cseg_off[k], c1 = ts->cseg_off[k + 1];
    int64_t g0 = ts->gseg_off[k], g1 = ts->gseg_off[k + 1];
    if (c0 < 0 || c1 < c0 || c1 > ts->n_csegs || c1 - c0 > MAX_SEGMENTS) { ok = 0; continue; }
    if (g0 < 0 || g1 < g0 || g1 > ts->n_gsegs || g1 - g0 > MAX_SEGMENTS) { ok = 0; continue; }
    if (ts->period[k] < 1 || ts->period[k] > MAX_TIME) ok = 0;
    if (ts->deadline[k] < 1 || ts->deadline[k] > ts->period[k]) ok = 0;
    if (ts->core[k] < 0 || ts->core[k] > MAX_CORE) ok = 0;
    for (int64_t j = c0; j < c1; ++j)
      if (ts->cseg_wcet[j] < 0 || ts->cseg_wcet[j] > MAX_TIME) ok = 0;
    for (int64_t j = g0; j < g1; ++j)
      if (ts->gseg_misc[j] < 0 || ts->gseg_misc[j] > MAX_TIME || ts->gseg_exec[j] < 0 ||
          ts->gseg_exec[j] > MAX_TIME)
        ok = 0;
  }
  return ok;
}

typedef struct {
  int n;
  wide C[MAX_TASKS], Gm[MAX_TASKS], Ge[MAX_TASKS], T[MAX_TASKS], D[MAX_TASKS];
  int64_t eta[MAX_TASKS], core[MAX_TASKS];
  int cpu_rank[MAX_TASKS]; /* 0 = highest CPU priority; ties by position */
} model_t;

/* Bound of task i when the tasks flagged in above_gpu[] have a higher GPU-segment priority.
 * Returns the converged bound, WCRT_MISS or WCRT_ITER_LIMIT. */
static int64_t bound_of(const model_t *m, int i, const unsigned char *above_gpu, int busy,
                        int literal, int64_t eps, int64_t iter_cap) {
  const int gi = m->eta[i] > 0;
  /* C_i + G*_i + B^C_i (Sec. 6.3, Lemma 8) */
  const wide base = m->C[i] + m->Gm[i] + m->Ge[i] + 2 * (wide)eps * m->eta[i] + ((wide)m->eta[i] + 1) * eps;
  wide R = base;
  int64_t sweeps = 0;
  for (;;) {
    if (R > m->D[i]) return WCRT_MISS;
    if (sweeps >= iter_cap) return WCRT_ITER_LIMIT;
    sweeps += 1;
    wide next = base;
    for (int h = 0; h < m->n; ++h) {
      if (h == i) continue;
      const int hpp = m->core[h] == m->core[i] && m->cpu_rank[h] < m->cpu_rank[i];
      const int hp_gpu = above_gpu[h] && !hpp; /* hp(tau_i) of Sec. 6.4 without hpp(tau_i) */
      const int gh = m->eta[h] > 0;
      const wide star = 2 * (wide)eps * m->eta[h];
      /* Sec. 6.4: D_h in place of R_h.  The substitution presumes R_h <= D_h; a task whose own
       * execution already exceeds its deadline has no such slack, and its jitter is taken as 0
       * (that task gets MISS on its own account, so the taskset fails either way). */
      wide Jc = m->D[h] - (m->C[h] + m->Gm[h]);
      wide Jg = m->D[h] - m->Ge[h];
      if (Jc < 0) Jc = 0;
      if (Jg < 0) Jg = 0;
      if (!busy) {
        if (hpp && !gh) next += ceil_div(R, m->T[h]) * m->C[h];                              /* Lemma 15 */
        if (hpp && gh) next += ceil_div(R + Jc, m->T[h]) * (m->C[h] + m->Gm[h] + star);      /* Lemma 15 */
        if (hpp && gh && gi) next += ceil_div(R + Jg, m->T[h]) * m->Ge[h];                   /* Lemma 13 */
        if (hp_gpu && gh && gi) next += ceil_div(R + Jg, m->T[h]) * (m->Ge[h] + star);       /* Lemma 13 */
      } else {
        if (hpp) next += ceil_div(R, m->T[h]) * (m->C[h] + m->Gm[h]);                        /* Lemma 12 */
        if (hpp && gh && (gi || !literal)) next += ceil_div(R, m->T[h]) * (m->Ge[h] + star); /* Lemma 10 */
        if (hp_gpu && gh) next += ceil_div(R + Jg, m->T[h]) * (m->Ge[h] + star);             /* Lemmas 10, 11 */
      }
    }
    if (next == R) return (int64_t)R;
    R = next;
  }
}

/*
 * Tasksets [first, first+count).  flags: FLAG_BUSY, FLAG_LITERAL, FLAG_ASSIGN.
 * Without FLAG_ASSIGN gpu_prio_in[k] (larger = higher, ties by position) gives the GPU-segment
 * priorities and out_gpu_prio may be NULL; with it gpu_prio_in is ignored and out_gpu_prio
 * receives levels 1..n (n = highest), 0 for tasks left unassigned.  Returns 0, or -1 on a bad
 * argument.
 */
int oracle_gpu_prio_range(const oracle_tasksets_t *ts, int64_t first, int64_t count, int flags,
                          int64_t eps, int64_t iter_cap, const int64_t *gpu_prio_in,
                          int64_t *out_gpu_prio, int64_t *out_wcrt, uint8_t *out_sched) {
  if (flags & ~(FLAG_BUSY | FLAG_LITERAL | FLAG_ASSIGN)) return -1;
  if (eps < 0 || eps > MAX_TIME) return -1;
  const int busy = (flags & FLAG_BUSY) != 0, literal = (flags & FLAG_LITERAL) != 0;
  const int assign = (flags & FLAG_ASSIGN) != 0;
  if (!assign && !gpu_prio_in) return -1;
  if (assign && !out_gpu_prio) return -1;
  for (int64_t t = first; t < first + count; ++t) {
    int range_ok;
    if (!taskset_is_valid(ts, t, &range_ok)) {
      if (range_ok)
        for (int64_t k = ts->task_off[t]; k < ts->task_off[t + 1]; ++k) {
          out_wcrt[k] = WCRT_INVALID;
          if (out_gpu_prio) out_gpu_prio[k] = 0;
        }
      out_sched[t] = SCHED_INVALID;
      continue;
    }
    const int64_t a = ts->task_off[t];
    model_t m;
    m.n = (int)(ts->task_off[t + 1] - a);
    for (int i = 0; i < m.n; ++i) {
      const int64_t k = a + i;
      m.C[i] = m.Gm[i] = m.Ge[i] = 0;
      for (int64_t j = ts->cseg_off[k]; j < ts->cseg_off[k + 1]; ++j) m.C[i] += ts->cseg_wcet[j];
      for (int64_t j = ts->gseg_off[k]; j < ts->gseg_off[k + 1]; ++j) {
        m.Gm[i] += ts->gseg_misc[j];
        m.Ge[i] += ts->gseg_exec[j];
      }
      m.eta[i] = ts->gseg_off[k + 1] - ts->gseg_off[k];
      m.T[i] = ts->period[k], m.D[i] = ts->deadline[k], m.core[i] = ts->core[k];
    }
    for (int i = 0; i < m.n; ++i) {
      int r = 0;
      for (int q = 0; q < m.n; ++q)
        if (ts->priority[a + q] > ts->priority[a + i] || (ts->priority[a + q] == ts->priority[a + i] && q < i)) r += 1;
      m.cpu_rank[i] = r;
    }
    unsigned char above[MAX_TASKS];
    int sched = SCHED_YES;
    if (!assign) {
      int gpu_rank[MAX_TASKS];
      for (int i = 0; i < m.n; ++i) {
        int r = 0;
        for (int q = 0; q < m.n; ++q)
          if (gpu_prio_in[a + q] > gpu_prio_in[a + i] || (gpu_prio_in[a + q] == gpu_prio_in[a + i] && q < i)) r += 1;
        gpu_rank[i] = r;
      }
      int rule_ok = 1; /* same core: GPU order equals CPU order (Sec. 5.3) */
      for (int i = 0; i < m.n; ++i)
        for (int q = 0; q < m.n; ++q)
          if (m.core[i] == m.core[q] && m.cpu_rank[q] < m.cpu_rank[i] && gpu_rank[q] > gpu_rank[i]) rule_ok = 0;
      if (!rule_ok) {
        for (int i = 0; i < m.n; ++i) out_wcrt[a + i] = WCRT_INVALID;
        out_sched[t] = SCHED_INVALID;
        continue;
      }
      for (int i = 0; i < m.n; ++i) {
        for (int q = 0; q < m.n; ++q) above[q] = gpu_rank[q] < gpu_rank[i];
        const int64_t r = bound_of(&m, i, above, busy, literal, eps, iter_cap);
        out_wcrt[a + i] = r;
        if (out_gpu_prio) out_gpu_prio[a + i] = gpu_prio_in[a + i];
        if (r < 0) sched = SCHED_NO;
      }
    } else {
      unsigned char unassigned[MAX_TASKS];
      for (int i = 0; i < m.n; ++i) unassigned[i] = 1, out_gpu_prio[a + i] = 0, out_wcrt[a + i] = WCRT_MISS;
      for (int level = 1; level <= m.n && sched == SCHED_YES; ++level) {
        int chosen = -1;
        /* candidates from the lowest CPU priority upwards */
        for (int want = m.n - 1; want >= 0 && chosen < 0; --want) {
          int c = -1;
          for (int i = 0; i < m.n; ++i)
            if (unassigned[i] && m.cpu_rank[i] == want) c = i;
          if (c < 0) continue;
          int lowest_on_core = 1;
          for (int q = 0; q < m.n; ++q)
            if (q != c && unassigned[q] && m.core[q] == m.core[c] && m.cpu_rank[q] > m.cpu_rank[c]) lowest_on_core = 0;
          if (!lowest_on_core) continue;
          for (int q = 0; q < m.n; ++q) above[q] = unassigned[q] && q != c;
          const int64_t r = bound_of(&m, c, above, busy, literal, eps, iter_cap);
          if (r >= 0) {
            chosen = c;
            out_wcrt[a + c] = r;
            out_gpu_prio[a + c] = level;
            unassigned[c] = 0;
          }
        }
        if (chosen < 0) sched = SCHED_NO;
      }
    }
    out_sched[t] = (uint8_t)sched;
  }
  return 0;
}
