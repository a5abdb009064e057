/*
 * rta_oracle.c -- plain, single-threaded CPU oracle of the GCAPS / round-robin response-time
 * analysis (GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 6).
 *
 * THIS IS TEST INFRASTRUCTURE.  It defines what the CUDA library must compute and is used only
 * by the tests, by the smoke check and by the benchmark's CPU-baseline leg.  It shares no code
 * with the CUDA path and is never called by it.
 *
 * The method is an iteration (the least fixed point of an integer recurrence), so the oracle is
 * the algorithm itself, step by step, in the paper's notation, one taskset and one task at a
 * time.  All arithmetic is exact: inputs are integer microseconds and every intermediate is
 * held in a 128-bit integer, so nothing can overflow inside the stated input domain.
 *
 * Readings taken where the paper is silent or inconsistent (each is a convention of this
 * build, identical in the CUDA path):
 *   - task-level G^m_i, G^e_i are sums over the task's GPU segments and G_i = G^m_i + G^e_i;
 *   - GCAPS charges tau_i its own C_i + G*_i (Sec. 6.3 folds 2*eps per GPU segment into G_i);
 *   - a larger priority value is a higher priority, ties go to the earlier task;
 *   - iteration: R^0 = base_i, R^{k+1} = base_i + sum of terms evaluated at R^k; stop when
 *     R^{k+1} = R^k (converged) or when an iterate exceeds D_i (deadline miss);
 *   - on the first miss (in priority order) the task gets MISS and all later tasks SKIPPED;
 *     after ITER_CAP sweeps without either outcome the task gets ITER_LIMIT instead;
 *   - without the LITERAL flag: Lemma 7's jitter J^c_h is 0 for a CPU-only tau_h, and
 *     Lemma 10's same-core term is charged to a CPU-only tau_i too;
 *   - Lemma 4's interleaving-set size is nu_i = N_g - |{h in hpp(i): eta^g_h > 0}| + 1 and
 *     Lemma 1's is N_g - 1 (N_g = number of GPU-using tasks of the taskset);
 *   - with FLAG_BEST_EFFORT a task whose priority value is <= 0 is a best-effort task (Table 4
 *     prints priority 0 for the two tasks "not assigned real-time priority"; Sec. 7.1 runs
 *     such tasks "with the lowest priority in the system"): it has no deadline to meet, is
 *     never analysed (BEST_EFFORT in out_wcrt) and, being below every real-time task, is in
 *     no hp() or hpp(); it still shares the time-sliced GPU under round robin, so it counts
 *     in N_g (Lemma 1, Lemma 4).  Under GCAPS it is preempted at once and adds nothing.
 * Parity unpinned: the sentinel convention, the iteration cap and the two repaired forms are
 * not fixed by the paper; the tests pin them only through hand-derived vectors.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef __int128 wide;

#define MAX_TASKS 256
#define MAX_SEGMENTS 65536
#define MAX_TIME (1LL << 40)
#define MAX_CORE ((1LL << 31) - 1)

#define POLICY_GCAPS 0
#define POLICY_RR 1
#define FLAG_BUSY 0x100
#define FLAG_LITERAL 0x200
#define FLAG_BEST_EFFORT 0x800

#define SCHED_NO 0
#define SCHED_YES 1
#define SCHED_INVALID 2
#define WCRT_MISS (-1)
#define WCRT_SKIPPED (-2)
#define WCRT_ITER_LIMIT (-3)
#define WCRT_INVALID (-4)
#define WCRT_BEST_EFFORT (-5)

typedef struct {
  int64_t n_tasks, n_csegs, n_gsegs;
  const int64_t *task_off, *period, *deadline, *priority, *core;
  const int64_t *cseg_off, *cseg_wcet, *gseg_off, *gseg_misc, *gseg_exec;
} oracle_tasksets_t;

typedef struct {
  int64_t sweeps; /* evaluations of the right-hand side of Eq. 1 (one per iterate)            */
  int64_t terms;  /* ceil((R+J)/T_h)*W products evaluated                                      */
  int64_t tasks;  /* tasks whose recurrence was started                                        */
} oracle_counts_t;

static wide ceil_div(wide a, wide b) { return (a + b - 1) / b; } /* a >= 0, b > 0 */

/* Domain check of one taskset (the task model of Sec. 4 with D_i <= T_i).  Returns a bit mask:
 * 1 task range, 2 segment range, 4 period, 8 deadline, 16 core, 32 WCET; 0 = valid. */
static int check_taskset(const oracle_tasksets_t *ts, int64_t t) {
  int64_t a = ts->task_off[t], b = ts->task_off[t + 1];
  if (a < 0 || b < a || b > ts->n_tasks || b - a > MAX_TASKS) return 1;
  int bad = 0;
  for (int64_t k = a; k < b; ++k) {
    int64_t c0 = ts->cseg_off[k], c1 = ts->cseg_off[k + 1];
    int64_t g0 = ts->gseg_off[k], g1 = ts->gseg_off[k + 1];
    int seg_ok = 1;
    if (c0 < 0 || c1 < c0 || c1 > ts->n_csegs || c1 - c0 > MAX_SEGMENTS) seg_ok = 0;
    if (g0 < 0 || g1 < g0 || g1 > ts->n_gsegs || g1 - g0 > MAX_SEGMENTS) seg_ok = 0;
    if (!seg_ok) bad |= 2;
    if (ts->period[k] < 1 || ts->period[k] > MAX_TIME) bad |= 4;
    if (ts->deadline[k] < 1 || ts->deadline[k] > ts->period[k]) bad |= 8;
    if (ts->core[k] < 0 || ts->core[k] > MAX_CORE) bad |= 16;
    if (seg_ok) {
      for (int64_t j = c0; j < c1; ++j)
        if (ts->cseg_wcet[j] < 0 || ts->cseg_wcet[j] > MAX_TIME) bad |= 32;
      for (int64_t j = g0; j < g1; ++j) {
        if (ts->gseg_misc[j] < 0 || ts->gseg_misc[j] > MAX_TIME) bad |= 32;
        if (ts->gseg_exec[j] < 0 || ts->gseg_exec[j] > MAX_TIME) bad |= 32;
      }
    }
  }
  return bad;
}

/*
 * Analyses taskset t.  Writes out_wcrt[task_off[t] .. task_off[t+1]) and returns the
 * schedulable flag.  L = TSG time-slice length (Eq. 3), ovh = theta for RR (Def. 1) and
 * epsilon for GCAPS (Def. 2).
 */
static int analyse_taskset(const oracle_tasksets_t *ts, int64_t t, int policy_flags, int64_t L,
                           int64_t ovh, int64_t iter_cap, int64_t *out_wcrt,
                           oracle_counts_t *cnt) {
  const int policy = policy_flags & 0xff;
  const int busy = (policy_flags & FLAG_BUSY) != 0;
  const int literal = (policy_flags & FLAG_LITERAL) != 0;
  const int best_effort = (policy_flags & FLAG_BEST_EFFORT) != 0;

  int bad = check_taskset(ts, t);
  if (bad) {
    if (!(bad & 1))
      for (int64_t k = ts->task_off[t]; k < ts->task_off[t + 1]; ++k) out_wcrt[k] = WCRT_INVALID;
    return SCHED_INVALID;
  }
  const int64_t first = ts->task_off[t];
  const int n = (int)(ts->task_off[t + 1] - first);

  /* ---- task-level quantities (Sec. 4): C_i, G^m_i, G^e_i, eta^g_i; RR slice count --------- */
  wide C[MAX_TASKS], Gm[MAX_TASKS], Ge[MAX_TASKS], slices[MAX_TASKS];
  int64_t eta[MAX_TASKS];
  int n_gpu = 0; /* N_g */
  for (int i = 0; i < n; ++i) {
    int64_t k = first + i;
    C[i] = Gm[i] = Ge[i] = slices[i] = 0;
    for (int64_t j = ts->cseg_off[k]; j < ts->cseg_off[k + 1]; ++j) C[i] += ts->cseg_wcet[j];
    for (int64_t j = ts->gseg_off[k]; j < ts->gseg_off[k + 1]; ++j) {
      Gm[i] += ts->gseg_misc[j];
      Ge[i] += ts->gseg_exec[j];
      if (policy == POLICY_RR) slices[i] += ceil_div(ts->gseg_exec[j], L); /* Eq. 3 */
    }
    eta[i] = ts->gseg_off[k + 1] - ts->gseg_off[k];
    if (eta[i] > 0) n_gpu += 1;
  }

  /* ---- priority order: larger pi first, ties by position --------------------------------- */
  int order[MAX_TASKS];
  for (int i = 0; i < n; ++i) order[i] = i;
  for (int a = 1; a < n; ++a) { /* stable insertion sort, descending priority */
    int x = order[a], b = a - 1;
    while (b >= 0 && ts->priority[first + order[b]] < ts->priority[first + x]) {
      order[b + 1] = order[b];
      b -= 1;
    }
    order[b + 1] = x;
  }

  wide R[MAX_TASKS]; /* converged response times of already analysed (higher-priority) tasks */
  int sched = SCHED_YES;
  for (int pos = 0; pos < n; ++pos) {
    const int i = order[pos];
    const int64_t k = first + i;
    if (best_effort && ts->priority[k] <= 0) { /* not a real-time task: nothing to bound */
      out_wcrt[k] = WCRT_BEST_EFFORT;
      continue;
    }
    if (sched != SCHED_YES) {
      out_wcrt[k] = WCRT_SKIPPED;
      continue;
    }
    const int gi = eta[i] > 0;
    const wide Di = ts->deadline[k];

    /* ---- the part of Eq. 1 that does not depend on R ---------------------------------- */
    wide base;
    wide nu_busy = 0; /* Lemma 4's interleaving-set size for this tau_i */
    if (policy == POLICY_GCAPS) {
      /* C_i + G*_i (Sec. 6.3) + B^C_i (Lemma 8); I^ie_i = 0 (Lemma 9) */
      base = C[i] + (Gm[i] + Ge[i] + 2 * (wide)ovh * eta[i]) + ((wide)eta[i] + 1) * ovh;
    } else {
      /* C_i + G_i + I^ie_i (Lemma 1, Eq. 3); I^dp_i = 0 (Lemma 2), B^C_i = 0 (Lemma 3) */
      wide I_ie = gi ? ((wide)L + ovh) * (n_gpu - 1) * slices[i] : 0;
      base = C[i] + Gm[i] + Ge[i] + I_ie;
      int hpp_gpu = 0;
      for (int q = 0; q < pos; ++q) {
        int h = order[q];
        if (ts->core[first + h] == ts->core[k] && eta[h] > 0) hpp_gpu += 1;
      }
      nu_busy = n_gpu - hpp_gpu + 1;
    }

    cnt->tasks += 1;
    wide Rcur = base;
    int64_t verdict = 0; /* 0 = converged */
    int64_t sweeps = 0;
    for (;;) {
      if (Rcur > Di) {
        verdict = WCRT_MISS;
        break;
      }
      if (sweeps >= iter_cap) {
        verdict = WCRT_ITER_LIMIT;
        break;
      }
      sweeps += 1;
      cnt->sweeps += 1;
      wide next = base;
      for (int q = 0; q < pos; ++q) { /* tau_h in hp(tau_i) */
        const int h = order[q];
        const int64_t kh = first + h;
        const wide Th = ts->period[kh];
        const int same = ts->core[kh] == ts->core[k]; /* tau_h in hpp(tau_i) */
        const int gh = eta[h] > 0;
        const wide Jc = R[h] - (C[h] + Gm[h]); /* Lemma 7 / Lemma 15 */
        const wide Jg = R[h] - Ge[h];          /* Lemma 10 */
        const wide star = 2 * (wide)ovh * eta[h];
        if (policy == POLICY_GCAPS && !busy) {
          if (same && !gh) { /* Lemma 15, first sum */
            next += ceil_div(Rcur, Th) * C[h];
            cnt->terms += 1;
          }
          if (same && gh) { /* Lemma 15, second sum */
            next += ceil_div(Rcur + Jc, Th) * (C[h] + Gm[h] + star);
            cnt->terms += 1;
          }
          if (same && gh && gi) { /* Lemma 13, first sum */
            next += ceil_div(Rcur + Jg, Th) * Ge[h];
            cnt->terms += 1;
          }
          if (!same && gh && gi) { /* Lemma 13, second sum */
            next += ceil_div(Rcur + Jg, Th) * (Ge[h] + star);
            cnt->terms += 1;
          }
          /* I^id_i = 0 (Lemma 14) */
        } else if (policy == POLICY_GCAPS && busy) {
          if (same) { /* Lemma 12 */
            next += ceil_div(Rcur, Th) * (C[h] + Gm[h]);
            cnt->terms += 1;
          }
          if (same && gh && (gi || !literal)) { /* Lemma 10, first sum */
            next += ceil_div(Rcur, Th) * (Ge[h] + star);
            cnt->terms += 1;
          }
          if (!same && gh) { /* Lemma 10 second sum (gi) / Lemma 11 (not gi) */
            next += ceil_div(Rcur + Jg, Th) * (Ge[h] + star);
            cnt->terms += 1;
          }
        } else if (policy == POLICY_RR && !busy) {
          if (same) { /* Lemma 7; I^id_i = 0 (Lemma 6) */
            wide J = (gh || literal) ? Jc : 0;
            next += ceil_div(Rcur + J, Th) * (C[h] + Gm[h]);
            cnt->terms += 1;
          }
        } else {
          if (same) { /* Lemma 5 plus, for a GPU-using tau_h, Lemma 4 */
            wide W = C[h] + Gm[h];
            if (gh) W += ((wide)L + ovh) * nu_busy * slices[h];
            next += ceil_div(Rcur, Th) * W;
            cnt->terms += 1;
          }
        }
      }
      if (next == Rcur) break; /* least fixed point reached */
      Rcur = next;
    }
    if (verdict == 0) {
      R[i] = Rcur;
      out_wcrt[k] = (int64_t)Rcur;
    } else {
      out_wcrt[k] = verdict;
      sched = SCHED_NO;
    }
  }
  return sched;
}

/* ---- exported entry points --------------------------------------------------------------- */

/* Analyses tasksets [first, first+count).  out_wcrt is indexed like the per-task arrays,
 * out_sched like the tasksets (absolute indices).  counts may be NULL.  Returns 0, or -1 on
 * an argument outside the domain of the analysis constants. */
int oracle_rta_range(const oracle_tasksets_t *ts, int64_t first, int64_t count, int policy_flags,
                     int64_t L, int64_t ovh, int64_t iter_cap, int64_t *out_wcrt,
                     uint8_t *out_sched, oracle_counts_t *counts) {
  const int policy = policy_flags & 0xff;
  if (policy != POLICY_GCAPS && policy != POLICY_RR) return -1;
  if (policy_flags & ~(0xff | FLAG_BUSY | FLAG_LITERAL | FLAG_BEST_EFFORT)) return -1;
  if (ovh < 0 || ovh > MAX_TIME) return -1;
  if (policy == POLICY_RR && (L < 1 || L > MAX_TIME)) return -1;
  oracle_counts_t local = {0, 0, 0};
  for (int64_t t = first; t < first + count; ++t)
    out_sched[t] = (uint8_t)analyse_taskset(ts, t, policy_flags, L, ovh, iter_cap, out_wcrt, &local);
  if (counts) *counts = local;
  return 0;
}

/* Domain check only: out_err[t] = bit mask (0 = valid). */
void oracle_validate_range(const oracle_tasksets_t *ts, int64_t first, int64_t count,
                           int32_t *out_err) {
  for (int64_t t = first; t < first + count; ++t) out_err[t] = check_taskset(ts, t);
}
