/*
 * des_sim.c -- tick-level discrete-event simulator of one taskset on omega CPU cores and one
 * GPU.  TEST INFRASTRUCTURE ONLY: it exists to check that the analytic bounds of the oracle are
 * never exceeded by an observed schedule on tiny tasksets.  It contains no response-time
 * analysis and shares no code with it.
 *
 * Model (paper Sec. 4 and Sec. 2/5.1, overheads epsilon = theta = 0):
 *   - every task releases jobs strictly periodically from a given offset; a job executes its
 *     segments in order  C_{i,1}, (G^m_{i,1}, G^e_{i,1}), C_{i,2}, ...  (CPU segment, then for
 *     each GPU segment its miscellaneous CPU part followed by its pure GPU part);
 *   - CPU: partitioned, preemptive, fixed priority per core.  C and G^m parts need the CPU.
 *     During a pure GPU part the job either keeps competing for its core although it has no
 *     CPU work to do (busy-waiting) or leaves the core (self-suspension);
 *   - GPU, GCAPS policy: the pending pure-GPU part of the highest-priority job owns the GPU,
 *     preemptively (the priority rule of the paper's Alg. 1 applied to real-time tasks);
 *   - GPU, RR policy: pending pure-GPU parts are served round robin in task-index order with a
 *     time slice of L ticks; the policy is work-conserving (an idle entry is skipped at once);
 *   - one tick = one time unit; decisions are taken at tick boundaries.
 * A job that is still running when the next job of its task is released delays that next job
 * (releases queue up); response times are measured from the nominal release instant.
 */
#include <stdint.h>
#include <string.h>

#define SIM_MAX_TASKS 16
#define SIM_MAX_PHASES 64

typedef struct {
  int n_phase;
  int kind[SIM_MAX_PHASES];    /* 0 = needs CPU, 1 = pure GPU */
  int64_t len[SIM_MAX_PHASES];
} job_shape_t;

/*
 * n tasks; per task: T, prio (larger = higher, ties by index), gpu_prio (the priority of the
 * task's GPU segments under the GCAPS policy, Sec. 5.3), core, offset, and the CSR segment
 * arrays restricted to this taskset (cseg_off/gseg_off have n+1 entries, relative to the given
 * cseg/gm/ge arrays).  policy 0 = GCAPS, 1 = RR; busy 0/1; L = RR slice in ticks.
 * Simulates ticks [0, horizon).  max_resp[i] receives the largest response time of a job of
 * task i that COMPLETED inside the horizon (0 if none), unfinished[i] the age of a job still
 * running at the horizon (0 if none).  Returns 0, or -1 if the taskset does not fit the limits.
 */
int des_simulate_gp(int n, const int64_t *T, const int64_t *prio, const int64_t *gpu_prio,
                    const int64_t *core, const int64_t *offset, const int64_t *cseg_off,
                    const int64_t *cseg, const int64_t *gseg_off, const int64_t *gm,
                    const int64_t *ge, int policy, int busy, int64_t L, int64_t horizon,
                    int64_t *max_resp, int64_t *unfinished) {
  if (n < 1 || n > SIM_MAX_TASKS) return -1;
  job_shape_t shape[SIM_MAX_TASKS];
  for (int i = 0; i < n; ++i) {
    int nc = (int)(cseg_off[i + 1] - cseg_off[i]);
    int ng = (int)(gseg_off[i + 1] - gseg_off[i]);
    int p = 0;
    int steps = nc > ng + 1 ? nc : ng + 1;
    if (2 * ng + nc + 2 > SIM_MAX_PHASES) return -1;
    /* interleave: C_1, (Gm_1, Ge_1), C_2, (Gm_2, Ge_2), ... ; surplus segments keep the order */
    for (int s = 0; s < steps; ++s) {
      if (s < nc) shape[i].kind[p] = 0, shape[i].len[p++] = cseg[cseg_off[i] + s];
      if (s < ng) {
        shape[i].kind[p] = 0, shape[i].len[p++] = gm[gseg_off[i] + s];
        shape[i].kind[p] = 1, shape[i].len[p++] = ge[gseg_off[i] + s];
      }
    }
    shape[i].n_phase = p;
  }
  int active[SIM_MAX_TASKS];      /* a job of the task is in progress                         */
  int phase[SIM_MAX_TASKS];
  int64_t rem[SIM_MAX_TASKS];     /* remaining length of the current phase                    */
  int64_t rel[SIM_MAX_TASKS];     /* nominal release of the job in progress                   */
  int64_t next_rel[SIM_MAX_TASKS];
  int64_t backlog[SIM_MAX_TASKS]; /* released jobs not yet started                            */
  for (int i = 0; i < n; ++i) {
    active[i] = 0, phase[i] = 0, rem[i] = 0, rel[i] = 0, backlog[i] = 0;
    next_rel[i] = offset[i];
    max_resp[i] = 0, unfinished[i] = 0;
  }
  int rr_cur = -1;
  int64_t rr_left = 0;

  for (int64_t now = 0; now < horizon; ++now) {
    /* releases, and start of queued jobs */
    for (int i = 0; i < n; ++i) {
      if (now == next_rel[i]) {
        backlog[i] += 1;
        next_rel[i] += T[i];
      }
    }
    for (int i = 0; i < n; ++i) {
      for (;;) {
        if (!active[i]) {
          if (backlog[i] == 0) break;
          backlog[i] -= 1;
          active[i] = 1;
          phase[i] = 0;
          rel[i] = next_rel[i] - T[i] * (backlog[i] + 1);
          rem[i] = shape[i].len[0];
        }
        /* skip empty phases; complete the job if nothing is left */
        while (phase[i] < shape[i].n_phase && rem[i] == 0) {
          phase[i] += 1;
          if (phase[i] < shape[i].n_phase) rem[i] = shape[i].len[phase[i]];
        }
        if (phase[i] < shape[i].n_phase) break;
        int64_t resp = now - rel[i];
        if (resp > max_resp[i]) max_resp[i] = resp;
        active[i] = 0;
      }
    }
    /* GPU arbitration among pending pure-GPU parts */
    int gpu_owner = -1;
    if (policy == 0) {
      for (int i = 0; i < n; ++i) {
        if (!active[i] || shape[i].kind[phase[i]] != 1) continue;
        if (gpu_owner < 0 || gpu_prio[i] > gpu_prio[gpu_owner]) gpu_owner = i;
      }
    } else {
      int cur_ready = rr_cur >= 0 && active[rr_cur] && shape[rr_cur].kind[phase[rr_cur]] == 1;
      if (!cur_ready || rr_left == 0) {
        int start = rr_cur < 0 ? 0 : rr_cur + 1, found = -1;
        for (int s = 0; s < n; ++s) {
          int i = (start + s) % n;
          if (active[i] && shape[i].kind[phase[i]] == 1) {
            found = i;
            break;
          }
        }
        if (found >= 0) rr_cur = found, rr_left = L;
        else rr_cur = -1, rr_left = 0;
      }
      gpu_owner = rr_cur;
    }
    /* CPU arbitration per core */
    int cpu_owner[SIM_MAX_TASKS];
    for (int i = 0; i < n; ++i) cpu_owner[i] = 0;
    for (int i = 0; i < n; ++i) {
      if (!active[i]) continue;
      int wants = shape[i].kind[phase[i]] == 0 || busy;
      if (!wants) continue;
      int best = 1;
      for (int k = 0; k < n; ++k) {
        if (k == i || !active[k] || core[k] != core[i]) continue;
        int kw = shape[k].kind[phase[k]] == 0 || busy;
        if (kw && (prio[k] > prio[i] || (prio[k] == prio[i] && k < i))) best = 0;
      }
      cpu_owner[i] = best;
    }
    /* advance one tick */
    for (int i = 0; i < n; ++i) {
      if (!active[i]) continue;
      if (shape[i].kind[phase[i]] == 0) {
        if (cpu_owner[i]) rem[i] -= 1;
      } else if (gpu_owner == i) {
        rem[i] -= 1;
        if (policy == 1) rr_left -= 1;
      }
    }
  }
  for (int i = 0; i < n; ++i) {
    if (active[i]) unfinished[i] = horizon - rel[i];
    else if (backlog[i] > 0) unfinished[i] = horizon - (next_rel[i] - T[i] * backlog[i]);
  }
  return 0;
}

/* The same with the GPU arbitrated by the tasks' CPU priorities. */
int des_simulate(int n, const int64_t *T, const int64_t *prio, const int64_t *core,
                 const int64_t *offset, const int64_t *cseg_off, const int64_t *cseg,
                 const int64_t *gseg_off, const int64_t *gm, const int64_t *ge, int policy,
                 int busy, int64_t L, int64_t horizon, int64_t *max_resp, int64_t *unfinished) {
  return des_simulate_gp(n, T, prio, prio, core, offset, cseg_off, cseg, gseg_off, gm, ge, policy,
                         busy, L, horizon, max_resp, unfinished);
}

/*
 * Brute force over release offsets: simulates the taskset once for EVERY offset vector
 * (o_0, ..., o_{n-1}) with o_i in {0, step, 2*step, ...} below T_i, each run over two
 * hyperperiods past the largest offset (hyper = lcm of the periods, passed in), and returns per
 * task the largest response time seen in any run, a job still unfinished at a horizon counting
 * with its age.  n_runs receives the number of offset vectors tried.  Arguments otherwise as
 * des_simulate_gp.  Returns 0, or -1 if a run does not fit the simulator's limits.
 */
int des_sweep_offsets(int n, const int64_t *T, const int64_t *prio, const int64_t *gpu_prio,
                      const int64_t *core, const int64_t *cseg_off, const int64_t *cseg,
                      const int64_t *gseg_off, const int64_t *gm, const int64_t *ge, int policy,
                      int busy, int64_t L, int64_t step, int64_t hyper, int64_t *worst,
                      int64_t *n_runs) {
  if (n < 1 || n > SIM_MAX_TASKS || step < 1) return -1;
  int64_t off[SIM_MAX_TASKS], resp[SIM_MAX_TASKS], unfinished[SIM_MAX_TASKS];
  for (int i = 0; i < n; ++i) off[i] = 0, worst[i] = 0;
  *n_runs = 0;
  for (;;) {
    int64_t max_off = 0;
    for (int i = 0; i < n; ++i)
      if (off[i] > max_off) max_off = off[i];
    if (des_simulate_gp(n, T, prio, gpu_prio, core, off, cseg_off, cseg, gseg_off, gm, ge, policy,
                        busy, L, 2 * hyper + max_off + 1, resp, unfinished) != 0)
      return -1;
    *n_runs += 1;
    for (int i = 0; i < n; ++i) {
      if (resp[i] > worst[i]) worst[i] = resp[i];
      if (unfinished[i] > worst[i]) worst[i] = unfinished[i];
    }
    int i = 0; /* next offset vector, first task fastest */
    while (i < n) {
      off[i] += step;
      if (off[i] < T[i]) break;
      off[i] = 0;
      i += 1;
    }
    if (i == n) break;
  }
  return 0;
}
