/*
 * gcaps_rta.h -- C ABI of the batched worst-case response-time analysis (RTA) library
 * for GPU-using real-time tasksets (GCAPS, ECRTS 2024, arXiv 2406.05221).
 *
 * One call analyses n_tasksets independent tasksets on one NVIDIA B200 (sm_100a).  For every
 * taskset it walks the tasks in decreasing priority and solves the integer fixed-point
 * response-time recurrence of the paper's Sec. 6 (Eq. 1, Eq. 2, Eq. 4 with the lemma set of
 * the chosen analysis), and writes one worst-case response time (WCRT) per task and one
 * schedulable flag per taskset.
 *
 * All times are integer microseconds held as int64_t.  Nothing in this header is a torch type;
 * device buffers are plain device pointers owned by the caller.
 *
 * Host threads.  Every entry point may be called from several host threads at once.  The calls
 * that work on device buffers keep no state between calls apart from per-device constants that
 * are looked up once under a lock; concurrent calls must use different workspaces (and, to
 * overlap on the GPU, different streams).  The host-buffer calls (gcaps_rta_batch_host,
 * gcaps_rta_batch_host_multi, gcaps_rta_release_host) share one set of staging buffers and are
 * serialised by a lock: a second thread waits until the first one's call has returned.
 *
 * Stream order.  The work of a call is complete, for everything enqueued on the same stream
 * afterwards, when the stream reaches that later work: a copy of the results, a kernel reading
 * them or the next call may follow without any host synchronisation.
 */
#ifndef GCAPS_RTA_H_
#define GCAPS_RTA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GCAPS_RTA_VERSION 100 /* major*100 + minor */

/* ---- limits of the input domain ------------------------------------------------------------ */
#define GCAPS_RTA_MAX_TASKS 256              /* tasks per taskset                                */
#define GCAPS_RTA_MAX_SEGMENTS 65536         /* CPU segments, and GPU segments, per task         */
#define GCAPS_RTA_MAX_TIME (1LL << 40)       /* every period, deadline, WCET, L and overhead     */
#define GCAPS_RTA_MAX_CORE ((1LL << 31) - 1) /* CPU core ids are 0 .. MAX_CORE                   */
#define GCAPS_RTA_ITER_CAP (1LL << 20)       /* fixed-point sweeps per task before ITER_LIMIT    */

/* ---- policy argument ------------------------------------------------------------------------
 * Low byte: the GPU arbitration policy that is analysed.
 *   GCAPS_POLICY_GCAPS  preemptive priority-based GPU context scheduling (Sec. 6.3, Lemmas 8-15)
 *   GCAPS_POLICY_RR     default work-conserving round-robin time-sliced driver (Sec. 6.2,
 *                       Lemmas 1-7)
 * OR-able flags:
 *   GCAPS_RTA_BUSY      tasks busy-wait on the CPU during pure GPU execution (the "busy-waiting
 *                       mode" lemmas); without it tasks self-suspend (the "self-suspension mode"
 *                       lemmas).
 *   GCAPS_RTA_LITERAL   evaluate the lemmas exactly as printed.  Without it two printed forms
 *                       are repaired: (a) RR self-suspension, Lemma 7: the jitter J^c_h is taken
 *                       as 0 for a CPU-only tau_h (a task without GPU segments never suspends);
 *                       (b) GCAPS busy-waiting, Lemma 10: the busy-wait G^{e*}_h of a same-core
 *                       GPU-using tau_h is charged to tau_i also when tau_i is CPU-only.
 *   GCAPS_RTA_BEST_EFFORT  tasks whose priority value is <= 0 are best-effort tasks: tasks
 *                       without a real-time priority that run below every real-time task (the
 *                       last experiment of Sec. 7.1; Table 4 prints priority 0 for them).  Such a
 *                       task has no deadline to meet: it is not analysed, gets
 *                       GCAPS_WCRT_BEST_EFFORT and never makes a taskset unschedulable.  It
 *                       interferes with no real-time task on the CPU, nor on the GPU under GCAPS
 *                       (it is preempted at once); under round robin it takes its turns on the
 *                       time-sliced GPU like any GPU-using task, i.e. it counts in the number of
 *                       GPU-using tasks of Lemma 1 and Lemma 4.  Real-time tasks then need
 *                       priorities > 0.  Without the flag a value <= 0 is an ordinary priority.
 */
#define GCAPS_POLICY_GCAPS 0
#define GCAPS_POLICY_RR 1
#define GCAPS_RTA_BUSY 0x100
#define GCAPS_RTA_LITERAL 0x200
#define GCAPS_RTA_ASSIGN 0x400 /* only for gcaps_rta_gpu_priority_batch: search the GPU priorities */
#define GCAPS_RTA_BEST_EFFORT 0x800 /* not accepted by gcaps_rta_gpu_priority_batch */

/* ---- values written to out_sched[t] --------------------------------------------------------- */
#define GCAPS_SCHED_NO 0      /* some task's bound exceeds its deadline (or hit ITER_LIMIT)      */
#define GCAPS_SCHED_YES 1     /* every task converged to R_i <= D_i (an empty taskset is YES)    */
#define GCAPS_SCHED_INVALID 2 /* the taskset is outside the input domain; nothing was analysed   */

/* ---- sentinels written to out_wcrt[k] (all negative; a converged bound is >= 0) ------------- */
#define GCAPS_WCRT_MISS (-1)       /* first task, in priority order, whose iterate exceeded D_i  */
#define GCAPS_WCRT_SKIPPED (-2)    /* every task after the first MISS / ITER_LIMIT in that order */
#define GCAPS_WCRT_ITER_LIMIT (-3) /* GCAPS_RTA_ITER_CAP sweeps without convergence or miss      */
#define GCAPS_WCRT_INVALID (-4)    /* task of an INVALID taskset (when its slot is addressable)  */
#define GCAPS_WCRT_BEST_EFFORT (-5) /* best-effort task (GCAPS_RTA_BEST_EFFORT): not analysed    */

/* ---- return codes ---------------------------------------------------------------------------- */
#define GCAPS_OK 0
#define GCAPS_ERR_INVALID_ARG (-1)   /* null pointer, negative count, unknown policy bits, L<=0
                                        for RR, overhead<0, a time argument above MAX_TIME      */
#define GCAPS_ERR_WORKSPACE (-2)     /* workspace null or smaller than gcaps_rta_workspace_bytes */
#define GCAPS_ERR_CUDA (-3)          /* a CUDA runtime call failed; see gcaps_rta_last_cuda_error */
#define GCAPS_ERR_NO_DEVICE (-4)     /* no CUDA device / not an sm_100 device                    */
#define GCAPS_ERR_TOO_LARGE (-5)     /* batch larger than GCAPS_RTA_STATIC_MAX_TASKSETS (only
                                        returned by gcaps_rta_batch_static)                     */

/*
 * A batch of tasksets in CSR structure-of-arrays form (task model: Sec. 4).
 *
 * Taskset t owns tasks task_off[t] .. task_off[t+1]-1 of the per-task arrays.  Task k owns CPU
 * segments cseg_off[k] .. cseg_off[k+1]-1 (eta^c_k of them) and GPU segments gseg_off[k] ..
 * gseg_off[k+1]-1 (eta^g_k of them; none for a CPU-only task).  GPU segment j of a task is the
 * pair (G^m = gseg_misc[j], G^e = gseg_exec[j]): miscellaneous CPU work and pure GPU work.
 * The task-level quantities of the paper are sums over the task's segments:
 *   C_i = sum cseg_wcet,  G^m_i = sum gseg_misc,  G^e_i = sum gseg_exec,  G_i = G^m_i + G^e_i.
 * A larger priority value means a higher priority; equal priorities are ordered by position
 * (the earlier task is the higher one).  The order of tasks inside a taskset is free.
 *
 * Every pointer of one struct is either a device pointer (gcaps_rta_batch, gcaps_rta_validate)
 * or a host pointer (gcaps_rta_batch_host).  The library only reads these arrays and keeps no
 * pointer after the call's work has completed.
 *
 * Domain of a valid taskset: 0 <= n <= GCAPS_RTA_MAX_TASKS tasks; offsets non-decreasing and
 * inside [0, n_tasks], [0, n_csegs], [0, n_gsegs]; at most GCAPS_RTA_MAX_SEGMENTS segments of a
 * kind per task; 1 <= D_i <= T_i <= GCAPS_RTA_MAX_TIME; 0 <= core <= GCAPS_RTA_MAX_CORE; every
 * segment WCET in [0, GCAPS_RTA_MAX_TIME].
 */
typedef struct gcaps_tasksets {
  int64_t n_tasks;          /* length of the per-task arrays (= task_off[n_tasksets])            */
  int64_t n_csegs;          /* length of cseg_wcet (= cseg_off[n_tasks])                         */
  int64_t n_gsegs;          /* length of gseg_misc and gseg_exec (= gseg_off[n_tasks])           */
  const int64_t *task_off;  /* [n_tasksets+1]                                                    */
  const int64_t *period;    /* [n_tasks]   T_i                                                   */
  const int64_t *deadline;  /* [n_tasks]   D_i                                                   */
  const int64_t *priority;  /* [n_tasks]   pi_i, larger = higher                                 */
  const int64_t *core;      /* [n_tasks]   CPU core the task is partitioned to                   */
  const int64_t *cseg_off;  /* [n_tasks+1]                                                       */
  const int64_t *cseg_wcet; /* [n_csegs]   C_{i,k}                                               */
  const int64_t *gseg_off;  /* [n_tasks+1]                                                       */
  const int64_t *gseg_misc; /* [n_gsegs]   G^m_{i,j}                                             */
  const int64_t *gseg_exec; /* [n_gsegs]   G^e_{i,j}                                             */
} gcaps_tasksets_t;

/*
 * gcaps_rta_batch -- response-time analysis of a device-resident batch (Sec. 6: Eq. 1-4 and
 * Lemmas 1-15; the fixed-point iteration is implied by R_i appearing on both sides of Eq. 1).
 *
 *   ts                      host struct whose pointers are DEVICE pointers (see above)
 *   n_tasksets              number of tasksets, >= 0 (0 is a no-op)
 *   policy                  GCAPS_POLICY_* | flags
 *   timeslice_us            L of Eq. 3; used by RR only, must be 1..MAX_TIME there
 *   ctx_switch_overhead_us  theta (Def. 1) for RR, epsilon = alpha + theta (Def. 2) for GCAPS;
 *                           0..MAX_TIME
 *   out_wcrt                DEVICE, [ts->n_tasks]: converged R_i, or a GCAPS_WCRT_* sentinel;
 *                           indexed like the per-task input arrays
 *   out_sched               DEVICE, [n_tasksets]: GCAPS_SCHED_*
 *   workspace               DEVICE scratch of at least gcaps_rta_workspace_bytes() bytes, 256-byte
 *                           aligned, caller-owned; contents are undefined afterwards.  It holds
 *                           the size-binned launch plan (a permutation of taskset indices).
 *   stream                  a cudaStream_t passed as void* (NULL = the default stream)
 *
 * For task i of a taskset, in decreasing priority:  R <- base_i;  repeat  R' <- base_i +
 * sum over interfering (J, W, T_h) of ceil((R + J) / T_h) * W  until R' = R (converged, R_i = R)
 * or R > D_i (MISS).  After the first MISS or ITER_LIMIT the remaining tasks are SKIPPED.
 *
 * Asynchronous: the work is enqueued on `stream`; no host synchronisation, no allocation.
 * Returns GCAPS_OK or a negative GCAPS_ERR_* (nothing is enqueued on an argument error).
 * Tasksets outside the input domain get GCAPS_SCHED_INVALID; the kernels never trap on them.
 */
int gcaps_rta_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                    int64_t timeslice_us, int64_t ctx_switch_overhead_us, int64_t *out_wcrt,
                    uint8_t *out_sched, void *workspace, size_t workspace_bytes, void *stream);

/*
 * gcaps_rta_workspace_bytes -- size of the scratch buffer gcaps_rta_batch needs for a batch of
 * n_tasksets tasksets (a pure host computation; 0 for a negative count).
 */
size_t gcaps_rta_workspace_bytes(int64_t n_tasksets);

/*
 * gcaps_rta_batch_host -- the same analysis for a batch held in HOST memory (task model: Sec. 4;
 * analysis: Sec. 6).  `ts` holds host pointers, out_wcrt / out_sched are host arrays.  The call
 * copies the inputs to the device in chunks of whole tasksets, runs gcaps_rta_batch on each
 * chunk, copies the results back and returns after everything has completed.  Device staging
 * memory is allocated on first use, grown on demand and kept until gcaps_rta_release_host();
 * page-locked host buffers give the best transfer rate but are not required.  On an error return
 * nothing of the call is still in flight: the caller's arrays may be freed at once (results of
 * chunks that had completed may have been written).  One host-buffer call runs at a time per
 * process; calls from other threads wait.
 */
int gcaps_rta_batch_host(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                         int64_t timeslice_us, int64_t ctx_switch_overhead_us, int64_t *out_wcrt,
                         uint8_t *out_sched);

/*
 * gcaps_rta_gpu_priority_batch -- the GCAPS analysis with a separate priority for the GPU
 * segments of every task (Sec. 5.3 "Separate Priority for GPU Segments", Sec. 6.4 "Analysis for
 * GPU Priority Assignment").  hp(tau_i) of Lemmas 10, 11 and 13 becomes the set of tasks with a
 * higher GPU-segment priority, hpp(tau_i) keeps its meaning (same core, higher CPU priority),
 * and every jitter uses D_h in place of R_h, so each task is analysed on its own:
 * J^c_h = D_h - (C_h + G^m_h), J^g_h = D_h - G^e_h (0 where the task's own execution exceeds
 * its deadline).
 *
 *   flags               GCAPS_RTA_BUSY, GCAPS_RTA_LITERAL (as for gcaps_rta_batch), GCAPS_RTA_ASSIGN
 *   runlist_update_us   epsilon (Def. 2), 0..MAX_TIME
 *   gpu_priority        DEVICE, [ts->n_tasks], larger = higher, ties by position; used unless
 *                       GCAPS_RTA_ASSIGN is set (may be NULL then).  Within one core the order
 *                       of the GPU priorities must equal the order of the CPU priorities (the
 *                       paper's deadlock rule); a taskset that breaks it is GCAPS_SCHED_INVALID.
 *   out_gpu_priority    DEVICE, [ts->n_tasks]; required with GCAPS_RTA_ASSIGN, else optional (a
 *                       copy of gpu_priority).  With GCAPS_RTA_ASSIGN it receives the levels the
 *                       Audsley-style search of Sec. 5.3 found: 1 (lowest) .. n (highest), 0 for
 *                       tasks it could not place.  Levels are filled from the lowest; at each
 *                       level the unplaced tasks are tried from the lowest CPU priority upwards
 *                       (only a task with no unplaced task of lower CPU priority on its core is a
 *                       candidate) and the first one whose bound meets its deadline with all
 *                       other unplaced tasks above it takes the level.
 *   out_wcrt            DEVICE, [ts->n_tasks]: the task's bound, GCAPS_WCRT_MISS (also: never
 *                       placed) or GCAPS_WCRT_ITER_LIMIT; nothing is SKIPPED here
 *   out_sched           DEVICE, [n_tasksets]: 1 if every task has a bound within its deadline
 *   workspace           DEVICE scratch as for gcaps_rta_batch (gcaps_rta_workspace_bytes() bytes,
 *                       256-byte aligned): the size-binned launch plan
 *
 * Asynchronous on `stream`, no allocation.  Same return codes as gcaps_rta_batch.
 */
int gcaps_rta_gpu_priority_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int flags,
                                 int64_t runlist_update_us, const int64_t *gpu_priority,
                                 int64_t *out_gpu_priority, int64_t *out_wcrt, uint8_t *out_sched,
                                 void *workspace, size_t workspace_bytes, void *stream);

/*
 * gcaps_rta_batch_host_multi -- gcaps_rta_batch_host for several analyses of the same batch (the
 * paper's experiments run every taskset through GCAPS and through round robin, Sec. 7.1): the
 * inputs cross the host-device link once per chunk and are analysed n_policies times on the
 * device.  policies[q] is a GCAPS_POLICY_* | flags word, 1 <= n_policies <=
 * GCAPS_RTA_MAX_HOST_POLICIES; out_wcrt[q] / out_sched[q] are the host arrays of analysis q
 * ([ts->n_tasks] and [n_tasksets]).  timeslice_us and ctx_switch_overhead_us apply to all of
 * them.  Same return codes and synchronous behaviour as gcaps_rta_batch_host.
 */
#define GCAPS_RTA_MAX_HOST_POLICIES 8
int gcaps_rta_batch_host_multi(const gcaps_tasksets_t *ts, int64_t n_tasksets, const int *policies,
                               int n_policies, int64_t timeslice_us, int64_t ctx_switch_overhead_us,
                               int64_t *const *out_wcrt, uint8_t *const *out_sched);

/*
 * gcaps_rta_sweep_batch -- one device-resident batch analysed under several (timeslice, overhead)
 * pairs in a single pass.  The paper's experiments re-run the same generated tasksets while one
 * parameter of the analysis varies (Sec. 7.1; L of Eq. 3, theta of Def. 1 and epsilon of Def. 2
 * are such parameters); doing that with gcaps_rta_batch reads every taskset once per pair.  Here
 * each taskset is read, ordered and aggregated once and then goes through the recurrence of
 * gcaps_rta_batch once per pair.  Results are those of n_points separate gcaps_rta_batch calls.
 *
 *   n_points                1 .. GCAPS_RTA_MAX_SWEEP
 *   timeslice_us            HOST array [n_points]: L of pair q (RR only; may be NULL for GCAPS)
 *   ctx_switch_overhead_us  HOST array [n_points]: theta (RR) or epsilon (GCAPS) of pair q
 *   out_wcrt                DEVICE, [n_points][ts->n_tasks] (pair-major), or NULL when only the
 *                           schedulable flags are wanted
 *   out_sched               DEVICE, [n_points][n_tasksets] (pair-major)
 *   policy, workspace, stream, return codes, asynchrony: as for gcaps_rta_batch; the two host
 *   arrays are read before the call returns.
 */
#define GCAPS_RTA_MAX_SWEEP 32
int gcaps_rta_sweep_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int n_points,
                          const int64_t *timeslice_us, const int64_t *ctx_switch_overhead_us,
                          int64_t *out_wcrt, uint8_t *out_sched, void *workspace,
                          size_t workspace_bytes, void *stream);

/*
 * gcaps_rta_multi_batch -- several analyses of one device-resident batch in a single pass.  The
 * paper's experiments put every generated taskset through the GCAPS analysis and through the
 * analysis of the default round-robin driver, in both waiting modes (Sec. 7.1; Sec. 6.2 and 6.3
 * each give a busy-waiting and a self-suspension lemma set).  Here a taskset is read, ordered
 * and aggregated once and then goes through the recurrence of gcaps_rta_batch once per requested
 * analysis and per (timeslice, overhead) pair; the two self-suspension analyses run in one
 * launch, the two busy-waiting ones in another.  Results are those of separate gcaps_rta_batch
 * calls.
 *
 *   analyses   OR of GCAPS_ANALYSIS_*; `flags`: GCAPS_RTA_LITERAL, GCAPS_RTA_BEST_EFFORT
 *   n_points, timeslice_us, ctx_switch_overhead_us: as for gcaps_rta_sweep_batch (the overhead of
 *              a pair is theta for the round-robin analyses and epsilon for the GCAPS ones)
 *   out_wcrt   DEVICE, [n_points][k][ts->n_tasks] or NULL; out_sched DEVICE, [n_points][k]
 *              [n_tasksets]; k = number of requested analyses, in the order of the constants below
 *   everything else as for gcaps_rta_batch.
 */
#define GCAPS_ANALYSIS_GCAPS_SUSPEND 1
#define GCAPS_ANALYSIS_GCAPS_BUSY 2
#define GCAPS_ANALYSIS_RR_SUSPEND 4
#define GCAPS_ANALYSIS_RR_BUSY 8
int gcaps_rta_multi_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int analyses, int flags,
                          int n_points, const int64_t *timeslice_us,
                          const int64_t *ctx_switch_overhead_us, int64_t *out_wcrt,
                          uint8_t *out_sched, void *workspace, size_t workspace_bytes, void *stream);

/*
 * gcaps_rta_batch_static -- gcaps_rta_batch for callers that are not able to allocate device
 * memory.  (The paper has no counterpart: this is a convenience of this library, not a step of
 * the analysis.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a host
 * application that owns the allocator and hands out only input and output buffers, a real-time
 * or safety-certified process that must not allocate after start-up, or a caller in a context
 * where an allocation would synchronise the device or fail outright.  Such a caller cannot
 * provide the workspace gcaps_rta_batch asks for.  Here the workspace is a fixed array that is
 * part of the library image itself: every GPU that loads the library holds
 * GCAPS_RTA_STATIC_SCRATCH_BYTES of device memory for it until the process exits.
 *
 * Arguments, results, error codes and asynchrony are those of gcaps_rta_batch, minus the two
 * workspace arguments, with these differences:
 *   - n_tasksets may not exceed GCAPS_RTA_STATIC_MAX_TASKSETS; a larger batch is refused with
 *     GCAPS_ERR_TOO_LARGE and nothing is enqueued (split the batch, or use gcaps_rta_batch);
 *   - the call allocates nothing and frees nothing, on the host or on the device;
 *   - the first call on each device looks up the device address of the array (one cheap runtime
 *     query with that device current).  Make that first call outside any stream capture.  The
 *     address is kept for the life of the process and does not survive a cudaDeviceReset of that
 *     device: do not call this entry point again after one;
 *   - every call on a device shares the one array and finds the previous call's plan in it.
 *     The kernels rewrite every word of it that they later read, so stale contents are harmless,
 *     but two calls whose kernels overlap on the GPU (different streams, or different host
 *     threads without ordering) race on it and give undefined results.  Calls issued to one
 *     stream, or otherwise ordered, are safe.
 */
#define GCAPS_RTA_STATIC_MAX_TASKSETS 65536
#define GCAPS_RTA_STATIC_SCRATCH_BYTES (256 + 3072 + 4 * GCAPS_RTA_STATIC_MAX_TASKSETS)
int gcaps_rta_batch_static(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                           int64_t timeslice_us, int64_t ctx_switch_overhead_us,
                           int64_t *out_wcrt, uint8_t *out_sched, void *stream);

/*
 * On-device taskset generation.  The paper's experiments analyse randomly generated tasksets
 * (Sec. 7.1, Table 3: tasks per CPU, utilisation per CPU split over its tasks, period, number of
 * GPU segments, segment parameters, rate-monotonic priorities, worst-fit-decreasing allocation).
 * These two calls produce such tasksets directly in device memory, in the layout of
 * gcaps_tasksets_t, so that a large sweep never moves its inputs over the host link.  The
 * generator is integer-only (fixed point with 32 fractional bits, SplitMix64 as a counter-based
 * random source): taskset `index` of a stream is a pure function of (seed, stream, index), and
 * the host generator of the package's taskgen module yields the same bits.
 *
 * gcaps_gen_params_t: all "Q32" fields are value * 2^32.
 */
typedef struct gcaps_gen_params {
  uint64_t seed, stream;
  int32_t cores_lo, cores_hi;    /* CPUs per taskset, uniform, at most 64                       */
  int32_t tpc_lo, tpc_hi;        /* tasks per CPU, uniform; at most 256 tasks per taskset       */
  uint64_t util_lo, util_hi;     /* utilisation per CPU, Q32, uniform, below 1                  */
  uint64_t log2_lo, log2_hi;     /* log2 of the period range (us), Q32: periods are log-uniform */
  uint64_t log2_hi0;             /* harmonic tasksets: upper end of log2 of the base period     */
  int64_t period_lo, period_hi;  /* us, clamp of every period; period_hi <= 2^30                */
  uint64_t harmonic;             /* Q32 share of tasksets whose periods are P0 * 2^k, k <= 10   */
  uint64_t gpu_frac;             /* Q32 share of GPU-using tasks (gpu_mode 0)                   */
  uint64_t ratio_lo, ratio_hi;   /* G_i / (C_i + G_i), Q32, uniform, below 1                    */
  int32_t gpu_mode;              /* 0: exactly round(gpu_frac * n) GPU-using tasks with seg_lo ..
                                    seg_hi segments; 1: every task draws seg_lo .. seg_hi       */
  int32_t seg_lo, seg_hi;        /* GPU segments per task, at most 16                           */
  int32_t wfd;                   /* 1: worst-fit-decreasing re-allocation of tasks to CPUs      */
} gcaps_gen_params_t;

/* Scratch of gcaps_gen_count / gcaps_gen_fill for `count` tasksets of these parameters (host
 * computation; 12 bytes per possible task of a taskset plus 64 bytes per taskset; 0 for a
 * non-positive count or parameters outside the limits). */
size_t gcaps_gen_workspace_bytes(const gcaps_gen_params_t *params, int64_t count);

/*
 * gcaps_gen_count -- sizes of tasksets first .. first+count-1 of the stream: writes their
 * offsets into `workspace` (kept for gcaps_gen_fill) and the three array lengths n_tasks,
 * n_csegs, n_gsegs to out_totals (DEVICE, 3 x int64; read them back to size the arrays).
 * workspace: DEVICE, gcaps_gen_workspace_bytes(params, count) bytes, 256-byte aligned.  Asynchronous on
 * `stream`; GCAPS_OK or a GCAPS_ERR_* (parameters outside the limits stated above:
 * GCAPS_ERR_INVALID_ARG).
 */
int gcaps_gen_count(const gcaps_gen_params_t *params, int64_t first, int64_t count,
                    int64_t *out_totals, void *workspace, size_t workspace_bytes, void *stream);

/*
 * gcaps_gen_fill -- writes the tasksets that gcaps_gen_count (same params, first, count and
 * workspace; the workspace must be untouched in between) sized into the DEVICE arrays of `ts`.
 * ts->n_tasks, n_csegs, n_gsegs state how many elements the caller's arrays hold: size them from
 * out_totals.  A taskset that would reach beyond one of them is left out (its task_off entry is
 * still written); the call cannot report that, being asynchronous.  task_off gets count + 1
 * entries, cseg_off and gseg_off one entry more than there are tasks.  D_i = T_i.  Asynchronous on
 * `stream`; GCAPS_OK or a GCAPS_ERR_*.
 */
int gcaps_gen_fill(const gcaps_gen_params_t *params, int64_t first, int64_t count,
                   const gcaps_tasksets_t *ts, void *workspace, size_t workspace_bytes,
                   void *stream);

/*
 * Measurement aids (not steps of the analysis; the paper reports no timing of its analysis at
 * all, so it has no counterpart for either).
 *
 * gcaps_rta_plan_batch -- enqueues only the planning step of gcaps_rta_batch for this batch (the
 * size-binned permutation of taskset indices in `workspace`), so that the cost of planning can
 * be timed apart from the analysis.  Arguments and return codes as for gcaps_rta_batch.
 *
 * gcaps_rta_int_issue_probe -- enqueues one launch of a register-only integer kernel that fills
 * every SM with independent arithmetic chains (8 per thread, 64 warps per SM) and reports how
 * many 32-bit integer lane-operations the launch executes; divided by the launch's duration
 * (CUDA events around the call) that is the device's integer issue rate, the bound beside HBM
 * bandwidth for the recurrence of Eq. 1.  kind 0: multiply-add chains; 1: add chains; 2: one
 * multiply-add and one add per step.  trips: 1 .. 2^24 loop trips of 16 chain steps each.
 * scratch: DEVICE, one uint32 (never written in practice).  out_lane_ops: HOST, receives the
 * count.  Asynchronous on `stream`.
 */
int gcaps_rta_plan_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, void *workspace,
                         size_t workspace_bytes, void *stream);
int gcaps_rta_int_issue_probe(int kind, int64_t trips, uint32_t *scratch, int64_t *out_lane_ops,
                              void *stream);

/* Frees the staging memory gcaps_rta_batch_host keeps on the current device. */
void gcaps_rta_release_host(void);

/*
 * gcaps_rta_validate -- per-taskset check of the input domain stated above (task model: Sec. 4,
 * D_i <= T_i).  out_err is a DEVICE array [n_tasksets]; 0 = valid, otherwise a bit mask of
 * GCAPS_BAD_*.  Asynchronous on `stream`.
 */
#define GCAPS_BAD_TASK_RANGE 0x01 /* task_off not monotone / outside [0,n_tasks] / n too large  */
#define GCAPS_BAD_SEG_RANGE 0x02  /* segment offsets not monotone / outside range / too many    */
#define GCAPS_BAD_PERIOD 0x04     /* T_i outside 1..MAX_TIME                                     */
#define GCAPS_BAD_DEADLINE 0x08   /* D_i outside 1..T_i                                          */
#define GCAPS_BAD_CORE 0x10       /* core outside 0..MAX_CORE                                    */
#define GCAPS_BAD_WCET 0x20       /* a segment WCET outside 0..MAX_TIME                          */
int gcaps_rta_validate(const gcaps_tasksets_t *ts, int64_t n_tasksets, int32_t *out_err,
                       void *stream);

/* Text for a return code; never NULL. */
const char *gcaps_rta_strerror(int code);

/* The cudaError_t (as int) of the last failed CUDA call made by this library on this thread. */
int gcaps_rta_last_cuda_error(void);

/* GCAPS_RTA_VERSION of the loaded library. */
int gcaps_rta_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GCAPS_RTA_H_ */
