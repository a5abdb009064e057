// gcaps_rta.cu -- batched worst-case response-time analysis of GPU-using real-time tasksets
// (GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 6) for NVIDIA B200 (sm_100a).
//
// One warp analyses one taskset at a time:
//   stage      coalesced loads of the taskset's per-task slices into registers (lane = task)
//   aggregate  coalesced loads of the segment arrays, warp prefix sums into shared memory; the
//              per-task sums C_i, G^m_i, G^e_i and the RR slice count of Eq. 3 are differences of
//              two prefix values
//   order      rank of every task by (priority desc, position asc); the per-task values move
//              through shared memory to the lane that owns the task's rank
//   iterate    for each task in rank order the recurrence of Eq. 1 with the lemma set of the
//              chosen analysis: lanes over the higher-priority interferers, each evaluating
//              ceil((R+J)/T_h)*W terms (division by the invariant T_h is a multiply-high by a
//              per-task reciprocal), summed across the warp
//   publish    the lane that owns the converged task keeps R_i and forms its jitters J^c, J^g
//   early exit the first deadline miss ends the taskset
//   write      out_wcrt (one value per task), out_sched (one byte per taskset)
// The fast path holds every time in 32 bits and is taken when all values of a taskset are below
// 2^26 us; any other taskset goes through an exact 64-bit path with saturating arithmetic.
// Tasksets are binned by size (a small plan pass writes a permutation into the workspace) so that
// the warps of a launch hold the same number of tasks per lane; inside a launch warps pull chunks
// of tasksets from a counter, because iteration counts differ widely.
//
// A "one warp" above is a group of 8 or 16 lanes for tasksets of up to 32 tasks (two or four
// tasksets per warp).  gcaps_rta_multi_batch / gcaps_rta_sweep_batch use the same code with one
// staging, ordering and aggregation per taskset and one recurrence per requested analysis and
// (timeslice, overhead) pair.
//
// Everything is integer arithmetic on microseconds.  No tensor cores: nothing here is a dense
// contraction.  No host synchronisation and no allocation in gcaps_rta_batch.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "rta_common.cuh"

using namespace gcaps_detail;

#ifndef GCAPS_PREFETCH_AHEAD
#define GCAPS_PREFETCH_AHEAD 0
#endif
#ifndef GCAPS_FIRST_RANKS
#define GCAPS_FIRST_RANKS 1
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// plan: counting sort of taskset indices by size bin (histogram per block, scan, scatter)
// ---------------------------------------------------------------------------------------------
__global__ void plan_count_kernel(KParams p) {
  __shared__ unsigned int cnt[kBinStride];
  if (threadIdx.x < kBinStride) cnt[threadIdx.x] = 0;
  __syncthreads();
  i64 t0 = (i64)blockIdx.x * kPlanItems;
  for (int k = threadIdx.x; k < kPlanItems; k += blockDim.x) {
    i64 t = t0 + k;
    if (t < p.n_tasksets) atomicAdd(&cnt[size_bin(p.task_off[t + 1] - p.task_off[t])], 1u);
  }
  __syncthreads();
  if (threadIdx.x < kBinStride)
    p.block_cnt[(size_t)blockIdx.x * kBinStride + threadIdx.x] = cnt[threadIdx.x];
}

// One block, one warp per bin.  Turns per-block counts into per-block write cursors and fills the
// header.
__global__ void plan_scan_kernel(KParams p, unsigned int n_blocks) {
  __shared__ unsigned int bin_total[kBinStride];
  const int lane = threadIdx.x & 31, b = threadIdx.x >> 5;
  if (b < kNumBins) {
    unsigned int carry = 0;
    for (unsigned int base = 0; base < n_blocks; base += 32) {
      const unsigned int i = base + lane;
      const unsigned int v = i < n_blocks ? p.block_cnt[(size_t)i * kBinStride + b] : 0u;
      unsigned int x = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int y = __shfl_up_sync(0xffffffffu, x, d);
        if (lane >= d) x += y;
      }
      if (i < n_blocks) p.block_cnt[(size_t)i * kBinStride + b] = carry + x - v;  // cursor within the bin
      carry += __shfl_sync(0xffffffffu, x, 31);
    }
    if (lane == 0) bin_total[b] = carry;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int s = 0;
    for (int k = 0; k < kBinStride; ++k) {
      const unsigned int c = k < kNumBins ? bin_total[k] : 0u;
      p.hdr->bin_start[k] = s;
      p.hdr->bin_count[k] = c;
      p.hdr->next[k] = 0;
      s += c;
    }
  }
}

__global__ void plan_scatter_kernel(KParams p) {
  __shared__ unsigned int cursor[kBinStride];
  if (threadIdx.x < kBinStride)
    cursor[threadIdx.x] = p.block_cnt[(size_t)blockIdx.x * kBinStride + threadIdx.x];
  __syncthreads();
  i64 t0 = (i64)blockIdx.x * kPlanItems;
  for (int k = threadIdx.x; k < kPlanItems; k += blockDim.x) {
    i64 t = t0 + k;
    if (t < p.n_tasksets) {
      int b = size_bin(p.task_off[t + 1] - p.task_off[t]);
      unsigned int slot = atomicAdd(&cursor[b], 1u);
      p.perm[p.hdr->bin_start[b] + slot] = (unsigned int)t;
    }
  }
}

// The three steps in one block, for batches small enough that launches cost more than the work.
__global__ void __launch_bounds__(1024) plan_small_kernel(KParams p) {
  __shared__ unsigned int cnt[kBinStride], start[kBinStride];
  if (threadIdx.x < kBinStride) cnt[threadIdx.x] = 0;
  __syncthreads();
  for (i64 t = threadIdx.x; t < p.n_tasksets; t += blockDim.x)
    atomicAdd(&cnt[size_bin(p.task_off[t + 1] - p.task_off[t])], 1u);
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned int s = 0;
    for (int k = 0; k < kBinStride; ++k) {
      const unsigned int c = k < kNumBins ? cnt[k] : 0u;
      p.hdr->bin_start[k] = s;
      p.hdr->bin_count[k] = c;
      p.hdr->next[k] = 0;
      start[k] = s;
      cnt[k] = 0;  // from here on the write cursor of the bin
      s += c;
    }
  }
  __syncthreads();
  for (i64 t = threadIdx.x; t < p.n_tasksets; t += blockDim.x) {
    const int b = size_bin(p.task_off[t + 1] - p.task_off[t]);
    p.perm[start[b] + atomicAdd(&cnt[b], 1u)] = (unsigned int)t;
  }
}

// Shared-memory image of one taskset, indexed by priority rank unless noted.
template <int MAXN>
struct GroupSmem {
  u64 T[MAXN];     // period
  u64 D[MAXN];     // deadline
  u64 A[MAXN];     // C + G^m
  u64 Ge[MAXN];    // G^e
  u64 Star[MAXN];  // 2 * eps * eta^g   (GCAPS)   /   (L + theta) * slices, clamped   (RR)
  u64 R[MAXN];     // converged response time
  i64 prio_out[MAXN];  // by position: priority while ranking, then the output value
  int core[MAXN];
  int eta[MAXN];
  unsigned short ord[MAXN];  // rank -> position
};

// ---------------------------------------------------------------------------------------------
// the analysis of one taskset by a group of LPT lanes (exact 64-bit arithmetic)
// ---------------------------------------------------------------------------------------------
template <int LPT, int MAXN>
__device__ void analyse_taskset(const KParams &p, i64 t, GroupSmem<MAXN> &s, int lane,
                                unsigned int mask) {
  const int policy = p.policy & 0xff;
  const bool busy = (p.policy & GCAPS_RTA_BUSY) != 0;
  const bool literal = (p.policy & GCAPS_RTA_LITERAL) != 0;
  const bool best_effort = (p.policy & GCAPS_RTA_BEST_EFFORT) != 0;
  const u64 L = (u64)p.L, ovh = (u64)p.ovh;

  const i64 a = p.task_off[t] - p.task_base, b = p.task_off[t + 1] - p.task_base;
  if (a < 0 || b < a || b > p.n_tasks || b - a > MAXN) {
    // a range this launch cannot hold is a broken or oversized taskset: nothing is addressable
    if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
    return;
  }
  const int n = (int)(b - a);

  // ---- stage: priorities by position, domain check of the per-task scalars -------------------
  int bad = 0;
  for (int i = lane; i < n; i += LPT) {
    const i64 k = a + i;
    s.prio_out[i] = p.priority[k];
    const i64 T = p.period[k], D = p.deadline[k], c = p.core[k];
    if (T < 1 || T > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_PERIOD;
    if (D < 1 || D > T) bad |= GCAPS_BAD_DEADLINE;
    if (c < 0 || c > GCAPS_RTA_MAX_CORE) bad |= GCAPS_BAD_CORE;
  }
  __syncwarp(mask);

  // ---- order + aggregate: each lane ranks its tasks, sums their segments, stores by rank ------
  int n_gpu_lane = 0;
  for (int i = lane; i < n; i += LPT) {
    const i64 k = a + i;
    const i64 pi = s.prio_out[i];
    int rank = 0;
    for (int q = 0; q < n; ++q) {
      const i64 pq = s.prio_out[q];
      rank += (pq > pi || (pq == pi && q < i)) ? 1 : 0;
    }
    const i64 c0 = p.cseg_off[k] - p.cseg_base, c1 = p.cseg_off[k + 1] - p.cseg_base;
    const i64 g0 = p.gseg_off[k] - p.gseg_base, g1 = p.gseg_off[k + 1] - p.gseg_base;
    bool seg_ok = !(c0 < 0 || c1 < c0 || c1 > p.n_csegs || c1 - c0 > GCAPS_RTA_MAX_SEGMENTS ||
                    g0 < 0 || g1 < g0 || g1 > p.n_gsegs || g1 - g0 > GCAPS_RTA_MAX_SEGMENTS);
    u64 C = 0, Gm = 0, Ge = 0, slices = 0;
    if (seg_ok) {
      for (i64 j = c0; j < c1; ++j) {
        const i64 w = p.cseg_wcet[j];
        if (w < 0 || w > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_WCET;
        C += (u64)w;
      }
      for (i64 j = g0; j < g1; ++j) {
        const i64 m = p.gseg_misc[j], e = p.gseg_exec[j];
        if (m < 0 || m > GCAPS_RTA_MAX_TIME || e < 0 || e > GCAPS_RTA_MAX_TIME)
          bad |= GCAPS_BAD_WCET;
        Gm += (u64)m;
        Ge += (u64)e;
        if (policy == GCAPS_POLICY_RR && e > 0) slices += ceil_div64((u64)e, L);  // Eq. 3
      }
    } else {
      bad |= GCAPS_BAD_SEG_RANGE;
    }
    const int eta = seg_ok ? (int)(g1 - g0) : 0;
    n_gpu_lane += eta > 0 ? 1 : 0;
    s.T[rank] = (u64)p.period[k];
    s.D[rank] = (u64)p.deadline[k];
    s.A[rank] = C + Gm;
    s.Ge[rank] = Ge;
    s.Star[rank] = policy == GCAPS_POLICY_GCAPS ? 2 * ovh * (u64)eta : sat_mul(L + ovh, slices);
    s.core[rank] = (int)p.core[k];
    s.eta[rank] = eta;
    // a best-effort task (flag set, priority <= 0) ranks behind every real-time task; bit 15
    s.ord[rank] = (unsigned short)(i | ((best_effort && pi <= 0) ? 0x8000 : 0));
  }
  bad = group_or<LPT>(bad, mask);
  const int n_gpu = group_sum_int<LPT>(n_gpu_lane, mask);  // N_g
  __syncwarp(mask);
  if (bad) {
    if (p.out_wcrt)
      for (int i = lane; i < n; i += LPT) p.out_wcrt[a + i] = GCAPS_WCRT_INVALID;
    if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
    return;
  }
  for (int i = lane; i < n; i += LPT)
    s.prio_out[i] = (best_effort && s.prio_out[i] <= 0) ? GCAPS_WCRT_BEST_EFFORT : GCAPS_WCRT_SKIPPED;
  __syncwarp(mask);

  // ---- iterate: tasks in decreasing priority ---------------------------------------------------
  int sched = GCAPS_SCHED_YES;
  for (int pos = 0; pos < n; ++pos) {
    if (s.ord[pos] & 0x8000) break;  // only best-effort tasks from here on: nothing to bound
    const u64 Di = s.D[pos];
    const int core_i = s.core[pos];
    const bool gi = s.eta[pos] > 0;
    u64 base;
    u64 nu = 0;  // Lemma 4's interleaving-set size
    if (policy == GCAPS_POLICY_GCAPS) {
      // C_i + G*_i + B^C_i  (Sec. 6.3, Lemma 8); Star = 2*eps*eta
      base = s.A[pos] + s.Ge[pos] + s.Star[pos] + ((u64)s.eta[pos] + 1) * ovh;
    } else {
      // C_i + G_i + I^ie_i  (Lemma 1); Star = (L+theta)*slices
      base = s.A[pos] + s.Ge[pos] + (gi ? sat_mul(s.Star[pos], (u64)(n_gpu - 1)) : 0);
      if (busy) {
        int c = 0;
        for (int h = lane; h < pos; h += LPT) c += (s.core[h] == core_i && s.eta[h] > 0) ? 1 : 0;
        nu = (u64)(n_gpu - group_sum_int<LPT>(c, mask) + 1);
      }
    }
    u64 R = base;
    i64 verdict = 0;
    i64 sweeps = 0;
    for (;;) {
      if (R > Di) {
        verdict = GCAPS_WCRT_MISS;
        break;
      }
      if (sweeps >= GCAPS_RTA_ITER_CAP) {
        verdict = GCAPS_WCRT_ITER_LIMIT;
        break;
      }
      sweeps += 1;
      u64 part = 0;
      for (int h = lane; h < pos; h += LPT) {
        const u64 Th = s.T[h];
        const bool same = s.core[h] == core_i;
        const bool gh = s.eta[h] > 0;
        const u64 Rh = s.R[h];
        const u64 Jc = Rh - s.A[h], Jg = Rh - s.Ge[h];
        u64 term = 0;
        if (policy == GCAPS_POLICY_GCAPS && !busy) {
          if (same && !gh) term = sat_mul(ceil_div64(R, Th), s.A[h]);  // Lemma 15 (G^m_h = 0)
          if (same && gh) term = sat_mul(ceil_div64(R + Jc, Th), s.A[h] + s.Star[h]);
          if (same && gh && gi) term += sat_mul(ceil_div64(R + Jg, Th), s.Ge[h]);   // Lemma 13
          if (!same && gh && gi) term = sat_mul(ceil_div64(R + Jg, Th), s.Ge[h] + s.Star[h]);
        } else if (policy == GCAPS_POLICY_GCAPS) {
          if (same) {
            u64 W = s.A[h];                                                        // Lemma 12
            if (gh && (gi || !literal)) W += s.Ge[h] + s.Star[h];                  // Lemma 10
            term = sat_mul(ceil_div64(R, Th), W);
          } else if (gh) {
            term = sat_mul(ceil_div64(R + Jg, Th), s.Ge[h] + s.Star[h]);           // Lemma 10/11
          }
        } else if (!busy) {
          if (same) term = sat_mul(ceil_div64(R + ((gh || literal) ? Jc : 0), Th), s.A[h]);  // L7
        } else {
          if (same) {
            u64 W = s.A[h];                                                        // Lemma 5
            if (gh) W += sat_mul(s.Star[h], nu);                                   // Lemma 4
            term = sat_mul(ceil_div64(R, Th), W);
          }
        }
        part += term;  // each term <= 2^51, at most 8 per lane: no overflow
      }
      const u64 next = base + group_sum<LPT>(part, mask);
      if (next == R) break;
      R = next;
    }
    if (verdict == 0) {
      if (lane == 0) {
        s.R[pos] = R;
        s.prio_out[s.ord[pos] & 0x7fff] = (i64)R;
      }
      __syncwarp(mask);
    } else {
      if (lane == 0) s.prio_out[s.ord[pos] & 0x7fff] = verdict;
      sched = GCAPS_SCHED_NO;
      break;
    }
  }
  __syncwarp(mask);
  if (p.out_wcrt)
    for (int i = lane; i < n; i += LPT) p.out_wcrt[a + i] = s.prio_out[i];
  if (lane == 0) p.out_sched[t] = (uint8_t)sched;
  __syncwarp(mask);
}

// ---------------------------------------------------------------------------------------------
// 32-bit fast path
// ---------------------------------------------------------------------------------------------
// ---- running sums of a segment array, 128 elements per step ------------------------------------
// Lane l takes four consecutive elements (two 16-byte loads), so a warp reads 1 KB contiguous.
// Loads must start on a 16-byte boundary: when the slice starts on an odd element the step begins
// one element early (`par` = 1).  Q[x] receives the sum (modulo 2^32) of elements -par .. x - par;
// Q[-1] is a guard word holding 0.  For 0 <= lo <= hi <= N the sum of elements [lo, hi) is
// Q[hi - 1 + par] - Q[lo - 1 + par]: a borrowed element in front only shifts every entry by the
// same amount, and elements behind the slice only reach entries that are never read.
struct Quad {
  i64 v[4];
};

// Elements e .. e+3 of X, for a slice whose 16-byte pairs all lie inside the array (the common
// case, checked once per taskset by the caller).  Pairs that start at or behind N are not read.
__device__ __forceinline__ void load_quad_inside(const i64 *__restrict__ X, int e, int N, Quad &q) {
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    longlong2 w = make_longlong2(0, 0);
    if (e + 2 * h < N) w = __ldg(reinterpret_cast<const longlong2 *>(X + e + 2 * h));
    q.v[2 * h] = w.x, q.v[2 * h + 1] = w.y;
  }
}

// The same for a slice at the very edge of its array: only wanted elements inside [lo, hi) are
// touched, everything else reads as 0.
__device__ __noinline__ Quad load_quad_edge(const i64 *__restrict__ X, int e, int N, const i64 *lo,
                                            const i64 *hi) {
  Quad q;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const i64 *ptr = X + e + j;
    q.v[j] = (e + j >= 0 && e + j < N && ptr >= lo && ptr < hi) ? __ldg(ptr) : 0;
  }
  return q;
}

// Narrows a quad to 32 bits, leaves the lane's own running sums in x[0..3] and records in `bad`
// whether a wanted element lies outside [0, 2^26).
__device__ __forceinline__ void narrow_quad(const Quad &q, int e, int N, u32 (&x)[4], u32 &bad) {
  const u32 hi_or = (u32)((u64)q.v[0] >> 32) | (u32)((u64)q.v[1] >> 32) | (u32)((u64)q.v[2] >> 32) |
                    (u32)((u64)q.v[3] >> 32);
  const u32 lo_or = (u32)q.v[0] | (u32)q.v[1] | (u32)q.v[2] | (u32)q.v[3];
  if (hi_or | (lo_or >> 26)) {  // rare: look again, this time only at the elements of this slice
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if ((u32)(e + j) < (u32)N) bad |= (u32)((u64)q.v[j] >> 32) | ((u32)q.v[j] >> 26);
  }
  x[0] = (u32)q.v[0];
  x[1] = x[0] + (u32)q.v[1];
  x[2] = x[1] + (u32)q.v[2];
  x[3] = x[2] + (u32)q.v[3];
}

// True if every 16-byte pair that load_quad_inside would read for this slice is inside the array.
__device__ __forceinline__ bool slice_is_inside(i64 first, int N, int par, i64 total) {
  return (par == 0 || first >= 1) && ((((N + par) & 1) == 0) || first + N < total);
}

template <int LPT, int SLOTS>
struct FastLayout {
  static constexpr int MAXN = LPT * SLOTS;
  static constexpr int kStep = 4 * LPT;  // elements one prefix step of the group covers
  // a prefix array takes slices of up to CAP-1 elements and is written kStep words at a time
  static constexpr int CAP = (6 * MAXN + kStep - 1) / kStep * kStep;
  static constexpr int kInfo = 0;  // uint4 per rank: deadline, core, base, position | GPU flag
  static constexpr int kQ0 = 4 * MAXN + 4;
  static constexpr int kQ1 = kQ0 + CAP + 4;
  static constexpr int kFastWords = kQ1 + CAP;
  static constexpr int kExactWords = (17 * MAXN + 3) / 4 * 4;  // the exact path: 66 B per task
  static constexpr int kWords = kFastWords > kExactWords ? kFastWords : kExactWords;
  static_assert(kWords % 4 == 0 && CAP % kStep == 0 && 4 * MAXN <= CAP, "16-byte aligned rows");
};

// One step (NB blocks of 4*LPT elements) of the running sums of up to two arrays that share their
// offsets, by a group of LPT lanes (`gmask`).
template <int LPT, int NB, bool TWO>
__device__ __forceinline__ void prefix_step(const i64 *__restrict__ X0, const i64 *__restrict__ X1,
                                            int e0, int N, int par0, int par1, bool inside,
                                            const i64 *lo0, const i64 *hi0, const i64 *lo1,
                                            const i64 *hi1, u32 *Q0, u32 *Q1, u32 &carry0,
                                            u32 &carry1, u32 &bad, int lane, unsigned int gmask) {
  Quad q0[NB], q1[NB];
  u32 x0[NB][4], x1[NB][4], i0[NB], i1[NB];
  if (inside) {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      load_quad_inside(X0, e0 + 4 * LPT * b + 4 * lane - par0, N, q0[b]);
      if (TWO) load_quad_inside(X1, e0 + 4 * LPT * b + 4 * lane - par1, N, q1[b]);
    }
  } else {
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      q0[b] = load_quad_edge(X0, e0 + 4 * LPT * b + 4 * lane - par0, N, lo0, hi0);
      if (TWO) q1[b] = load_quad_edge(X1, e0 + 4 * LPT * b + 4 * lane - par1, N, lo1, hi1);
    }
  }
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    narrow_quad(q0[b], e0 + 4 * LPT * b + 4 * lane - par0, N, x0[b], bad);
    i0[b] = x0[b][3];
    if (TWO) {
      narrow_quad(q1[b], e0 + 4 * LPT * b + 4 * lane - par1, N, x1[b], bad);
      i1[b] = x1[b][3];
    }
  }
#pragma unroll
  for (int d = 1; d < LPT; d <<= 1) {  // the warp scans of all blocks side by side
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      const u32 y0 = __shfl_up_sync(gmask, i0[b], d, LPT);
      if (lane >= d) i0[b] += y0;
      if (TWO) {
        const u32 y1 = __shfl_up_sync(gmask, i1[b], d, LPT);
        if (lane >= d) i1[b] += y1;
      }
    }
  }
#pragma unroll
  for (int b = 0; b < NB; ++b) {
    if (e0 + 4 * LPT * b < N + 1) {
      const u32 b0 = i0[b] - x0[b][3] + carry0;
      *reinterpret_cast<uint4 *>(Q0 + e0 + 4 * LPT * b + 4 * lane) =
          make_uint4(x0[b][0] + b0, x0[b][1] + b0, x0[b][2] + b0, x0[b][3] + b0);
      carry0 += __shfl_sync(gmask, i0[b], LPT - 1, LPT);
      if (TWO) {
        const u32 b1 = i1[b] - x1[b][3] + carry1;
        *reinterpret_cast<uint4 *>(Q1 + e0 + 4 * LPT * b + 4 * lane) =
            make_uint4(x1[b][0] + b1, x1[b][1] + b1, x1[b][2] + b1, x1[b][3] + b1);
        carry1 += __shfl_sync(gmask, i1[b], LPT - 1, LPT);
      }
    }
  }
}

// Range check of segment slices without running sums: `bad` collects whether a wanted element lies
// outside [0, 2^26), and the elements, narrowed to 32 bits, go to shared memory as they are
// (D[w] = element w - par; same loads and store pattern as prefix_step).  NB blocks of 128
// elements per array in flight together (TWO: two arrays that share their offsets).
template <int NB, bool TWO>
__device__ __forceinline__ void check_slices(const i64 *__restrict__ X0, const i64 *__restrict__ X1, int N,
                                             int par0, int par1, bool inside, const i64 *lo0,
                                             const i64 *hi0, const i64 *lo1, const i64 *hi1, u32 *D0,
                                             u32 *D1, int lane, u32 &bad) {
  for (int e0 = 0; e0 < N + (par0 > par1 ? par0 : par1); e0 += 128 * NB) {
    Quad q0[NB], q1[NB];
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      if (inside) {
        load_quad_inside(X0, e0 + 128 * b + 4 * lane - par0, N, q0[b]);
        if (TWO) load_quad_inside(X1, e0 + 128 * b + 4 * lane - par1, N, q1[b]);
      } else {
        q0[b] = load_quad_edge(X0, e0 + 128 * b + 4 * lane - par0, N, lo0, hi0);
        if (TWO) q1[b] = load_quad_edge(X1, e0 + 128 * b + 4 * lane - par1, N, lo1, hi1);
      }
    }
#pragma unroll
    for (int b = 0; b < NB; ++b) {
      if (e0 + 128 * b < N + 1) {
        u32 x[4];
        narrow_quad(q0[b], e0 + 128 * b + 4 * lane - par0, N, x, bad);
        *reinterpret_cast<uint4 *>(D0 + e0 + 128 * b + 4 * lane) =
            make_uint4((u32)q0[b].v[0], (u32)q0[b].v[1], (u32)q0[b].v[2], (u32)q0[b].v[3]);
        if (TWO) {
          narrow_quad(q1[b], e0 + 128 * b + 4 * lane - par1, N, x, bad);
          *reinterpret_cast<uint4 *>(D1 + e0 + 128 * b + 4 * lane) =
              make_uint4((u32)q1[b].v[0], (u32)q1[b].v[1], (u32)q1[b].v[2], (u32)q1[b].v[3]);
        }
      }
    }
  }
}

// The first kFirstRanks tasks of the priority order, analysed before anything is summed for the
// rest of the taskset (a warp per taskset).  Where tasksets are far from schedulable the first
// deadline miss comes within a handful of ranks, and the per-task sums of all the other tasks
// would never be used: here every segment value is still read and range-checked (a value outside
// the 32-bit path's range sends the taskset to the exact path, as always), but sums are formed
// only for these ranks: four lanes per rank add up the rank's own few segments, all ranks at once
// (one trip to memory), and lane r then holds everything about rank r, as the task under analysis
// and as an interferer of the ranks behind it.  The recurrence over these ranks needs registers
// and warp collectives only.  Same arithmetic, same sequence of iterates, same sentinels as the
// full pass.  `first8[r]` = (first, end) of rank r's CPU segments and of its GPU segments within
// the taskset's slices; info[r] = (deadline, core, period, position).
// Returns 1: the taskset is finished (a miss among these ranks, or no other real-time task), its
// outputs are written; 0: all these ranks converged, the caller runs the full pass (which repeats
// them); -1: a value does not fit the 32-bit path.
constexpr int kFirstRanks = 8;
template <int SLOTS, int MODE>
__device__ __forceinline__ int first_ranks(const KParams &p, i64 t, i64 a, int n, const uint4 *info,
                                           const uint4 *first8, u32 *Q0, u32 *Q1, int n_rt,
                                           const int (&rank)[SLOTS], const int (&g0)[SLOTS],
                                           const int (&g1)[SLOTS], const i64 *__restrict__ Xc,
                                           const i64 *__restrict__ Xm, const i64 *__restrict__ Xe, int Nc,
                                           int Ng, int parc, int parm, int pare, i64 cfirst, i64 gfirst,
                                           int lane, bool literal) {
  const int limit = n_rt < kFirstRanks ? n_rt : kFirstRanks;
  // lanes 4r .. 4r+3 add up the segments of rank r
  const int r4 = lane >> 2, sub = lane & 3;
  uint4 seg = make_uint4(0u, 0u, 0u, 0u);
  if (r4 < limit) seg = first8[r4];
  u32 bad = 0, sum_c = 0, sum_m = 0, sum_e = 0, sum_s = 0;
  // every segment value of the taskset must be in [0, 2^26); on the way the values stop over in
  // shared memory, where the eight ranks find their own
  check_slices<(SLOTS < 3 ? SLOTS : 3), false>(Xc, Xc, Nc, parc, parc, slice_is_inside(cfirst, Nc, parc, p.n_csegs),
                                               p.cseg_wcet, p.cseg_wcet + p.n_csegs, p.cseg_wcet, p.cseg_wcet,
                                               Q0, Q0, lane, bad);
  __syncwarp();
  for (int j = (int)seg.x + parc + sub; j < (int)seg.y + parc; j += 4) sum_c += Q0[j];
  __syncwarp();
  check_slices<2, true>(Xm, Xe, Ng, parm, pare,
                        slice_is_inside(gfirst, Ng, parm, p.n_gsegs) && slice_is_inside(gfirst, Ng, pare, p.n_gsegs),
                        p.gseg_misc, p.gseg_misc + p.n_gsegs, p.gseg_exec, p.gseg_exec + p.n_gsegs, Q1, Q0,
                        lane, bad);
  __syncwarp();
  for (int j = (int)seg.z + sub; j < (int)seg.w; j += 4) {
    sum_m += Q1[j + parm];
    const u32 e = Q0[j + pare] & (kFastLimit - 1);  // (checked above; keeps the division exact)
    sum_e += e;
    if (MODE >= 2) {  // Eq. 3: slices of the pure GPU part
      if (p.l_mode == 0) sum_s += __umulhi(e + (u32)p.L - 1u, p.l_magic) >> p.l_shift;
      else if (p.l_mode == 1) sum_s += e;
      else sum_s += e > 0 ? 1u : 0u;
    }
  }
  int n_gpu = 0;  // N_g
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) n_gpu += __popc(__ballot_sync(kFull, g1[s] > g0[s]));
#pragma unroll
  for (int d = 1; d <= 2; d <<= 1) {
    sum_c += __shfl_xor_sync(kFull, sum_c, d), sum_m += __shfl_xor_sync(kFull, sum_m, d);
    sum_e += __shfl_xor_sync(kFull, sum_e, d);
    if (MODE >= 2) sum_s += __shfl_xor_sync(kFull, sum_s, d);
  }
  // lane r takes rank r from lane 4r (a task has fewer than 64 segments of a kind, every value is
  // below 2^26: no overflow)
  const int src = (4 * lane) & 31;
  sum_c = __shfl_sync(kFull, sum_c, src), sum_m = __shfl_sync(kFull, sum_m, src);
  sum_e = __shfl_sync(kFull, sum_e, src);
  if (MODE >= 2) sum_s = __shfl_sync(kFull, sum_s, src);
  const u32 eta_r = __shfl_sync(kFull, seg.w - seg.z, src);
  const bool mine = lane < limit;
  const uint4 f = mine ? info[lane] : make_uint4(1u, 0xffffffffu, 2u, 0u);  // deadline, core, period, position
  const u32 ovh = (u32)p.ovh;  // below 2^20 on this path
  const u32 D_r = f.x, core_r = f.y, Tm1 = f.z - 1, A_r = sum_c + sum_m, Ge_r = sum_e;
  const bool gpu_r = eta_r > 0;
  u32 S_r, base_r;
  if (MODE < 2) {
    S_r = 2 * ovh * eta_r;                               // eta < 64: below 2^27
    base_r = A_r + Ge_r + S_r + (eta_r + 1) * ovh;       // C_i + G*_i + B^C_i, below 2^29
    if (mine) bad |= S_r >> 26;
  } else {
    const u64 lt = (u64)p.L + ovh;                       // <= 2^41
    u64 B = sum_s == 0 ? 0 : (lt >= kFastClamp ? kFastClamp : lt * (u64)sum_s);
    if (B > kFastClamp) B = kFastClamp;
    S_r = (u32)B;
    const u64 b64 = (u64)A_r + Ge_r + (gpu_r ? B * (u64)(n_gpu - 1) : 0);  // Lemma 1
    base_r = b64 > (u64)(2 * kFastClamp) ? 2 * kFastClamp : (u32)b64;
  }
  base_r = base_r > 2 * kFastClamp ? 2 * kFastClamp : base_r;
  if (mine) bad |= (sum_c | sum_m | A_r | Ge_r) >> 26;
  if (__any_sync(kFull, bad != 0)) return -1;
  u32 magic, shift;
  make_reciprocal(f.z, magic, shift);
  // what rank r contributes as an interferer (the jitters follow when it has converged)
  u32 Wa, Wb;
  if (MODE == 0) {
    Wa = A_r + (gpu_r ? S_r : 0u);    // Lemma 15: C_h, or C_h + G^{m*}_h
    Wb = gpu_r ? Ge_r + S_r : 0u;     // Lemma 13, other cores: G^{e*}_h
  } else if (MODE == 1) {
    Wa = A_r;                         // Lemma 12
    Wb = gpu_r ? Ge_r + S_r : 0u;     // Lemmas 10, 11: G^{e*}_h
  } else {
    Wa = A_r;                         // Lemmas 5, 7
    Wb = gpu_r ? S_r : 0u;            // Lemma 4: (L+theta) * slices
  }
  u32 Jc = Tm1, Jg = Tm1;
  // ---- the recurrence of Eq. 1 over these ranks -----------------------------------------------------
  int verdict = 0, pos = 0;
  for (; pos < limit; ++pos) {
    const u32 Di = __shfl_sync(kFull, D_r, pos), core_i = __shfl_sync(kFull, core_r, pos);
    const u32 base_i = __shfl_sync(kFull, base_r, pos);
    const bool gi = __shfl_sync(kFull, (int)gpu_r, pos) != 0;
    const bool act = lane < pos, same = core_r == core_i;
    u32 j1, w1, w2 = 0;
    if (MODE == 0) {
      w1 = same ? Wa : (gi ? Wb : 0u);            // Lemma 15 / Lemma 13 (other cores)
      j1 = same ? Jc : Jg;
      w2 = (same && gi && gpu_r) ? Ge_r : 0u;     // Lemma 13 (same core), jitter J^g
    } else if (MODE == 1) {
      w1 = same ? Wa + ((gi || !literal) ? Wb : 0u) : Wb;  // Lemmas 12+10 / 10, 11
      j1 = same ? Tm1 : Jg;
    } else if (MODE == 2) {
      w1 = same ? Wa : 0u;                        // Lemma 7
      j1 = Jc;
    } else {
      // Lemma 4: N_g - |{h in hpp(i): GPU-using}| + 1
      const u32 nu = (u32)(n_gpu - __popc(__ballot_sync(kFull, act && same && gpu_r)) + 1);
      const u64 w = (u64)Wa + (u64)Wb * nu;       // Lemmas 5 and 4
      w1 = same ? (w > kFastClamp ? kFastClamp : (u32)w) : 0u;
      j1 = Tm1;
    }
    if (!act) w1 = 0, w2 = 0;
    u32 R = base_i;
    int sweeps = 0;
    for (;;) {
      if (R > Di) {
        verdict = GCAPS_WCRT_MISS;
        break;
      }
      if (sweeps >= (int)GCAPS_RTA_ITER_CAP) {
        verdict = GCAPS_WCRT_ITER_LIMIT;
        break;
      }
      sweeps += 1;
      u32 next = base_i;
      if (pos > 0) {
        u64 acc = (u64)(__umulhi(R + j1, magic) >> shift) * w1;
        if (MODE == 0) acc += (u64)(__umulhi(R + Jg, magic) >> shift) * w2;
        const u32 part = acc > (u64)kFastClamp ? kFastClamp : (u32)acc;
        next += __reduce_add_sync(kFull, part);
      }
      if (next == R) break;
      R = next;
    }
    if (verdict != 0) break;
    // publish: R_i goes out; lane `pos` forms the jitters J^c = R - (C+G^m), J^g = R - G^e (a
    // CPU-only task has no J^c unless the printed form of Lemma 7 is asked for)
    if (lane == pos) {
      if (p.out_wcrt) p.out_wcrt[a + f.w] = (i64)R;
      if (MODE == 0 ? gpu_r : (MODE == 2 ? (gpu_r || literal) : false)) Jc = R - A_r + Tm1;
      Jg = R - Ge_r + Tm1;
    }
  }
  if (verdict == 0 && limit < n_rt) return 0;  // undecided: the full pass takes over
  const int n_done = pos;  // ranks that converged (= n_rt without a verdict)
  if (p.out_wcrt) {
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const int r = rank[s];
      if (lane + 32 * s < n && r >= n_done)
        p.out_wcrt[a + lane + 32 * s] = r >= n_rt ? (i64)GCAPS_WCRT_BEST_EFFORT
                                                  : (r == n_done ? (i64)verdict : (i64)GCAPS_WCRT_SKIPPED);
    }
  }
  if (lane == 0) p.out_sched[t] = verdict == 0 ? GCAPS_SCHED_YES : GCAPS_SCHED_NO;
  return 1;
}

// An analysis mode known at compile time (converts to int like a run-time mode does).
template <int V>
struct ModeTag {
  __host__ __device__ constexpr operator int() const { return V; }
};

// MODE: 0 GCAPS self-suspension, 1 GCAPS busy-waiting, 2 RR self-suspension, 3 RR busy-waiting.
// Returns false, having written nothing, if the taskset is not eligible for 32-bit arithmetic
// (or is invalid): the caller then runs the exact 64-bit path, which also does the validation.
//
// A group of LPT lanes (8, 16 or a whole warp) works on one taskset.  Until the per-task sums are
// known lane l of the group holds the tasks at positions l, l+LPT, ... ("slots").
// Then every task's values move through shared memory to the lane that owns its rank, so that the
// interferers of the task of rank `pos` sit in lanes (pos-1) % LPT downwards of slots up to
// (pos-1) / LPT and higher slots can be skipped.
//
// MASK: bit m set = analysis MODE m is compiled in.  SWEEP: the taskset is staged, ordered and
// aggregated once and then analysed under every (timeslice, overhead) pair q of `sw` and every
// mode m of MASK that sw->enabled names; that analysis writes result block
// q * sw->block_stride + sw->block_of_mode[m] (out_wcrt + block * n_tasks, skipped when out_wcrt
// is null; out_sched + block * n_tasksets).  Without SWEEP, MASK has one bit and the analysis
// takes its constants and outputs from `p`.
//
// Returns kFastDone (outputs written), kFastDeclined (nothing written that matters: the caller runs
// the exact path) or, with FIRST_ONLY, kFastUndecided.  FIRST_ONLY (one analysis, a warp per
// taskset): only the first ranks of the priority order are analysed (first_ranks below); if they
// all converge and more ranks follow, nothing is decided and the caller runs the full pass.
constexpr int kFastDeclined = 0, kFastDone = 1, kFastUndecided = 2;
template <int LPT, int SLOTS, int MASK, bool SWEEP = false, bool FIRST_ONLY = false>
__device__ __forceinline__ int analyse_fast(const KParams &p, i64 t, i64 a, int n, u32 *buf, int lane,
                                            unsigned int gmask, const SweepArgs *sw = nullptr) {
  static_assert(!FIRST_ONLY || (LPT == 32 && !SWEEP), "the first ranks' own pass: a warp per taskset");
  typedef FastLayout<LPT, SLOTS> Lay;
  constexpr int kLog = LPT == 32 ? 5 : LPT == 16 ? 4 : 3;  // log2 of the lanes per taskset
  constexpr int MAXN = Lay::MAXN, CAP = Lay::CAP;
  // prefix blocks of the CPU segments whose loads are issued together.  Tasksets of 65..96 tasks
  // with a few GPU segments per task have 200..400 CPU segments: three blocks of 128 cover them
  // in one step where two need a second, mostly empty one (80-task tasksets: -4 % for a GCAPS
  // kernel; the RR kernels, which carry the slice sums too, lose as much to the registers it takes)
  constexpr int BC = SLOTS <= 2 ? SLOTS : ((SLOTS == 3 && (MASK & 12) == 0 && !SWEEP) ? 3 : 2);
#ifdef GCAPS_BG2
  constexpr int BG = (SLOTS == 3 && (MASK & 12) == 0 && !SWEEP) ? 2 : 1;
#else
  constexpr int BG = 1;
#endif
  constexpr bool kAnyGcaps = (MASK & 3) != 0;
  constexpr bool kMulti = (MASK & (MASK - 1)) != 0;
  static_assert(!kMulti || SWEEP, "several analyses per taskset use the sweep loop");
  const bool literal = (p.policy & GCAPS_RTA_LITERAL) != 0;
  const bool best_effort = (p.policy & GCAPS_RTA_BEST_EFFORT) != 0;
  uint4 *info = reinterpret_cast<uint4 *>(buf + Lay::kInfo);
  u32 *Q0 = buf + Lay::kQ0, *Q1 = buf + Lay::kQ1;

  // ---- stage: per-task scalars, lane = position; rank ----------------------------------------
  u32 T[SLOTS];
  int rank[SLOTS], c0[SLOTS], g0[SLOTS];
  bool ok = true;
  int Nc, Ng;
  i64 cfirst, gfirst;
  {
    i64 t64[SLOTS], d64[SLOTS], pr[SLOTS], c64[SLOTS], co[SLOTS], go[SLOTS];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {  // all loads of the taskset's per-task arrays in flight
      const i64 k = a + (lane + LPT * s < n ? lane + LPT * s : 0);
      t64[s] = p.period[k], d64[s] = p.deadline[k], pr[s] = p.priority[k], c64[s] = p.core[k];
      co[s] = p.cseg_off[k], go[s] = p.gseg_off[k];
    }
    const i64 cend = p.cseg_off[a + n] - p.cseg_base, gend = p.gseg_off[a + n] - p.gseg_base;
    cfirst = __shfl_sync(gmask, co[0], 0, LPT) - p.cseg_base;
    gfirst = __shfl_sync(gmask, go[0], 0, LPT) - p.gseg_base;
    const i64 Nc64 = cend - cfirst, Ng64 = gend - gfirst;
    if (cfirst < 0 || Nc64 < 0 || cend > p.n_csegs || Nc64 >= CAP || gfirst < 0 || Ng64 < 0 ||
        gend > p.n_gsegs || Ng64 >= CAP)
      return kFastDeclined;
    Nc = (int)Nc64, Ng = (int)Ng64;
    u32 high = 0;  // any set bit: some value does not fit the 32-bit path
    u32 D[SLOTS], core[SLOTS];
    int prio[SLOTS];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const bool v = lane + LPT * s < n;
      const i64 rc = co[s] - p.cseg_base - cfirst, rg = go[s] - p.gseg_base - gfirst;
      const u32 h = (u32)((u64)t64[s] >> 32) | (u32)((u64)d64[s] >> 32) | (u32)((u64)c64[s] >> 32) |
                    (u32)((u64)rc >> 32) | (u32)((u64)rg >> 32) |
                    (u32)(((u64)pr[s] + 0x80000000ull) >> 32);
      T[s] = v ? (u32)t64[s] : 2u;
      D[s] = (u32)d64[s];
      core[s] = (u32)c64[s];
      prio[s] = v ? (int)pr[s] : (int)0x80000000;
      c0[s] = v ? (int)rc : Nc;
      g0[s] = v ? (int)rg : Ng;
      high |= v ? h : 0u;
      // 2 <= T < 2^26, 1 <= D <= T, core < 2^31, offsets inside the slice
      ok &= T[s] - 2u < kFastLimit - 2u && (!v || (D[s] - 1u < T[s] && (int)core[s] >= 0)) &&
            (u32)c0[s] <= (u32)Nc && (u32)g0[s] <= (u32)Ng;
    }
    if (__any_sync(gmask, high != 0 || !ok)) return kFastDeclined;  // (a wide priority also lands here)
    // order: rank by (priority desc, position asc)
    int m = prio[0];
#pragma unroll
    for (int s = 1; s < SLOTS; ++s) m = prio[s] > m ? prio[s] : m;
    const int pmax = __reduce_max_sync(gmask, m);
    bool dense = true;  // distinct priorities max-n+1 .. max: the rank is max - priority
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const u32 r = (u32)pmax - (u32)prio[s];
      const bool v = lane + LPT * s < n;
      dense &= !v || r < (u32)n;
      rank[s] = v ? (int)r : MAXN;
    }
    dense = __all_sync(gmask, dense);
    if (dense) {
#pragma unroll
      for (int s = 0; s < SLOTS; ++s)
        if (lane + LPT * s < n) Q0[rank[s]] = (u32)(lane + LPT * s);
      __syncwarp(gmask);
      bool uniq = true;
#pragma unroll
      for (int s = 0; s < SLOTS; ++s)
        if (lane + LPT * s < n) uniq &= Q0[rank[s]] == (u32)(lane + LPT * s);
      dense = __all_sync(gmask, uniq);
      __syncwarp(gmask);
    }
    if (!dense) {  // any priorities: count the tasks that come before
#pragma unroll
      for (int s = 0; s < SLOTS; ++s) {
        const int i = lane + LPT * s;
        int r = 0;
        for (int q = 0; q < n; ++q) {
          const int pq = (int)p.priority[a + q];
          r += (pq > prio[s] || (pq == prio[s] && q < i)) ? 1 : 0;
        }
        rank[s] = i < n ? r : MAXN;
      }
    }
    // best-effort tasks (flag set, priority <= 0) rank behind every real-time task: the ranks
    // from n_rt on are theirs
    // (kept in a spare word in front of Q0's guard entry until the recurrence starts)
    {
      int n_rt = n;
      if (best_effort) {
#pragma unroll
        for (int s = 0; s < SLOTS; ++s)
          n_rt -= __popc(__ballot_sync(gmask, lane + LPT * s < n && prio[s] <= 0));
      }
      if (lane == 0) Q0[-2] = (u32)n_rt;
    }
    // what every lane must know about the task of a given rank (base and GPU flag follow; the
    // first ranks' own pass keeps the period and the position there instead)
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      if constexpr (FIRST_ONLY) {
        if (rank[s] < kFirstRanks) info[rank[s]] = make_uint4(D[s], core[s], T[s], (u32)(lane + LPT * s));
      } else {
        if (lane + LPT * s < n) *reinterpret_cast<uint2 *>(&info[rank[s]]) = make_uint2(D[s], core[s]);
      }
    }
  }
  // end offsets: the next task's start (positions beyond n hold the total)
  int c1[SLOTS], g1[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const int cn = __shfl_down_sync(gmask, c0[s], 1, LPT), gn = __shfl_down_sync(gmask, g0[s], 1, LPT);
    const int ch = __shfl_sync(gmask, s + 1 < SLOTS ? c0[s + 1 < SLOTS ? s + 1 : s] : Nc, 0, LPT);
    const int gh = __shfl_sync(gmask, s + 1 < SLOTS ? g0[s + 1 < SLOTS ? s + 1 : s] : Ng, 0, LPT);
    c1[s] = lane == LPT - 1 ? ch : cn;
    g1[s] = lane == LPT - 1 ? gh : gn;
    ok &= (u32)(c1[s] - c0[s]) < 64u && (u32)(g1[s] - g0[s]) < 64u;
  }
  if (!__all_sync(gmask, ok)) return kFastDeclined;

  // ---- aggregate: running sums of the segment arrays; per-task sums are differences --------
  u32 A[SLOTS], Ge[SLOTS], S[SLOTS];  // C+G^m, G^e, and 2*eps*eta (GCAPS) or (L+theta)*slices (RR)
  u32 bad = 0;
  const i64 *__restrict__ Xc = p.cseg_wcet + cfirst;
  const i64 *__restrict__ Xm = p.gseg_misc + gfirst, *__restrict__ Xe = p.gseg_exec + gfirst;
  const int parc = (int)(((uintptr_t)Xc >> 3) & 1), parm = (int)(((uintptr_t)Xm >> 3) & 1);
  const int pare = (int)(((uintptr_t)Xe >> 3) & 1);
  if constexpr (FIRST_ONLY) {
    constexpr int MODE = (MASK & 1) ? 0 : (MASK & 2) ? 1 : (MASK & 4) ? 2 : 3;
    uint4 *first8 = info + kFirstRanks;  // (only the first ranks' rows of `info` are used here)
#pragma unroll
    for (int s = 0; s < SLOTS; ++s)
      if (rank[s] < kFirstRanks) first8[rank[s]] = make_uint4((u32)c0[s], (u32)c1[s], (u32)g0[s], (u32)g1[s]);
    __syncwarp(gmask);
    const int r = first_ranks<SLOTS, MODE>(p, t, a, n, info, first8, Q0, Q1, (int)Q0[-2], rank, g0, g1, Xc, Xm, Xe,
                                           Nc, Ng, parc, parm, pare, cfirst, gfirst, lane, literal);
    __syncwarp(gmask);
    return r > 0 ? kFastDone : (r == 0 ? kFastUndecided : kFastDeclined);
  }
  if (lane == 0) Q0[-1] = 0, Q1[-1] = 0;
  {  // CPU segments -> Q0
    const bool inside = slice_is_inside(cfirst, Nc, parc, p.n_csegs);
    u32 carry = 0, unused = 0;
    for (int e0 = 0; e0 < Nc + parc; e0 += Lay::kStep * BC)
      prefix_step<LPT, BC, false>(Xc, Xc, e0, Nc, parc, parc, inside, p.cseg_wcet, p.cseg_wcet + p.n_csegs,
                             p.cseg_wcet, p.cseg_wcet, Q0, Q0, carry, unused, bad, lane, gmask);
  }
  __syncwarp(gmask);
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) A[s] = Q0[c1[s] - 1 + parc] - Q0[c0[s] - 1 + parc];
  __syncwarp(gmask);
  {  // G^m -> Q0, G^e -> Q1
    const bool inside = slice_is_inside(gfirst, Ng, parm, p.n_gsegs) &&
                        slice_is_inside(gfirst, Ng, pare, p.n_gsegs);
    u32 cm = 0, ce = 0;
    for (int e0 = 0; e0 < Ng + 1; e0 += Lay::kStep * BG)
      prefix_step<LPT, BG, true>(Xm, Xe, e0, Ng, parm, pare, inside, p.gseg_misc, p.gseg_misc + p.n_gsegs,
                            p.gseg_exec, p.gseg_exec + p.n_gsegs, Q0, Q1, cm, ce, bad, lane, gmask);
  }
  __syncwarp(gmask);
  u32 eta[SLOTS];
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const u32 Gm = Q0[g1[s] - 1 + parm] - Q0[g0[s] - 1 + parm];
    Ge[s] = Q1[g1[s] - 1 + pare] - Q1[g0[s] - 1 + pare];
    eta[s] = (u32)(g1[s] - g0[s]);
    bad |= (A[s] | Gm | Ge[s]) >> 26;
    A[s] += Gm;
    bad |= A[s] >> 26;
  }
  __syncwarp(gmask);
  // ---- what does not depend on the timeslice or the overhead ---------------------------------
  int n_gpu = 0;  // N_g
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) n_gpu += __popc(__ballot_sync(gmask, eta[s] > 0));
  if (kAnyGcaps) {  // 2 * eps * eta must stay below 2^26 (eta < 64, eps < 2^20: no overflow here)
    const u32 ovh_max = SWEEP ? (u32)sw->max_ovh : (u32)p.ovh;
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) bad |= (2 * ovh_max * eta[s]) >> 26;
  }
  if (__any_sync(gmask, bad != 0)) return kFastDeclined;
  const int n_rt_all = (int)Q0[-2];  // real-time tasks: the ranks that are analysed
  uint4 *xch = reinterpret_cast<uint4 *>(Q0);  // by rank: T, C+G^m, G^e, S  (Q0 is dead by now)

  // Eq. 3: running sums of the slices of every pure GPU part for timeslice L (values already
  // checked) into Ps
  auto slice_sums = [&](u32 *Ps, i64 L64, u32 l_mode, u32 l_magic, u32 l_shift) {
    // Eq. 3: slices of every pure GPU part, summed per task (values already checked)
    const bool inside = slice_is_inside(gfirst, Ng, pare, p.n_gsegs);
    u32 carry = 0;
    if (lane == 0) Ps[-1] = 0;
    for (int e0 = 0; e0 < Ng + 1; e0 += Lay::kStep * BG) {
      Quad qe[BG];
      u32 x[BG][4], incl[BG];
#pragma unroll
      for (int b = 0; b < BG; ++b) {
        if (inside) load_quad_inside(Xe, e0 + 4 * LPT * b + 4 * lane - pare, Ng, qe[b]);
        else qe[b] = load_quad_edge(Xe, e0 + 4 * LPT * b + 4 * lane - pare, Ng, p.gseg_exec, p.gseg_exec + p.n_gsegs);
      }
#pragma unroll
      for (int b = 0; b < BG; ++b) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          // a neighbour's element may be large: keep it below 2^26 so the division stays exact
          const u32 w = (u32)qe[b].v[j] & (kFastLimit - 1);
          u32 sq;
          if (l_mode == 0) sq = __umulhi(w + (u32)L64 - 1u, l_magic) >> l_shift;
          else if (l_mode == 1) sq = w;
          else sq = w > 0 ? 1u : 0u;
          x[b][j] = sq + (j > 0 ? x[b][j - 1] : 0u);
        }
        incl[b] = x[b][3];
      }
#pragma unroll
      for (int d = 1; d < LPT; d <<= 1) {
#pragma unroll
        for (int b = 0; b < BG; ++b) {
          const u32 y = __shfl_up_sync(gmask, incl[b], d, LPT);
          if (lane >= d) incl[b] += y;
        }
      }
#pragma unroll
      for (int b = 0; b < BG; ++b) {
        if (e0 + 4 * LPT * b < Ng + 1) {
          const u32 before = incl[b] - x[b][3] + carry;
          *reinterpret_cast<uint4 *>(Ps + e0 + 4 * LPT * b + 4 * lane) =
              make_uint4(x[b][0] + before, x[b][1] + before, x[b][2] + before, x[b][3] + before);
          carry += __shfl_sync(gmask, incl[b], LPT - 1, LPT);
        }
      }
    }
    __syncwarp(gmask);
  };

  // The recurrence of Eq. 1 for every real-time task in rank order under analysis MODE, once the
  // tasks sit in the lanes of their ranks: Sr = 2*eps*eta (GCAPS) or (L+theta)*slices (RR) of this
  // lane's tasks, info[rank].z = base.  Writes out_wcrt (unless null in a sweep) and out_sched.
  auto recurrence = [&](auto mode_tag, i64 *out_wcrt, uint8_t *out_sched) {
  constexpr int MODE = mode_tag;  // a ModeTag: every analysis of a kernel gets its own copy
  const int n_rt = n_rt_all;
  // by rank from here on: period - 1, C+G^m, G^e, core, position, GPU-using, and the two weights
  // of the analysis' pairs
  u32 Tm1[SLOTS], Ar[SLOTS], Ger[SLOTS], pos_of[SLOTS], core[SLOTS], Wa[SLOTS], Wb[SLOTS];
  bool gpu[SLOTS];
  u32 magic[SLOTS], shift[SLOTS];  // reciprocal of T_h, made when the slot is first needed
  int slots_made = 0;
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) {
    const int r = lane + LPT * s;
    const uint4 x = r < n ? xch[r] : make_uint4(2u, 0u, 0u, 0u);
    const uint4 f = r < n ? info[r] : make_uint4(0u, 0xffffffffu, 0u, 0u);
    const u32 Sr = x.w;  // 2*eps*eta (GCAPS) or (L+theta)*slices (RR) of this rank's task
    Tm1[s] = x.x - 1, Ar[s] = x.y, Ger[s] = x.z;
    core[s] = f.y, pos_of[s] = f.w & 0xffffu, gpu[s] = (f.w & 0x10000u) != 0;
    magic[s] = 0, shift[s] = 0;
    if (MODE == 0) {
      Wa[s] = Ar[s] + (gpu[s] ? Sr : 0u);    // Lemma 15: C_h, or C_h + G^{m*}_h
      Wb[s] = gpu[s] ? Ger[s] + Sr : 0u;     // Lemma 13, other cores: G^{e*}_h
    } else if (MODE == 1) {
      Wa[s] = Ar[s];                            // Lemma 12
      Wb[s] = gpu[s] ? Ger[s] + Sr : 0u;     // Lemmas 10, 11: G^{e*}_h
    } else {
      Wa[s] = Ar[s];                            // Lemmas 5, 7
      Wb[s] = gpu[s] ? Sr : 0u;              // Lemma 4: (L+theta) * slices
    }
  }

  // ---- iterate in rank order ------------------------------------------------------------------
  u32 Jc[SLOTS], Jg[SLOTS];               // jitters with T_h - 1 folded in (ceiling)
#pragma unroll
  for (int s = 0; s < SLOTS; ++s) Jc[s] = Jg[s] = Tm1[s];
  int n_done = n_rt;
  int verdict = 0;
  for (int pos = 0; pos < n_rt; ++pos) {
    const uint4 f = info[pos];
    const u32 Di = f.x, core_i = f.y, base_i = f.z;
    const bool gi = (f.w & 0x10000u) != 0;
    const int smax = (pos - 1) >> kLog;  // -1 for the first task: nothing interferes
    if (smax >= slots_made) {              // the first task that looks at slot smax
#pragma unroll
      for (int s = 0; s < SLOTS; ++s)
        if (s == smax) make_reciprocal(Tm1[s] + 1, magic[s], shift[s]);
      slots_made = smax + 1;
    }
    u32 nu = 0;
    if (MODE == 3) {  // Lemma 4: N_g - |{h in hpp(i): GPU-using}| + 1
      int c = 0;
#pragma unroll
      for (int s = 0; s < SLOTS; ++s)
        if (s <= smax) c += __popc(__ballot_sync(gmask, lane + LPT * s < pos && core[s] == core_i && gpu[s]));
      nu = (u32)(n_gpu - c + 1);
    }
    // the (J, W) pairs of this task's interferers; W = 0 where a pair does not apply
    u32 J1[SLOTS], W1[SLOTS], W2[SLOTS];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      J1[s] = 0, W1[s] = 0, W2[s] = 0;
      if (s <= smax) {
        const bool act = lane + LPT * s < pos;
        const bool same = core[s] == core_i;
        u32 w1, w2 = 0, j1;
        if (MODE == 0) {
          w1 = same ? Wa[s] : (gi ? Wb[s] : 0u);           // Lemma 15 / Lemma 13 (other cores)
          j1 = same ? Jc[s] : Jg[s];
          w2 = (same && gi && gpu[s]) ? Ger[s] : 0u;       // Lemma 13 (same core), jitter J^g
        } else if (MODE == 1) {
          w1 = same ? Wa[s] + ((gi || !literal) ? Wb[s] : 0u) : Wb[s];  // Lemmas 12+10 / 10, 11
          j1 = same ? Tm1[s] : Jg[s];
        } else if (MODE == 2) {
          w1 = same ? Wa[s] : 0u;                          // Lemma 7
          j1 = Jc[s];
        } else {
          const u64 w = (u64)Wa[s] + (u64)Wb[s] * nu;      // Lemmas 5 and 4
          w1 = same ? (w > kFastClamp ? kFastClamp : (u32)w) : 0u;
          j1 = Tm1[s];
        }
        J1[s] = j1, W1[s] = act ? w1 : 0u, W2[s] = act ? w2 : 0u;
      }
    }
    u32 R = base_i;
    int v = 0;
    int sweeps = 0;
    for (;;) {
      if (R > Di) {
        v = GCAPS_WCRT_MISS;
        break;
      }
      if (sweeps >= (int)GCAPS_RTA_ITER_CAP) {
        v = GCAPS_WCRT_ITER_LIMIT;
        break;
      }
      sweeps += 1;
      u32 next = base_i;
      if (smax >= 0) {
        u64 acc = 0;
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) {
          if (s <= smax) {
            acc += (u64)(__umulhi(R + J1[s], magic[s]) >> shift[s]) * W1[s];
            if (MODE == 0) acc += (u64)(__umulhi(R + Jg[s], magic[s]) >> shift[s]) * W2[s];
          }
        }
        const u32 part = acc > (u64)kFastClamp ? kFastClamp : (u32)acc;
        next += __reduce_add_sync(gmask, part);
      }
      if (next == R) break;
      R = next;
    }
    if (v != 0) {
      n_done = pos;
      verdict = v;
      break;
    }
    // publish: the owner writes R_i and forms its jitters J^c = R - (C+G^m), J^g = R - G^e (a
    // CPU-only task has no J^c unless the printed form of Lemma 7 is asked for)
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      if (lane + LPT * s == pos) {
        if (!SWEEP || out_wcrt) out_wcrt[a + pos_of[s]] = (i64)R;
        if (MODE == 0 ? gpu[s] : (MODE == 2 ? (gpu[s] || literal) : false)) Jc[s] = R - Ar[s] + Tm1[s];
        Jg[s] = R - Ger[s] + Tm1[s];
      }
    }
  }
  // ---- write the sentinels of the tasks that did not converge ---------------------------------
  if (!SWEEP || out_wcrt) {
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      const int r = lane + LPT * s;
      if (r < n && r >= n_done)
        out_wcrt[a + pos_of[s]] = r >= n_rt ? (i64)GCAPS_WCRT_BEST_EFFORT
                                          : (r == n_done ? (i64)verdict : (i64)GCAPS_WCRT_SKIPPED);
    }
  }
  if (lane == 0) out_sched[t] = verdict == 0 ? GCAPS_SCHED_YES : GCAPS_SCHED_NO;
  __syncwarp(gmask);
  };  // recurrence

  if constexpr (!SWEEP) {
    // ---- one analysis: constants by position, then everything moves to the rank's lane ---------
    constexpr int MODE = (MASK & 1) ? 0 : (MASK & 2) ? 1 : (MASK & 4) ? 2 : 3;
    constexpr bool kGcaps = MODE < 2;
    const u32 ovh = (u32)p.ovh;  // the fast path needs eps, theta < 2^20
    u32 sl[SLOTS];               // RR: slices of the task's pure GPU parts (Eq. 3)
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) sl[s] = 0;
    if (!kGcaps) {
      slice_sums(Q0, p.L, p.l_mode, p.l_magic, p.l_shift);
      __syncwarp(gmask);
#pragma unroll
      for (int s = 0; s < SLOTS; ++s) sl[s] = Q0[g1[s] - 1 + pare] - Q0[g0[s] - 1 + pare];
      __syncwarp(gmask);
    }
    u32 base[SLOTS];
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      if (kGcaps) {
        S[s] = 2 * ovh * eta[s];                                 // eta < 64: below 2^27
        base[s] = A[s] + Ge[s] + S[s] + (eta[s] + 1) * ovh;        // C_i + G*_i + B^C_i, below 2^29
      } else {
        const u64 slices = sl[s];
        const u64 lt = (u64)p.L + ovh;  // <= 2^41
        u64 B = slices == 0 ? 0 : (lt >= kFastClamp ? kFastClamp : lt * slices);  // < 2^26 * 2^32
        if (B > kFastClamp) B = kFastClamp;
        S[s] = (u32)B;
        const u64 b64 = (u64)A[s] + Ge[s] + (eta[s] > 0 ? B * (u64)(n_gpu - 1) : 0);  // Lemma 1
        base[s] = b64 > (u64)(2 * kFastClamp) ? 2 * kFastClamp : (u32)b64;
      }
      base[s] = base[s] > 2 * kFastClamp ? 2 * kFastClamp : base[s];
    }
    __syncwarp(gmask);
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      if (lane + LPT * s < n) {
        *(reinterpret_cast<uint2 *>(&info[rank[s]]) + 1) =
            make_uint2(base[s], (u32)(lane + LPT * s) | (eta[s] > 0 ? 0x10000u : 0u));
        xch[rank[s]] = make_uint4(T[s], A[s], Ge[s], S[s]);
      }
    }
    __syncwarp(gmask);
    recurrence(ModeTag<MODE>(), p.out_wcrt, p.out_sched);
  } else {
    // ---- several analyses: the tasks move to the rows of their ranks once; for every analysis
    // the lane of a rank then makes that task's S and base from the row and the recurrence
    // starts from the rows again, so nothing per task is held in registers across analyses ------
    // second row by rank: GPU segment range (11 bits each) and number of GPU segments (6 bits)
    // packed in .x, slices of Eq. 3 for the timeslice sl_L in .y
    uint2 *xch2 = reinterpret_cast<uint2 *>(Q0 + 4 * MAXN);
    static_assert(Lay::CAP <= 2048 && Lay::CAP >= 6 * MAXN, "packed segment range, room for the second row");
#pragma unroll
    for (int s = 0; s < SLOTS; ++s) {
      if (lane + LPT * s < n) {
        info[rank[s]].w = (u32)(lane + LPT * s) | (eta[s] > 0 ? 0x10000u : 0u);
        xch[rank[s]] = make_uint4(T[s], A[s], Ge[s], 0u);
        xch2[rank[s]] = make_uint2((u32)g0[s] | ((u32)g1[s] << 11) | (eta[s] << 22), 0u);
      }
    }
    __syncwarp(gmask);
    i64 sl_L = -1;
    constexpr bool kMultiModes = (MASK & (MASK - 1)) != 0;
    const int enabled = kMultiModes ? sw->enabled : MASK;
    for (int q = 0; q < sw->n; ++q) {
      const i64 L64 = sw->q[q].L;
      const u32 ovh = (u32)sw->q[q].ovh;  // the fast path needs eps, theta < 2^20
      auto analyse_as = [&](auto mode_tag) {
        constexpr int MODE = mode_tag;
        constexpr bool kGcaps = MODE < 2;
        const int block = q * sw->block_stride + sw->block_of_mode[MODE];
        i64 *const out_wcrt = p.out_wcrt ? p.out_wcrt + (i64)block * p.n_tasks : nullptr;
        uint8_t *const out_sched = p.out_sched + (i64)block * p.n_tasksets;
        if (!kGcaps && L64 != sl_L) {
          sl_L = L64;
          slice_sums(Q1, L64, sw->q[q].l_mode, sw->q[q].l_magic, sw->q[q].l_shift);
          __syncwarp(gmask);
#pragma unroll
          for (int s = 0; s < SLOTS; ++s) {
            const int r = lane + LPT * s;
            if (r < n) {
              const u32 g = xch2[r].x;
              xch2[r].y = Q1[(int)((g >> 11) & 0x7ffu) - 1 + pare] - Q1[(int)(g & 0x7ffu) - 1 + pare];
            }
          }
        }
#pragma unroll
        for (int s = 0; s < SLOTS; ++s) {
          const int r = lane + LPT * s;
          if (r < n) {
            const uint4 x = xch[r];
            const uint2 g = xch2[r];
            const u32 eta_r = g.x >> 22;
            u32 Sr, base;
            if (kGcaps) {
              Sr = 2 * ovh * eta_r;                                 // eta < 64: below 2^27
              base = x.y + x.z + Sr + (eta_r + 1) * ovh;             // C_i + G*_i + B^C_i, below 2^29
            } else {
              const u64 slices = g.y;
              const u64 lt = (u64)L64 + ovh;  // <= 2^41
              u64 B = slices == 0 ? 0 : (lt >= kFastClamp ? kFastClamp : lt * slices);
              if (B > kFastClamp) B = kFastClamp;
              Sr = (u32)B;
              const u64 b64 = (u64)x.y + x.z + (eta_r > 0 ? B * (u64)(n_gpu - 1) : 0);  // Lemma 1
              base = b64 > (u64)(2 * kFastClamp) ? 2 * kFastClamp : (u32)b64;
            }
            base = base > 2 * kFastClamp ? 2 * kFastClamp : base;
            xch[r].w = Sr;
            info[r].z = base;
          }
        }
        __syncwarp(gmask);
        recurrence(mode_tag, out_wcrt, out_sched);
      };
      if ((MASK & 1) && (enabled & 1)) analyse_as(ModeTag<0>());
      if ((MASK & 2) && (enabled & 2)) analyse_as(ModeTag<1>());
      if ((MASK & 4) && (enabled & 4)) analyse_as(ModeTag<2>());
      if ((MASK & 8) && (enabled & 8)) analyse_as(ModeTag<3>());
    }
  }
  return kFastDone;
}

__device__ __forceinline__ void prefetch_l2(const void *ptr) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(ptr));
}

// What a warp knows in advance about one taskset of a chunk (kept in shared memory).
struct Ahead {
  i64 a;           // first task
  i64 c_lo, g_lo;  // first CPU segment, first GPU segment
  u32 t;           // taskset index
  u32 packed;      // tasks (bits 0-8) | CPU segments (9-19) | GPU segments (20-30) | fast (31)
};
static_assert(sizeof(Ahead) == 32, "two 16-byte rows");
constexpr int kMaxAhead = 16;  // tasksets of one pull
constexpr int kAheadWords = 2 * kMaxAhead * (int)(sizeof(Ahead) / sizeof(u32));  // two chunks

// blocks per SM the register allocation aims at: more warps in flight matter more here than a
// few spilled values, because every phase is a chain of dependent instructions and the loads of
// a taskset can only be hidden behind the work of other warps
__host__ __device__ constexpr int min_blocks(int slots) {
  return slots <= 3 ? 6 : slots == 4 ? 4 : slots == 6 ? 3 : 2;
}

// One size bin, worked through by all warps of a persistent launch.  A warp is 32/LPT groups of
// LPT lanes; every group analyses one taskset at a time.  Warps pull chunks of taskset indices
// from the bin's counter; the index, task range and first segment offsets of the next chunk are
// fetched while the current one is analysed.
template <int LPT, int SLOTS, int MASK, bool SWEEP = false>
__device__ __forceinline__ void run_bin(const KParams &p, int bin, u32 *warp_buf, Ahead *ahead,
                                        const SweepArgs *sw = nullptr) {
  typedef FastLayout<LPT, SLOTS> Lay;
  constexpr int MAXN = LPT * SLOTS;
  constexpr int G = 32 / LPT;  // groups per warp
  static_assert(sizeof(GroupSmem<MAXN>) <= sizeof(u32) * Lay::kWords, "exact path fits");
  const int lane32 = threadIdx.x & 31, group = lane32 / LPT, lane = lane32 % LPT;
  const unsigned int gmask = LPT == 32 ? kFull : (((1u << LPT) - 1u) << (group * LPT));
  u32 *buf = warp_buf + group * Lay::kWords;
  const unsigned int start = p.hdr->bin_start[bin], count = p.hdr->bin_count[bin];
  if (count == 0) return;
  // keeps 2*eps*eta and (eta+1)*eps in 32 bits
  const bool fast_call = (SWEEP ? sw->max_ovh : p.ovh) < (1 << 20);
  // tasksets per pull: up to 8 per group when the bin is large, fewer when that would leave warps
  // without work
  const unsigned int n_groups = gridDim.x * (kBlockThreads / 32) * G;
  const int rounds = count >= 32 * n_groups ? (G == 1 ? 8 : kMaxAhead / G)
                                            : (count >= 8 * n_groups ? 4 / (G > 2 ? 2 : 1) : 1);
  const int chunk = rounds * G;  // <= kMaxAhead

  // lanes 0..chunk-1 each look up one taskset of a chunk and leave what they found in `slot`
  auto look_up = [&](unsigned int first, Ahead *slot) {
    if (lane32 < chunk) {
      Ahead me;
      me.a = 0, me.c_lo = me.g_lo = 0, me.t = 0, me.packed = 0;
      if (first < count && first + lane32 < count) {
        me.t = p.perm[start + first + lane32];
        me.a = p.task_off[me.t] - p.task_base;
        const i64 b = p.task_off[(i64)me.t + 1] - p.task_base;
        if (me.a >= 0 && b > me.a && b <= p.n_tasks && b - me.a <= MAXN) {
          u32 nc = 0, ng = 0;
          me.c_lo = p.cseg_off[me.a] - p.cseg_base, me.g_lo = p.gseg_off[me.a] - p.gseg_base;
          const i64 c_hi = p.cseg_off[b] - p.cseg_base, g_hi = p.gseg_off[b] - p.gseg_base;
          if (me.c_lo >= 0 && c_hi <= p.n_csegs && c_hi - me.c_lo < Lay::CAP && c_hi > me.c_lo)
            nc = (u32)(c_hi - me.c_lo);
          if (me.g_lo >= 0 && g_hi <= p.n_gsegs && g_hi - me.g_lo < Lay::CAP && g_hi > me.g_lo)
            ng = (u32)(g_hi - me.g_lo);
          me.packed = (u32)(b - me.a) | (nc << 9) | (ng << 20) | 0x80000000u;
        }
      }
      slot[lane32] = me;
    }
    __syncwarp();
  };
  static_assert(MAXN <= 256 && Lay::CAP <= 2048, "fields of Ahead::packed");

  int undecided_run = 0, tried_since = 0;  // (the first ranks' own pass, see below)
  unsigned int first = 0;
  if (lane32 == 0) first = atomicAdd(&p.hdr->next[bin], (unsigned int)chunk);
  first = __shfl_sync(kFull, first, 0);
  int which = 0;
  look_up(first, ahead);
  while (first < count) {
    unsigned int nfirst = 0;
    if (lane32 == 0) nfirst = atomicAdd(&p.hdr->next[bin], (unsigned int)chunk);
    const Ahead *cur = ahead + which * kMaxAhead;
    Ahead *nxt = ahead + (which ^ 1) * kMaxAhead;
    const int in_chunk = count - first < (unsigned int)chunk ? (int)(count - first) : chunk;
    const int in_rounds = (in_chunk + G - 1) / G;
    for (int c = 0; c < in_rounds; ++c) {
      if (c == 1 || in_rounds == 1) {  // the next chunk's index has arrived by now
        nfirst = __shfl_sync(kFull, nfirst, 0);
        look_up(nfirst, nxt);
      }
      const int mine = c * G + group;
      if (mine < in_chunk) {
        const Ahead me = cur[mine];
        const i64 t = (i64)me.t;
        const int n = (int)(me.packed & 0x1ffu), nc = (int)((me.packed >> 9) & 0x7ffu);
        const int ng = (int)((me.packed >> 20) & 0x7ffu);
        // the segment slices start their way into L2 now; the per-task loads follow at once, so
        // that the running sums later wait for L2 rather than for DRAM (16 elements per line,
        // only addresses inside the arrays)
        for (int e = 16 * lane; e < nc; e += 16 * LPT) prefetch_l2(p.cseg_wcet + me.c_lo + e);
        for (int e = 16 * lane; e < ng; e += 16 * LPT)
          prefetch_l2(p.gseg_misc + me.g_lo + e), prefetch_l2(p.gseg_exec + me.g_lo + e);
#if GCAPS_PREFETCH_AHEAD
        // the per-task arrays of the group's next taskset of this pull start their way into L2 while
        // this one is analysed (one 128-byte line per lane and array; a taskset has at most 256
        // tasks, i.e. 17 lines of an array)
        if (mine + G < in_chunk) {
          const Ahead nx = cur[mine + G];
          const int nn = (int)(nx.packed & 0x1ffu);
          if ((nx.packed >> 31) != 0 && lane < 17) {
            const i64 *arrays[6] = {p.period, p.deadline, p.priority, p.core, p.cseg_off, p.gseg_off};
#pragma unroll
            for (int k = 0; k < 6; ++k) {
              const uintptr_t lo = reinterpret_cast<uintptr_t>(arrays[k] + nx.a);
              const uintptr_t line = (lo & ~(uintptr_t)127) + 128u * (unsigned)lane;
              if (line < lo + 8u * (unsigned)(nn + (k >= 4 ? 1 : 0))) prefetch_l2(reinterpret_cast<const void *>(line));
            }
          }
#if GCAPS_PREFETCH_AHEAD > 1
          const int nnc = (int)((nx.packed >> 9) & 0x7ffu), nng = (int)((nx.packed >> 20) & 0x7ffu);
          for (int e = 16 * lane; e < nnc; e += 16 * LPT) prefetch_l2(p.cseg_wcet + nx.c_lo + e);
          for (int e = 16 * lane; e < nng; e += 16 * LPT)
            prefetch_l2(p.gseg_misc + nx.g_lo + e), prefetch_l2(p.gseg_exec + nx.g_lo + e);
#endif
        }
#endif
        bool done = false;
        if (fast_call && (me.packed >> 31) != 0) {
          int how = kFastUndecided;
          if constexpr (LPT == 32 && !SWEEP && (MASK & 12) != 0 && GCAPS_FIRST_RANKS != 0) {
            // Far from schedulable, a taskset ends with a miss among its first ranks; nearly
            // schedulable, looking at them first is wasted.  Tasksets of a batch tend to be alike:
            // after four undecided ones in a row only every sixteenth taskset is tried that way.
            // (Round robin only: with tens of GPU-using tasks taking turns on the GPU the first or
            // second rank already misses, and the pass pays; under GCAPS the first miss comes a few
            // ranks later and the pass was measured slower than the full one.)
            if (undecided_run < 4 || (tried_since & 15) == 0) {
              how = analyse_fast<LPT, SLOTS, MASK, false, true>(p, t, me.a, n, buf, lane, gmask);
              undecided_run = how == kFastUndecided ? undecided_run + 1 : 0;
              __syncwarp(gmask);
            }
            tried_since += 1;
          }
          if (how == kFastUndecided) how = analyse_fast<LPT, SLOTS, MASK, SWEEP>(p, t, me.a, n, buf, lane, gmask, sw);
          done = how == kFastDone;
        }
        __syncwarp(gmask);
        if (!done && !SWEEP) {
          // the exact path reads task_off again and validates everything itself
          analyse_taskset<LPT, MAXN>(p, t, *reinterpret_cast<GroupSmem<MAXN> *>(buf), lane, gmask);
        }
        if (!done && SWEEP) {  // the exact path once per (timeslice, overhead) pair
          constexpr bool kMulti = (MASK & (MASK - 1)) != 0;
          const int enabled = kMulti ? sw->enabled : MASK;
          for (int q = 0; q < sw->n; ++q) {
            for (int m = 0; m < 4; ++m) {
              if (!((MASK & enabled) >> m & 1)) continue;
              const int block = q * sw->block_stride + sw->block_of_mode[m];
              KParams pq = p;
              pq.policy = (p.policy & ~(0xff | GCAPS_RTA_BUSY)) | (m >= 2 ? GCAPS_POLICY_RR : GCAPS_POLICY_GCAPS) |
                          ((m & 1) ? GCAPS_RTA_BUSY : 0);
              pq.L = sw->q[q].L, pq.ovh = sw->q[q].ovh;
              pq.out_wcrt = p.out_wcrt ? p.out_wcrt + (i64)block * p.n_tasks : nullptr;
              pq.out_sched = p.out_sched + (i64)block * p.n_tasksets;
              analyse_taskset<LPT, MAXN>(pq, t, *reinterpret_cast<GroupSmem<MAXN> *>(buf), lane, gmask);
              __syncwarp(gmask);
            }
          }
        }
      }
      __syncwarp();
    }
    first = nfirst;
    which ^= 1;
  }
}

// shared memory of one warp for the bins a kernel covers
template <int LPT, int SLOTS>
__host__ __device__ constexpr int bin_warp_words() {
  return (32 / LPT) * FastLayout<LPT, SLOTS>::kWords;
}
__host__ __device__ constexpr int cmax(int a, int b) { return a > b ? a : b; }
constexpr int kSmallWarpWords =
    cmax(cmax(bin_warp_words<8, 1>(), bin_warp_words<8, 2>()),
         cmax(bin_warp_words<8, 3>(), bin_warp_words<16, 2>())) + kAheadWords;

// The bins of up to 32 tasks in one persistent launch, largest tasksets first: (lanes per
// taskset, tasks per lane) = (16,2) (8,3) (8,2) (8,1) for at most 32, 24, 16, 8 tasks, i.e. two or
// four tasksets per warp.
template <int MODE>
__global__ void __launch_bounds__(kBlockThreads, min_blocks(3)) rta_small_kernel(KParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();  // the kernel of the next size bin shares no data with this one
  u32 *warp_buf = reinterpret_cast<u32 *>(smem_raw) + (threadIdx.x >> 5) * kSmallWarpWords;
  Ahead *ahead = reinterpret_cast<Ahead *>(warp_buf + kSmallWarpWords - kAheadWords);
  run_bin<16, 2, 1 << MODE>(p, 3, warp_buf, ahead);
  run_bin<8, 3, 1 << MODE>(p, 2, warp_buf, ahead);
  run_bin<8, 2, 1 << MODE>(p, 1, warp_buf, ahead);
  run_bin<8, 1, 1 << MODE>(p, 0, warp_buf, ahead);
  wait_for_previous_grid();
}

// One bin of larger tasksets (a warp per taskset, 2, 3, 4, 6 or 8 tasks per lane) per launch.
template <int SLOTS, int MODE>
__global__ void __launch_bounds__(kBlockThreads, min_blocks(SLOTS)) rta_big_kernel(KParams p, int bin) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();  // the kernel of the next size bin shares no data with this one
  constexpr int kWarpWords = bin_warp_words<32, SLOTS>() + kAheadWords;
  u32 *warp_buf = reinterpret_cast<u32 *>(smem_raw) + (threadIdx.x >> 5) * kWarpWords;
  Ahead *ahead = reinterpret_cast<Ahead *>(warp_buf + kWarpWords - kAheadWords);
  run_bin<32, SLOTS, 1 << MODE>(p, bin, warp_buf, ahead);
  wait_for_previous_grid();
}

// All nine bins in one launch, for batches so small (at most kPlanSmall tasksets) that the
// launches of a call cost more than its work: a call is then the one-block plan kernel and this.
// Registers and shared memory are those of the largest bin, which such a batch can afford.
#ifdef GCAPS_RTA_ANY_TU
constexpr int kAnyWarpWords = cmax(kSmallWarpWords, bin_warp_words<32, 8>() + kAheadWords);
template <int MODE>
__global__ void __launch_bounds__(kBlockThreads, 2) rta_any_kernel(KParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();
  u32 *warp_buf = reinterpret_cast<u32 *>(smem_raw) + (threadIdx.x >> 5) * kAnyWarpWords;
  Ahead *ahead = reinterpret_cast<Ahead *>(warp_buf + kAnyWarpWords - kAheadWords);
  run_bin<32, 8, 1 << MODE>(p, 8, warp_buf, ahead);
  run_bin<32, 6, 1 << MODE>(p, 7, warp_buf, ahead);
  run_bin<32, 4, 1 << MODE>(p, 6, warp_buf, ahead);
  run_bin<32, 3, 1 << MODE>(p, 5, warp_buf, ahead);
  run_bin<32, 2, 1 << MODE>(p, 4, warp_buf, ahead);
  run_bin<16, 2, 1 << MODE>(p, 3, warp_buf, ahead);
  run_bin<8, 3, 1 << MODE>(p, 2, warp_buf, ahead);
  run_bin<8, 2, 1 << MODE>(p, 1, warp_buf, ahead);
  run_bin<8, 1, 1 << MODE>(p, 0, warp_buf, ahead);
  wait_for_previous_grid();
}
#endif  // GCAPS_RTA_ANY_TU

// The same launches for a fused sweep: every taskset is read once and analysed under all the
// (timeslice, overhead) pairs of `sw`.
template <int MASK>
__global__ void __launch_bounds__(kBlockThreads, min_blocks(3))
rta_small_sweep_kernel(KParams p, const __grid_constant__ SweepArgs sw) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();  // the kernel of the next size bin shares no data with this one
  u32 *warp_buf = reinterpret_cast<u32 *>(smem_raw) + (threadIdx.x >> 5) * kSmallWarpWords;
  Ahead *ahead = reinterpret_cast<Ahead *>(warp_buf + kSmallWarpWords - kAheadWords);
  run_bin<16, 2, MASK, true>(p, 3, warp_buf, ahead, &sw);
  run_bin<8, 3, MASK, true>(p, 2, warp_buf, ahead, &sw);
  run_bin<8, 2, MASK, true>(p, 1, warp_buf, ahead, &sw);
  run_bin<8, 1, MASK, true>(p, 0, warp_buf, ahead, &sw);
  wait_for_previous_grid();
}

template <int SLOTS, int MASK>
__global__ void __launch_bounds__(kBlockThreads, min_blocks(SLOTS))
rta_big_sweep_kernel(KParams p, int bin, const __grid_constant__ SweepArgs sw) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();  // the kernel of the next size bin shares no data with this one
  constexpr int kWarpWords = bin_warp_words<32, SLOTS>() + kAheadWords;
  u32 *warp_buf = reinterpret_cast<u32 *>(smem_raw) + (threadIdx.x >> 5) * kWarpWords;
  Ahead *ahead = reinterpret_cast<Ahead *>(warp_buf + kWarpWords - kAheadWords);
  run_bin<32, SLOTS, MASK, true>(p, bin, warp_buf, ahead, &sw);
  wait_for_previous_grid();
}

// ---------------------------------------------------------------------------------------------
// validation kernel: one thread per taskset
// ---------------------------------------------------------------------------------------------
__global__ void validate_kernel(KParams p, int32_t *out_err) {
  const i64 t = (i64)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= p.n_tasksets) return;
  const i64 a = p.task_off[t], b = p.task_off[t + 1];
  if (a < 0 || b < a || b > p.n_tasks || b - a > GCAPS_RTA_MAX_TASKS) {
    out_err[t] = GCAPS_BAD_TASK_RANGE;
    return;
  }
  int bad = 0;
  for (i64 k = a; k < b; ++k) {
    const i64 c0 = p.cseg_off[k], c1 = p.cseg_off[k + 1], g0 = p.gseg_off[k], g1 = p.gseg_off[k + 1];
    const bool seg_ok = !(c0 < 0 || c1 < c0 || c1 > p.n_csegs || c1 - c0 > GCAPS_RTA_MAX_SEGMENTS ||
                          g0 < 0 || g1 < g0 || g1 > p.n_gsegs || g1 - g0 > GCAPS_RTA_MAX_SEGMENTS);
    if (!seg_ok) bad |= GCAPS_BAD_SEG_RANGE;
    const i64 T = p.period[k], D = p.deadline[k], c = p.core[k];
    if (T < 1 || T > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_PERIOD;
    if (D < 1 || D > T) bad |= GCAPS_BAD_DEADLINE;
    if (c < 0 || c > GCAPS_RTA_MAX_CORE) bad |= GCAPS_BAD_CORE;
    if (seg_ok) {
      for (i64 j = c0; j < c1; ++j)
        if (p.cseg_wcet[j] < 0 || p.cseg_wcet[j] > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_WCET;
      for (i64 j = g0; j < g1; ++j)
        if (p.gseg_misc[j] < 0 || p.gseg_misc[j] > GCAPS_RTA_MAX_TIME || p.gseg_exec[j] < 0 ||
            p.gseg_exec[j] > GCAPS_RTA_MAX_TIME)
          bad |= GCAPS_BAD_WCET;
    }
  }
  out_err[t] = bad;
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t plan_blocks(int64_t n_tasksets) { return (size_t)((n_tasksets + kPlanItems - 1) / kPlanItems); }

}  // namespace

#ifdef GCAPS_RTA_ANY_TU
// This file compiled as gcaps_rta_any.cu: only the all-bins kernels and their launcher (they
// hold one copy of the device code per size bin and analysis, and compiling them beside the
// other kernels rather than after them shortens the build).
namespace gcaps_detail {

cudaError_t launch_any_bins(int mode, const KParams &p, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  static int blocks_per_sm[4][64] = {{0}};
  const size_t smem = sizeof(u32) * kAnyWarpWords * kWarps;
  const long long want = (p.n_tasksets + kWarps - 1) / kWarps;
  switch (mode) {
    case 0: return launch_persistent(rta_any_kernel<0>, blocks_per_sm[0], smem, want, sm_count, st, p);
    case 1: return launch_persistent(rta_any_kernel<1>, blocks_per_sm[1], smem, want, sm_count, st, p);
    case 2: return launch_persistent(rta_any_kernel<2>, blocks_per_sm[2], smem, want, sm_count, st, p);
    case 3: return launch_persistent(rta_any_kernel<3>, blocks_per_sm[3], smem, want, sm_count, st, p);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace gcaps_detail
#else

// ---------------------------------------------------------------------------------------------
// host side shared with the other translation units of the library
// ---------------------------------------------------------------------------------------------
namespace gcaps_detail {

thread_local int g_last_cuda_error = 0;
std::mutex g_init_mutex;

static DeviceInfo g_dev[64];

int device_info(DeviceInfo *out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_NO_DEVICE;
  }
  if (dev < 0 || dev >= 64) return GCAPS_ERR_NO_DEVICE;
  std::lock_guard<std::mutex> lock(g_init_mutex);
  if (g_dev[dev].ok == 0) {
    int major = 0, sms = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) {
      g_last_cuda_error = (int)e;
      return GCAPS_ERR_NO_DEVICE;
    }
    g_dev[dev].sm_count = sms;
    g_dev[dev].ok = major == 10 ? 1 : -1;
  }
  if (g_dev[dev].ok != 1) return GCAPS_ERR_NO_DEVICE;
  *out = g_dev[dev];
  return GCAPS_OK;
}

int check_args(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int64_t L, int64_t ovh) {
  if (!ts || n_tasksets < 0 || n_tasksets > 0x7fffffffLL) return GCAPS_ERR_INVALID_ARG;
  const int pol = policy & 0xff;
  if (pol != GCAPS_POLICY_GCAPS && pol != GCAPS_POLICY_RR) return GCAPS_ERR_INVALID_ARG;
  if (policy & ~(0xff | GCAPS_RTA_BUSY | GCAPS_RTA_LITERAL | GCAPS_RTA_BEST_EFFORT))
    return GCAPS_ERR_INVALID_ARG;
  if (ovh < 0 || ovh > GCAPS_RTA_MAX_TIME) return GCAPS_ERR_INVALID_ARG;
  if (pol == GCAPS_POLICY_RR && (L < 1 || L > GCAPS_RTA_MAX_TIME)) return GCAPS_ERR_INVALID_ARG;
  if (ts->n_tasks < 0 || ts->n_csegs < 0 || ts->n_gsegs < 0) return GCAPS_ERR_INVALID_ARG;
  if (n_tasksets > 0) {
    if (!ts->task_off) return GCAPS_ERR_INVALID_ARG;
    if (ts->n_tasks > 0 && (!ts->period || !ts->deadline || !ts->priority || !ts->core ||
                            !ts->cseg_off || !ts->gseg_off))
      return GCAPS_ERR_INVALID_ARG;
    if (ts->n_csegs > 0 && !ts->cseg_wcet) return GCAPS_ERR_INVALID_ARG;
    if (ts->n_gsegs > 0 && (!ts->gseg_misc || !ts->gseg_exec)) return GCAPS_ERR_INVALID_ARG;
  }
  return GCAPS_OK;
}

void fill_params(KParams *p, const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int64_t L,
                 int64_t ovh, int64_t *out_wcrt, uint8_t *out_sched) {
  memset(p, 0, sizeof(*p));
  p->task_off = (const i64 *)ts->task_off;
  p->period = (const i64 *)ts->period;
  p->deadline = (const i64 *)ts->deadline;
  p->priority = (const i64 *)ts->priority;
  p->core = (const i64 *)ts->core;
  p->cseg_off = (const i64 *)ts->cseg_off;
  p->cseg_wcet = (const i64 *)ts->cseg_wcet;
  p->gseg_off = (const i64 *)ts->gseg_off;
  p->gseg_misc = (const i64 *)ts->gseg_misc;
  p->gseg_exec = (const i64 *)ts->gseg_exec;
  p->n_tasks = ts->n_tasks;
  p->n_csegs = ts->n_csegs;
  p->n_gsegs = ts->n_gsegs;
  p->n_tasksets = n_tasksets;
  p->policy = policy;
  p->L = (policy & 0xff) == GCAPS_POLICY_RR ? L : 1;
  p->ovh = ovh;
  if (p->L == 1) {
    p->l_mode = 1;
  } else if (p->L >= (i64)kFastLimit) {
    p->l_mode = 2;
  } else {
    p->l_mode = 0;
    make_reciprocal((u32)p->L, p->l_magic, p->l_shift);
  }
  p->out_wcrt = (i64 *)out_wcrt;
  p->out_sched = out_sched;
}

int enqueue_plan(KParams &p, void *workspace, size_t workspace_bytes, cudaStream_t st) {
  const size_t need = gcaps_rta_workspace_bytes(p.n_tasksets);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255u))
    return GCAPS_ERR_WORKSPACE;
  unsigned char *w = (unsigned char *)workspace;
  const size_t nb = plan_blocks(p.n_tasksets);
  p.hdr = (PlanHeader *)w;
  p.block_cnt = (unsigned int *)(w + 256);
  p.perm = (unsigned int *)(w + 256 + align_up(nb * kBinStride * sizeof(unsigned int), 256));
  if (p.n_tasksets <= kPlanSmall) {
    plan_small_kernel<<<1, 1024, 0, st>>>(p);
    return GCAPS_OK;
  }
  plan_count_kernel<<<(unsigned int)nb, 256, 0, st>>>(p);
  plan_scan_kernel<<<1, 32 * kNumBins, 0, st>>>(p, (unsigned int)nb);
  plan_scatter_kernel<<<(unsigned int)nb, 256, 0, st>>>(p);
  return GCAPS_OK;
}

}  // namespace gcaps_detail

namespace {

template <int SLOTS, int MODE>
cudaError_t launch_big(const KParams &p, int bin, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  static int blocks_per_sm[64] = {0};
  const size_t smem = sizeof(u32) * (bin_warp_words<32, SLOTS>() + kAheadWords) * kWarps;
  return launch_persistent_ex(true, rta_big_kernel<SLOTS, MODE>, blocks_per_sm, smem,
                           (p.n_tasksets + kWarps - 1) / kWarps, sm_count, st, p, bin);
}

template <int MODE>
cudaError_t launch_all_bins(const KParams &p, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  if (p.n_tasksets <= kPlanSmall) return launch_any_bins(MODE, p, sm_count, st);  // one launch for every bin
  static int blocks_per_sm[64] = {0};
  const size_t smem = sizeof(u32) * kSmallWarpWords * kWarps;
  cudaError_t e = launch_persistent(rta_small_kernel<MODE>, blocks_per_sm, smem,
                                    (p.n_tasksets + kWarps - 1) / kWarps, sm_count, st, p);
  if (e == cudaSuccess) e = launch_big<2, MODE>(p, 4, sm_count, st);
  if (e == cudaSuccess) e = launch_big<3, MODE>(p, 5, sm_count, st);
  if (e == cudaSuccess) e = launch_big<4, MODE>(p, 6, sm_count, st);
  if (e == cudaSuccess) e = launch_big<6, MODE>(p, 7, sm_count, st);
  if (e == cudaSuccess) e = launch_big<8, MODE>(p, 8, sm_count, st);
  return e;
}

template <int SLOTS, int MASK>
cudaError_t launch_big_sweep(const KParams &p, const SweepArgs &sw, int bin, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  static int blocks_per_sm[64] = {0};
  const size_t smem = sizeof(u32) * (bin_warp_words<32, SLOTS>() + kAheadWords) * kWarps;
  return launch_persistent_ex(true, rta_big_sweep_kernel<SLOTS, MASK>, blocks_per_sm, smem,
                           (p.n_tasksets + kWarps - 1) / kWarps, sm_count, st, p, bin, sw);
}

template <int MASK>
cudaError_t launch_all_bins_sweep(const KParams &p, const SweepArgs &sw, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  static int blocks_per_sm[64] = {0};
  const size_t smem = sizeof(u32) * kSmallWarpWords * kWarps;
  cudaError_t e = launch_persistent(rta_small_sweep_kernel<MASK>, blocks_per_sm, smem,
                                    (p.n_tasksets + kWarps - 1) / kWarps, sm_count, st, p, sw);
  if (e == cudaSuccess) e = launch_big_sweep<2, MASK>(p, sw, 4, sm_count, st);
  if (e == cudaSuccess) e = launch_big_sweep<3, MASK>(p, sw, 5, sm_count, st);
  if (e == cudaSuccess) e = launch_big_sweep<4, MASK>(p, sw, 6, sm_count, st);
  if (e == cudaSuccess) e = launch_big_sweep<6, MASK>(p, sw, 7, sm_count, st);
  if (e == cudaSuccess) e = launch_big_sweep<8, MASK>(p, sw, 8, sm_count, st);
  return e;
}

cudaError_t launch_sweep_set(const KParams &p, const SweepArgs &sw, int sm_count, cudaStream_t st) {
  switch (sw.enabled) {
    case 1: return launch_all_bins_sweep<1>(p, sw, sm_count, st);
    case 2: return launch_all_bins_sweep<2>(p, sw, sm_count, st);
    case 4: return launch_all_bins_sweep<4>(p, sw, sm_count, st);
    case 8: return launch_all_bins_sweep<8>(p, sw, sm_count, st);
    case 5: return launch_all_bins_sweep<5>(p, sw, sm_count, st);   // GCAPS + RR, self-suspension
    case 10: return launch_all_bins_sweep<10>(p, sw, sm_count, st);  // GCAPS + RR, busy-waiting
    default: return cudaErrorInvalidValue;
  }
}

// Plan + analysis launches of one call.  `sw` null: one analysis (p.policy).  Otherwise the
// analyses named in `analyses` (bit m = mode m) for every pair of `sw`: the self-suspension
// modes in one set of launches, the busy-waiting modes in another (the plan is shared, the work
// counters are cleared in between).
int enqueue_batch(KParams p, void *workspace, size_t workspace_bytes, int sm_count, cudaStream_t st,
                  const SweepArgs *sw = nullptr, int analyses = 0) {
  if (p.n_tasksets == 0) return GCAPS_OK;
  const int rc = enqueue_plan(p, workspace, workspace_bytes, st);
  if (rc != GCAPS_OK) return rc;
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess && sw) {
    SweepArgs set = *sw;
    set.block_stride = __builtin_popcount(analyses);
    for (int m = 0, k = 0; m < 4; ++m) {
      set.block_of_mode[m] = k;
      k += (analyses >> m) & 1;
    }
    bool first = true;
    for (int half = 0; half < 2 && e == cudaSuccess; ++half) {
      set.enabled = analyses & (half == 0 ? 5 : 10);
      if (set.enabled == 0) continue;
      if (!first) e = cudaMemsetAsync(p.hdr->next, 0, sizeof(p.hdr->next), st);
      first = false;
      if (e == cudaSuccess) e = launch_sweep_set(p, set, sm_count, st);
    }
  } else if (e == cudaSuccess) {
    const bool rr = (p.policy & 0xff) == GCAPS_POLICY_RR, busy = (p.policy & GCAPS_RTA_BUSY) != 0;
    if (!rr && !busy) e = launch_all_bins<0>(p, sm_count, st);
    else if (!rr) e = launch_all_bins<1>(p, sm_count, st);
    else if (!busy) e = launch_all_bins<2>(p, sm_count, st);
    else e = launch_all_bins<3>(p, sm_count, st);
  }
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}

// staging memory of the host-buffer entry point (one set per process, current device)
struct HostStage {
  void *dev[2];
  size_t dev_bytes[2];
  cudaStream_t stream[2];
  int device;
  bool streams_ok;
};
HostStage g_stage = {{nullptr, nullptr}, {0, 0}, {nullptr, nullptr}, -1, false};
std::mutex g_stage_mutex;  // one host-buffer call at a time owns the staging slots

void release_stage_locked() {
  for (int k = 0; k < 2; ++k) {
    if (g_stage.dev[k]) cudaFree(g_stage.dev[k]);
    g_stage.dev[k] = nullptr;
    g_stage.dev_bytes[k] = 0;
    if (g_stage.streams_ok && g_stage.stream[k]) cudaStreamDestroy(g_stage.stream[k]);
    g_stage.stream[k] = nullptr;
  }
  g_stage.streams_ok = false;
  g_stage.device = -1;
}

// Workspace of gcaps_rta_batch_static: lives in the library image, one copy per device that
// loads it.  In host code this name is only a handle for cudaGetSymbolAddress, never an address
// a kernel may be given.
static __device__ __align__(256) unsigned char g_static_scratch[GCAPS_RTA_STATIC_SCRATCH_BYTES];
void *g_static_scratch_ptr[64];  // device address of the array, per device, once looked up

}  // namespace

extern "C" {

size_t gcaps_rta_workspace_bytes(int64_t n_tasksets) {
  if (n_tasksets <= 0) return 0;
  const size_t nb = plan_blocks(n_tasksets);
  return 256 + align_up(nb * kBinStride * sizeof(unsigned int), 256) +
         align_up((size_t)n_tasksets * sizeof(unsigned int), 256);
}

int gcaps_rta_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                    int64_t timeslice_us, int64_t ctx_switch_overhead_us, int64_t *out_wcrt,
                    uint8_t *out_sched, void *workspace, size_t workspace_bytes, void *stream) {
  int rc = check_args(ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us);
  if (rc != GCAPS_OK) return rc;
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_sched || (ts->n_tasks > 0 && !out_wcrt)) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  KParams p;
  fill_params(&p, ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us, out_wcrt, out_sched);
  return enqueue_batch(p, workspace, workspace_bytes, di.sm_count, (cudaStream_t)stream);
}

int gcaps_rta_multi_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int analyses, int flags,
                          int n_points, const int64_t *timeslice_us,
                          const int64_t *ctx_switch_overhead_us, int64_t *out_wcrt,
                          uint8_t *out_sched, void *workspace, size_t workspace_bytes, void *stream) {
  if (analyses < 1 || analyses > 15 || (flags & ~(GCAPS_RTA_LITERAL | GCAPS_RTA_BEST_EFFORT)))
    return GCAPS_ERR_INVALID_ARG;
  if (n_points < 1 || n_points > GCAPS_RTA_MAX_SWEEP || !ctx_switch_overhead_us)
    return GCAPS_ERR_INVALID_ARG;
  const bool rr = (analyses & (GCAPS_ANALYSIS_RR_SUSPEND | GCAPS_ANALYSIS_RR_BUSY)) != 0;
  if (rr && !timeslice_us) return GCAPS_ERR_INVALID_ARG;
  const int policy = (rr ? GCAPS_POLICY_RR : GCAPS_POLICY_GCAPS) | flags;  // (for the argument checks)
  SweepArgs sw;
  memset(&sw, 0, sizeof(sw));
  sw.n = n_points;
  for (int q = 0; q < n_points; ++q) {
    const int64_t L = rr ? timeslice_us[q] : 1;
    int rc = check_args(ts, n_tasksets, policy, L, ctx_switch_overhead_us[q]);
    if (rc != GCAPS_OK) return rc;
    KParams one;  // (fills the reciprocal of L exactly as a single call would)
    fill_params(&one, ts, n_tasksets, policy, L, ctx_switch_overhead_us[q], nullptr, nullptr);
    sw.q[q].L = one.L, sw.q[q].ovh = one.ovh;
    sw.q[q].l_mode = one.l_mode, sw.q[q].l_magic = one.l_magic, sw.q[q].l_shift = one.l_shift;
    if (one.ovh > sw.max_ovh) sw.max_ovh = one.ovh;
  }
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_sched) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  KParams p;
  fill_params(&p, ts, n_tasksets, policy, sw.q[0].L, sw.q[0].ovh, out_wcrt, out_sched);
  return enqueue_batch(p, workspace, workspace_bytes, di.sm_count, (cudaStream_t)stream, &sw, analyses);
}

int gcaps_rta_sweep_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int n_points,
                          const int64_t *timeslice_us, const int64_t *ctx_switch_overhead_us,
                          int64_t *out_wcrt, uint8_t *out_sched, void *workspace,
                          size_t workspace_bytes, void *stream) {
  const int pol = policy & 0xff;
  if (pol != GCAPS_POLICY_GCAPS && pol != GCAPS_POLICY_RR) return GCAPS_ERR_INVALID_ARG;
  if (policy & ~(0xff | GCAPS_RTA_BUSY | GCAPS_RTA_LITERAL | GCAPS_RTA_BEST_EFFORT)) return GCAPS_ERR_INVALID_ARG;
  const int mode = (pol == GCAPS_POLICY_RR ? 2 : 0) + ((policy & GCAPS_RTA_BUSY) ? 1 : 0);
  return gcaps_rta_multi_batch(ts, n_tasksets, 1 << mode, policy & (GCAPS_RTA_LITERAL | GCAPS_RTA_BEST_EFFORT),
                               n_points, timeslice_us, ctx_switch_overhead_us, out_wcrt, out_sched,
                               workspace, workspace_bytes, stream);
}

int gcaps_rta_batch_static(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                           int64_t timeslice_us, int64_t ctx_switch_overhead_us,
                           int64_t *out_wcrt, uint8_t *out_sched, void *stream) {
  int rc = check_args(ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us);
  if (rc != GCAPS_OK) return rc;
  if (n_tasksets > GCAPS_RTA_STATIC_MAX_TASKSETS ||
      gcaps_rta_workspace_bytes(n_tasksets) > (size_t)GCAPS_RTA_STATIC_SCRATCH_BYTES)
    return GCAPS_ERR_TOO_LARGE;
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_sched || (ts->n_tasks > 0 && !out_wcrt)) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess || dev < 0 || dev >= 64) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_NO_DEVICE;
  }
  void *scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_init_mutex);
    if (!g_static_scratch_ptr[dev]) {
      // once per device, with that device current: the array's address on this device
      void *ptr = nullptr;
      e = cudaGetSymbolAddress(&ptr, g_static_scratch);
      if (e != cudaSuccess || !ptr) {
        g_last_cuda_error = (int)e;
        return GCAPS_ERR_CUDA;
      }
      g_static_scratch_ptr[dev] = ptr;
    }
    scratch = g_static_scratch_ptr[dev];
  }
  KParams p;
  fill_params(&p, ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us, out_wcrt, out_sched);
  // Nothing in the array has to be cleared first: the plan kernels write the header (counts,
  // starts, zeroed work counters), every per-block count and every permutation entry that the
  // analysis kernels of this call read.
  return enqueue_batch(p, scratch, (size_t)GCAPS_RTA_STATIC_SCRATCH_BYTES, di.sm_count,
                       (cudaStream_t)stream);
}

int gcaps_rta_validate(const gcaps_tasksets_t *ts, int64_t n_tasksets, int32_t *out_err,
                       void *stream) {
  int rc = check_args(ts, n_tasksets, GCAPS_POLICY_GCAPS, 1, 0);
  if (rc != GCAPS_OK) return rc;
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_err) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  KParams p;
  fill_params(&p, ts, n_tasksets, GCAPS_POLICY_GCAPS, 1, 0, nullptr, nullptr);
  validate_kernel<<<(unsigned int)((n_tasksets + 127) / 128), 128, 0, (cudaStream_t)stream>>>(p, out_err);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}

#define HOST_TRY(call)                    \
  do {                                    \
    cudaError_t e_ = (call);              \
    if (e_ != cudaSuccess) {              \
      g_last_cuda_error = (int)e_;        \
      return GCAPS_ERR_CUDA;              \
    }                                     \
  } while (0)

void gcaps_rta_release_host(void) {
  std::lock_guard<std::mutex> lock(g_stage_mutex);
  release_stage_locked();
}

constexpr int kMaxHostPolicies = GCAPS_RTA_MAX_HOST_POLICIES;

// Copies tasksets [t, t1) (tasks [k0, k1)) to the staging slot, enqueues their analysis under
// every requested policy and the copies of the results back.  The offsets of the range are known to be monotone and in range.
static int host_chunk(const gcaps_tasksets_t *ts, int64_t t, int64_t t1, const int *policies,
                      int n_pol, int64_t L, int64_t ovh, int64_t *const *out_wcrt,
                      uint8_t *const *out_sched, int slot, int sm_count) {
  const int64_t k0 = ts->task_off[t], k1 = ts->task_off[t1];
  const int64_t nt = t1 - t, nk = k1 - k0;
  const int64_t c0 = ts->cseg_off[k0], nc = ts->cseg_off[k1] - c0;
  const int64_t g0 = ts->gseg_off[k0], ng = ts->gseg_off[k1] - g0;
  size_t off = 0;
  auto take = [&](size_t n_bytes) {
    size_t o = off;
    off += align_up(n_bytes, 256);
    return o;
  };
  const size_t o_task_off = take((nt + 1) * 8), o_period = take(nk * 8), o_deadline = take(nk * 8);
  const size_t o_priority = take(nk * 8), o_core = take(nk * 8), o_cseg_off = take((nk + 1) * 8);
  const size_t o_cseg = take(nc * 8), o_gseg_off = take((nk + 1) * 8), o_gm = take(ng * 8);
  const size_t o_ge = take(ng * 8);
  size_t o_wcrt[kMaxHostPolicies], o_sched[kMaxHostPolicies];
  for (int q = 0; q < n_pol; ++q) o_wcrt[q] = take(nk * 8), o_sched[q] = take(nt);
  const size_t ws_bytes = gcaps_rta_workspace_bytes(nt);
  const size_t o_ws = take(ws_bytes);
  cudaStream_t st = g_stage.stream[slot];
  HOST_TRY(cudaStreamSynchronize(st));  // the slot's previous chunk has left the buffer
  if (g_stage.dev_bytes[slot] < off) {
    if (g_stage.dev[slot]) HOST_TRY(cudaFree(g_stage.dev[slot]));
    g_stage.dev[slot] = nullptr;
    g_stage.dev_bytes[slot] = 0;
    const size_t want = off + (off >> 3);
    HOST_TRY(cudaMalloc(&g_stage.dev[slot], want));
    g_stage.dev_bytes[slot] = want;
  }
  unsigned char *d = (unsigned char *)g_stage.dev[slot];
#define H2D(dst_off, src, count) \
  HOST_TRY(cudaMemcpyAsync(d + (dst_off), (src), (size_t)(count) * 8, cudaMemcpyHostToDevice, st))
  H2D(o_task_off, ts->task_off + t, nt + 1);
  if (nk > 0) {
    H2D(o_period, ts->period + k0, nk);
    H2D(o_deadline, ts->deadline + k0, nk);
    H2D(o_priority, ts->priority + k0, nk);
    H2D(o_core, ts->core + k0, nk);
  }
  H2D(o_cseg_off, ts->cseg_off + k0, nk + 1);
  H2D(o_gseg_off, ts->gseg_off + k0, nk + 1);
  if (nc > 0) H2D(o_cseg, ts->cseg_wcet + c0, nc);
  if (ng > 0) {
    H2D(o_gm, ts->gseg_misc + g0, ng);
    H2D(o_ge, ts->gseg_exec + g0, ng);
  }
#undef H2D
  gcaps_tasksets_t dts;
  dts.n_tasks = nk, dts.n_csegs = nc, dts.n_gsegs = ng;
  dts.task_off = (const int64_t *)(d + o_task_off);
  dts.period = (const int64_t *)(d + o_period);
  dts.deadline = (const int64_t *)(d + o_deadline);
  dts.priority = (const int64_t *)(d + o_priority);
  dts.core = (const int64_t *)(d + o_core);
  dts.cseg_off = (const int64_t *)(d + o_cseg_off);
  dts.cseg_wcet = (const int64_t *)(d + o_cseg);
  dts.gseg_off = (const int64_t *)(d + o_gseg_off);
  dts.gseg_misc = (const int64_t *)(d + o_gm);
  dts.gseg_exec = (const int64_t *)(d + o_ge);
  for (int q = 0; q < n_pol; ++q) {  // one copy of the inputs, one analysis per policy
    KParams p;
    fill_params(&p, &dts, nt, policies[q], L, ovh, (int64_t *)(d + o_wcrt[q]), d + o_sched[q]);
    p.task_base = k0, p.cseg_base = c0, p.gseg_base = g0;
    int rc = enqueue_batch(p, d + o_ws, ws_bytes, sm_count, st);
    if (rc != GCAPS_OK) return rc;
    if (nk > 0)
      HOST_TRY(cudaMemcpyAsync(out_wcrt[q] + k0, d + o_wcrt[q], (size_t)nk * 8,
                               cudaMemcpyDeviceToHost, st));
    HOST_TRY(cudaMemcpyAsync(out_sched[q] + t, d + o_sched[q], (size_t)nt, cudaMemcpyDeviceToHost, st));
  }
  return GCAPS_OK;
}

// An error in a later chunk: earlier chunks' copies into the caller's arrays may still be in
// flight on the staging streams; nothing of this call may touch the caller's memory once it has
// returned.  Keeps the CUDA error code the failing step recorded.
static int drain_stage(int rc) {
  const int keep = g_last_cuda_error;
  for (int k = 0; k < 2; ++k)
    if (g_stage.streams_ok && g_stage.stream[k]) cudaStreamSynchronize(g_stage.stream[k]);
  g_last_cuda_error = keep;
  return rc;
}

// True if the task range [k0, k1] is inside the arrays and both segment offset arrays are
// non-decreasing and in range over it.
static bool host_range_is_canonical(const gcaps_tasksets_t *ts, int64_t k0, int64_t k1) {
  if (k0 < 0 || k1 < k0 || k1 > ts->n_tasks) return false;
  if (ts->cseg_off[k0] < 0 || ts->cseg_off[k1] > ts->n_csegs) return false;
  if (ts->gseg_off[k0] < 0 || ts->gseg_off[k1] > ts->n_gsegs) return false;
  int ok = 1;
  for (int64_t k = k0; k < k1; ++k)
    ok &= (ts->cseg_off[k] <= ts->cseg_off[k + 1]) & (ts->gseg_off[k] <= ts->gseg_off[k + 1]);
  return ok != 0;
}

int gcaps_rta_batch_host(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy,
                         int64_t timeslice_us, int64_t ctx_switch_overhead_us, int64_t *out_wcrt,
                         uint8_t *out_sched) {
  return gcaps_rta_batch_host_multi(ts, n_tasksets, &policy, 1, timeslice_us, ctx_switch_overhead_us,
                                    &out_wcrt, &out_sched);
}

int gcaps_rta_batch_host_multi(const gcaps_tasksets_t *ts, int64_t n_tasksets, const int *policies,
                               int n_policies, int64_t timeslice_us, int64_t ctx_switch_overhead_us,
                               int64_t *const *out_wcrt, uint8_t *const *out_sched) {
  if (!policies || n_policies < 1 || n_policies > kMaxHostPolicies || !out_wcrt || !out_sched)
    return GCAPS_ERR_INVALID_ARG;
  int rc = GCAPS_OK;
  for (int q = 0; q < n_policies; ++q) {
    rc = check_args(ts, n_tasksets, policies[q], timeslice_us, ctx_switch_overhead_us);
    if (rc != GCAPS_OK) return rc;
  }
  if (n_tasksets == 0) return GCAPS_OK;
  for (int q = 0; q < n_policies; ++q)
    if (!out_sched[q] || (ts->n_tasks > 0 && !out_wcrt[q])) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  std::lock_guard<std::mutex> lock(g_stage_mutex);
  int dev = 0;
  HOST_TRY(cudaGetDevice(&dev));
  if (g_stage.device != dev) {
    release_stage_locked();
    g_stage.device = dev;
  }
  if (!g_stage.streams_ok) {
    HOST_TRY(cudaStreamCreateWithFlags(&g_stage.stream[0], cudaStreamNonBlocking));
    HOST_TRY(cudaStreamCreateWithFlags(&g_stage.stream[1], cudaStreamNonBlocking));
    g_stage.streams_ok = true;
  }
  const int64_t kChunkTasksets = 1 << 16;
  const int64_t kChunkTasks = 3 << 20;  // ~ 200-400 MB of staging per slot
  int64_t t = 0;
  int slot = 0;
  while (t < n_tasksets) {
    // a chunk is a run of whole tasksets whose task ranges follow one another
    int64_t t1 = t;
    const int64_t k0 = ts->task_off[t];
    int64_t k1 = k0;
    while (t1 < n_tasksets && t1 - t < kChunkTasksets) {
      const int64_t kn = ts->task_off[t1 + 1];
      if (kn < k1 || (t1 > t && kn - k0 > kChunkTasks)) break;
      k1 = kn;
      t1 += 1;
    }
    if (t1 > t && host_range_is_canonical(ts, k0, k1)) {
      rc = host_chunk(ts, t, t1, policies, n_policies, timeslice_us, ctx_switch_overhead_us,
                      out_wcrt, out_sched, slot, di.sm_count);
      if (rc != GCAPS_OK) return drain_stage(rc);
      slot ^= 1;
      t = t1;
      continue;
    }
    // Malformed offsets somewhere in the run: go through it one taskset at a time, so that each
    // taskset is judged on its own offsets alone.
    const int64_t stop = t1 > t ? t1 : t + 1;
    for (; t < stop; ++t) {
      const int64_t a = ts->task_off[t], b = ts->task_off[t + 1];
      if (a < 0 || b < a || b > ts->n_tasks || b - a > GCAPS_RTA_MAX_TASKS) {
        for (int q = 0; q < n_policies; ++q) out_sched[q][t] = GCAPS_SCHED_INVALID;
      } else if (!host_range_is_canonical(ts, a, b)) {
        for (int q = 0; q < n_policies; ++q) {
          out_sched[q][t] = GCAPS_SCHED_INVALID;
          for (int64_t k = a; k < b; ++k) out_wcrt[q][k] = GCAPS_WCRT_INVALID;
        }
      } else {
        rc = host_chunk(ts, t, t + 1, policies, n_policies, timeslice_us, ctx_switch_overhead_us,
                        out_wcrt, out_sched, slot, di.sm_count);
        if (rc != GCAPS_OK) return drain_stage(rc);
        slot ^= 1;
      }
    }
  }
  HOST_TRY(cudaStreamSynchronize(g_stage.stream[0]));
  HOST_TRY(cudaStreamSynchronize(g_stage.stream[1]));
  return GCAPS_OK;
}

const char *gcaps_rta_strerror(int code) {
  switch (code) {
    case GCAPS_OK: return "ok";
    case GCAPS_ERR_INVALID_ARG: return "invalid argument";
    case GCAPS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GCAPS_ERR_CUDA: return "CUDA runtime error (see gcaps_rta_last_cuda_error)";
    case GCAPS_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
    case GCAPS_ERR_TOO_LARGE:
      return "batch exceeds GCAPS_RTA_STATIC_MAX_TASKSETS: split it or use gcaps_rta_batch";
    default: return "unknown error code";
  }
}

int gcaps_rta_last_cuda_error(void) { return g_last_cuda_error; }

int gcaps_rta_version(void) { return GCAPS_RTA_VERSION; }

}  // extern "C"
#endif  // GCAPS_RTA_ANY_TU
