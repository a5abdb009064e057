// gcaps_gpu_priority.cu -- the GCAPS analysis with a separate priority for GPU segments, and the
// Audsley-style search for those priorities (GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 5.3 and
// Sec. 6.4), for NVIDIA B200 (sm_100a).
//
// Sec. 6.4 replaces R_h by D_h in every jitter, so each pair (J, W) of an interferer is a
// constant of the taskset and the tasks of a taskset can be bounded in any order.  A group of 8,
// 16 or 32 lanes works on one taskset (tasksets are binned by size with the same plan as the
// default analysis); lane l of the group keeps, in registers, what its tasks (positions l,
// l + lanes, ...) contribute as interferers: the reciprocal of T_h, the same-core pairs
// (J^c_h, C_h + G^{m*}_h) and (J^g_h, G^e_h), and the other-core pair (J^g_h, G^{e*}_h).
// Bounding one task is then: a per-lane choice of which pairs apply (same core and higher CPU
// priority; or higher GPU priority, which during the search means "still without a level"), and
// sweeps of multiply-high / shift / multiply-add summed across the group.  All values of a
// taskset below 2^26 us: 32-bit arithmetic; otherwise the same loop in saturating 64-bit.
#include <cuda_runtime.h>
#include <stdint.h>

#include "rta_common.cuh"

using namespace gcaps_detail;

namespace {

struct GpParams {
  KParams k;
  const i64 *gpu_prio_in;
  i64 *gpu_prio_out;
  int assign;
};

// Per-taskset shared memory of a group, by position.
template <int MAXN>
struct GpSmem {
  i64 key[MAXN];   // priorities while ranking
  i64 base[MAXN];  // C_i + G*_i + B^C_i
  i64 D[MAXN];
  int core[MAXN];
  short cpu_rank[MAXN];     // 0 = highest CPU priority, ties by position
  short gpu_rank[MAXN];     // the same for the given GPU priorities
  short by_cpu_rank[MAXN];  // CPU rank -> position
  unsigned char uses_gpu[MAXN];
  // search: bit r set = the task of CPU rank r has no level yet and no task of lower CPU priority
  // on its core is without one, i.e. it may take the next level (the same-core rule of Sec. 5.3)
  unsigned int cand[8];
};

// Largest r < below with bit r set in the 256-bit set `bits`, or -1.
__device__ __forceinline__ int highest_below(const unsigned int *bits, int below) {
  for (int w = (below - 1) >> 5; w >= 0; --w) {
    unsigned int m = bits[w];
    if (w == (below - 1) >> 5) m &= (2u << ((below - 1) & 31)) - 1u;  // (2u << 31 wraps to 0: all ones)
    if (m) return 32 * w + 31 - __clz((int)m);
  }
  return -1;
}

// What a lane knows about its S tasks as interferers (slot s: position lane + LPT * s).
template <int S>
struct GpLane {
  u64 T[S];
  u64 Kc[S], Kg[S];          // J^c_h + T_h - 1, J^g_h + T_h - 1 (the ceiling folded in)
  u64 Wc[S], We[S], Wes[S];  // C_h + G^m_h (+ 2 eps eta_h unless busy-waiting), G^e_h, G^{e*}_h
  u32 magic[S], shift[S];    // reciprocal of T_h (32-bit path)
  int core[S], cpu_rank[S];
  bool gpu[S], valid[S];
};

template <int LPT>
__device__ __forceinline__ u32 sum32(u32 v, unsigned int gmask) {
  if constexpr (LPT == 32) {
    return __reduce_add_sync(gmask, v);
  } else {
#pragma unroll
    for (int d = LPT / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(gmask, v, d, LPT);
    return v;
  }
}

// Bound of task i (core_i, CPU rank rank_i, GPU-using gi, constant part `base`, deadline Di) when
// the tasks flagged in above[] have a higher GPU-segment priority: the recurrence of Sec. 6.3
// with hp() by GPU priority and D_h in the jitters (Sec. 6.4).  Returns the bound,
// GCAPS_WCRT_MISS or GCAPS_WCRT_ITER_LIMIT, the same value in every lane of the group.
template <int LPT, int S, bool FAST>
__device__ __forceinline__ i64 bound_of(const GpLane<S> &me, int lane, unsigned int gmask, int i,
                                        int core_i, int rank_i, bool gi, u64 base, u64 Di,
                                        const bool (&above)[S], bool busy, bool literal) {
  // the (J, W) pairs of this lane's tasks; W = 0 where a pair does not apply
  u64 Ka[S], Wa[S], Wb[S];
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const int h = lane + LPT * s;
    const bool hpp = me.valid[s] && h != i && me.core[s] == core_i && me.cpu_rank[s] < rank_i;
    const bool hpg = me.valid[s] && h != i && above[s] && !hpp;  // hp(tau_i) of Sec. 6.4 minus hpp
    Ka[s] = me.Kc[s], Wa[s] = 0, Wb[s] = 0;
    if (!busy) {
      if (hpp) Wa[s] = me.Wc[s];                      // Lemma 15 (jitter 0 for a CPU-only tau_h)
      if (hpp && me.gpu[s] && gi) Wb[s] = me.We[s];   // Lemma 13, same core
      if (hpg && me.gpu[s] && gi) Wb[s] = me.Wes[s];  // Lemma 13, other cores
    } else {
      if (hpp) {
        Ka[s] = me.T[s] - 1;                                                       // no jitter
        Wa[s] = me.Wc[s] + ((me.gpu[s] && (gi || !literal)) ? me.Wes[s] : 0);      // Lemmas 12, 10
      } else if (hpg && me.gpu[s]) {
        Wb[s] = me.Wes[s];                                                         // Lemmas 10, 11
      }
    }
  }
  u64 R = base;
  i64 sweeps = 0;
  for (;;) {
    if (R > Di) return GCAPS_WCRT_MISS;
    if (sweeps >= GCAPS_RTA_ITER_CAP) return GCAPS_WCRT_ITER_LIMIT;
    sweeps += 1;
    u64 next;
    if (FAST) {  // R <= D_i < 2^26, K < 2^27: the dividend stays below 2^28
      u64 acc = 0;
#pragma unroll
      for (int s = 0; s < S; ++s) {
        acc += (u64)(__umulhi((u32)R + (u32)Ka[s], me.magic[s]) >> me.shift[s]) * (u32)Wa[s];
        acc += (u64)(__umulhi((u32)R + (u32)me.Kg[s], me.magic[s]) >> me.shift[s]) * (u32)Wb[s];
      }
      const u32 part = acc > (u64)kFastClamp ? kFastClamp : (u32)acc;
      next = base + sum32<LPT>(part, gmask);
    } else {
      u64 part = 0;
#pragma unroll
      for (int s = 0; s < S; ++s) {
        if (Wa[s]) part += sat_mul((R + Ka[s]) / me.T[s], Wa[s]);
        if (Wb[s]) part += sat_mul((R + me.Kg[s]) / me.T[s], Wb[s]);
      }
      next = base + group_sum<LPT>(part > kClamp ? kClamp : part, gmask);
    }
    if (next == R) return (i64)R;
    R = next;
  }
}

template <int LPT, int S>
__device__ void analyse_gpu_priority(const GpParams &g, i64 t, GpSmem<LPT * S> &sm, int lane,
                                     unsigned int gmask) {
  constexpr int MAXN = LPT * S;
  const KParams &p = g.k;
  const bool busy = (p.policy & GCAPS_RTA_BUSY) != 0, literal = (p.policy & GCAPS_RTA_LITERAL) != 0;
  const u64 eps = (u64)p.ovh;
  const i64 a = p.task_off[t], b = p.task_off[t + 1];
  if (a < 0 || b < a || b > p.n_tasks || b - a > MAXN) {
    // (a taskset of more than MAXN tasks can only reach the largest bin, where MAXN is the limit)
    if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
    return;
  }
  const int n = (int)(b - a);

  // ---- stage, validate, aggregate (task model of Sec. 4) ------------------------------------
  int bad = 0;
  bool fits32 = eps < (1u << 20);
  u64 T[S], D[S], A[S], Ge[S], Star[S];
  int eta[S], core[S];
  bool valid[S];
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const int i = lane + LPT * s;
    valid[s] = i < n;
    T[s] = 2, D[s] = 1, A[s] = 0, Ge[s] = 0, Star[s] = 0, eta[s] = 0, core[s] = -1;
    if (valid[s]) {
      const i64 k = a + i;
      const i64 Ti = p.period[k], Di = p.deadline[k], c = p.core[k];
      if (Ti < 1 || Ti > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_PERIOD;
      if (Di < 1 || Di > Ti) bad |= GCAPS_BAD_DEADLINE;
      if (c < 0 || c > GCAPS_RTA_MAX_CORE) bad |= GCAPS_BAD_CORE;
      const i64 c0 = p.cseg_off[k], c1 = p.cseg_off[k + 1], g0 = p.gseg_off[k], g1 = p.gseg_off[k + 1];
      const bool seg_ok = !(c0 < 0 || c1 < c0 || c1 > p.n_csegs || c1 - c0 > GCAPS_RTA_MAX_SEGMENTS ||
                            g0 < 0 || g1 < g0 || g1 > p.n_gsegs || g1 - g0 > GCAPS_RTA_MAX_SEGMENTS);
      u64 C = 0, Gm = 0, Gx = 0;
      if (seg_ok) {
#pragma unroll 4
        for (i64 j = c0; j < c1; ++j) {
          const i64 w = p.cseg_wcet[j];
          if (w < 0 || w > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_WCET;
          C += (u64)w;
        }
#pragma unroll 4
        for (i64 j = g0; j < g1; ++j) {
          const i64 m = p.gseg_misc[j], e = p.gseg_exec[j];
          if (m < 0 || m > GCAPS_RTA_MAX_TIME || e < 0 || e > GCAPS_RTA_MAX_TIME) bad |= GCAPS_BAD_WCET;
          Gm += (u64)m, Gx += (u64)e;
        }
      } else {
        bad |= GCAPS_BAD_SEG_RANGE;
      }
      eta[s] = seg_ok ? (int)(g1 - g0) : 0;
      T[s] = (u64)Ti, D[s] = (u64)Di, A[s] = C + Gm, Ge[s] = Gx, core[s] = (int)c;
      Star[s] = 2 * eps * (u64)eta[s];
      sm.key[i] = p.priority[k];
      sm.core[i] = (int)c;
      fits32 = fits32 && Ti >= 2 && Ti < (i64)kFastLimit && eta[s] < 64 && A[s] + Star[s] < kFastLimit &&
               Gx + Star[s] < kFastLimit;
    }
  }
  bad = group_or<LPT>(bad, gmask);
  fits32 = __all_sync(gmask, fits32);
  __syncwarp(gmask);
  if (bad) {
#pragma unroll
    for (int s = 0; s < S; ++s)
      if (valid[s]) {
        p.out_wcrt[a + lane + LPT * s] = GCAPS_WCRT_INVALID;
        if (g.gpu_prio_out) g.gpu_prio_out[a + lane + LPT * s] = 0;
      }
    if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
    return;
  }
  // ---- CPU ranks: larger priority first, ties by position -----------------------------------
  GpLane<S> me;
  // distinct priorities hi-n+1 .. hi (what a numbering by period gives): the rank is hi - priority
  i64 hi = INT64_MIN;
#pragma unroll
  for (int s = 0; s < S; ++s)
    if (valid[s] && sm.key[lane + LPT * s] > hi) hi = sm.key[lane + LPT * s];
#pragma unroll
  for (int d = LPT / 2; d >= 1; d >>= 1) {
    const i64 other = __shfl_xor_sync(gmask, hi, d, LPT);
    hi = other > hi ? other : hi;
  }
  bool dense = true;
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const u64 r = valid[s] ? (u64)hi - (u64)sm.key[lane + LPT * s] : 0;
    dense &= r < (u64)n;
    me.cpu_rank[s] = (int)(r < (u64)n ? r : 0);
  }
  dense = __all_sync(gmask, dense);
  if (dense) {  // ... and no rank taken twice
#pragma unroll
    for (int s = 0; s < S; ++s)
      if (valid[s]) sm.by_cpu_rank[me.cpu_rank[s]] = (short)(lane + LPT * s);
    __syncwarp(gmask);
    bool uniq = true;
#pragma unroll
    for (int s = 0; s < S; ++s)
      if (valid[s]) uniq &= sm.by_cpu_rank[me.cpu_rank[s]] == (short)(lane + LPT * s);
    dense = __all_sync(gmask, uniq);
    __syncwarp(gmask);
  }
  if (!dense) {  // any priorities: count the tasks that come before
    i64 mine[S];
#pragma unroll
    for (int s = 0; s < S; ++s) mine[s] = valid[s] ? sm.key[lane + LPT * s] : 0, me.cpu_rank[s] = 0;
    for (int q = 0; q < n; ++q) {
      const i64 kq = sm.key[q];
#pragma unroll
      for (int s = 0; s < S; ++s)
        me.cpu_rank[s] += (valid[s] && (kq > mine[s] || (kq == mine[s] && q < lane + LPT * s))) ? 1 : 0;
    }
  }
  __syncwarp(gmask);
#pragma unroll
  for (int s = 0; s < S; ++s) {
    const int i = lane + LPT * s;
    const bool gh = eta[s] > 0;
    // Sec. 6.4: J^c_h = D_h - (C_h + G^m_h), J^g_h = D_h - G^e_h (a task whose own execution
    // exceeds its deadline has no such slack: 0); a CPU-only tau_h has no J^c (Lemma 15)
    const u64 Jc = (gh && D[s] > A[s]) ? D[s] - A[s] : 0, Jg = D[s] > Ge[s] ? D[s] - Ge[s] : 0;
    me.T[s] = T[s], me.Kc[s] = Jc + T[s] - 1, me.Kg[s] = Jg + T[s] - 1;
    me.Wc[s] = A[s] + ((gh && !busy) ? Star[s] : 0);  // Lemma 15: C_h + G^{m*}_h; Lemma 12: C_h + G^m_h
    me.We[s] = Ge[s], me.Wes[s] = Ge[s] + Star[s];
    me.core[s] = core[s], me.gpu[s] = gh, me.valid[s] = valid[s];
    me.magic[s] = 0, me.shift[s] = 0;
    if (fits32) make_reciprocal((u32)T[s], me.magic[s], me.shift[s]);
    if (valid[s]) {
      sm.cpu_rank[i] = (short)me.cpu_rank[s];
      sm.by_cpu_rank[me.cpu_rank[s]] = (short)i;
      sm.uses_gpu[i] = gh ? 1 : 0;
      sm.base[i] = (i64)(A[s] + Ge[s] + Star[s] + ((u64)eta[s] + 1) * eps);  // C_i + G*_i + B^C_i
      sm.D[i] = (i64)D[s];
    }
  }
  __syncwarp(gmask);
  auto bound = [&](int i, const bool(&above)[S]) -> i64 {
    const int core_i = sm.core[i], rank_i = sm.cpu_rank[i];
    const bool gi = sm.uses_gpu[i] != 0;
    const u64 bi = (u64)sm.base[i], Di = (u64)sm.D[i];
    if (fits32 && bi < kFastClamp)
      return bound_of<LPT, S, true>(me, lane, gmask, i, core_i, rank_i, gi, bi, Di, above, busy, literal);
    return bound_of<LPT, S, false>(me, lane, gmask, i, core_i, rank_i, gi, bi, Di, above, busy, literal);
  };

  int sched = GCAPS_SCHED_YES;
  if (!g.assign) {
    // ---- the given GPU priorities ---------------------------------------------------------------
#pragma unroll
    for (int s = 0; s < S; ++s)
      if (valid[s]) sm.key[lane + LPT * s] = g.gpu_prio_in[a + lane + LPT * s];
    __syncwarp(gmask);
    int gpu_rank[S];
    {
      i64 mine[S];
#pragma unroll
      for (int s = 0; s < S; ++s) mine[s] = valid[s] ? sm.key[lane + LPT * s] : 0, gpu_rank[s] = 0;
      for (int q = 0; q < n; ++q) {
        const i64 kq = sm.key[q];
#pragma unroll
        for (int s = 0; s < S; ++s)
          gpu_rank[s] += (valid[s] && (kq > mine[s] || (kq == mine[s] && q < lane + LPT * s))) ? 1 : 0;
      }
#pragma unroll
      for (int s = 0; s < S; ++s)
        if (valid[s]) sm.gpu_rank[lane + LPT * s] = (short)gpu_rank[s];
    }
    __syncwarp(gmask);
    int broken = 0;  // same core: the GPU order must equal the CPU order (Sec. 5.3)
    for (int q = 0; q < n; ++q) {
      const int core_q = sm.core[q], crank_q = sm.cpu_rank[q], grank_q = sm.gpu_rank[q];
#pragma unroll
      for (int s = 0; s < S; ++s)
        if (valid[s] && core_q == core[s] && crank_q < me.cpu_rank[s] && grank_q > gpu_rank[s]) broken = 1;
    }
    if (group_or<LPT>(broken, gmask)) {
#pragma unroll
      for (int s = 0; s < S; ++s)
        if (valid[s]) p.out_wcrt[a + lane + LPT * s] = GCAPS_WCRT_INVALID;
      if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
      return;
    }
    for (int i = 0; i < n; ++i) {
      const int rank_i = sm.gpu_rank[i];
      bool above[S];
#pragma unroll
      for (int s = 0; s < S; ++s) above[s] = gpu_rank[s] < rank_i;
      const i64 r = bound(i, above);
      if (lane == 0) {
        p.out_wcrt[a + i] = r;
        if (g.gpu_prio_out) g.gpu_prio_out[a + i] = g.gpu_prio_in[a + i];
      }
      if (r < 0) sched = GCAPS_SCHED_NO;
    }
  } else {
    // ---- the search of Sec. 5.3: levels from the lowest ----------------------------------------
    bool unplaced[S];
    if (lane < 8) sm.cand[lane] = 0;
#pragma unroll
    for (int s = 0; s < S; ++s) {
      unplaced[s] = valid[s];
      if (valid[s]) {
        p.out_wcrt[a + lane + LPT * s] = GCAPS_WCRT_MISS;
        g.gpu_prio_out[a + lane + LPT * s] = 0;
      }
    }
    __syncwarp(gmask);
    {  // the lowest CPU priority of every core starts as a candidate
      bool lowest[S];
#pragma unroll
      for (int s = 0; s < S; ++s) lowest[s] = valid[s];
      for (int q = 0; q < n; ++q) {
        const int core_q = sm.core[q], rank_q = sm.cpu_rank[q];
#pragma unroll
        for (int s = 0; s < S; ++s) lowest[s] &= !(core_q == core[s] && rank_q > me.cpu_rank[s]);
      }
#pragma unroll
      for (int s = 0; s < S; ++s)
        if (lowest[s]) atomicOr(&sm.cand[me.cpu_rank[s] >> 5], 1u << (me.cpu_rank[s] & 31));
    }
    __syncwarp(gmask);
    for (int level = 1; level <= n && sched == GCAPS_SCHED_YES; ++level) {
      bool placed = false;
      int want = n;
      while (!placed) {  // candidates from the lowest CPU priority upwards
        want = highest_below(sm.cand, want);
        if (want < 0) break;
        const int c = sm.by_cpu_rank[want];
        const i64 r = bound(c, unplaced);  // every other unplaced task above c (c itself is skipped)
        if (r >= 0) {
          placed = true;
          const int core_c = sm.core[c];
          int next = -1;  // the task of c's core that becomes a candidate now
#pragma unroll
          for (int s = 0; s < S; ++s) {
            if (lane + LPT * s == c) {
              unplaced[s] = false;
              p.out_wcrt[a + c] = r;
              g.gpu_prio_out[a + c] = (i64)level;
            }
            if (unplaced[s] && core[s] == core_c && me.cpu_rank[s] < want && me.cpu_rank[s] > next)
              next = me.cpu_rank[s];
          }
#pragma unroll
          for (int d = LPT / 2; d >= 1; d >>= 1) {
            const int other = __shfl_xor_sync(gmask, next, d, LPT);
            next = other > next ? other : next;
          }
          __syncwarp(gmask);
          if (lane == 0) {
            sm.cand[want >> 5] &= ~(1u << (want & 31));
            if (next >= 0) sm.cand[next >> 5] |= 1u << (next & 31);
          }
          __syncwarp(gmask);
        }
      }
      if (!placed) sched = GCAPS_SCHED_NO;
    }
  }
  if (lane == 0) p.out_sched[t] = (uint8_t)sched;
  __syncwarp(gmask);
}

// The tasksets of one size bin, pulled from the bin's counter by the warps of the launch.
// `warp_smem` is this warp's own shared memory (the same stride for every bin a kernel covers:
// the warps of a block may be working on different bins at the same time).
template <int LPT, int S>
__device__ __forceinline__ void run_bin(const GpParams &g, int bin, unsigned char *warp_smem) {
  constexpr int G = 32 / LPT;  // tasksets per warp
  typedef GpSmem<LPT * S> Sm;
  const KParams &p = g.k;
  const int lane32 = threadIdx.x & 31, group = lane32 / LPT, lane = lane32 % LPT;
  const unsigned int gmask = LPT == 32 ? kFull : (((1u << LPT) - 1u) << (group * LPT));
  Sm &sm = reinterpret_cast<Sm *>(warp_smem)[group];
  const unsigned int start = p.hdr->bin_start[bin], count = p.hdr->bin_count[bin];
  for (;;) {
    unsigned int first = 0;
    if (lane32 == 0) first = atomicAdd(&p.hdr->next[bin], (unsigned int)G);
    first = __shfl_sync(kFull, first, 0);
    if (first >= count) break;
    if (first + group < count)
      analyse_gpu_priority<LPT, S>(g, (i64)p.perm[start + first + group], sm, lane, gmask);
    __syncwarp();
  }
}

template <int LPT, int S>
__host__ __device__ constexpr size_t warp_bytes() {
  return (size_t)(32 / LPT) * sizeof(GpSmem<LPT * S>);
}
constexpr size_t cmax(size_t x, size_t y) { return x > y ? x : y; }
constexpr size_t kSmallWarpBytes =
    cmax(cmax(warp_bytes<16, 2>(), warp_bytes<8, 3>()), cmax(warp_bytes<8, 2>(), warp_bytes<8, 1>()));
static_assert(kSmallWarpBytes % 16 == 0, "every warp's area starts 16-byte aligned");

// the four bins of up to 32 tasks: (lanes per taskset, tasks per lane) as in the default analysis
__global__ void __launch_bounds__(kBlockThreads) gpu_priority_small_kernel(GpParams g) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();  // the kernel of the next size bin shares no data with this one
  unsigned char *mine = smem_raw + (threadIdx.x >> 5) * kSmallWarpBytes;
  run_bin<16, 2>(g, 3, mine);
  run_bin<8, 3>(g, 2, mine);
  run_bin<8, 2>(g, 1, mine);
  run_bin<8, 1>(g, 0, mine);
  wait_for_previous_grid();
}

// one bin of larger tasksets, a warp per taskset.  Five blocks per SM (96 registers): the search is
// bound by instruction issue and dependent latency, and 20 warps hide more of it than the 16 that
// the unbounded 127 registers allow, spills included (-7 % on 80-task tasksets).
template <int S>
__global__ void __launch_bounds__(kBlockThreads, 5) gpu_priority_big_kernel(GpParams g, int bin) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  let_dependents_start();
  run_bin<32, S>(g, bin, smem_raw + (threadIdx.x >> 5) * warp_bytes<32, S>());
  wait_for_previous_grid();
}

template <int S>
cudaError_t launch_big(const GpParams &g, int bin, int sm_count, cudaStream_t st) {
  constexpr int kWarps = kBlockThreads / 32;
  static int blocks_per_sm[64] = {0};
  return launch_persistent_ex(true, gpu_priority_big_kernel<S>, blocks_per_sm, warp_bytes<32, S>() * kWarps,
                           (g.k.n_tasksets + kWarps - 1) / kWarps, sm_count, st, g, bin);
}

}  // namespace

extern "C" int gcaps_rta_gpu_priority_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, int flags,
                                            int64_t runlist_update_us, const int64_t *gpu_priority,
                                            int64_t *out_gpu_priority, int64_t *out_wcrt,
                                            uint8_t *out_sched, void *workspace,
                                            size_t workspace_bytes, void *stream) {
  if (flags & ~(GCAPS_RTA_BUSY | GCAPS_RTA_LITERAL | GCAPS_RTA_ASSIGN)) return GCAPS_ERR_INVALID_ARG;
  const int policy = GCAPS_POLICY_GCAPS | (flags & (GCAPS_RTA_BUSY | GCAPS_RTA_LITERAL));
  int rc = check_args(ts, n_tasksets, policy, 1, runlist_update_us);
  if (rc != GCAPS_OK) return rc;
  const bool assign = (flags & GCAPS_RTA_ASSIGN) != 0;
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_sched || (ts->n_tasks > 0 && (!out_wcrt || (assign ? !out_gpu_priority : !gpu_priority))))
    return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  GpParams g;
  fill_params(&g.k, ts, n_tasksets, policy, 1, runlist_update_us, out_wcrt, out_sched);
  g.gpu_prio_in = (const i64 *)gpu_priority;
  g.gpu_prio_out = (i64 *)out_gpu_priority;
  g.assign = assign ? 1 : 0;
  cudaStream_t st = (cudaStream_t)stream;
  rc = enqueue_plan(g.k, workspace, workspace_bytes, st);
  if (rc != GCAPS_OK) return rc;
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) {
    constexpr int kWarps = kBlockThreads / 32;
    static int blocks_per_sm[64] = {0};
    e = launch_persistent(gpu_priority_small_kernel, blocks_per_sm, kSmallWarpBytes * kWarps,
                          (n_tasksets + kWarps - 1) / kWarps, di.sm_count, st, g);
  }
  if (e == cudaSuccess) e = launch_big<2>(g, 4, di.sm_count, st);
  if (e == cudaSuccess) e = launch_big<3>(g, 5, di.sm_count, st);
  if (e == cudaSuccess) e = launch_big<4>(g, 6, di.sm_count, st);
  if (e == cudaSuccess) e = launch_big<6>(g, 7, di.sm_count, st);
  if (e == cudaSuccess) e = launch_big<8>(g, 8, di.sm_count, st);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}
