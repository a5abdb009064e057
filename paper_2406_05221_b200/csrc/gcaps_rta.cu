// gcaps_rta.cu -- batched worst-case response-time analysis of GPU-using real-time tasksets
// (GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 6) for NVIDIA B200 (sm_100a).
//
// One group of LPT lanes (a warp or a slice of one) analyses one taskset at a time:
//   stage      coalesced loads of the taskset's per-task slices; per-task sums over its segments
//              (C_i, G^m_i, G^e_i, RR slice count of Eq. 3) go to shared memory in priority order
//   order      rank of every task by (priority desc, position asc)
//   iterate    for each task in that order the recurrence of Eq. 1 with the lemma set of the
//              chosen analysis: lanes over the higher-priority interferers, each evaluating
//              ceil((R+J)/T_h)*W terms, summed across the group with __shfl_xor
//   publish    R_i feeds the jitters J^c, J^g of later tasks; first deadline miss ends the taskset
//   write      out_wcrt through shared memory (coalesced), out_sched one byte
// Tasksets are binned by size (a small plan pass writes a permutation into the caller's
// workspace) so that groups of a launch see similar amounts of work; inside a launch groups pull
// chunks of tasksets from a counter, because iteration counts differ widely.
//
// Everything is integer arithmetic on microseconds.  No tensor cores: nothing here is a dense
// contraction.  No host synchronisation and no allocation in gcaps_rta_batch.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "../../include/gcaps_rta.h"

namespace {

typedef unsigned long long u64;
typedef long long i64;

constexpr int kNumBins = 6;
// largest taskset size of each bin and the lanes that cooperate on one taskset of it
__host__ __device__ constexpr int bin_max_n(int b) {
  return b == 0 ? 8 : b == 1 ? 16 : b == 2 ? 32 : b == 3 ? 64 : b == 4 ? 96 : GCAPS_RTA_MAX_TASKS;
}
constexpr int kBlockThreads = 128;
constexpr int kPlanItems = 1024;  // tasksets per plan block
constexpr u64 kClamp = 1ull << 50;  // any quantity >= 2^50 exceeds every deadline (<= 2^40)

struct PlanHeader {
  unsigned int bin_start[8];
  unsigned int bin_count[8];
  unsigned int next[8];  // work counters of the analysis launches
  unsigned int pad[8];
};
static_assert(sizeof(PlanHeader) == 128, "header layout");

struct KParams {
  const i64 *task_off, *period, *deadline, *priority, *core;
  const i64 *cseg_off, *cseg_wcet, *gseg_off, *gseg_misc, *gseg_exec;
  i64 n_tasks, n_csegs, n_gsegs;        // lengths of the arrays the pointers address
  i64 task_base, cseg_base, gseg_base;  // subtracted from the stored offsets (chunked host path)
  i64 n_tasksets;
  int policy;  // GCAPS_POLICY_* | flags
  i64 L, ovh;
  i64 *out_wcrt;
  uint8_t *out_sched;
  PlanHeader *hdr;
  unsigned int *block_cnt;  // [plan blocks][8]
  unsigned int *perm;       // [n_tasksets]
};

__device__ __forceinline__ int size_bin(i64 n) {
  if (n <= 8) return 0;  // also negative / broken ranges: rejected by the analysis kernel
  if (n <= 16) return 1;
  if (n <= 32) return 2;
  if (n <= 64) return 3;
  if (n <= 96) return 4;
  if (n <= GCAPS_RTA_MAX_TASKS) return 5;
  return 0;
}

// ---------------------------------------------------------------------------------------------
// plan: counting sort of taskset indices by size bin (histogram per block, scan, scatter)
// ---------------------------------------------------------------------------------------------
__global__ void plan_count_kernel(KParams p) {
  __shared__ unsigned int cnt[8];
  if (threadIdx.x < 8) cnt[threadIdx.x] = 0;
  __syncthreads();
  i64 t0 = (i64)blockIdx.x * kPlanItems;
  for (int k = threadIdx.x; k < kPlanItems; k += blockDim.x) {
    i64 t = t0 + k;
    if (t < p.n_tasksets) atomicAdd(&cnt[size_bin(p.task_off[t + 1] - p.task_off[t])], 1u);
  }
  __syncthreads();
  if (threadIdx.x < 8) p.block_cnt[(size_t)blockIdx.x * 8 + threadIdx.x] = cnt[threadIdx.x];
}

// One block.  Turns per-block counts into per-block write cursors and fills the header.
__global__ void plan_scan_kernel(KParams p, unsigned int n_blocks) {
  __shared__ unsigned int warp_tot[32];
  __shared__ unsigned int carry;
  __shared__ unsigned int bin_total[8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, n_warps = blockDim.x >> 5;
  for (int b = 0; b < kNumBins; ++b) {
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    for (unsigned int base = 0; base < n_blocks; base += blockDim.x) {
      unsigned int i = base + threadIdx.x;
      unsigned int v = i < n_blocks ? p.block_cnt[(size_t)i * 8 + b] : 0u;
      unsigned int x = v;
      for (int d = 1; d < 32; d <<= 1) {
        unsigned int y = __shfl_up_sync(0xffffffffu, x, d);
        if (lane >= d) x += y;
      }
      if (lane == 31) warp_tot[warp] = x;
      __syncthreads();
      unsigned int before = 0;
      for (int w = 0; w < warp; ++w) before += warp_tot[w];
      unsigned int excl = carry + before + x - v;
      if (i < n_blocks) p.block_cnt[(size_t)i * 8 + b] = excl;  // cursor relative to the bin
      __syncthreads();
      if (threadIdx.x == blockDim.x - 1) {
        unsigned int tot = 0;
        for (int w = 0; w < n_warps; ++w) tot += warp_tot[w];
        carry += tot;
      }
      __syncthreads();
    }
    if (threadIdx.x == 0) bin_total[b] = carry;
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    unsigned int s = 0;
    for (int b = 0; b < 8; ++b) {
      unsigned int c = b < kNumBins ? bin_total[b] : 0u;
      p.hdr->bin_start[b] = s;
      p.hdr->bin_count[b] = c;
      p.hdr->next[b] = 0;
      s += c;
    }
  }
}

__global__ void plan_scatter_kernel(KParams p) {
  __shared__ unsigned int cursor[8];
  if (threadIdx.x < 8) cursor[threadIdx.x] = p.block_cnt[(size_t)blockIdx.x * 8 + threadIdx.x];
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

// ---------------------------------------------------------------------------------------------
// exact saturating helpers of the 64-bit path
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ u64 sat_mul(u64 a, u64 b) {  // min(a*b, kClamp)
  u64 lo = a * b;
  return (__umul64hi(a, b) != 0 || lo > kClamp) ? kClamp : lo;
}
__device__ __forceinline__ u64 ceil_div64(u64 a, u64 b) { return (a + b - 1) / b; }

template <int LPT>
__device__ __forceinline__ u64 group_sum(u64 v, unsigned int mask) {
#pragma unroll
  for (int d = LPT / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(mask, v, d, LPT);
  return v;
}
template <int LPT>
__device__ __forceinline__ int group_or(int v, unsigned int mask) {
#pragma unroll
  for (int d = LPT / 2; d >= 1; d >>= 1) v |= __shfl_xor_sync(mask, v, d, LPT);
  return v;
}
template <int LPT>
__device__ __forceinline__ int group_sum_int(int v, unsigned int mask) {
#pragma unroll
  for (int d = LPT / 2; d >= 1; d >>= 1) v += __shfl_xor_sync(mask, v, d, LPT);
  return v;
}

// Shared-memory image of one taskset, indexed by priority rank unless noted.
template <int MAXN>
struct GroupSmem {
  u64 T[MAXN];     // period
  u64 D[MAXN];     // deadline
  u64 A[MAXN];     // C + G^m
  u64 Cc[MAXN];    // C
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
    s.Cc[rank] = C;
    s.Ge[rank] = Ge;
    s.Star[rank] = policy == GCAPS_POLICY_GCAPS ? 2 * ovh * (u64)eta : sat_mul(L + ovh, slices);
    s.core[rank] = (int)p.core[k];
    s.eta[rank] = eta;
    s.ord[rank] = (unsigned short)i;
  }
  bad = group_or<LPT>(bad, mask);
  const int n_gpu = group_sum_int<LPT>(n_gpu_lane, mask);  // N_g
  __syncwarp(mask);
  if (bad) {
    for (int i = lane; i < n; i += LPT) p.out_wcrt[a + i] = GCAPS_WCRT_INVALID;
    if (lane == 0) p.out_sched[t] = GCAPS_SCHED_INVALID;
    return;
  }
  for (int i = lane; i < n; i += LPT) s.prio_out[i] = GCAPS_WCRT_SKIPPED;
  __syncwarp(mask);

  // ---- iterate: tasks in decreasing priority ---------------------------------------------------
  int sched = GCAPS_SCHED_YES;
  for (int pos = 0; pos < n; ++pos) {
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
          if (same && !gh) term = sat_mul(ceil_div64(R, Th), s.Cc[h]);             // Lemma 15
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
        s.prio_out[s.ord[pos]] = (i64)R;
      }
      __syncwarp(mask);
    } else {
      if (lane == 0) s.prio_out[s.ord[pos]] = verdict;
      sched = GCAPS_SCHED_NO;
      break;
    }
  }
  __syncwarp(mask);
  for (int i = lane; i < n; i += LPT) p.out_wcrt[a + i] = s.prio_out[i];
  if (lane == 0) p.out_sched[t] = (uint8_t)sched;
  __syncwarp(mask);
}

// Persistent launch over one size bin: groups pull chunks of tasksets from the bin's counter.
template <int LPT, int MAXN>
__global__ void __launch_bounds__(kBlockThreads) rta_bin_kernel(KParams p, int bin) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int kGroupsPerWarp = 32 / LPT;
  constexpr int kChunk = 4;  // tasksets per group per pull
  GroupSmem<MAXN> *all = reinterpret_cast<GroupSmem<MAXN> *>(smem_raw);
  const int warp_in_block = threadIdx.x >> 5, lane32 = threadIdx.x & 31;
  const int group_in_warp = lane32 / LPT, lane = lane32 % LPT;
  GroupSmem<MAXN> &s = all[warp_in_block * kGroupsPerWarp + group_in_warp];
  const unsigned int mask =
      LPT == 32 ? 0xffffffffu : (((1u << LPT) - 1u) << (group_in_warp * LPT));
  const unsigned int start = p.hdr->bin_start[bin], count = p.hdr->bin_count[bin];
  for (;;) {
    unsigned int first = 0;
    if (lane32 == 0) first = atomicAdd(&p.hdr->next[bin], (unsigned int)(kChunk * kGroupsPerWarp));
    first = __shfl_sync(0xffffffffu, first, 0);
    if (first >= count) break;
    for (int c = 0; c < kChunk; ++c) {
      const unsigned int idx = first + c * kGroupsPerWarp + group_in_warp;
      if (idx < count) analyse_taskset<LPT, MAXN>(p, (i64)p.perm[start + idx], s, lane, mask);
    }
    __syncwarp();
  }
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

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
thread_local int g_last_cuda_error = 0;

struct DeviceInfo {
  int sm_count;
  int ok;  // 1 = usable sm_100 device, -1 = not usable
};
DeviceInfo g_dev[64];

int device_info(DeviceInfo *out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_NO_DEVICE;
  }
  if (dev < 0 || dev >= 64) return GCAPS_ERR_NO_DEVICE;
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

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

size_t plan_blocks(int64_t n_tasksets) { return (size_t)((n_tasksets + kPlanItems - 1) / kPlanItems); }

int check_args(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int64_t L, int64_t ovh) {
  if (!ts || n_tasksets < 0 || n_tasksets > 0x7fffffffLL) return GCAPS_ERR_INVALID_ARG;
  const int pol = policy & 0xff;
  if (pol != GCAPS_POLICY_GCAPS && pol != GCAPS_POLICY_RR) return GCAPS_ERR_INVALID_ARG;
  if (policy & ~(0xff | GCAPS_RTA_BUSY | GCAPS_RTA_LITERAL)) return GCAPS_ERR_INVALID_ARG;
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
  p->out_wcrt = (i64 *)out_wcrt;
  p->out_sched = out_sched;
}

template <int LPT, int MAXN>
cudaError_t launch_bin(const KParams &p, int bin, int sm_count, cudaStream_t st) {
  constexpr int kGroups = kBlockThreads / LPT;
  const size_t smem = sizeof(GroupSmem<MAXN>) * kGroups;
  static bool attr_done[64] = {false};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_done[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(rta_bin_kernel<LPT, MAXN>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    attr_done[dev & 63] = true;
  }
  int per_sm = 1;
  cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(
      &per_sm, rta_bin_kernel<LPT, MAXN>, kBlockThreads, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  // never more blocks than the bin could feed (the exact bin population lives on the device)
  long long want = (p.n_tasksets + kGroups - 1) / kGroups;
  long long grid = (long long)sm_count * per_sm;
  if (grid > want) grid = want;
  if (grid < 1) grid = 1;
  rta_bin_kernel<LPT, MAXN><<<(unsigned int)grid, kBlockThreads, smem, st>>>(p, bin);
  return cudaGetLastError();
}

int enqueue_batch(KParams p, void *workspace, size_t workspace_bytes, int sm_count, cudaStream_t st) {
  if (p.n_tasksets == 0) return GCAPS_OK;
  const size_t need = gcaps_rta_workspace_bytes(p.n_tasksets);
  if (!workspace || workspace_bytes < need || ((uintptr_t)workspace & 255u))
    return GCAPS_ERR_WORKSPACE;
  unsigned char *w = (unsigned char *)workspace;
  const size_t nb = plan_blocks(p.n_tasksets);
  p.hdr = (PlanHeader *)w;
  p.block_cnt = (unsigned int *)(w + 256);
  p.perm = (unsigned int *)(w + 256 + align_up(nb * 8 * sizeof(unsigned int), 256));
  plan_count_kernel<<<(unsigned int)nb, 256, 0, st>>>(p);
  plan_scan_kernel<<<1, 1024, 0, st>>>(p, (unsigned int)nb);
  plan_scatter_kernel<<<(unsigned int)nb, 256, 0, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) e = launch_bin<8, 8>(p, 0, sm_count, st);
  if (e == cudaSuccess) e = launch_bin<16, 16>(p, 1, sm_count, st);
  if (e == cudaSuccess) e = launch_bin<32, 32>(p, 2, sm_count, st);
  if (e == cudaSuccess) e = launch_bin<32, 64>(p, 3, sm_count, st);
  if (e == cudaSuccess) e = launch_bin<32, 96>(p, 4, sm_count, st);
  if (e == cudaSuccess) e = launch_bin<32, GCAPS_RTA_MAX_TASKS>(p, 5, sm_count, st);
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
  return 256 + align_up(nb * 8 * sizeof(unsigned int), 256) +
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
  KParams p;
  fill_params(&p, ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us, out_wcrt, out_sched);
  // Nothing in the array has to be cleared first: the plan kernels write the header (counts,
  // starts, zeroed work counters), every per-block count and every permutation entry that the
  // analysis kernels of this call read.
  return enqueue_batch(p, g_static_scratch_ptr[dev], (size_t)GCAPS_RTA_STATIC_SCRATCH_BYTES,
                       di.sm_count, (cudaStream_t)stream);
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

// Copies tasksets [t, t1) (tasks [k0, k1)) to the staging slot, enqueues their analysis and the
// copies of the results back.  The offsets of the range are known to be monotone and in range.
static int host_chunk(const gcaps_tasksets_t *ts, int64_t t, int64_t t1, int policy, int64_t L,
                      int64_t ovh, int64_t *out_wcrt, uint8_t *out_sched, int slot, int sm_count) {
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
  const size_t o_ge = take(ng * 8), o_wcrt = take(nk * 8), o_sched = take(nt);
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
  KParams p;
  fill_params(&p, &dts, nt, policy, L, ovh, (int64_t *)(d + o_wcrt), d + o_sched);
  p.task_base = k0, p.cseg_base = c0, p.gseg_base = g0;
  int rc = enqueue_batch(p, d + o_ws, ws_bytes, sm_count, st);
  if (rc != GCAPS_OK) return rc;
  if (nk > 0)
    HOST_TRY(cudaMemcpyAsync(out_wcrt + k0, d + o_wcrt, (size_t)nk * 8, cudaMemcpyDeviceToHost, st));
  HOST_TRY(cudaMemcpyAsync(out_sched + t, d + o_sched, (size_t)nt, cudaMemcpyDeviceToHost, st));
  return GCAPS_OK;
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
  int rc = check_args(ts, n_tasksets, policy, timeslice_us, ctx_switch_overhead_us);
  if (rc != GCAPS_OK) return rc;
  if (n_tasksets == 0) return GCAPS_OK;
  if (!out_sched || (ts->n_tasks > 0 && !out_wcrt)) return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  int dev = 0;
  HOST_TRY(cudaGetDevice(&dev));
  if (g_stage.device != dev) {
    gcaps_rta_release_host();
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
      rc = host_chunk(ts, t, t1, policy, timeslice_us, ctx_switch_overhead_us, out_wcrt, out_sched,
                      slot, di.sm_count);
      if (rc != GCAPS_OK) return rc;
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
        out_sched[t] = GCAPS_SCHED_INVALID;
      } else if (!host_range_is_canonical(ts, a, b)) {
        out_sched[t] = GCAPS_SCHED_INVALID;
        for (int64_t k = a; k < b; ++k) out_wcrt[k] = GCAPS_WCRT_INVALID;
      } else {
        rc = host_chunk(ts, t, t + 1, policy, timeslice_us, ctx_switch_overhead_us, out_wcrt,
                        out_sched, slot, di.sm_count);
        if (rc != GCAPS_OK) return rc;
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
