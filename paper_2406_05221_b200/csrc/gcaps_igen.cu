// gcaps_igen.cu -- on-device generation of synthetic tasksets (the generation procedure of
// GCAPS, ECRTS 2024, arXiv 2406.05221, Sec. 7.1 / Table 3) for NVIDIA B200 (sm_100a).
//
// The generator itself is igen.h (integer-only; the host generator compiles the same
// definition).  gcaps_gen_count: one thread per taskset runs the per-task part of the generator
// (igen_begin), writes the three sizes of the taskset and leaves what it drew per task (period,
// execution demand, priority, core, GPU segments: 12 bytes per task) and the position of the
// random stream in the workspace; three exclusive scans turn the sizes into offsets (block sums,
// one block over the block sums, block-local scan).  gcaps_gen_fill: one warp per taskset, lane =
// task; the random draws of a task start at a position that is a prefix sum over the tasks
// before it (the random source is counter-based), so every lane splits its own task's demand
// into segments (igen_task_segments) and writes them at offsets that are prefix sums again.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include "igen.h"
#include "rta_common.cuh"

using namespace gcaps_detail;

static_assert(sizeof(gcaps_gen_params_t) == sizeof(igen_params_t), "same layout");

namespace {

constexpr int kGenThreads = 128;
constexpr int kScanThreads = 256;
constexpr int kScanItems = 4 * kScanThreads;  // elements of one scan block

// workspace: off[3][count + 1] (tasks, CPU segments, GPU segments), block sums [3][blocks], then
// the per-taskset state: state_stride 32-bit words each -- key and counter of the random stream
// (4 words), then per task T, E and (priority | core << 16 | GPU segments << 24)
struct GenSpace {
  i64 *off[3];
  i64 *block_sum[3];
  i64 n_blocks;
  u32 *state;
  i64 state_stride;
};

__host__ __device__ inline i64 max_tasks_of(const igen_params_t &p) {
  const i64 m = (i64)p.cores_hi * (i64)p.tpc_hi;
  return m > IGEN_MAX_TASKS ? IGEN_MAX_TASKS : m;
}

__host__ __device__ inline i64 scan_blocks(i64 count) { return (count + kScanItems - 1) / kScanItems; }

__global__ void __launch_bounds__(kGenThreads) gen_count_kernel(igen_params_t p, i64 first, i64 count,
                                                                 GenSpace w) {
  const i64 t = (i64)blockIdx.x * kGenThreads + threadIdx.x;
  if (t >= count) return;
  igen_state_t s;
  igen_begin(&p, (uint64_t)(first + t), &s);
  w.off[0][t] = s.n, w.off[1][t] = s.n_csegs, w.off[2][t] = s.n_gsegs;
  u32 *st = w.state + t * w.state_stride;
  st[0] = (u32)s.rng.key, st[1] = (u32)(s.rng.key >> 32);
  st[2] = (u32)s.rng.ctr, st[3] = (u32)(s.rng.ctr >> 32);
  for (int i = 0; i < s.n; ++i) {
    st[4 + 3 * i] = s.T[i];
    st[5 + 3 * i] = s.E[i];
    st[6 + 3 * i] = (u32)s.prio[i] | ((u32)s.core[i] << 16) | ((u32)s.eta[i] << 24);
  }
}

__device__ __forceinline__ i64 block_exclusive_scan(i64 v, i64 *total, i64 *warp_sums) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  i64 x = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const i64 y = __shfl_up_sync(kFull, x, d);
    if (lane >= d) x += y;
  }
  if (lane == 31) warp_sums[warp] = x;
  __syncthreads();
  if (warp == 0) {
    i64 ws = lane < kScanThreads / 32 ? warp_sums[lane] : 0;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const i64 y = __shfl_up_sync(kFull, ws, d);
      if (lane >= d) ws += y;
    }
    if (lane < kScanThreads / 32) warp_sums[lane] = ws;  // inclusive sums of the warps
  }
  __syncthreads();
  const i64 before = warp > 0 ? warp_sums[warp - 1] : 0;
  *total = warp_sums[kScanThreads / 32 - 1];
  __syncthreads();
  return before + x - v;
}

// sums of every block of kScanItems sizes, for the three arrays (blockIdx.y)
__global__ void __launch_bounds__(kScanThreads) scan_sums_kernel(GenSpace w, i64 count) {
  __shared__ i64 warp_sums[kScanThreads / 32];
  const i64 *in = w.off[blockIdx.y];
  const i64 base = (i64)blockIdx.x * kScanItems + 4 * threadIdx.x;
  i64 v = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    if (base + j < count) v += in[base + j];
  i64 total;
  block_exclusive_scan(v, &total, warp_sums);
  if (threadIdx.x == 0) w.block_sum[blockIdx.y][blockIdx.x] = total;
}

// one block per array: block sums -> exclusive offsets of the blocks; the grand total goes to
// off[a][count] and to out_totals[a]
__global__ void __launch_bounds__(kScanThreads) scan_blocks_kernel(GenSpace w, i64 count, i64 *out_totals) {
  __shared__ i64 warp_sums[kScanThreads / 32];
  i64 *bs = w.block_sum[blockIdx.x];
  i64 carry = 0;
  for (i64 b0 = 0; b0 < w.n_blocks; b0 += kScanThreads) {
    const i64 b = b0 + threadIdx.x;
    const i64 v = b < w.n_blocks ? bs[b] : 0;
    i64 total;
    const i64 ex = block_exclusive_scan(v, &total, warp_sums);
    if (b < w.n_blocks) bs[b] = carry + ex;
    carry += total;
  }
  if (threadIdx.x == 0) {
    w.off[blockIdx.x][count] = carry;
    out_totals[blockIdx.x] = carry;
  }
}

// sizes -> exclusive offsets, in place
__global__ void __launch_bounds__(kScanThreads) scan_apply_kernel(GenSpace w, i64 count) {
  __shared__ i64 warp_sums[kScanThreads / 32];
  i64 *io = w.off[blockIdx.y];
  const i64 base = (i64)blockIdx.x * kScanItems + 4 * threadIdx.x;
  i64 x[4], v = 0;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    x[j] = base + j < count ? io[base + j] : 0;
    v += x[j];
  }
  i64 total;
  i64 run = w.block_sum[blockIdx.y][blockIdx.x] + block_exclusive_scan(v, &total, warp_sums);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    if (base + j < count) io[base + j] = run;
    run += x[j];
  }
}

struct GenOut {
  i64 *task_off, *period, *deadline, *priority, *core, *cseg_off, *cseg_wcet, *gseg_off, *gseg_misc, *gseg_exec;
  i64 cap_tasks, cap_csegs, cap_gsegs;
};

__device__ __forceinline__ u32 warp_exclusive(u32 v, int lane, u32 *total) {
  u32 x = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const u32 y = __shfl_up_sync(kFull, x, d);
    if (lane >= d) x += y;
  }
  *total = __shfl_sync(kFull, x, 31);
  return x - v;
}

__global__ void __launch_bounds__(kGenThreads) gen_fill_kernel(igen_params_t p, i64 first, i64 count,
                                                                GenSpace w, GenOut o) {
  const int lane = threadIdx.x & 31;
  const i64 t = (i64)blockIdx.x * (kGenThreads / 32) + (threadIdx.x >> 5);
  if (t >= count) return;
  const i64 k0 = w.off[0][t], n = w.off[0][t + 1] - k0;
  const i64 c_start = w.off[1][t], g_start = w.off[2][t];
  if (lane == 0) o.task_off[t] = k0;
  const bool fits = k0 + n <= o.cap_tasks && w.off[1][t + 1] <= o.cap_csegs && w.off[2][t + 1] <= o.cap_gsegs;
  if (fits) {
    const u32 *st = w.state + t * w.state_stride;
    const uint64_t key = (uint64_t)st[0] | ((uint64_t)st[1] << 32);
    uint64_t ctr = (uint64_t)st[2] | ((uint64_t)st[3] << 32);
    u32 c_run = 0, g_run = 0;  // segments of the tasks before this round of 32
    for (i64 i0 = 0; i0 < n; i0 += 32) {
      const i64 i = i0 + lane;
      const bool mine = i < n;
      u32 T = 0, E = 0, pk = 0;
      if (mine) T = st[4 + 3 * i], E = st[5 + 3 * i], pk = st[6 + 3 * i];
      const int eta = (int)(pk >> 24);
      u32 draws_total, c_total, g_total;
      const u32 draws_before = warp_exclusive(mine ? igen_task_draws(eta) : 0u, lane, &draws_total);
      const u32 c_before = warp_exclusive(mine ? (u32)eta + 1u : 0u, lane, &c_total);
      const u32 g_before = warp_exclusive(mine ? (u32)eta : 0u, lane, &g_total);
      if (mine) {
        igen_rng_t rng;
        rng.key = key, rng.ctr = ctr + draws_before;
        const i64 c0 = c_start + c_run + c_before, g0 = g_start + g_run + g_before;
        // the segment values go straight to their places in the output arrays
        igen_task_segments(&rng, (int64_t)E, eta, p.ratio_lo, p.ratio_hi, (int64_t *)(o.cseg_wcet + c0),
                           (int64_t *)(o.gseg_misc + g0), (int64_t *)(o.gseg_exec + g0));
        o.period[k0 + i] = T;
        o.deadline[k0 + i] = T;
        o.priority[k0 + i] = pk & 0xffffu;
        o.core[k0 + i] = (pk >> 16) & 0xffu;
        o.cseg_off[k0 + i] = c0;
        o.gseg_off[k0 + i] = g0;
      }
      ctr += draws_total, c_run += c_total, g_run += g_total;
    }
  }
  if (t == count - 1 && lane == 0) {
    o.task_off[count] = w.off[0][count];
    if (w.off[0][count] <= o.cap_tasks) {
      o.cseg_off[w.off[0][count]] = w.off[1][count];
      o.gseg_off[w.off[0][count]] = w.off[2][count];
    }
  }
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

bool params_ok(const gcaps_gen_params_t *p) {
  return p && p->cores_lo >= 1 && p->cores_hi >= p->cores_lo && p->cores_hi <= IGEN_MAX_CORES &&
         p->tpc_lo >= 0 && p->tpc_hi >= p->tpc_lo && p->tpc_hi <= IGEN_MAX_TASKS &&
         p->util_lo <= p->util_hi && p->util_hi < (1ULL << 32) && p->log2_lo <= p->log2_hi &&
         p->log2_hi0 >= p->log2_lo && p->log2_hi < (31ULL << 32) && p->log2_hi0 < (31ULL << 32) &&
         p->period_lo >= 1 && p->period_hi >= p->period_lo && p->period_hi <= (1LL << 30) &&
         p->harmonic <= (1ULL << 32) && p->gpu_frac <= (1ULL << 32) && p->ratio_lo <= p->ratio_hi &&
         p->ratio_hi < (1ULL << 32) && (p->gpu_mode == 0 || p->gpu_mode == 1) && p->seg_lo >= 0 &&
         p->seg_hi >= p->seg_lo && p->seg_hi <= IGEN_MAX_SEGS;
}

int make_space(GenSpace *w, const gcaps_gen_params_t *params, int64_t count, void *workspace,
               size_t workspace_bytes) {
  if (!workspace || workspace_bytes < gcaps_gen_workspace_bytes(params, count) || ((uintptr_t)workspace & 255u))
    return GCAPS_ERR_WORKSPACE;
  unsigned char *b = (unsigned char *)workspace;
  const size_t off_bytes = align256((size_t)(count + 1) * sizeof(i64));
  w->n_blocks = scan_blocks(count);
  const size_t sum_bytes = align256((size_t)w->n_blocks * sizeof(i64));
  for (int a = 0; a < 3; ++a) {
    w->off[a] = (i64 *)(b + a * off_bytes);
    w->block_sum[a] = (i64 *)(b + 3 * off_bytes + a * sum_bytes);
  }
  igen_params_t p;
  memcpy(&p, params, sizeof(p));
  w->state = (u32 *)(b + 3 * off_bytes + 3 * sum_bytes);
  w->state_stride = 4 + 3 * max_tasks_of(p);
  return GCAPS_OK;
}

}  // namespace

extern "C" {

size_t gcaps_gen_workspace_bytes(const gcaps_gen_params_t *params, int64_t count) {
  if (count <= 0 || !params_ok(params)) return 0;
  igen_params_t p;
  memcpy(&p, params, sizeof(p));
  return 3 * align256((size_t)(count + 1) * sizeof(i64)) +
         3 * align256((size_t)scan_blocks(count) * sizeof(i64)) +
         align256((size_t)count * (size_t)(4 + 3 * max_tasks_of(p)) * sizeof(u32));
}

int gcaps_gen_count(const gcaps_gen_params_t *params, int64_t first, int64_t count,
                    int64_t *out_totals, void *workspace, size_t workspace_bytes, void *stream) {
  if (!params_ok(params) || first < 0 || count < 0 || count > 0x7fffffffLL || !out_totals)
    return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (count == 0) {
    cudaError_t e = cudaMemsetAsync(out_totals, 0, 3 * sizeof(int64_t), st);
    if (e != cudaSuccess) {
      g_last_cuda_error = (int)e;
      return GCAPS_ERR_CUDA;
    }
    return GCAPS_OK;
  }
  GenSpace w;
  rc = make_space(&w, params, count, workspace, workspace_bytes);
  if (rc != GCAPS_OK) return rc;
  igen_params_t p;
  memcpy(&p, params, sizeof(p));
  gen_count_kernel<<<(unsigned int)((count + kGenThreads - 1) / kGenThreads), kGenThreads, 0, st>>>(p, first, count, w);
  scan_sums_kernel<<<dim3((unsigned int)w.n_blocks, 3), kScanThreads, 0, st>>>(w, count);
  scan_blocks_kernel<<<3, kScanThreads, 0, st>>>(w, count, (i64 *)out_totals);
  scan_apply_kernel<<<dim3((unsigned int)w.n_blocks, 3), kScanThreads, 0, st>>>(w, count);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}

int gcaps_gen_fill(const gcaps_gen_params_t *params, int64_t first, int64_t count,
                   const gcaps_tasksets_t *ts, void *workspace, size_t workspace_bytes, void *stream) {
  if (!params_ok(params) || first < 0 || count < 0 || count > 0x7fffffffLL || !ts) return GCAPS_ERR_INVALID_ARG;
  if (count == 0) return GCAPS_OK;
  if (!ts->task_off || ts->n_tasks < 0 || ts->n_csegs < 0 || ts->n_gsegs < 0 || !ts->cseg_off || !ts->gseg_off ||
      (ts->n_tasks > 0 && (!ts->period || !ts->deadline || !ts->priority || !ts->core)) ||
      (ts->n_csegs > 0 && !ts->cseg_wcet) || (ts->n_gsegs > 0 && (!ts->gseg_misc || !ts->gseg_exec)))
    return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  GenSpace w;
  rc = make_space(&w, params, count, workspace, workspace_bytes);
  if (rc != GCAPS_OK) return rc;
  igen_params_t p;
  memcpy(&p, params, sizeof(p));
  GenOut o;
  o.task_off = (i64 *)ts->task_off, o.period = (i64 *)ts->period, o.deadline = (i64 *)ts->deadline;
  o.priority = (i64 *)ts->priority, o.core = (i64 *)ts->core, o.cseg_off = (i64 *)ts->cseg_off;
  o.cseg_wcet = (i64 *)ts->cseg_wcet, o.gseg_off = (i64 *)ts->gseg_off;
  o.gseg_misc = (i64 *)ts->gseg_misc, o.gseg_exec = (i64 *)ts->gseg_exec;
  o.cap_tasks = ts->n_tasks, o.cap_csegs = ts->n_csegs, o.cap_gsegs = ts->n_gsegs;
  constexpr int kWarps = kGenThreads / 32;
  gen_fill_kernel<<<(unsigned int)((count + kWarps - 1) / kWarps), kGenThreads, 0, (cudaStream_t)stream>>>(
      p, first, count, w, o);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}

}  // extern "C"
