// rta_common.cuh -- what the translation units of the library share: integer types, the launch
// plan's header, the kernel parameter block, the exact and the reciprocal arithmetic helpers, and
// the host-side argument checks.  Internal; the public interface is include/gcaps_rta.h.
#ifndef GCAPS_RTA_COMMON_CUH_
#define GCAPS_RTA_COMMON_CUH_

#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/gcaps_rta.h"

namespace gcaps_detail {

typedef unsigned long long u64;
typedef long long i64;

constexpr int kNumBins = 9;
constexpr int kBinStride = 12;  // counters per plan block and per header array
typedef unsigned int u32;
// size bins: at most 8, 16, 24, 32, 64, 96, 128, 192, 256 tasks
constexpr u32 kFastLimit = 1u << 26;  // fast path: every time of the taskset is below this
constexpr u32 kFastClamp = 1u << 26;  // ... so a sum clamped here still exceeds every deadline
constexpr int kBlockThreads = 128;
constexpr int kPlanItems = 1024;  // tasksets per plan block
constexpr int kPlanSmall = 8192;  // batches up to this size are planned by one block in one launch
constexpr u64 kClamp = 1ull << 50;  // any quantity >= 2^50 exceeds every deadline (<= 2^40)

struct PlanHeader {
  unsigned int bin_start[kBinStride];
  unsigned int bin_count[kBinStride];
  unsigned int next[kBinStride];  // work counters of the analysis launches
};
static_assert(sizeof(PlanHeader) <= 256, "header layout");

struct KParams {
  const i64 *task_off, *period, *deadline, *priority, *core;
  const i64 *cseg_off, *cseg_wcet, *gseg_off, *gseg_misc, *gseg_exec;
  i64 n_tasks, n_csegs, n_gsegs;        // lengths of the arrays the pointers address
  i64 task_base, cseg_base, gseg_base;  // subtracted from the stored offsets (chunked host path)
  i64 n_tasksets;
  int policy;  // GCAPS_POLICY_* | flags
  i64 L, ovh;
  // division by L in the 32-bit path: 0 = multiply-high by l_magic then shift, 1 = L is 1,
  // 2 = L >= 2^26 (every non-empty pure GPU part takes one slice)
  u32 l_mode, l_magic, l_shift;
  i64 *out_wcrt;
  uint8_t *out_sched;
  PlanHeader *hdr;
  unsigned int *block_cnt;  // [plan blocks][kBinStride]
  unsigned int *perm;       // [n_tasksets]
};

// The (timeslice, overhead) pairs of a fused sweep: one staging and aggregation of a taskset,
// one analysis per pair.  Passed to the sweep kernels by value.
struct SweepPoint {
  i64 L, ovh;
  u32 l_mode, l_magic, l_shift, pad;  // division by L in the 32-bit path, as in KParams
};
struct SweepArgs {
  int n;        // pairs, 1 .. GCAPS_RTA_MAX_SWEEP
  int enabled;  // analyses this launch runs per pair: bit m = mode m (0 GCAPS self-suspension,
                // 1 GCAPS busy-waiting, 2 RR self-suspension, 3 RR busy-waiting)
  // the analysis of pair q under mode m writes result block q * block_stride + block_of_mode[m]
  int block_stride;
  int block_of_mode[4];
  i64 max_ovh;  // largest overhead of the sweep
  SweepPoint q[GCAPS_RTA_MAX_SWEEP];
};

__device__ __forceinline__ int size_bin(i64 n) {
  if (n <= 8) return 0;  // also negative / broken ranges: rejected by the analysis kernel
  if (n <= 16) return 1;
  if (n <= 24) return 2;
  if (n <= 32) return 3;
  if (n <= 64) return 4;
  if (n <= 96) return 5;
  if (n <= 128) return 6;
  if (n <= 192) return 7;
  if (n <= GCAPS_RTA_MAX_TASKS) return 8;
  return 0;
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

constexpr unsigned int kFull = 0xffffffffu;

// Reciprocal of a divisor d in [2, 2^26): floor(x / d) = umulhi(x, magic) >> shift for every
// x < 2^28.  With s = ceil(log2 d) and k = max(28 + s, 32), magic = ceil(2^k / d) < 2^32 and its
// error magic*d - 2^k < d <= 2^s, so x * error < 2^k and the quotient is exact.
__host__ __device__ __forceinline__ void make_reciprocal(u32 d, u32 &magic, u32 &shift) {
#ifdef __CUDA_ARCH__
  const int s = 32 - __clz((int)(d - 1));
#else
  int s = 0;
  while ((1u << s) < d) ++s;
#endif
  const int k = (28 + s) > 32 ? (28 + s) : 32;
  shift = (u32)(k - 32);
#ifdef __CUDA_ARCH__
  // estimate 2^k / d in single precision (off by less than 2^10), correct the estimate once with
  // the same approximate reciprocal (off by at most 1 then), and finish with integers.  Checked
  // against the exact quotient for every d in [2, 2^26), also with the reciprocal off by 8 ulp.
  float inv;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(__uint2float_rn(d)));
  const u32 q0 = __float2uint_rd(inv * __int_as_float((127 + k) << 23));
  const i64 rem0 = (i64)(1ull << k) - (i64)((u64)q0 * d);
  const int c = __float2int_rd(__ll2float_rn(rem0) * inv);
  u32 q = q0 + (u32)c;
  i64 rem = rem0 - (i64)c * (i64)d;
  if (rem < 0) {
    q -= 1;
    rem += d;
  } else if (rem >= (i64)d) {
    q += 1;
    rem -= d;
  }
  magic = rem == 0 ? q : q + 1;
#else
  const u64 two_k = 1ull << k;
  magic = (u32)((two_k + d - 1) / d);
#endif
}

// The kernels of the size bins of one call follow one another in the caller's stream and share no
// data.  Each lets its dependents go at entry, and all but the first are launched with
// programmatic stream serialisation, so the next bin's blocks start as this one's leave.  A grid
// launched that way could otherwise also COMPLETE before its predecessor, and whatever the stream
// runs next (a copy of the results, the plan kernels of the next call rewriting the workspace)
// would then overtake a kernel that is still writing.  So every kernel ends with
// griddepcontrol.wait: no grid retires before the grid in front of it has completed and its writes
// are visible, completion is transitive along the chain, and the first kernel of the chain is an
// ordinary launch that waited for everything before it.
__device__ __forceinline__ void let_dependents_start() {
  asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void wait_for_previous_grid() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Launches `kernel` (a persistent kernel of kBlockThreads threads needing `smem` bytes) with as
// many blocks as the device keeps resident, but never more than the batch could feed.
// overlap_previous: the kernel launched just before on this stream works on other data (another
// size bin) and has let its dependents go (let_dependents_start), so this one is launched with
// programmatic stream serialisation and fills the SMs as that one's blocks leave instead of
// waiting for its last block.  It needs nothing that kernel writes, and it must end with
// wait_for_previous_grid().
extern std::mutex g_init_mutex;  // guards the once-per-device set-up steps of the library

template <typename... Args>
cudaError_t launch_persistent_ex(bool overlap_previous, void (*kernel)(Args...), int *blocks_per_sm,
                                 size_t smem, long long want, int sm_count, cudaStream_t st, Args... args) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  dev &= 63;
  int resident = __atomic_load_n(&blocks_per_sm[dev], __ATOMIC_ACQUIRE);
  if (resident == 0) {  // first use on this device (host threads may get here together)
    std::lock_guard<std::mutex> lock(g_init_mutex);
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kBlockThreads, smem);
    if (e != cudaSuccess) return e;
    resident = per_sm < 1 ? 1 : per_sm;
    __atomic_store_n(&blocks_per_sm[dev], resident, __ATOMIC_RELEASE);
  }
  long long grid = (long long)sm_count * resident;
  if (grid > want) grid = want;
  if (grid < 1) grid = 1;
  if (!overlap_previous) {
    kernel<<<(unsigned int)grid, kBlockThreads, smem, st>>>(args...);
    return cudaGetLastError();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned int)grid), cfg.blockDim = dim3(kBlockThreads);
  cfg.dynamicSmemBytes = smem, cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr, cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <typename... Args>
cudaError_t launch_persistent(void (*kernel)(Args...), int *blocks_per_sm, size_t smem, long long want,
                              int sm_count, cudaStream_t st, Args... args) {
  return launch_persistent_ex(false, kernel, blocks_per_sm, smem, want, sm_count, st, args...);
}


// ---- host side (defined in gcaps_rta.cu) -------------------------------------------------------
struct DeviceInfo {
  int sm_count;
  int ok;  // 1 = usable sm_100 device, -1 = not usable
};

extern thread_local int g_last_cuda_error;
int device_info(DeviceInfo *out);
int check_args(const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int64_t L, int64_t ovh);
void fill_params(KParams *p, const gcaps_tasksets_t *ts, int64_t n_tasksets, int policy, int64_t L,
                 int64_t ovh, int64_t *out_wcrt, uint8_t *out_sched);
// Points p at the plan areas of `workspace` and enqueues the three plan kernels (size bins, a
// permutation of the taskset indices, zeroed work counters).  GCAPS_OK or GCAPS_ERR_WORKSPACE.
int enqueue_plan(KParams &p, void *workspace, size_t workspace_bytes, cudaStream_t st);
// One launch over all size bins for analysis `mode` (0 GCAPS self-suspension, 1 GCAPS
// busy-waiting, 2 RR self-suspension, 3 RR busy-waiting); defined in gcaps_rta_any.cu.
cudaError_t launch_any_bins(int mode, const KParams &p, int sm_count, cudaStream_t st);

}  // namespace gcaps_detail
#endif  // GCAPS_RTA_COMMON_CUH_
