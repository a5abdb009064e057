// gcaps_diag.cu -- measurement aids of the library: the integer issue rate of the device (the
// second roofline of the analysis: its inner loop is plain integer arithmetic, no tensor cores)
// and the planning step of a call on its own (so that "plan" and "analysis" can be timed apart).
// Neither is part of the analysis path.
#include <cuda_runtime.h>
#include <stdint.h>

#include "rta_common.cuh"

using namespace gcaps_detail;

namespace {

constexpr int kProbeThreads = 256;
constexpr int kProbeBlocksPerSm = 8;
constexpr int kChains = 8;   // independent dependency chains per thread
constexpr int kUnroll = 16;  // chain steps per loop trip

// KIND 0: multiply-add chains  a <- a * m + c
// KIND 1: add chains           a <- a + b, b <- b + a
// KIND 2: one of each          a <- a * m + b, b <- b + a
// Every chain depends only on itself, eight chains per thread and 64 warps per SM keep the issue
// slots full; nothing touches memory until the end.  The result is compared with a value it
// cannot be proven different from, so the arithmetic stays.
template <int KIND>
__global__ void __launch_bounds__(kProbeThreads) int_issue_kernel(u32 *out, u32 trips, u32 m, u32 c) {
  u32 a[kChains], b[kChains];
#pragma unroll
  for (int j = 0; j < kChains; ++j) {
    a[j] = (blockIdx.x * kProbeThreads + threadIdx.x) * 2654435761u + (u32)j * 40503u + c;
    b[j] = a[j] ^ m;
  }
  for (u32 t = 0; t < trips; ++t) {
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
      for (int j = 0; j < kChains; ++j) {
        if (KIND == 0) {
          a[j] = a[j] * m + c;
        } else if (KIND == 1) {
          a[j] = a[j] + b[j];
          b[j] = b[j] + a[j];
        } else {
          a[j] = a[j] * m + b[j];
          b[j] = b[j] + a[j];
        }
      }
    }
  }
  u32 x = 0;
#pragma unroll
  for (int j = 0; j < kChains; ++j) x ^= a[j] + b[j];
  if (x == 0x9e3779b9u && m == 1u) atomicAdd(out, 1u);
}

}  // namespace

extern "C" int gcaps_rta_int_issue_probe(int kind, int64_t trips, uint32_t *scratch, int64_t *out_lane_ops,
                                         void *stream) {
  if (kind < 0 || kind > 2 || trips < 1 || trips > (1 << 24) || !scratch || !out_lane_ops)
    return GCAPS_ERR_INVALID_ARG;
  DeviceInfo di;
  const int rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  const unsigned int grid = (unsigned int)(di.sm_count * kProbeBlocksPerSm);
  const u32 m = 2891336453u, c = 12345u;
  cudaStream_t st = (cudaStream_t)stream;
  if (kind == 0) int_issue_kernel<0><<<grid, kProbeThreads, 0, st>>>(scratch, (u32)trips, m, c);
  else if (kind == 1) int_issue_kernel<1><<<grid, kProbeThreads, 0, st>>>(scratch, (u32)trips, m, c);
  else int_issue_kernel<2><<<grid, kProbeThreads, 0, st>>>(scratch, (u32)trips, m, c);
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  const int64_t per_step = kind == 0 ? 1 : 2;  // arithmetic instructions per chain step
  *out_lane_ops = (int64_t)grid * kProbeThreads * kChains * kUnroll * trips * per_step;
  return GCAPS_OK;
}

extern "C" int gcaps_rta_plan_batch(const gcaps_tasksets_t *ts, int64_t n_tasksets, void *workspace,
                                    size_t workspace_bytes, void *stream) {
  int rc = check_args(ts, n_tasksets, GCAPS_POLICY_GCAPS, 1, 0);
  if (rc != GCAPS_OK) return rc;
  if (n_tasksets == 0) return GCAPS_OK;
  DeviceInfo di;
  rc = device_info(&di);
  if (rc != GCAPS_OK) return rc;
  KParams p;
  fill_params(&p, ts, n_tasksets, GCAPS_POLICY_GCAPS, 1, 0, nullptr, nullptr);
  rc = enqueue_plan(p, workspace, workspace_bytes, (cudaStream_t)stream);
  if (rc != GCAPS_OK) return rc;
  const cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return GCAPS_ERR_CUDA;
  }
  return GCAPS_OK;
}
