// Shared host/device helpers of the library: status codes, launch accounting.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>

#include "../../include/pcm_b200.h"

namespace pcm {

extern std::atomic<long long> g_launches;

// Device status word bits (latched with atomicOr, read by pcm_poll_status).
constexpr unsigned STATUS_TIMEOUT = 1u;       // a bounded wait expired
constexpr unsigned STATUS_BAD_PHASE = 2u;     // phase label >= n_phases
constexpr unsigned STATUS_TOO_LONG = 4u;      // trajectory longer than max_len
constexpr unsigned STATUS_BAD_OFFSETS = 8u;   // traj_off / kept_idx inconsistent with host sizes
constexpr unsigned STATUS_BAD_ACTION = 16u;   // continuous action not finite or beyond the fixed-point range

#define PCM_CUDA_TRY(expr)                         \
  do {                                             \
    cudaError_t e__ = (expr);                      \
    if (e__ != cudaSuccess) return PCM_ERR_CUDA;   \
  } while (0)

// Counts the launch and reports a launch-configuration error immediately.
#define PCM_LAUNCH_CHECK()                                   \
  do {                                                       \
    pcm::g_launches.fetch_add(1, std::memory_order_relaxed); \
    if (cudaPeekAtLastError() != cudaSuccess) {              \
      cudaGetLastError();                                    \
      return PCM_ERR_CUDA;                                   \
    }                                                        \
  } while (0)

static inline int ceil_div(long long a, long long b) { return (int)((a + b - 1) / b); }

// Per-device bookkeeping.  cudaFuncSetAttribute and the SM count belong to the current device, so a process that
// drives several GPUs needs them once per device, not once per process.
// First use of `seen_mask` on device `dev` (0..63) returns true and marks the device; devices outside that range
// always return true (the attribute is then simply set again).
static inline bool first_use_on_device(unsigned long long* seen_mask, int dev) {
  if (dev < 0 || dev >= 64) return true;
  if (*seen_mask & (1ull << dev)) return false;
  *seen_mask |= 1ull << dev;
  return true;
}
static inline bool attr_needed(unsigned long long* seen_mask) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return true;
  return first_use_on_device(seen_mask, dev);
}
// SM count of the current device, cached per device; 148 when the query fails.
static inline int sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 148;
  if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  if (dev >= 0 && dev < 64) cached[dev] = n;
  return n;
}

}  // namespace pcm
