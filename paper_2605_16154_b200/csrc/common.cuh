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

}  // namespace pcm
