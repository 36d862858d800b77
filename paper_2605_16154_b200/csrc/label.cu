// Gripper-based phase labelling (Sec. 5.1 "Phase Labeling", App. E.2): every chunk gets one of five phases
// from the fraction of its timesteps with the gripper-close command active.  Thresholds are compared through
// integer counts, so the labels are exact.  One thread per trajectory: the rule is a short sequential scan.
#include "internal.h"

struct pcm_ctx;
namespace pcm { unsigned* ctx_status(pcm_ctx*); }

namespace pcm {

// phases and their priority when windows overlap: active-grip > pre-grasp > release-ramp > approach > tail
enum { PH_APPROACH = 0, PH_PRE = 1, PH_ACTIVE = 2, PH_RELEASE = 3, PH_TAIL = 4 };
__device__ __forceinline__ int phase_priority(int ph) {
  return ph == PH_ACTIVE ? 4 : ph == PH_PRE ? 3 : ph == PH_RELEASE ? 2 : ph == PH_APPROACH ? 1 : 0;
}

// scratch encoding in the output byte while a trajectory is being labelled:
//   bits 0..1: closure class 0: g < 0.1, 1: 0.1 <= g < 0.5, 2: 0.5 <= g < 0.75, 3: g >= 0.75
//   bits 4..6: label + 1 (0 = not claimed yet)
__global__ void label_phases_kernel(const int32_t* __restrict__ traj_off, const int32_t* __restrict__ step_off,
                                    const uint8_t* __restrict__ grip_close, int n_traj, int chunk_len,
                                    uint8_t* __restrict__ phase, unsigned* __restrict__ status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_traj) return;
  const int t0 = step_off[i], T = step_off[i + 1] - t0;
  const int a = traj_off[i], N = traj_off[i + 1] - a;
  if (T < 0 || N != (T + chunk_len - 1) / chunk_len) {
    atomicOr(status, STATUS_BAD_OFFSETS);
    return;
  }
  uint8_t* out = phase + a;
  for (int j = 0; j < N; ++j) {
    const int lo = j * chunk_len, hi = min(T, lo + chunk_len), n = hi - lo;
    int cnt = 0;
    for (int t = lo; t < hi; ++t) cnt += grip_close[t0 + t] ? 1 : 0;
    const int cls = (4 * cnt >= 3 * n) ? 3 : (2 * cnt >= n) ? 2 : (10 * cnt >= n) ? 1 : 0;
    out[j] = (uint8_t)(cls | (cls >= 2 ? ((PH_ACTIVE + 1) << 4) : 0));
  }
  auto claim = [&](int j, int ph) {
    const int cur = (out[j] >> 4) & 7;
    if (cur == 0 || phase_priority(ph) > phase_priority(cur - 1)) out[j] = (uint8_t)((out[j] & 3) | ((ph + 1) << 4));
  };
  int last_start = -1, last_end = -1;
  for (int j = 0; j < N; ++j) {
    if ((out[j] & 3) != 3) continue;
    const int s = j;
    while (j + 1 < N && (out[j + 1] & 3) == 3) ++j;
    const int e = j;
    for (int k = max(0, s - 3); k < s; ++k)
      if ((out[k] & 3) == 1) claim(k, PH_PRE);
    for (int k = e + 1; k < min(N, e + 4); ++k)
      if ((out[k] & 3) < 2) claim(k, PH_RELEASE);
    last_start = s;
    last_end = e;
  }
  for (int j = 0; j < N; ++j) {
    const int cur = (out[j] >> 4) & 7, cls = out[j] & 3;
    int ph;
    if (cur) ph = cur - 1;
    else if (j < last_start) ph = PH_APPROACH;
    else if (last_end >= 0 && j > last_end && cls == 0) ph = PH_TAIL;
    else ph = PH_APPROACH;
    out[j] = (uint8_t)ph;
  }
}

}  // namespace pcm

using namespace pcm;

extern "C" int pcm_label_phases(pcm_ctx* ctx, int32_t n_traj, const int32_t* traj_off, const int32_t* step_off,
                                const uint8_t* grip_close, int32_t chunk_len, uint8_t* phase, pcm_stream stream) {
  if (!ctx || !traj_off || !step_off || !grip_close || !phase || n_traj < 1 || chunk_len < 1) return PCM_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  label_phases_kernel<<<ceil_div(n_traj, 64), 64, 0, s>>>(traj_off, step_off, grip_close, n_traj, chunk_len, phase,
                                                           ctx_status(ctx));
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}
