// Optional per-kernel-class timing with CUDA events on the launching stream.  Off by default; when
// on, every instrumented launch is bracketed by an event pair and pcm_profile_read() adds up the
// elapsed times together with the algorithmic flops / bytes the caller declared for the launch.
#include <cstring>
#include <mutex>
#include <vector>

#include "internal.h"

namespace pcm {

struct ProfRecord { int cls; cudaEvent_t a, b; double flops, bytes; };

static bool g_prof_on = false;
static std::mutex g_prof_mu;
static std::vector<ProfRecord> g_prof_open;          // begun, end not yet recorded (used as a stack)
static std::vector<ProfRecord> g_prof_done;
static std::vector<cudaEvent_t> g_prof_pool;

bool prof_enabled() { return g_prof_on; }

static cudaEvent_t take_event() {
  if (!g_prof_pool.empty()) {
    cudaEvent_t e = g_prof_pool.back();
    g_prof_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

void prof_begin(int cls, cudaStream_t s) {
  if (!g_prof_on) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  ProfRecord r{cls, take_event(), take_event(), 0.0, 0.0};
  cudaEventRecord(r.a, s);
  g_prof_open.push_back(r);
}

void prof_end(cudaStream_t s, double flops, double bytes) {
  if (!g_prof_on) return;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  if (g_prof_open.empty()) return;
  ProfRecord r = g_prof_open.back();
  g_prof_open.pop_back();
  cudaEventRecord(r.b, s);
  r.flops = flops; r.bytes = bytes;
  g_prof_done.push_back(r);
}

}  // namespace pcm

using namespace pcm;

extern "C" int pcm_profile_enable(int32_t on) {
  std::lock_guard<std::mutex> lk(g_prof_mu);
  g_prof_on = on != 0;
  return PCM_OK;
}

extern "C" int pcm_profile_read(pcm_profile* out) {
  if (!out) return PCM_ERR_ARG;
  PCM_CUDA_TRY(cudaDeviceSynchronize());
  std::lock_guard<std::mutex> lk(g_prof_mu);
  memset(out, 0, sizeof(*out));
  for (const ProfRecord& r : g_prof_done) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, r.a, r.b) != cudaSuccess) ms = 0.f;
    if (r.cls >= 0 && r.cls < PCM_PROFILE_CLASSES) {
      out->ms[r.cls] += ms; out->flops[r.cls] += r.flops; out->bytes[r.cls] += r.bytes; out->launches[r.cls] += 1;
    }
    g_prof_pool.push_back(r.a);
    g_prof_pool.push_back(r.b);
  }
  g_prof_done.clear();
  return PCM_OK;
}

extern "C" int32_t pcm_first_use_on_device(uint64_t* seen_mask, int32_t device) {
  if (!seen_mask) return 1;
  unsigned long long m = *seen_mask;
  const bool first = first_use_on_device(&m, device);
  *seen_mask = m;
  return first ? 1 : 0;
}
