// PCM control plane on the device: advantages (Eq. 1), phase scores (Eq. 5), online keep-probability
// update (Eq. 7-9), fixed-budget weighted sampling on a Philox stream (Eq. 10), and the context that
// holds the persistent state.
#include <cstring>
#include <mutex>
#include <new>

#include "async_ptx.cuh"
#include "internal.h"

namespace pcm {
std::atomic<long long> g_launches{0};

constexpr int ACT = PCM_ACT_DIM;           // 56 action tokens per chunk
constexpr int WORDS = ACT / 4;             // 14 32-bit words per chunk
constexpr int STATE_VERSION = 1;

struct KeepState {                         // persistent, device resident
  double buf[PCM_MAX_PHASES][PCM_MAX_TRC]; // phase-score buffers B_c
  double p[PCM_MAX_PHASES];                // keep-probabilities p_c
  long long step;
  int count;                               // entries currently in every buffer
  int n_refresh;
};

struct StateBlob {                         // host representation for export / import
  int version;
  int n_phases;
  int t_rc;
  int pad;
  KeepState st;
};

}  // namespace pcm

struct pcm_ctx {
  pcm_config cfg;
  int max_traj;
  int device;
  pcm::KeepState* state;       // device
  unsigned* status;            // device status word
  double* c_group;             // device [max_groups][n_phases]
  uint8_t* valid_group;        // device [max_groups][n_phases]
  int32_t* n_pos;              // device [max_traj]: chunks of positive weight per trajectory (sampler scratch)
};

namespace pcm {

unsigned* ctx_status(pcm_ctx* c) { return c->status; }

// ------------------------------------------------------------------------------------------------
// Eq. 5, per group: integer token sums per (phase, outcome), then C_{c,g}
// ------------------------------------------------------------------------------------------------
// One CTA per group, a warp per trajectory.  The trajectory's tokens are staged in shared memory by asynchronous
// copies (slabs of 32 chunks, two in flight per warp, about 170 KB per SM over all resident warps).  The sums
// per (phase, dimension) of a slab are an integer contraction over its chunks,
//     Sum[dim][phase] += tok^T[dim][chunk] * onehot[chunk][phase],
// and run on the tensor cores as mma.sync m16n8k32 (u8 x u8 -> s32): per slab a lane reads eight 8-byte vectors,
// transposes bytes in registers (the data has dimensions contiguous, the contraction index must be), builds the
// one-hot operand from the slab's labels with byte compares, and issues 4 x NT MMAs (NT = ceil(n_phases / 8)).
// Dimension 56 of the padded 64 is the constant 1, so the chunk counts come out of the same products.  Labels may
// come in any order: nothing depends on runs.  Accumulators stay in registers for the whole trajectory and are
// flushed once, with 32-bit shared-memory adds.  Integer sums are exact, so any order gives the same result.
// (A byte costs one ALU operation per lane in a packed-add scheme, which left the kernel instruction-bound at less
// than half of the copy bandwidth; the contraction costs a fraction of that.)
constexpr int SC_SLAB = 32;                              // chunks per staged slab = the contraction length of one MMA
constexpr int SC_SLAB_BYTES = SC_SLAB * ACT;             // 1792
constexpr int SC_WARPS = 8;

__device__ __forceinline__ void cp_async_8(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// D (16 x 8, s32) += A (16 x 32, u8, row) * B (32 x 8, u8, col).  Lane = 4 g + t: A registers hold rows g, g + 8 and
// contraction indices 4 t .. 4 t + 3 (a0, a1) and 16 + 4 t .. (a2, a3), lowest byte first; B registers hold column g
// and the same contraction indices; D registers hold rows g (c0, c1) and g + 8 (c2, c3), columns 2 t and 2 t + 1.
__device__ __forceinline__ void imma_16x8x32(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                             uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// r[m] = byte m of w0, w1, w2, w3 (lowest byte first): a 4 x 4 byte transpose
__device__ __forceinline__ void transpose4(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3, uint32_t (&r)[4]) {
  const uint32_t t0 = __byte_perm(w0, w1, 0x5140), t1 = __byte_perm(w2, w3, 0x5140);
  const uint32_t t2 = __byte_perm(w0, w1, 0x7362), t3 = __byte_perm(w2, w3, 0x7362);
  r[0] = __byte_perm(t0, t1, 0x5410); r[1] = __byte_perm(t0, t1, 0x7632);
  r[2] = __byte_perm(t2, t3, 0x5410); r[3] = __byte_perm(t2, t3, 0x7632);
}

template <int NT>
__global__ void __launch_bounds__(SC_WARPS * 32, NT <= 2 ? 4 : 2)
score_groups_kernel(const int32_t* __restrict__ traj_off, const uint8_t* __restrict__ tok,
                    const uint8_t* __restrict__ phase, const uint8_t* __restrict__ reward, int G,
                    int n_phases, double* __restrict__ c_group, uint8_t* __restrict__ valid_group,
                    unsigned* __restrict__ status) {
  extern __shared__ __align__(16) unsigned sm[];
  const int n_cnt = (n_phases * 2 * (ACT + 1) + 3) & ~3; // counters, padded to 16 bytes
  unsigned* sums = sm;                                   // [n_phases][2][56]
  unsigned* cnt = sm + n_phases * 2 * ACT;               // [n_phases][2]
  uint8_t* stage = reinterpret_cast<uint8_t*>(sm + n_cnt);   // [SC_WARPS][2][SC_SLAB_BYTES]
  __shared__ __align__(16) unsigned char lab_s[SC_WARPS][SC_SLAB];   // the current slab's labels, 0x40 = no chunk / bad label
  const int g = blockIdx.x;
  for (int i = threadIdx.x; i < n_phases * 2 * (ACT + 1); i += blockDim.x) sm[i] = 0;
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gid = lane >> 2, tig = lane & 3;             // fragment coordinates: rows gid, gid + 8; contraction indices 4 tig ..
  uint8_t* mybuf = stage + (size_t)warp * 2 * SC_SLAB_BYTES;
  unsigned char* lab = lab_s[warp];

  for (int i = g * G + warp; i < (g + 1) * G; i += SC_WARPS) {
    const int o = reward[i] ? 1 : 0;
    const int a = traj_off[i], b = traj_off[i + 1];
    const int n_slab = (b - a + SC_SLAB - 1) / SC_SLAB;
    // stage slab k (chunks a + 32 k ..) into buffer k & 1, one commit group per slab: 16-byte pieces when the slab
    // starts at an even chunk (56 c is then a multiple of 16), 8-byte pieces otherwise and for an odd tail
    auto issue = [&](int k) {
      const int c0 = a + k * SC_SLAB, nc = min(SC_SLAB, b - c0);
      const uint8_t* src = tok + (size_t)c0 * ACT;
      uint8_t* dst = mybuf + (k & 1) * SC_SLAB_BYTES;
      const int bytes = nc * ACT;
      if ((c0 & 1) == 0) {
        const int n16 = bytes >> 4;
        for (int piece = lane; piece < n16; piece += 32) cp_async_16(dst + piece * 16, src + piece * 16);
        if ((bytes & 8) && lane == 0) cp_async_8(dst + n16 * 16, src + n16 * 16);
      } else {
        for (int piece = lane; piece < (bytes >> 3); piece += 32) cp_async_8(dst + piece * 8, src + piece * 8);
      }
      cp_async_commit();
    };
    if (n_slab > 0) issue(0);
    if (n_slab > 1) issue(1);
    // acc[j][n]: rows = dimensions 8 gid + 2 j (c0, c1) and 8 gid + 2 j + 1 (c2, c3); columns = phases 8 n + 2 tig, + 1
    int acc[4][NT][4];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int n = 0; n < NT; ++n) acc[j][n][0] = acc[j][n][1] = acc[j][n][2] = acc[j][n][3] = 0;
    for (int k = 0; k < n_slab; ++k) {
      const int c0 = a + k * SC_SLAB, nc = min(SC_SLAB, b - c0);
      // this slab's labels, one per lane, requested before the wait so that they overlap the copies
      int l0 = lane < nc ? (int)__ldg(phase + c0 + lane) : 0x40;
      const bool bad = lane < nc && l0 >= n_phases;        // reported; the chunk matches no phase and drops out
      if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, STATUS_BAD_PHASE);
      if (bad) l0 = 0x40;
      __syncwarp();                                      // the previous slab's labels have been read by every lane
      lab[lane] = (unsigned char)l0;
      if (k + 1 < n_slab) cp_async_wait<1>(); else cp_async_wait<0>();
      __syncwarp();
      const uint8_t* buf = mybuf + (k & 1) * SC_SLAB_BYTES;
      // A operand: T[h][m] = dimension 8 gid + m of chunks 16 h + 4 tig .. + 3.  The group gid = 7 holds the padding
      // dimensions 56 .. 63: dimension 56 is the constant 1 (it counts chunks), the others are 0.
      uint32_t T[2][8];
      if (gid < 7) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint2 w[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) w[q] = *reinterpret_cast<const uint2*>(buf + (16 * h + 4 * tig + q) * ACT + 8 * gid);
          uint32_t lo[4], hi[4];
          transpose4(w[0].x, w[1].x, w[2].x, w[3].x, lo);
          transpose4(w[0].y, w[1].y, w[2].y, w[3].y, hi);
#pragma unroll
          for (int m = 0; m < 4; ++m) { T[h][m] = lo[m]; T[h][4 + m] = hi[m]; }
        }
      } else {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          T[h][0] = 0x01010101u;
#pragma unroll
          for (int m = 1; m < 8; ++m) T[h][m] = 0u;
        }
      }
      // B operand: one-hot of the labels against phase 8 n + gid
      const uint32_t lab_lo = *reinterpret_cast<const uint32_t*>(lab + 4 * tig);
      const uint32_t lab_hi = *reinterpret_cast<const uint32_t*>(lab + 16 + 4 * tig);
#pragma unroll
      for (int n = 0; n < NT; ++n) {
        // byte-wise "label == phase": labels are below 0x60 (a phase, or the 0x40 of a chunk that takes no part), so
        // x = label ^ phase is below 0x80 and x + 0x7f sets bit 7 exactly where x != 0, without carrying into the next byte
        const uint32_t rep = (uint32_t)(8 * n + gid) * 0x01010101u;
        const uint32_t b0 = (~((lab_lo ^ rep) + 0x7f7f7f7fu) >> 7) & 0x01010101u;
        const uint32_t b1 = (~((lab_hi ^ rep) + 0x7f7f7f7fu) >> 7) & 0x01010101u;
#pragma unroll
        for (int j = 0; j < 4; ++j) imma_16x8x32(acc[j][n], T[0][2 * j], T[0][2 * j + 1], T[1][2 * j], T[1][2 * j + 1], b0, b1);
      }
      __syncwarp();                                      // every lane is done with the buffer before it is refilled
      if (k + 2 < n_slab) issue(k + 2);
    }
    // flush the trajectory's sums: this lane holds dimensions 8 gid + 2 j, + 1 for phases 8 n + 2 tig, + 1
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int dim = 8 * gid + 2 * j + (e >> 1), ph = 8 * n + 2 * tig + (e & 1);
          const int v = acc[j][n][e];
          if (ph < n_phases && v != 0) {
            if (dim < ACT) atomicAdd(sums + (ph * 2 + o) * ACT + dim, (unsigned)v);
            else if (dim == ACT) atomicAdd(cnt + ph * 2 + o, (unsigned)v);
          }
        }
  }
  __syncthreads();

  // C_{c,g}: individually rounded fp64 operations.  All threads form the squared differences of the phases present
  // in both outcomes; then lane c of the first warp adds phase c's 56 values in ascending-dimension order, which is
  // the order the result is defined with (the chains of all phases run side by side).
  double* sq = reinterpret_cast<double*>(stage);         // [n_phases][56], over the token slabs (no longer needed)
  for (int idx = threadIdx.x; idx < n_phases * ACT; idx += blockDim.x) {
    const int c = idx / ACT, dim = idx - c * ACT;
    const unsigned n_succ = cnt[c * 2 + 1], n_fail = cnt[c * 2 + 0];
    if (n_succ && n_fail) {
      const double m1 = __ddiv_rn((double)sums[(c * 2 + 1) * ACT + dim], (double)n_succ);
      const double m0 = __ddiv_rn((double)sums[(c * 2 + 0) * ACT + dim], (double)n_fail);
      const double diff = __dsub_rn(m1, m0);
      sq[idx] = __dmul_rn(diff, diff);
    }
  }
  __syncthreads();
  if (threadIdx.x < n_phases) {
    const int c = threadIdx.x;
    const bool both = cnt[c * 2 + 1] && cnt[c * 2 + 0];
    double val = 0.0;
    if (both) {
      double acc = 0.0;
      for (int dim = 0; dim < ACT; ++dim) acc = __dadd_rn(acc, sq[c * ACT + dim]);
      val = __dmul_rn(__dsqrt_rn(acc), 2.0 / 256.0);
    }
    c_group[(size_t)g * n_phases + c] = val;
    valid_group[(size_t)g * n_phases + c] = both ? 1 : 0;
  }
}

// ------------------------------------------------------------------------------------------------
// Eq. 5 on continuous actions (float32 [n_chunks][56]).  Every value is read as the integer
// round-half-even(a * 2^32); sums over chunks are then exact 64-bit integers, independent of their order.
// One CTA per group, a warp per trajectory; a chunk is 14 float4, so lanes 0..13 and 14..27 each walk one
// contiguous half of the trajectory and keep four running sums per lane while the phase does not change.
// ------------------------------------------------------------------------------------------------
constexpr float ACT_ABS_MAX = 4096.f;                     // |a| * 2^32 <= 2^44; 2^18 chunks per group stay below 2^63
constexpr int ACT_MAX_GROUP_CHUNKS = 1 << 18;

__global__ void __launch_bounds__(256)
score_groups_f32_kernel(const int32_t* __restrict__ traj_off, const float* __restrict__ act,
                        const uint8_t* __restrict__ phase, const uint8_t* __restrict__ reward, int G, int n_phases,
                        int max_len, double* __restrict__ c_group, uint8_t* __restrict__ valid_group,
                        unsigned* __restrict__ status) {
  extern __shared__ unsigned long long smf[];
  unsigned long long* sums = smf;                                           // [n_phases][2][56], two's complement
  unsigned* cnt = reinterpret_cast<unsigned*>(smf + n_phases * 2 * ACT);    // [n_phases][2]
  const int g = blockIdx.x;
  for (int i = threadIdx.x; i < n_phases * 2 * ACT; i += blockDim.x) sums[i] = 0ull;
  for (int i = threadIdx.x; i < n_phases * 2; i += blockDim.x) cnt[i] = 0u;
  __syncthreads();

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  const int slot = lane / 14, vec = lane - slot * 14;     // slots 0, 1 active; lanes 28..31 idle
  for (int i = g * G + warp; i < (g + 1) * G; i += nwarps) {
    const int o = reward[i] ? 1 : 0;
    const int a = traj_off[i], b = traj_off[i + 1];
    if (b - a > max_len || b < a) {
      if (lane == 0) atomicOr(status, STATUS_TOO_LONG);
      continue;
    }
    if (slot >= 2) continue;
    const int per = (b - a + 1) >> 1;
    const int c_lo = a + slot * per, c_hi = min(b, c_lo + per);
    long long acc[4] = {0, 0, 0, 0};
    unsigned run = 0;
    int cur = -1;
    auto flush = [&]() {
      if (run) {
        unsigned long long* sp = sums + (cur * 2 + o) * ACT + 4 * vec;
#pragma unroll
        for (int e = 0; e < 4; ++e) atomicAdd(sp + e, (unsigned long long)acc[e]);
        if (vec == 0) atomicAdd(cnt + cur * 2 + o, run);
      }
      acc[0] = acc[1] = acc[2] = acc[3] = 0;
      run = 0;
    };
    constexpr int UNROLL = 4;
    for (int c0 = c_lo; c0 < c_hi; c0 += UNROLL) {
      float4 v[UNROLL];
      int ph[UNROLL];
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        const int ch = c0 + u;
        if (ch < c_hi) {
          v[u] = __ldg(reinterpret_cast<const float4*>(act + (size_t)ch * ACT) + vec);
          ph[u] = __ldg(phase + ch);
        } else {
          v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
          ph[u] = -1;
        }
      }
#pragma unroll
      for (int u = 0; u < UNROLL; ++u) {
        if (ph[u] < 0) continue;
        if (ph[u] >= n_phases) {
          atomicOr(status, STATUS_BAD_PHASE);
          continue;
        }
        if (ph[u] != cur) {
          flush();
          cur = ph[u];
        }
        const float x[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (fabsf(x[e]) <= ACT_ABS_MAX)                  // false for NaN as well
            acc[e] += __double2ll_rn(__dmul_rn((double)x[e], 4294967296.0));
          else
            atomicOr(status, STATUS_BAD_ACTION);           // counted as 0
        }
        ++run;
      }
    }
    flush();
  }
  __syncthreads();

  __shared__ double sq[8][ACT];
  for (int c = warp; c < n_phases; c += nwarps) {
    const unsigned n_succ = cnt[c * 2 + 1], n_fail = cnt[c * 2 + 0];
    const bool both = n_succ && n_fail;
    if (both) {
      const unsigned long long* s1 = sums + (c * 2 + 1) * ACT;
      const unsigned long long* s0 = sums + (c * 2 + 0) * ACT;
      for (int dim = lane; dim < ACT; dim += 32) {
        const double m1 = __ddiv_rn(__ll2double_rn((long long)s1[dim]), (double)n_succ);
        const double m0 = __ddiv_rn(__ll2double_rn((long long)s0[dim]), (double)n_fail);
        const double diff = __dsub_rn(m1, m0);
        sq[warp][dim] = __dmul_rn(diff, diff);
      }
    }
    __syncwarp();
    if (lane == 0) {
      double val = 0.0;
      if (both) {
        double acc = 0.0;
        for (int dim = 0; dim < ACT; ++dim) acc = __dadd_rn(acc, sq[warp][dim]);
        val = __dmul_rn(__dsqrt_rn(acc), 1.0 / 4294967296.0);
      }
      c_group[(size_t)g * n_phases + c] = val;
      valid_group[(size_t)g * n_phases + c] = both ? 1 : 0;
    }
    __syncwarp();
  }
}

// Blocks 0 .. n_phases-1: mean of C_{c,g} over valid groups.  One warp per phase loads 32 groups at a
// time in parallel and adds them in ascending g (every lane runs the same chain, so the order of the
// fp64 additions is exactly the sequential one).
// Blocks n_phases ..: Eq. 1 advantages, one thread per group.
__global__ void score_finalize_kernel(const double* __restrict__ c_group,
                                      const uint8_t* __restrict__ valid_group, int n_groups, int n_phases,
                                      double* __restrict__ C, uint8_t* __restrict__ valid,
                                      int32_t* __restrict__ n_valid, const uint8_t* __restrict__ reward,
                                      int G, double eps, float* __restrict__ adv) {
  if ((int)blockIdx.x < n_phases) {
    if (threadIdx.x >= 32) return;
    const int c = blockIdx.x, lane = threadIdx.x;
    double s = 0.0;
    int k = 0;
    for (int g0 = 0; g0 < n_groups; g0 += 32) {
      const int g = g0 + lane;
      const bool ok = g < n_groups && valid_group[(size_t)g * n_phases + c];
      const double x = ok ? c_group[(size_t)g * n_phases + c] : 0.0;
      const unsigned m = __ballot_sync(0xffffffffu, ok);
      for (int l = 0; l < 32; ++l) {
        const double xl = __shfl_sync(0xffffffffu, x, l);
        if (m & (1u << l)) { s = __dadd_rn(s, xl); ++k; }
      }
    }
    if (lane == 0) {
      C[c] = k ? __ddiv_rn(s, (double)k) : 0.0;
      valid[c] = k ? 1 : 0;
      if (n_valid) n_valid[c] = k;
    }
    return;
  }
  if (!adv) return;
  const int g = (blockIdx.x - n_phases) * blockDim.x + threadIdx.x;
  if (g >= n_groups) return;
  double s = 0.0;
  for (int j = 0; j < G; ++j) s = __dadd_rn(s, reward[g * G + j] ? 1.0 : 0.0);
  const double mu = __ddiv_rn(s, (double)G);
  double v = 0.0;
  for (int j = 0; j < G; ++j) {
    const double dl = __dsub_rn(reward[g * G + j] ? 1.0 : 0.0, mu);
    v = __dadd_rn(v, __dmul_rn(dl, dl));
  }
  const double denom = __dadd_rn(__dsqrt_rn(__ddiv_rn(v, (double)G)), eps);
  for (int j = 0; j < G; ++j)
    adv[g * G + j] = (float)__ddiv_rn(__dsub_rn(reward[g * G + j] ? 1.0 : 0.0, mu), denom);
}

// ------------------------------------------------------------------------------------------------
// Eq. 7-9: online update (one thread; O(n_phases * t_rc) scalar fp64 operations in a fixed order)
// ------------------------------------------------------------------------------------------------
__global__ void update_keep_probs_kernel(KeepState* st, const double* __restrict__ C,
                                         const uint8_t* __restrict__ valid, int n_phases, int t_rc,
                                         double p_min, int mode, float* __restrict__ p_out,
                                         uint32_t* __restrict__ q_out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  for (int c = 0; c < n_phases; ++c) st->buf[c][st->count] = valid[c] ? C[c] : 0.0;
  st->count += 1;
  if (st->step == 0 || st->count == t_rc) {
    double S[PCM_MAX_PHASES];
    double tot = 0.0;
    for (int c = 0; c < n_phases; ++c) {
      double s = 0.0;
      for (int t = 0; t < st->count; ++t) s = __dadd_rn(s, st->buf[c][t]);
      S[c] = s;
    }
    for (int c = 0; c < n_phases; ++c) tot = __dadd_rn(tot, S[c]);
    if (mode != PCM_MASK_RANDOM && tot > 0.0) {
      double rho_max = 0.0;
      int c_max = 0;
      for (int c = 0; c < n_phases; ++c) {
        S[c] = __ddiv_rn(S[c], tot);                      // share rho_c
        if (S[c] > rho_max) { rho_max = S[c]; c_max = c; }
      }
      for (int c = 0; c < n_phases; ++c) {
        if (mode == PCM_MASK_FULL) {
          st->p[c] = c == c_max ? 1.0 : 0.0;              // only the highest-S_c phase survives
        } else {
          const double r = __ddiv_rn(S[c], rho_max);      // rho~_c
          st->p[c] = r > p_min ? r : p_min;
        }
      }
    }
    st->count = 0;
    st->n_refresh += 1;
  }
  st->step += 1;
  for (int c = 0; c < n_phases; ++c) {
    p_out[c] = (float)st->p[c];
    q_out[c] = (uint32_t)__double2ll_rn(__dmul_rn(st->p[c], 16777216.0));   // round half to even
  }
}

// ------------------------------------------------------------------------------------------------
// Eq. 10: sampling
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t& o0, uint32_t& o1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  o0 = c0; o1 = c1;
}

// n_pos[i] = chunks of trajectory i whose phase has a positive weight; one warp per trajectory
__global__ void count_positive_kernel(const int32_t* __restrict__ traj_off, const uint8_t* __restrict__ phase,
                                      const uint32_t* __restrict__ q, int n_traj, int n_phases,
                                      int32_t* __restrict__ n_pos) {
  const int i = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (i >= n_traj) return;
  const int a = traj_off[i], b = traj_off[i + 1];
  int c = 0;
  for (int k = a + lane; k < b; k += 32) {
    const int ph = phase[k];
    c += (ph < n_phases && q[ph] != 0) ? 1 : 0;
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) c += __shfl_xor_sync(0xffffffffu, c, off);
  if (lane == 0) n_pos[i] = c;
}

// kept_off = exclusive prefix sum of min(budget, n_pos[i]); single block.
__global__ void kept_offsets_kernel(const int32_t* __restrict__ n_pos, int n_traj, int budget,
                                    int32_t* __restrict__ kept_off) {
  __shared__ int part[1024];
  const int t = threadIdx.x, nt = blockDim.x;
  const int per = (n_traj + nt - 1) / nt;
  const int lo = min(t * per, n_traj), hi = min(lo + per, n_traj);
  int s = 0;
  for (int i = lo; i < hi; ++i) s += min(budget, n_pos[i]);
  part[t] = s;
  __syncthreads();
  for (int off = 1; off < nt; off <<= 1) {               // Hillis-Steele inclusive scan
    int v = (t >= off) ? part[t - off] : 0;
    __syncthreads();
    part[t] += v;
    __syncthreads();
  }
  int run = part[t] - s;
  for (int i = lo; i < hi; ++i) {
    kept_off[i] = run;
    run += min(budget, n_pos[i]);
  }
  if (t == nt - 1) kept_off[n_traj] = part[nt - 1];
}

// One warp per trajectory.  Weights sit in shared memory; bit 31 marks a chunk already drawn.
__global__ void __launch_bounds__(128)
sample_chunks_kernel(const int32_t* __restrict__ traj_off, const uint8_t* __restrict__ phase,
                     const uint32_t* __restrict__ q, int n_traj, int n_phases, int budget, int max_len,
                     uint32_t seed_lo, uint32_t seed_hi, uint32_t it_lo, uint32_t it_hi,
                     const int32_t* __restrict__ kept_off, int32_t* __restrict__ kept_idx,
                     int32_t* __restrict__ kept_per_phase, unsigned* __restrict__ status) {
  extern __shared__ unsigned wsm[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = blockIdx.x * (blockDim.x >> 5) + warp;
  if (i >= n_traj) return;
  unsigned* w = wsm + (size_t)warp * max_len;
  const int a = traj_off[i], N = traj_off[i + 1] - a;
  if (N > max_len || N < 0) {
    if (lane == 0) atomicOr(status, STATUS_TOO_LONG);
    return;
  }
  unsigned long long W = 0;
  int n_pos = 0;                                          // chunks that can be kept at all (weight > 0)
  for (int k = lane; k < N; k += 32) {
    const int ph = phase[a + k];
    unsigned wk = 0;
    if (ph < n_phases) wk = q[ph]; else atomicOr(status, STATUS_BAD_PHASE);
    w[k] = wk;
    W += wk;
    n_pos += wk ? 1 : 0;
  }
#pragma unroll
  for (int off = 16; off; off >>= 1) {
    W += __shfl_xor_sync(0xffffffffu, W, off);
    n_pos += __shfl_xor_sync(0xffffffffu, n_pos, off);
  }
  __syncwarp();
  const int m = min(budget, n_pos);

  if (m < n_pos) {
    for (int r = 0; r < m; ++r) {
      uint32_t b0, b1;
      philox4x32_10(it_lo, (uint32_t)i, (uint32_t)r, it_hi, seed_lo, seed_hi, b0, b1);
      const unsigned long long bits = ((unsigned long long)b1 << 32) | b0;
      const unsigned long long x = __umul64hi(bits, W);
      unsigned long long base = 0;
      int pick = -1;
      for (int k0 = 0; k0 < N; k0 += 32) {
        const int k = k0 + lane;
        unsigned v = (k < N) ? (w[k] & 0x7FFFFFFFu) : 0u;
        unsigned incl = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const unsigned up = __shfl_up_sync(0xffffffffu, incl, off);
          if (lane >= off) incl += up;
        }
        const unsigned tot = __shfl_sync(0xffffffffu, incl, 31);
        if (base + tot > x) {
          const unsigned hit = __ballot_sync(0xffffffffu, base + incl > x);
          pick = k0 + __ffs(hit) - 1;
          break;
        }
        base += tot;
      }
      if (pick < 0) {                                    // cannot happen while weights are >= 1
        if (lane == 0) atomicOr(status, STATUS_BAD_PHASE);
        break;
      }
      const unsigned wp = w[pick] & 0x7FFFFFFFu;
      __syncwarp();
      if (lane == 0) w[pick] = 0x80000000u;
      W -= wp;
      __syncwarp();
    }
  } else {
    for (int k = lane; k < N; k += 32)
      if (w[k]) w[k] = 0x80000000u;                       // every chunk of positive weight is kept
    __syncwarp();
  }

  // compaction in index order = ascending chunk ids
  int out = kept_off[i];
  for (int k0 = 0; k0 < N; k0 += 32) {
    const int k = k0 + lane;
    const bool kept = (k < N) && (w[k] & 0x80000000u);
    const unsigned mask = __ballot_sync(0xffffffffu, kept);
    if (kept) {
      kept_idx[out + __popc(mask & ((1u << lane) - 1u))] = a + k;
      if (kept_per_phase) atomicAdd(kept_per_phase + phase[a + k], 1);
    }
    out += __popc(mask);
  }
}

static int check_batch(const pcm_ctx* ctx, const pcm_batch* b) {
  if (!ctx || !b || !b->traj_off || !b->phase) return PCM_ERR_ARG;
  if (b->n_traj <= 0 || b->n_traj > ctx->max_traj || b->n_traj % ctx->cfg.group_size) return PCM_ERR_ARG;
  if (b->n_chunks < 0 || b->max_len < 0) return PCM_ERR_ARG;
  return PCM_OK;
}

}  // namespace pcm

using namespace pcm;

// score_groups_kernel with its shared memory: the counters plus two 32-chunk slabs per warp (29 KB, with 32 phases
// 43 KB; the attribute is set once per device so that any count stays legal).  Allocates nothing.
template <int NT>
static int launch_score_groups_nt(const pcm_batch* b, int G, int n_phases, int n_groups, double* c_group,
                                  uint8_t* valid_group, unsigned* status, cudaStream_t s) {
  const size_t n_cnt = ((size_t)n_phases * 2 * (ACT + 1) + 3) & ~(size_t)3;
  const size_t smem = n_cnt * sizeof(unsigned) + (size_t)SC_WARPS * 2 * SC_SLAB_BYTES;
  static unsigned long long attr_devices = 0;
  static std::mutex mu;
  {
    std::lock_guard<std::mutex> lk(mu);
    if (attr_needed(&attr_devices))
      PCM_CUDA_TRY(cudaFuncSetAttribute(score_groups_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)(((size_t)PCM_MAX_PHASES * 2 * (ACT + 1) + 3) * sizeof(unsigned) +
                                              (size_t)SC_WARPS * 2 * SC_SLAB_BYTES)));
  }
  score_groups_kernel<NT><<<n_groups, SC_WARPS * 32, smem, s>>>(b->traj_off, b->tok, b->phase, b->reward, G, n_phases,
                                                              c_group, valid_group, status);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

static int launch_score_groups(const pcm_batch* b, int G, int n_phases, int n_groups, double* c_group, uint8_t* valid_group,
                               unsigned* status, cudaStream_t s) {
  switch ((n_phases + 7) / 8) {                          // phase columns come in MMA tiles of 8
    case 1: return launch_score_groups_nt<1>(b, G, n_phases, n_groups, c_group, valid_group, status, s);
    case 2: return launch_score_groups_nt<2>(b, G, n_phases, n_groups, c_group, valid_group, status, s);
    case 3: return launch_score_groups_nt<3>(b, G, n_phases, n_groups, c_group, valid_group, status, s);
    default: return launch_score_groups_nt<4>(b, G, n_phases, n_groups, c_group, valid_group, status, s);
  }
}

extern "C" {

int pcm_create(pcm_ctx** out, const pcm_config* cfg, int32_t max_traj) {
  if (!out || !cfg) return PCM_ERR_ARG;
  if (cfg->n_phases < 1 || cfg->n_phases > PCM_MAX_PHASES || cfg->budget < 1 || cfg->group_size < 1 ||
      cfg->t_rc < 1 || cfg->t_rc > PCM_MAX_TRC || !(cfg->p_min > 0.0) || cfg->p_min > 1.0 ||
      !(cfg->adv_eps >= 0.0) || max_traj < cfg->group_size || cfg->mode < PCM_MASK_PCM || cfg->mode > PCM_MASK_FULL)
    return PCM_ERR_ARG;
  pcm_ctx* c = new (std::nothrow) pcm_ctx();
  if (!c) return PCM_ERR_ARG;
  c->cfg = *cfg;
  c->max_traj = max_traj;
  c->state = nullptr; c->status = nullptr; c->c_group = nullptr; c->valid_group = nullptr; c->n_pos = nullptr;
  const size_t ng = (size_t)max_traj / cfg->group_size;
  bool ok = cudaGetDevice(&c->device) == cudaSuccess &&
            cudaMalloc(&c->state, sizeof(KeepState)) == cudaSuccess &&
            cudaMalloc(&c->status, 256) == cudaSuccess &&
            cudaMalloc(&c->c_group, ng * cfg->n_phases * sizeof(double)) == cudaSuccess &&
            cudaMalloc(&c->valid_group, ng * cfg->n_phases) == cudaSuccess &&
            cudaMalloc(&c->n_pos, (size_t)max_traj * sizeof(int32_t)) == cudaSuccess;
  if (ok) {
    KeepState init;
    memset(&init, 0, sizeof(init));
    for (int k = 0; k < PCM_MAX_PHASES; ++k) init.p[k] = 1.0;
    ok = cudaMemcpy(c->state, &init, sizeof(init), cudaMemcpyHostToDevice) == cudaSuccess &&
         cudaMemset(c->status, 0, 256) == cudaSuccess;
  }
  if (!ok) {
    pcm_destroy(c);
    return PCM_ERR_CUDA;
  }
  *out = c;
  return PCM_OK;
}

int pcm_destroy(pcm_ctx* c) {
  if (!c) return PCM_ERR_ARG;
  cudaFree(c->state); cudaFree(c->status); cudaFree(c->c_group); cudaFree(c->valid_group); cudaFree(c->n_pos);
  delete c;
  return PCM_OK;
}

int pcm_poll_status(pcm_ctx* ctx, pcm_stream stream) {
  if (!ctx) return PCM_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  unsigned h = 0;
  PCM_CUDA_TRY(cudaMemcpyAsync(&h, ctx->status, sizeof(h), cudaMemcpyDeviceToHost, s));
  PCM_CUDA_TRY(cudaMemsetAsync(ctx->status, 0, sizeof(unsigned), s));
  PCM_CUDA_TRY(cudaStreamSynchronize(s));
  if (h & STATUS_TIMEOUT) return PCM_ERR_DEVICE_TIMEOUT;
  if (h) return PCM_ERR_DEVICE_DATA;
  return PCM_OK;
}

int pcm_state_export(pcm_ctx* ctx, void* host_buf, size_t* bytes) {
  if (!ctx || !bytes) return PCM_ERR_ARG;
  const size_t need = sizeof(StateBlob);
  if (!host_buf || *bytes < need) {
    *bytes = need;
    return host_buf ? PCM_ERR_STATE : PCM_OK;
  }
  StateBlob* b = (StateBlob*)host_buf;
  b->version = STATE_VERSION; b->n_phases = ctx->cfg.n_phases; b->t_rc = ctx->cfg.t_rc; b->pad = 0;
  PCM_CUDA_TRY(cudaDeviceSynchronize());
  PCM_CUDA_TRY(cudaMemcpy(&b->st, ctx->state, sizeof(KeepState), cudaMemcpyDeviceToHost));
  *bytes = need;
  return PCM_OK;
}

int pcm_state_import(pcm_ctx* ctx, const void* host_buf, size_t bytes) {
  if (!ctx || !host_buf) return PCM_ERR_ARG;
  const StateBlob* b = (const StateBlob*)host_buf;
  if (bytes != sizeof(StateBlob) || b->version != STATE_VERSION || b->n_phases != ctx->cfg.n_phases ||
      b->t_rc != ctx->cfg.t_rc || b->st.count < 0 || b->st.count >= ctx->cfg.t_rc)
    return PCM_ERR_STATE;
  PCM_CUDA_TRY(cudaDeviceSynchronize());
  PCM_CUDA_TRY(cudaMemcpy(ctx->state, &b->st, sizeof(KeepState), cudaMemcpyHostToDevice));
  return PCM_OK;
}

int pcm_score_phases(pcm_ctx* ctx, const pcm_batch* b, double* C, uint8_t* valid, int32_t* n_valid_groups,
                     float* adv, pcm_stream stream) {
  int rc = check_batch(ctx, b);
  if (rc) return rc;
  if (!b->tok || !b->reward || !C || !valid) return PCM_ERR_ARG;
  if (((uintptr_t)b->tok) & 15) return PCM_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  const int G = ctx->cfg.group_size, Kc = ctx->cfg.n_phases, ng = b->n_traj / G;
  prof_begin(PC_SCORE, s);
  rc = launch_score_groups(b, G, Kc, ng, ctx->c_group, ctx->valid_group, ctx->status, s);
  if (rc) return rc;
  prof_end(s, 0.0, (double)b->n_chunks * (ACT + 1));
  const int adv_blocks = adv ? ceil_div(ng, 128) : 0;
  score_finalize_kernel<<<Kc + adv_blocks, 128, 0, s>>>(ctx->c_group, ctx->valid_group, ng, Kc, C, valid,
                                                       n_valid_groups, b->reward, G, ctx->cfg.adv_eps, adv);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

int pcm_score_phases_f32(pcm_ctx* ctx, const pcm_batch* b, const float* act, double* C, uint8_t* valid,
                         int32_t* n_valid_groups, float* adv, pcm_stream stream) {
  int rc = check_batch(ctx, b);
  if (rc) return rc;
  if (!act || !b->reward || !C || !valid) return PCM_ERR_ARG;
  if (((uintptr_t)act) & 15) return PCM_ERR_ARG;
  const int G = ctx->cfg.group_size, Kc = ctx->cfg.n_phases, ng = b->n_traj / G;
  if ((long long)G * b->max_len > ACT_MAX_GROUP_CHUNKS) return PCM_ERR_SHAPE;
  cudaStream_t s = (cudaStream_t)stream;
  const size_t smem = (size_t)Kc * 2 * ACT * sizeof(unsigned long long) + (size_t)Kc * 2 * sizeof(unsigned);
  prof_begin(PC_SCORE, s);
  score_groups_f32_kernel<<<ng, 256, smem, s>>>(b->traj_off, act, b->phase, b->reward, G, Kc, b->max_len, ctx->c_group,
                                                 ctx->valid_group, ctx->status);
  PCM_LAUNCH_CHECK();
  prof_end(s, 0.0, (double)b->n_chunks * (ACT * 4 + 1));
  const int adv_blocks = adv ? ceil_div(ng, 128) : 0;
  score_finalize_kernel<<<Kc + adv_blocks, 128, 0, s>>>(ctx->c_group, ctx->valid_group, ng, Kc, C, valid,
                                                       n_valid_groups, b->reward, G, ctx->cfg.adv_eps, adv);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

int pcm_update_keep_probs(pcm_ctx* ctx, const double* C, const uint8_t* valid, float* p, uint32_t* q,
                          pcm_stream stream) {
  if (!ctx || !C || !valid || !p || !q) return PCM_ERR_ARG;
  update_keep_probs_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(ctx->state, C, valid, ctx->cfg.n_phases,
                                                               ctx->cfg.t_rc, ctx->cfg.p_min, ctx->cfg.mode, p, q);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

int pcm_sample_chunks(pcm_ctx* ctx, const pcm_batch* b, const uint32_t* q, uint64_t iter, int32_t* kept_idx,
                      int32_t* kept_off, int32_t* kept_per_phase, pcm_stream stream) {
  int rc = check_batch(ctx, b);
  if (rc) return rc;
  if (!q || !kept_idx || !kept_off) return PCM_ERR_ARG;
  if (b->max_len < 1 || b->max_len > 12000) return PCM_ERR_SHAPE;     // 4 warps x max_len x 4 B <= 192 KB
  cudaStream_t s = (cudaStream_t)stream;
  count_positive_kernel<<<ceil_div(b->n_traj, 8), 256, 0, s>>>(b->traj_off, b->phase, q, b->n_traj, ctx->cfg.n_phases,
                                                               ctx->n_pos);
  PCM_LAUNCH_CHECK();
  kept_offsets_kernel<<<1, 1024, 0, s>>>(ctx->n_pos, b->n_traj, ctx->cfg.budget, kept_off);
  PCM_LAUNCH_CHECK();
  if (kept_per_phase) PCM_CUDA_TRY(cudaMemsetAsync(kept_per_phase, 0, ctx->cfg.n_phases * sizeof(int32_t), s));
  const int warps = 4;
  const size_t smem = (size_t)warps * b->max_len * sizeof(unsigned);
  if (smem > 48 * 1024)
    PCM_CUDA_TRY(cudaFuncSetAttribute(sample_chunks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  prof_begin(PC_SAMPLE, s);
  sample_chunks_kernel<<<ceil_div(b->n_traj, warps), warps * 32, smem, s>>>(
      b->traj_off, b->phase, q, b->n_traj, ctx->cfg.n_phases, ctx->cfg.budget, b->max_len,
      (uint32_t)(ctx->cfg.seed & 0xFFFFFFFFu), (uint32_t)(ctx->cfg.seed >> 32), (uint32_t)(iter & 0xFFFFFFFFu),
      (uint32_t)(iter >> 32), kept_off, kept_idx, kept_per_phase, ctx->status);
  PCM_LAUNCH_CHECK();
  prof_end(s, 0.0, (double)b->n_chunks + 4.0 * b->n_traj * ctx->cfg.budget);
  return PCM_OK;
}

int64_t pcm_launch_count(void) { return (int64_t)g_launches.load(); }

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Allocation-free scoring: the per-group scratch is a fixed device array owned by the library.
// ------------------------------------------------------------------------------------------------
namespace pcm {

constexpr size_t NA_CGROUP_BYTES = (size_t)PCM_STATIC_MAX_GROUPS * PCM_MAX_PHASES * sizeof(double);
constexpr size_t NA_VALID_BYTES = (size_t)PCM_STATIC_MAX_GROUPS * PCM_MAX_PHASES;
static_assert(NA_CGROUP_BYTES + NA_VALID_BYTES + 256 == PCM_STATIC_SCRATCH_BYTES, "scratch layout and header disagree");

// [C_{c,g} as fp64][validity bytes][status word]; held by every device that loads the library.
static __device__ __align__(256) unsigned char g_static_scratch[PCM_STATIC_SCRATCH_BYTES];

// In host code the symbol above is only a handle, not a device address: the address a kernel can use
// is looked up once per device (with that device current) and cached here.
constexpr int NA_MAX_DEVICES = 64;
static std::mutex g_na_mu;
static unsigned char* g_na_addr[NA_MAX_DEVICES] = {};

static int static_scratch_address(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return PCM_ERR_CUDA;
  if (dev < 0 || dev >= NA_MAX_DEVICES) return PCM_ERR_ARG;
  std::lock_guard<std::mutex> lk(g_na_mu);
  if (!g_na_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return PCM_ERR_CUDA;
    }
    g_na_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_na_addr[dev];
  return PCM_OK;
}

}  // namespace pcm

extern "C" int pcm_score_phases_static(int32_t n_phases, int32_t group_size, double adv_eps, const pcm_batch* b,
                                       double* C, uint8_t* valid, int32_t* n_valid_groups, float* adv,
                                       uint32_t* device_status, pcm_stream stream) {
  if (!b || !b->traj_off || !b->phase || !b->tok || !b->reward || !C || !valid) return PCM_ERR_ARG;
  if (n_phases < 1 || n_phases > PCM_MAX_PHASES || group_size < 1 || !(adv_eps >= 0.0)) return PCM_ERR_ARG;
  if (b->n_traj <= 0 || b->n_traj % group_size || b->n_chunks < 0) return PCM_ERR_ARG;
  if (((uintptr_t)b->tok) & 15) return PCM_ERR_ARG;
  const int ng = b->n_traj / group_size;
  if (ng > PCM_STATIC_MAX_GROUPS) return PCM_ERR_SHAPE;          // beyond the fixed scratch: refuse, do not truncate
  unsigned char* base = nullptr;
  const int rc = static_scratch_address(&base);
  if (rc != PCM_OK) return rc;
  double* c_group = reinterpret_cast<double*>(base);
  uint8_t* valid_group = base + NA_CGROUP_BYTES;
  unsigned* status = reinterpret_cast<unsigned*>(base + NA_CGROUP_BYTES + NA_VALID_BYTES);
  cudaStream_t s = (cudaStream_t)stream;
  PCM_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(unsigned), s));   // the only part that must start at zero
  const int rc_launch = launch_score_groups(b, group_size, n_phases, ng, c_group, valid_group, status, s);
  if (rc_launch) return rc_launch;
  const int adv_blocks = adv ? ceil_div(ng, 128) : 0;
  score_finalize_kernel<<<n_phases + adv_blocks, 128, 0, s>>>(c_group, valid_group, ng, n_phases, C, valid, n_valid_groups,
                                                       b->reward, group_size, adv_eps, adv);
  PCM_LAUNCH_CHECK();
  if (device_status)
    PCM_CUDA_TRY(cudaMemcpyAsync(device_status, status, sizeof(unsigned), cudaMemcpyDeviceToDevice, s));
  return PCM_OK;
}
