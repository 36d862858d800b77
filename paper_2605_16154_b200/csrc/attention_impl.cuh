// Causal softmax attention inside each chunk's sequence, forward and backward, flash style: the
// probability matrix is never stored; the backward pass rebuilds it from the saved row
// log-sum-exp.  One CTA per (sequence, head); a warp owns one query row (or one key row in the
// dK/dV pass) at a time.  Two operand matrices of the head live in shared memory, rows padded by
// one 32-bit word so that "lane = row" accesses are conflict free.
#pragma once
#include "internal.h"

namespace pcm {

constexpr int AT_MAX_TILES = 12;            // S <= 384
constexpr int AT_WARPS = 8;

template <typename T> struct Pack;          // 32-bit shared-memory word holding W elements
template <> struct Pack<float> { static constexpr int W = 1; };
template <> struct Pack<__nv_bfloat16> { static constexpr int W = 2; };

template <typename T> __device__ __forceinline__ float ld_f32(const T* p);
template <> __device__ __forceinline__ float ld_f32<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_f32<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st_f32(T* p, float v);
template <> __device__ __forceinline__ void st_f32<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void st_f32<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Copies an [S][DH] matrix with global row stride `ld` into shared memory with row stride DH + W.
template <typename T, int DH>
__device__ __forceinline__ void load_matrix(T* dst, const T* __restrict__ src, long long ld, int S) {
  constexpr int RS = DH + Pack<T>::W;
  for (int idx = threadIdx.x; idx < S * DH; idx += blockDim.x) {
    const int r = idx / DH, c = idx - r * DH;
    dst[r * RS + c] = src[(long long)r * ld + c];
  }
}

// dot of a register-resident vector (all DH values in every lane) with a shared-memory row
template <typename T, int DH>
__device__ __forceinline__ float dot_row(const float* __restrict__ v, const T* __restrict__ row) {
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < DH; ++c) s = fmaf(v[c], ld_f32(row + c), s);
  return s;
}

template <typename T, int DH>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_fwd_kernel(const T* __restrict__ qkv, T* __restrict__ out, float* __restrict__ lse, int S, int H, float scale) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + Pack<T>::W;
  T* Ks = reinterpret_cast<T*>(smraw);
  T* Vs = Ks + (size_t)S * RS;
  const int seq = blockIdx.y, h = blockIdx.x, d = H * DH;
  const long long ld = 3LL * d;
  const T* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  load_matrix<T, DH>(Ks, base + d, ld, S);
  load_matrix<T, DH>(Vs, base + 2 * d, ld, S);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = warp; i < S; i += AT_WARPS) {
    float q[DH];
#pragma unroll
    for (int c = 0; c < DH; ++c) q[c] = ld_f32(base + (long long)i * ld + c) * scale;
    float sc[AT_MAX_TILES];
    float mx = -INFINITY;
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      const int j = t * 32 + lane;
      sc[t] = -INFINITY;
      if (t * 32 <= i && j <= i) sc[t] = dot_row<T, DH>(q, Ks + (size_t)j * RS);
      mx = fmaxf(mx, sc[t]);
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
    float sum = 0.f;
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      sc[t] = (sc[t] == -INFINITY) ? 0.f : __expf(sc[t] - mx);
      sum += sc[t];
    }
#pragma unroll
    for (int off = 16; off; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
    const float inv = 1.f / sum;
    float o[DH / 32];
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) o[e] = 0.f;
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      if (t * 32 > i) break;
      const int jn = min(32, i + 1 - t * 32);
      for (int jj = 0; jj < jn; ++jj) {
        const float p = __shfl_sync(0xffffffffu, sc[t], jj);
        const T* vr = Vs + (size_t)(t * 32 + jj) * RS;
#pragma unroll
        for (int e = 0; e < DH / 32; ++e) o[e] = fmaf(p, ld_f32(vr + lane + 32 * e), o[e]);
      }
    }
    T* orow = out + ((long long)seq * S + i) * d + (long long)h * DH;
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) st_f32(orow + lane + 32 * e, o[e] * inv);
    if (lane == 0) lse[((long long)seq * H + h) * S + i] = mx + logf(sum);
  }
}

// D_i = sum_c dO_i[c] * O_i[c] for every (sequence, head, row); one warp per row
template <typename T, int DH>
__global__ void attn_dsum_kernel(const T* __restrict__ out, const T* __restrict__ dout, float* __restrict__ dsum,
                                 int n_seq, int S, int H) {
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);   // over n_seq*S*H
  const int lane = threadIdx.x & 31;
  if (row >= (long long)n_seq * S * H) return;
  const long long tokrow = row / H;
  const int h = (int)(row - tokrow * H);
  const T* o = out + tokrow * (long long)(H * DH) + (long long)h * DH;
  const T* g = dout + tokrow * (long long)(H * DH) + (long long)h * DH;
  float s = 0.f;
#pragma unroll
  for (int e = 0; e < DH / 32; ++e) s = fmaf(ld_f32(o + lane + 32 * e), ld_f32(g + lane + 32 * e), s);
#pragma unroll
  for (int off = 16; off; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (lane == 0) {
    const long long seq = tokrow / S;
    const int i = (int)(tokrow - seq * S);
    dsum[(seq * H + h) * S + i] = s;
  }
}

// dQ pass: K and V of the head in shared memory, a warp per query row.
template <typename T, int DH>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_bwd_dq_kernel(const T* __restrict__ qkv, const T* __restrict__ dout, const float* __restrict__ lse,
                   const float* __restrict__ dsum, T* __restrict__ dqkv, int S, int H, float scale) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + Pack<T>::W;
  T* Ks = reinterpret_cast<T*>(smraw);
  T* Vs = Ks + (size_t)S * RS;
  const int seq = blockIdx.y, h = blockIdx.x, d = H * DH;
  const long long ld = 3LL * d;
  const T* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  load_matrix<T, DH>(Ks, base + d, ld, S);
  load_matrix<T, DH>(Vs, base + 2 * d, ld, S);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = warp; i < S; i += AT_WARPS) {
    float q[DH], g[DH];
    const T* grow = dout + ((long long)seq * S + i) * d + (long long)h * DH;
#pragma unroll
    for (int c = 0; c < DH; ++c) {
      q[c] = ld_f32(base + (long long)i * ld + c) * scale;
      g[c] = ld_f32(grow + c);
    }
    const float l = lse[((long long)seq * H + h) * S + i];
    const float Di = dsum[((long long)seq * H + h) * S + i];
    float ds[AT_MAX_TILES];
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      const int j = t * 32 + lane;
      ds[t] = 0.f;
      if (t * 32 <= i && j <= i) {
        const float p = __expf(dot_row<T, DH>(q, Ks + (size_t)j * RS) - l);
        const float dp = dot_row<T, DH>(g, Vs + (size_t)j * RS);
        ds[t] = p * (dp - Di) * scale;
      }
    }
    float acc[DH / 32];
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) acc[e] = 0.f;
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      if (t * 32 > i) break;
      const int jn = min(32, i + 1 - t * 32);
      for (int jj = 0; jj < jn; ++jj) {
        const float w = __shfl_sync(0xffffffffu, ds[t], jj);
        const T* kr = Ks + (size_t)(t * 32 + jj) * RS;
#pragma unroll
        for (int e = 0; e < DH / 32; ++e) acc[e] = fmaf(w, ld_f32(kr + lane + 32 * e), acc[e]);
      }
    }
    T* dq = dqkv + ((long long)seq * S + i) * ld + (long long)h * DH;
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) st_f32(dq + lane + 32 * e, acc[e]);
  }
}

// dK / dV pass: Q and dO of the head in shared memory, a warp per key row.
template <typename T, int DH>
__global__ void __launch_bounds__(AT_WARPS * 32)
attn_bwd_dkv_kernel(const T* __restrict__ qkv, const T* __restrict__ dout, const float* __restrict__ lse,
                    const float* __restrict__ dsum, T* __restrict__ dqkv, int S, int H, float scale) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + Pack<T>::W;
  T* Qs = reinterpret_cast<T*>(smraw);
  T* Gs = Qs + (size_t)S * RS;
  float* Ls = reinterpret_cast<float*>(Gs + (size_t)S * RS);
  float* Ds = Ls + S;
  const int seq = blockIdx.y, h = blockIdx.x, d = H * DH;
  const long long ld = 3LL * d;
  const T* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  load_matrix<T, DH>(Qs, base, ld, S);
  load_matrix<T, DH>(Gs, dout + (long long)seq * S * d + (long long)h * DH, d, S);
  for (int i = threadIdx.x; i < S; i += blockDim.x) {
    Ls[i] = lse[((long long)seq * H + h) * S + i];
    Ds[i] = dsum[((long long)seq * H + h) * S + i];
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = warp; j < S; j += AT_WARPS) {
    float k[DH], v[DH];
#pragma unroll
    for (int c = 0; c < DH; ++c) {
      k[c] = ld_f32(base + d + (long long)j * ld + c) * scale;
      v[c] = ld_f32(base + 2 * d + (long long)j * ld + c);
    }
    float pr[AT_MAX_TILES], ds[AT_MAX_TILES];
    const int t_first = j >> 5;
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      const int i = t * 32 + lane;
      pr[t] = 0.f; ds[t] = 0.f;
      if (t >= t_first && i >= j && i < S) {
        const float p = __expf(dot_row<T, DH>(k, Qs + (size_t)i * RS) - Ls[i]);
        const float dp = dot_row<T, DH>(v, Gs + (size_t)i * RS);
        pr[t] = p;
        ds[t] = p * (dp - Ds[i]) * scale;
      }
    }
    float dk[DH / 32], dv[DH / 32];
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) { dk[e] = 0.f; dv[e] = 0.f; }
#pragma unroll
    for (int t = 0; t < AT_MAX_TILES; ++t) {
      if (t < t_first || t * 32 >= S) continue;
      const int i_lo = max(j - t * 32, 0), i_hi = min(32, S - t * 32);
      for (int ii = i_lo; ii < i_hi; ++ii) {
        const float p = __shfl_sync(0xffffffffu, pr[t], ii);
        const float w = __shfl_sync(0xffffffffu, ds[t], ii);
        const T* qr = Qs + (size_t)(t * 32 + ii) * RS;
        const T* gr = Gs + (size_t)(t * 32 + ii) * RS;
#pragma unroll
        for (int e = 0; e < DH / 32; ++e) {
          dv[e] = fmaf(p, ld_f32(gr + lane + 32 * e), dv[e]);
          dk[e] = fmaf(w, ld_f32(qr + lane + 32 * e), dk[e]);
        }
      }
    }
    T* dkp = dqkv + ((long long)seq * S + j) * ld + d + (long long)h * DH;
    T* dvp = dkp + d;
#pragma unroll
    for (int e = 0; e < DH / 32; ++e) {
      st_f32(dkp + lane + 32 * e, dk[e]);
      st_f32(dvp + lane + 32 * e, dv[e]);
    }
  }
}

template <typename T, int DH>
static int attn_fwd_launch(const void* qkv, void* out, float* lse, int n_seq, int S, int H, cudaStream_t s) {
  const size_t smem = 2ull * S * (DH + Pack<T>::W) * sizeof(T);
  if (smem > 227 * 1024) return PCM_ERR_SHAPE;
  PCM_CUDA_TRY(cudaFuncSetAttribute(attn_fwd_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  attn_fwd_kernel<T, DH><<<dim3(H, n_seq), AT_WARPS * 32, smem, s>>>((const T*)qkv, (T*)out, lse, S, H,
                                                                   1.0f / sqrtf((float)DH));
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

template <typename T, int DH>
static int attn_bwd_launch(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum,
                           void* dqkv, int n_seq, int S, int H, cudaStream_t s) {
  const size_t smem_q = 2ull * S * (DH + Pack<T>::W) * sizeof(T);
  const size_t smem_kv = smem_q + 2ull * S * sizeof(float);
  if (smem_kv > 227 * 1024) return PCM_ERR_SHAPE;
  const float scale = 1.0f / sqrtf((float)DH);
  const long long rows = (long long)n_seq * S * H;
  attn_dsum_kernel<T, DH><<<ceil_div(rows, 8), 256, 0, s>>>((const T*)out, (const T*)dout, dsum, n_seq, S, H);
  PCM_LAUNCH_CHECK();
  PCM_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dq_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_q));
  attn_bwd_dq_kernel<T, DH><<<dim3(H, n_seq), AT_WARPS * 32, smem_q, s>>>((const T*)qkv, (const T*)dout, lse, dsum,
                                                                        (T*)dqkv, S, H, scale);
  PCM_LAUNCH_CHECK();
  PCM_CUDA_TRY(cudaFuncSetAttribute(attn_bwd_dkv_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_kv));
  attn_bwd_dkv_kernel<T, DH><<<dim3(H, n_seq), AT_WARPS * 32, smem_kv, s>>>((const T*)qkv, (const T*)dout, lse, dsum,
                                                                          (T*)dqkv, S, H, scale);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

// Per-dtype entry points, each compiled in its own translation unit.
template <typename T>
static int attention_fwd_t(const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh, cudaStream_t s) {
  if (dh == 32) return attn_fwd_launch<T, 32>(qkv, out, lse, n_seq, S, H, s);
  if (dh == 64) return attn_fwd_launch<T, 64>(qkv, out, lse, n_seq, S, H, s);
  if (dh == 128) return attn_fwd_launch<T, 128>(qkv, out, lse, n_seq, S, H, s);
  return PCM_ERR_SHAPE;
}
template <typename T>
static int attention_bwd_t(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum,
                           void* dqkv, int n_seq, int S, int H, int dh, cudaStream_t s) {
  if (dh == 32) return attn_bwd_launch<T, 32>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, s);
  if (dh == 64) return attn_bwd_launch<T, 64>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, s);
  if (dh == 128) return attn_bwd_launch<T, 128>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, s);
  return PCM_ERR_SHAPE;
}

}  // namespace pcm
