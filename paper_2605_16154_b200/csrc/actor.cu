// grpo_actor_fwd_bwd: forward and backward of the decoder policy on the packed batch of kept
// chunks under the masked, clipped GRPO objective (Eq. 11).  This file holds the orchestration and
// the memory-bound kernels (RMSNorm, rotary embedding, SwiGLU, the loss over the 256-bin head,
// embedding gradient); the contractions live in gemm_*.cu and attention*.cu.
#include <cstdlib>
#include <cstring>

#include "internal.h"

namespace pcm {

constexpr int ACT = PCM_ACT_DIM;
constexpr int NB = PCM_N_BINS;
constexpr float RMS_EPS = 1e-5f;
constexpr int NORM_BWD_BLOCKS = 592;         // 4 CTAs per SM on 148 SMs

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void stf(T* p, float v);
template <> __device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int off = 16; off; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  return v;
}

// four consecutive elements of T <-> floats (8- or 16-byte accesses)
template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&v)[4]) {
  if constexpr (sizeof(T) == 2) {
    const uint2 raw = *reinterpret_cast<const uint2*>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
    v[0] = a.x; v[1] = a.y; v[2] = b.x; v[3] = b.y;
  } else {
    const float4 f = *reinterpret_cast<const float4*>(p);
    v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
  }
}
template <typename T>
__device__ __forceinline__ void store4(T* p, float a, float b, float c, float d) {
  if constexpr (sizeof(T) == 2) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 raw;
    raw.x = *reinterpret_cast<uint32_t*>(&lo);
    raw.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = raw;
  } else {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
  }
}

// Row r of a [rows][d] tensor that holds only the scored positions maps to token row
// (r / 56) * S + P - 1 + r % 56 of the full activation; map_S == 0 means identity.
__device__ __forceinline__ long long map_row(long long r, int map_S, int map_P) {
  if (map_S == 0) return r;
  const long long j = r / ACT;
  return j * map_S + map_P - 1 + (r - j * ACT);
}

// ------------------------------------------------------------------------------------------------
// packed batch (model dtype) -> fp32 residual stream
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void to_residual_kernel(const T* __restrict__ x, float* __restrict__ y, long long n) {
  const long long i = ((long long)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i + 3 < n) {
    float v[4];
    load4<T>(x + i, v);
    *reinterpret_cast<float4*>(y + i) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
    for (long long k = i; k < n; ++k) y[k] = ldf(x + k);
  }
}

// ------------------------------------------------------------------------------------------------
// Scored rows of the last layer.  Only positions P-1 .. P+54 of a chunk feed the head, so after the last attention
// the layer continues on those 56 rows per chunk.  gather: compact row r <- full row map_row(r); scatter: the
// reverse (the caller zeroes the full tensors first).  One thread moves four columns of both tensors.
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void gather_scored_rows_kernel(const T* __restrict__ a_full, const float* __restrict__ x_full, T* __restrict__ a_s,
                                          float* __restrict__ x_s, long long rows, int S, int P, int d) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = d / 4;
  if (idx >= rows * per_row) return;
  const long long r = idx / per_row;
  const int c = (int)(idx - r * per_row) * 4;
  const long long src = map_row(r, S, P) * d + c, dst = r * d + c;
  float v[4];
  load4<T>(a_full + src, v);
  store4<T>(a_s + dst, v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(x_s + dst) = *reinterpret_cast<const float4*>(x_full + src);
}

template <typename T>
__global__ void scatter_scored_rows_kernel(const T* __restrict__ a_s, const float* __restrict__ x_s, T* __restrict__ a_full,
                                           float* __restrict__ x_full, long long rows, int S, int P, int d) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = d / 4;
  if (idx >= rows * per_row) return;
  const long long r = idx / per_row;
  const int c = (int)(idx - r * per_row) * 4;
  const long long dst = map_row(r, S, P) * d + c, src = r * d + c;
  float v[4];
  load4<T>(a_s + src, v);
  store4<T>(a_full + dst, v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(x_full + dst) = *reinterpret_cast<const float4*>(x_s + src);
}

// ------------------------------------------------------------------------------------------------
// RMSNorm forward: one warp per row.  x fp32 [.][d] (rows optionally gathered), h T [rows][d].
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
rmsnorm_fwd_kernel(const float* __restrict__ x, const T* __restrict__ gamma, T* __restrict__ h,
                   float* __restrict__ rstd, long long rows, int d, int map_S, int map_P) {
  const long long r = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (r >= rows) return;
  const float* xr = x + map_row(r, map_S, map_P) * d;
  float ss = 0.f;
  for (int c = lane * 4; c < d; c += 128) {
    const float4 v = *reinterpret_cast<const float4*>(xr + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  const float rs = rsqrtf(ss / (float)d + RMS_EPS);
  if (lane == 0) rstd[r] = rs;
  T* hr = h + r * d;
  for (int c = lane * 4; c < d; c += 128) {
    const float4 v = *reinterpret_cast<const float4*>(xr + c);
    float gm[4];
    load4<T>(gamma + c, gm);
    store4<T>(hr + c, v.x * rs * gm[0], v.y * rs * gm[1], v.z * rs * gm[2], v.w * rs * gm[3]);
  }
}

// ------------------------------------------------------------------------------------------------
// RMSNorm backward.  dy [rows][d] in fp32 or in the activation type T; x fp32 (rows optionally gathered); dx_out = dx_in + dx is
// written through the same row map, in fp32 and in T.  Per-CTA partial sums of
// dgamma = sum_rows dy * x * rstd go to part[blockIdx][d]; a second kernel adds them up in a fixed order.
// ------------------------------------------------------------------------------------------------
template <typename T, typename DY>
__global__ void __launch_bounds__(256)
rmsnorm_bwd_kernel(const DY* __restrict__ dy, const float* __restrict__ x, const float* __restrict__ rstd,
                   const T* __restrict__ gamma, const float* dx_in, float* dx_out, T* __restrict__ dx_out_t,
                   float* __restrict__ part, long long rows, int d, int map_S, int map_P) {
  extern __shared__ float red[];                         // [8 warps][d]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* mine = red + (size_t)warp * d;
  for (int c = lane; c < d; c += 32) mine[c] = 0.f;
  __syncwarp();
  for (long long r = (long long)blockIdx.x * 8 + warp; r < rows; r += (long long)gridDim.x * 8) {
    const long long xr_i = map_row(r, map_S, map_P);
    const float* xr = x + xr_i * d;
    const DY* dyr = dy + r * d;
    const float rs = rstd[r];
    float dot = 0.f;
    for (int c = lane * 4; c < d; c += 128) {
      const float4 xv = *reinterpret_cast<const float4*>(xr + c);
      float gm[4], gy[4];
      load4<DY>(dyr + c, gy);
      load4<T>(gamma + c, gm);
      dot += gy[0] * gm[0] * xv.x + gy[1] * gm[1] * xv.y + gy[2] * gm[2] * xv.z + gy[3] * gm[3] * xv.w;
    }
    dot = warp_sum(dot);
    const float coef = dot * rs * rs * rs / (float)d;    // mean(dn * n) * rstd, with n = x * rstd
    for (int c = lane * 4; c < d; c += 128) {
      const float4 xv = *reinterpret_cast<const float4*>(xr + c);
      const float xa[4] = {xv.x, xv.y, xv.z, xv.w};
      float ga[4];
      load4<DY>(dyr + c, ga);
      float o[4], gm[4];
      load4<T>(gamma + c, gm);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        o[e] = rs * ga[e] * gm[e] - coef * xa[e];
        mine[c + e] += ga[e] * xa[e] * rs;
      }
      if (dx_in) {
        const float4 pv = *reinterpret_cast<const float4*>(dx_in + xr_i * d + c);
        o[0] += pv.x; o[1] += pv.y; o[2] += pv.z; o[3] += pv.w;
      }
      *reinterpret_cast<float4*>(dx_out + xr_i * d + c) = make_float4(o[0], o[1], o[2], o[3]);
      store4<T>(dx_out_t + xr_i * d + c, o[0], o[1], o[2], o[3]);
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[(size_t)w * d + c];
    part[(size_t)blockIdx.x * d + c] = s;
  }
}

// The same for d = 128 NV WPR with the whole row in registers: every load of a row (x, dy, the incoming residual
// gradient) is issued before the first use, nothing is read twice, gamma and the dgamma partial sums of this lane's
// columns stay in registers for the life of the CTA.  Fewer, fatter warps: the kernel is HBM-bound and needs bytes
// in flight, not occupancy.  WPR warps share a row (WPR = 2 for d = 2048: a warp holds 1024 columns): they add their
// parts of the row's dot product through shared memory and a named barrier of their own.
template <typename T, typename DY, int NV, int WPR>
__global__ void __launch_bounds__(256)
rmsnorm_bwd_rows_kernel(const DY* __restrict__ dy, const float* __restrict__ x, const float* __restrict__ rstd,
                        const T* __restrict__ gamma, const float* dx_in, float* dx_out, T* __restrict__ dx_out_t,
                        float* __restrict__ part, long long rows, int map_S, int map_P) {
  constexpr int d = NV * 128 * WPR, RPB = 8 / WPR;        // row width; rows a CTA works on at a time
  extern __shared__ float red[];                         // [8 warps][NV * 128]
  __shared__ float dots[2][8];                           // partial dot products, double-buffered over a warp group's rows
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = warp / WPR, part_i = warp - grp * WPR;  // row slot of this warp, and which part of the row it holds
  const int col0 = part_i * NV * 128 + lane * 4;
  float gm[NV][4], acc[NV][4];
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    load4<T>(gamma + col0 + k * 128, gm[k]);
    acc[k][0] = acc[k][1] = acc[k][2] = acc[k][3] = 0.f;
  }
  int it = 0;
  for (long long r = (long long)blockIdx.x * RPB + grp; r < rows; r += (long long)gridDim.x * RPB, ++it) {
    const long long xr_i = map_row(r, map_S, map_P);
    const float* xr = x + xr_i * d + col0;
    const DY* dyr = dy + r * d + col0;
    float4 xv[NV], pv[NV];
    float gy[NV][4];
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      xv[k] = *reinterpret_cast<const float4*>(xr + k * 128);
      load4<DY>(dyr + k * 128, gy[k]);
    }
    if (dx_in) {
#pragma unroll
      for (int k = 0; k < NV; ++k) pv[k] = *reinterpret_cast<const float4*>(dx_in + xr_i * d + col0 + k * 128);
    } else {
#pragma unroll
      for (int k = 0; k < NV; ++k) pv[k] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    const float rs = rstd[r];
    float dot = 0.f;
#pragma unroll
    for (int k = 0; k < NV; ++k)
      dot += gy[k][0] * gm[k][0] * xv[k].x + gy[k][1] * gm[k][1] * xv[k].y + gy[k][2] * gm[k][2] * xv[k].z +
             gy[k][3] * gm[k][3] * xv[k].w;
    dot = warp_sum(dot);
    if constexpr (WPR > 1) {
      // the group's warps run the same trip count (same r), so the barrier is reached by all of them
      if (lane == 0) dots[it & 1][warp] = dot;
      asm volatile("bar.sync %0, %1;" ::"r"(1 + grp), "r"(WPR * 32) : "memory");
      dot = 0.f;
#pragma unroll
      for (int w = 0; w < WPR; ++w) dot += dots[it & 1][grp * WPR + w];
    }
    const float coef = dot * rs * rs * rs / (float)d;    // mean(dn * n) * rstd, with n = x * rstd
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      const float xa[4] = {xv[k].x, xv[k].y, xv[k].z, xv[k].w};
      const float pa[4] = {pv[k].x, pv[k].y, pv[k].z, pv[k].w};
      float o[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        o[e] = rs * gy[k][e] * gm[k][e] - coef * xa[e] + pa[e];
        acc[k][e] += gy[k][e] * xa[e] * rs;
      }
      *reinterpret_cast<float4*>(dx_out + xr_i * d + col0 + k * 128) = make_float4(o[0], o[1], o[2], o[3]);
      store4<T>(dx_out_t + xr_i * d + col0 + k * 128, o[0], o[1], o[2], o[3]);
    }
  }
#pragma unroll
  for (int k = 0; k < NV; ++k)
    *reinterpret_cast<float4*>(red + (size_t)warp * (NV * 128) + k * 128 + lane * 4) = make_float4(acc[k][0], acc[k][1], acc[k][2], acc[k][3]);
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const int pi = c / (NV * 128), cc = c - pi * (NV * 128);   // which part of the row, column inside it
    float s = 0.f;
#pragma unroll
    for (int g = 0; g < RPB; ++g) s += red[(size_t)(g * WPR + pi) * (NV * 128) + cc];
    part[(size_t)blockIdx.x * d + c] = s;
  }
}

// out[c] += sum_b part[b][c].  A CTA takes 32 columns; its eight warps each add every eighth row in ascending order
// (coalesced 128-byte reads), and the eight partial sums are then added in warp order: a fixed association, so the
// result does not depend on timing.
__global__ void __launch_bounds__(256)
colsum_accumulate_kernel(const float* __restrict__ part, int nblk, int d, float* __restrict__ out) {
  __shared__ float red[8][32];
  const int lane = threadIdx.x & 31, slice = threadIdx.x >> 5;
  const int c = blockIdx.x * 32 + lane;
  float s = 0.f;
  if (c < d)
    for (int b = slice; b < nblk; b += 8) s += part[(size_t)b * d + c];
  red[slice][lane] = s;
  __syncthreads();
  if (slice == 0 && c < d) {
    float t = red[0][lane];
#pragma unroll
    for (int w = 1; w < 8; ++w) t += red[w][lane];
    out[c] += t;
  }
}

// ------------------------------------------------------------------------------------------------
// rotary embedding on the q and k parts of qkv [rows][3d], in place; table [S][dh/2] of (cos, sin)
// built in fp64.  sign = +1 forward, -1 backward (the transpose of a rotation).
// ------------------------------------------------------------------------------------------------
__global__ void rope_table_kernel(float2* __restrict__ tab, int S, int dh) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  const int half = dh / 2;
  if (idx >= S * half) return;
  const int pos = idx / half, i = idx - pos * half;
  const double inv_freq = pow(10000.0, -(2.0 * (double)i) / (double)dh);
  const double ang = (double)pos * inv_freq;
  tab[idx] = make_float2((float)cos(ang), (float)sin(ang));
}

// 16-byte vectors of T: 8 bf16 or 4 fp32
template <typename T> struct Vec16 { static constexpr int N = 16 / sizeof(T); };
template <typename T>
__device__ __forceinline__ void load_vec(const T* p, float (&v)[Vec16<T>::N]) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  if constexpr (sizeof(T) == 2) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int e = 0; e < 4; ++e) { const float2 f = __bfloat1622float2(h[e]); v[2 * e] = f.x; v[2 * e + 1] = f.y; }
  } else {
    v[0] = __uint_as_float(raw.x); v[1] = __uint_as_float(raw.y); v[2] = __uint_as_float(raw.z); v[3] = __uint_as_float(raw.w);
  }
}
template <typename T>
__device__ __forceinline__ void store_vec(T* p, const float (&v)[Vec16<T>::N]) {
  uint4 raw;
  if constexpr (sizeof(T) == 2) {
    __nv_bfloat162 h[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) h[e] = __floats2bfloat162_rn(v[2 * e], v[2 * e + 1]);
    raw = *reinterpret_cast<uint4*>(h);
  } else {
    raw = make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
  }
  *reinterpret_cast<uint4*>(p) = raw;
}

// One thread rotates VEC consecutive pairs (i, i + dh/2) of one head of q or k.
template <typename T>
__global__ void rope_kernel(T* __restrict__ qkv, const float2* __restrict__ tab, long long rows, int S, int H,
                            int dh, float sign) {
  constexpr int VEC = Vec16<T>::N;
  const int half = dh / 2, d = H * dh, per_head = half / VEC;
  const long long per_row = 2LL * H * per_head;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * per_row) return;
  const long long r = idx / per_row;
  const int rem = (int)(idx - r * per_row);
  const int which = rem / (H * per_head);                // 0 = q, 1 = k
  const int hh = (rem - which * H * per_head) / per_head;
  const int i0 = (rem % per_head) * VEC;
  const int pos = (int)(r % S);
  T* p = qkv + r * 3LL * d + (long long)which * d + (long long)hh * dh + i0;
  float a[VEC], b[VEC];
  load_vec<T>(p, a);
  load_vec<T>(p + half, b);
  const float2* cs = tab + pos * half + i0;
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    const float2 t = cs[e];
    const float sn = t.y * sign, x = a[e], y = b[e];
    a[e] = x * t.x - y * sn;
    b[e] = y * t.x + x * sn;
  }
  store_vec<T>(p, a);
  store_vec<T>(p + half, b);
}

// ------------------------------------------------------------------------------------------------
// SwiGLU: gu [rows][8d] = gate | up; one thread handles one 16-byte vector of the hidden dimension
// ------------------------------------------------------------------------------------------------
template <typename T>
__global__ void swiglu_fwd_kernel(const T* __restrict__ gu, T* __restrict__ act, long long rows, int f) {
  constexpr int VEC = Vec16<T>::N;
  const int fv = f / VEC;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * fv) return;
  const long long r = idx / fv;
  const int c = (int)(idx - r * fv) * VEC;
  float g[VEC], u[VEC];
  load_vec<T>(gu + r * 2LL * f + c, g);
  load_vec<T>(gu + r * 2LL * f + f + c, u);
#pragma unroll
  for (int e = 0; e < VEC; ++e) g[e] = g[e] / (1.f + __expf(-g[e])) * u[e];
  store_vec<T>(act + r * (long long)f + c, g);
}

template <typename T>
__global__ void swiglu_bwd_kernel(const T* __restrict__ gu, const T* __restrict__ dact, T* __restrict__ dgu,
                                  long long rows, int f) {
  constexpr int VEC = Vec16<T>::N;
  const int fv = f / VEC;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * fv) return;
  const long long r = idx / fv;
  const int c = (int)(idx - r * fv) * VEC;
  float g[VEC], u[VEC], da[VEC];
  load_vec<T>(gu + r * 2LL * f + c, g);
  load_vec<T>(gu + r * 2LL * f + f + c, u);
  load_vec<T>(dact + r * (long long)f + c, da);
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    const float sg = 1.f / (1.f + __expf(-g[e]));
    const float dg = da[e] * u[e] * sg * (1.f + g[e] * (1.f - sg));
    u[e] = da[e] * g[e] * sg;
    g[e] = dg;
  }
  store_vec<T>(dgu + r * 2LL * f + c, g);
  store_vec<T>(dgu + r * 2LL * f + f + c, u);
}

// ------------------------------------------------------------------------------------------------
// Head + loss without tensor cores (fp32 mode, or widths the tensor-core GEMM does not take): one CTA computes the
// logits of HL_ROWS scored rows, thread v holding bin v of every row in a register, and applies the same row
// functions as the tensor-core epilogue.  hs [rows][d] and W_h [256][d] in T; dz [rows][256] in T.  The logits never
// leave registers.  part[blockIdx][4] receives the CTA's sums {surrogate, clipped terms, ratio, entropy}.
// ------------------------------------------------------------------------------------------------
constexpr int HL_ROWS = 8;
constexpr int HL_KT = 32;

template <typename T>
__global__ void __launch_bounds__(NB)
head_loss_simt_kernel(const T* __restrict__ hs, const T* __restrict__ w_h, int rows, int d, HeadLossArgs h,
                      T* __restrict__ dz) {
  __shared__ float Ws[HL_KT][NB + 1];
  __shared__ float Hs[HL_ROWS][HL_KT];
  __shared__ float red[3][HL_ROWS][NB / 32];
  __shared__ float zt_s[HL_ROWS];
  __shared__ float sums[HL_ROWS][4];
  const int v = threadIdx.x, warp = v >> 5, lane = v & 31;
  const long long r0 = (long long)blockIdx.x * HL_ROWS;
  float z[HL_ROWS];
#pragma unroll
  for (int i = 0; i < HL_ROWS; ++i) z[i] = 0.f;
  for (int k0 = 0; k0 < d; k0 += HL_KT) {
    for (int i = 0; i < 32; ++i) {                        // W_h rows warp*32 .. +31, 32 consecutive k each
      const int row = warp * 32 + i;
      Ws[lane][row] = k0 + lane < d ? ldf(w_h + (long long)row * d + k0 + lane) : 0.f;
    }
    {
      const int i = v >> 5;                               // 8 rows x 32 k = one element per thread
      Hs[i][lane] = (r0 + i < rows && k0 + lane < d) ? ldf(hs + (r0 + i) * d + k0 + lane) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < HL_KT; ++k) {
      const float wv = Ws[k][v];
#pragma unroll
      for (int i = 0; i < HL_ROWS; ++i) z[i] += Hs[i][k] * wv;
    }
    __syncthreads();
  }
  // row statistics over the 256 threads: maximum first, then the two sums against it
  float mx[HL_ROWS];
#pragma unroll
  for (int i = 0; i < HL_ROWS; ++i) {
    float m = z[i];
#pragma unroll
    for (int off = 16; off; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (lane == 0) red[0][i][warp] = m;
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < HL_ROWS; ++i) {
    float m = red[0][i][0];
#pragma unroll
    for (int w = 1; w < NB / 32; ++w) m = fmaxf(m, red[0][i][w]);
    mx[i] = m;
    const float ex = expf(z[i] - m);
    const float se = warp_sum(ex), sz = warp_sum(ex * (z[i] - m));
    if (lane == 0) { red[1][i][warp] = se; red[2][i][warp] = sz; }
    const long long r = r0 + i;
    if (r < rows && v == (int)h.tgt[r]) zt_s[i] = z[i];
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < HL_ROWS; ++i) {
    const long long r = r0 + i;
    const bool valid = r < rows;
    RowStats st{mx[i], 0.f, 0.f};
#pragma unroll
    for (int w = 0; w < NB / 32; ++w) { st.se += red[1][i][w]; st.sz += red[2][i][w]; }
    const float lse = hl_lse(st), ent = hl_entropy(st);
    const float logp = valid ? zt_s[i] - lse : 0.f;
    RowTerms tm{0.f, 0.f, 0.f, 0.f};
    if (valid) {
      if (h.mode == HL_TOKEN) tm = hl_token_terms(logp, h.lpo[r], h.adv_c[r / ACT], h.lo, h.hi, h.loss_scale);
      else if (h.mode == HL_COEF) tm.dlogp = h.coef[r];
    }
    if (v == 0) {
      if (valid && h.logp && h.mode != HL_COEF) h.logp[r] = logp;
      sums[i][0] = tm.surrogate; sums[i][1] = tm.clipped; sums[i][2] = tm.ratio; sums[i][3] = valid ? ent : 0.f;
    }
    if (valid && h.want_dz) stf(dz + r * NB + v, hl_dz(z[i], lse, ent, tm.dlogp, h.ent_scale, v == (int)h.tgt[r]));
  }
  __syncthreads();
  if (h.part && v < 4) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < HL_ROWS; ++i) t += sums[i][v];
    h.part[(size_t)blockIdx.x * 4 + v] = t;
  }
}

// Chunk-level importance ratio (Eq. 2 / Eq. 11 as written): one warp per chunk adds the 56 log-ratios in a fixed
// order, forms r = exp(sum), clips once, and hands every row of the chunk the same d loss / d logp.
// part[chunk][4] = {surrogate, clipped, ratio, 0}.
__global__ void __launch_bounds__(256)
chunk_ratio_kernel(const float* __restrict__ logp, const float* __restrict__ lpo, const float* __restrict__ adv_c,
                   int n_chunks, float lo, float hi, float loss_scale, float* __restrict__ coef, float* __restrict__ part) {
  const int chunk = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (chunk >= n_chunks) return;
  const long long base = (long long)chunk * ACT;
  float a = logp[base + lane] - lpo[base + lane];
  if (lane + 32 < ACT) a += logp[base + lane + 32] - lpo[base + lane + 32];
  const float tot = warp_sum(a);
  const RowTerms tm = hl_token_terms(tot, 0.f, adv_c[chunk], lo, hi, loss_scale);     // ratio = exp(tot)
  coef[base + lane] = tm.dlogp;
  if (lane + 32 < ACT) coef[base + lane + 32] = tm.dlogp;
  if (lane == 0) *reinterpret_cast<float4*>(part + (size_t)chunk * 4) = make_float4(tm.surrogate, tm.clipped, tm.ratio, 0.f);
}

// acc[0..3] += ordered sums of part; loss[0] = -loss_scale * acc[0] - ent_scale * acc[3]   (single CTA, fixed order)
__global__ void loss_reduce_kernel(const float* __restrict__ part, int nblk, float loss_scale, float ent_scale,
                                   float* __restrict__ acc, float* __restrict__ loss) {
  __shared__ double sh[256][4];
  double s[4] = {0, 0, 0, 0};
  for (int b = threadIdx.x; b < nblk; b += blockDim.x)
    for (int e = 0; e < 4; ++e) s[e] += (double)part[(size_t)b * 4 + e];
  for (int e = 0; e < 4; ++e) sh[threadIdx.x][e] = s[e];
  __syncthreads();
  for (int off = 128; off; off >>= 1) {
    if (threadIdx.x < off)
      for (int e = 0; e < 4; ++e) sh[threadIdx.x][e] += sh[threadIdx.x + off][e];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    for (int e = 0; e < 4; ++e) acc[e] += (float)sh[0][e];
    loss[0] = -loss_scale * acc[0] - ent_scale * acc[3];
  }
}

// ------------------------------------------------------------------------------------------------
// Embedding gradient: dE[v][:] += sum over action positions whose token is v of dx[row][:],
// visited in ascending row order (deterministic).  grid = (256 tokens, column tiles of 256).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
embed_grad_kernel(const float* __restrict__ dx, const uint8_t* __restrict__ tgt, int n_chunks, int S, int P, int d,
                  float* __restrict__ dE) {
  const int v = blockIdx.x;
  const int c = blockIdx.y * 256 + threadIdx.x;
  __shared__ int hits[256];
  __shared__ int wcount[8];
  __shared__ int n_hits;
  float acc = 0.f;
  const int total = n_chunks * ACT;
  for (int base = 0; base < total; base += 256) {
    const int idx = base + threadIdx.x;
    const bool hit = idx < total && tgt[idx] == v;
    // ordered compaction: warp ballots, then warp offsets in warp order
    const unsigned m = __ballot_sync(0xffffffffu, hit);
    if ((threadIdx.x & 31) == 0) wcount[threadIdx.x >> 5] = __popc(m);
    __syncthreads();
    int off = 0;
    for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) off += wcount[w];
    if (hit) hits[off + __popc(m & ((1u << (threadIdx.x & 31)) - 1u))] = idx;
    if (threadIdx.x == 255) n_hits = off + __popc(m);
    __syncthreads();
    if (c < d) {
      for (int k = 0; k < n_hits; ++k) {
        const int id = hits[k];
        const int j = id / ACT, t = id - j * ACT;
        acc += dx[((long long)j * S + P + t) * d + c];
      }
    }
    __syncthreads();
  }
  if (c < d) dE[(long long)v * d + c] += acc;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Arena {
  unsigned char* base;
  size_t off;
  void* take(size_t bytes) {
    void* p = base ? base + off : nullptr;
    off += align_up(bytes, 256);
    return p;
  }
};

// The four linear maps of a decoder layer, in the order the adapter tensors of grpo_lora use.
enum { PJ_QKV = 0, PJ_O = 1, PJ_GU = 2, PJ_D = 3 };

struct LayerActs {
  void* h1; void* qkv; void* attn; float* lse; float* rstd1; float* x_mid; float* rstd2; void* h2; void* gu; void* act;
  void* lt[4];                   // adapters: alpha/r * (input of the projection) A^T, kept for dB
};

struct Workspace {
  float2* rope_tab;
  float* x[129];                 // residual stream, x[0..L]; x[L] holds the scored rows only
  LayerActs la[128];
  void* hs; float* rstdf; void* dz; float* loss_part; float* loss_acc; float* logp_tmp; float* coef;
  float* dx; void* dx_t; void* dact; void* dgu; float* dh; void* dattn; void* dqkv; float* dsum;
  float* norm_part; float* dhs;
  // the last layer's post-attention part runs on the scored rows only (nothing reads the others)
  void* attn_s; float* xin_s; float* dxs; void* dxs_t; void* dattn_s;
  void* lu;                      // adapters: alpha/r * (output gradient of the projection) B
  size_t bytes;
};

// lora_r: adapter rank (0: none).  keep_dact: the SwiGLU backward is not fused into the GEMM epilogue.
static void carve(Workspace& w, unsigned char* base, const grpo_model_cfg& c, int mb, bool fwd_only, int lora_r,
                  bool keep_dact) {
  Arena a{base, 0};
  const size_t es = c.dtype == GRPO_BF16 ? 2 : 4;
  const int S = c.prefix_len + ACT, d = c.d, H = c.n_heads, L = c.n_layers;
  const size_t M = (size_t)mb * S, R = (size_t)mb * ACT, r = (size_t)lora_r;
  w.rope_tab = (float2*)a.take((size_t)S * (d / H / 2) * sizeof(float2));
  // with backward every layer keeps its activations; forward-only reuses one layer's worth
  const int kept_layers = fwd_only ? 1 : L;
  for (int l = 0; l <= (fwd_only ? 1 : L); ++l) w.x[l] = (float*)a.take(((!fwd_only && l == L) ? R : M) * d * 4);
  for (int l = 0; l < kept_layers; ++l) {
    LayerActs& la = w.la[l];
    const size_t Mp = (!fwd_only && l == L - 1) ? R : M;          // rows of the post-attention part
    la.h1 = a.take(M * d * es); la.qkv = a.take(M * 3 * d * es); la.attn = a.take(M * d * es);
    la.lse = (float*)a.take((size_t)mb * H * S * 4); la.rstd1 = (float*)a.take(M * 4);
    la.x_mid = (float*)a.take(Mp * d * 4); la.rstd2 = (float*)a.take(Mp * 4); la.h2 = a.take(Mp * d * es);
    la.gu = a.take(Mp * 8 * d * es); la.act = a.take(Mp * 4 * d * es);
    la.lt[PJ_QKV] = a.take(M * r * es);
    for (int pj = PJ_O; pj <= PJ_D; ++pj) la.lt[pj] = a.take(Mp * r * es);
  }
  if (fwd_only) {
    for (int l = 1; l < L; ++l) w.la[l] = w.la[0];
    for (int l = 2; l <= L; ++l) w.x[l] = w.x[l & 1];
  }
  w.hs = a.take(R * d * es); w.rstdf = (float*)a.take(R * 4);
  w.dz = a.take(R * NB * es);
  // loss partial sums: one entry of 4 per head block (at most one per 8 rows) plus one per chunk
  w.loss_part = (float*)a.take(((size_t)mb * (ACT / HL_ROWS) + (size_t)mb + 8) * 4 * 4); w.loss_acc = (float*)a.take(256);
  w.logp_tmp = (float*)a.take(R * 4); w.coef = (float*)a.take(R * 4);
  w.attn_s = a.take(R * d * es); w.xin_s = (float*)a.take(R * d * 4);
  if (!fwd_only) {
    w.dx = (float*)a.take(M * d * 4); w.dx_t = a.take(M * d * es);
    w.dact = keep_dact ? a.take(M * 4 * d * es) : nullptr;
    w.dgu = a.take(M * 8 * d * es); w.dh = (float*)a.take(M * d * 4); w.dattn = a.take(M * d * es);
    w.dqkv = a.take(M * 3 * d * es); w.dsum = (float*)a.take((size_t)mb * H * S * 4);
    w.norm_part = (float*)a.take((size_t)NORM_BWD_BLOCKS * d * 4); w.dhs = (float*)a.take(R * d * 4);
    w.dxs = (float*)a.take(R * d * 4); w.dxs_t = a.take(R * d * es); w.dattn_s = a.take(R * d * es);
    w.lu = a.take(M * r * es);
  }
  w.bytes = a.off;
}

static int check_cfg(const grpo_model_cfg* c) {
  if (!c) return PCM_ERR_ARG;
  if (c->dtype != GRPO_F32 && c->dtype != GRPO_BF16) return PCM_ERR_ARG;
  if (c->d < 8 || c->n_layers < 1 || c->n_layers > 128 || c->n_heads < 1 || c->prefix_len < 1) return PCM_ERR_ARG;
  if (c->d % c->n_heads) return PCM_ERR_SHAPE;
  const int dh = c->d / c->n_heads;
  if (dh != 32 && dh != 64 && dh != 128) return PCM_ERR_SHAPE;
  if (c->d % 8) return PCM_ERR_SHAPE;
  if (c->prefix_len + ACT > 384) return PCM_ERR_SHAPE;
  return PCM_OK;
}

static int check_lora(const grpo_lora* lo) {
  if (!lo) return PCM_ERR_ARG;
  if (lo->rank < 8 || lo->rank > 64 || (lo->rank % 8)) return PCM_ERR_SHAPE;
  if (!(lo->alpha > 0.f)) return PCM_ERR_ARG;
  if (!lo->a_qkv || !lo->b_qkv || !lo->a_o || !lo->b_o || !lo->a_gu || !lo->b_gu || !lo->a_d || !lo->b_d) return PCM_ERR_ARG;
  return PCM_OK;
}

static GemmBackend backend_from_env();

// bf16 on the tensor-core path: SwiGLU and the rotary embedding run inside GEMM / attention epilogues
static void fused_epilogues(const grpo_model_cfg& c, bool* swiglu, bool* rope) {
  *swiglu = *rope = false;
  if (c.dtype != GRPO_BF16 || backend_from_env() == GEMM_SIMT) return;
  const int d = c.d, dh = d / c.n_heads;
  // operand addresses only have to be aligned like real ones for the probe
  void* any = reinterpret_cast<void*>(uintptr_t(4096));
  GemmArgs probe{128, 8 * d, d, any, d, true, any, d, true, DT_BF16, any, 8 * d, DT_BF16, nullptr, 0};
  probe.epi.kind = EPI_SWIGLU_FWD; probe.epi.out2 = any; probe.epi.ld_out2 = 4 * d;
  *swiglu = gemm_epilogue_supported(probe);
  GemmArgs probe2{128, 3 * d, d, any, d, true, any, d, true, DT_BF16, any, 3 * d, DT_BF16, nullptr, 0};
  probe2.epi.kind = EPI_ROPE; probe2.epi.rope_tab = reinterpret_cast<const float2*>(any);
  probe2.epi.S = c.prefix_len + ACT; probe2.epi.dh = dh; probe2.epi.d = d;
  *rope = gemm_epilogue_supported(probe2);
}

template <typename T>
static int run(const grpo_model* m, const grpo_lora* lo, const grpo_packed* pk, const grpo_loss_cfg* lc, grpo_grads* gr,
               grpo_lora_grads* lg, float* loss, float* logp, grpo_stats* stats, void* workspace, size_t workspace_bytes,
               cudaStream_t s) {
  const grpo_model_cfg& c = m->cfg;
  const int d = c.d, L = c.n_layers, H = c.n_heads, dh = d / H, P = c.prefix_len, S = P + ACT;
  const int dt = c.dtype == GRPO_BF16 ? DT_BF16 : DT_F32;
  const bool fwd_only = lc->flags & GRPO_FWD_ONLY;
  const int n = pk->n_kept;
  const int mb_max = lc->mb_chunks < n ? lc->mb_chunks : (n > 0 ? n : 1);
  const bool chunk_ratio = lc->flags & GRPO_CHUNK_RATIO;
  const float n_terms = (chunk_ratio ? 1.f : (float)ACT) * (float)(n > 0 ? n : 1);
  const float loss_scale = lc->loss_scale > 0.f ? lc->loss_scale : 1.0f / n_terms;
  const float ent_scale = lc->entropy_coef / ((float)ACT * (float)(n > 0 ? n : 1));   // coefficient x token mean
  const long long launches0 = g_launches.load();
  const int r = lo ? lo->rank : 0;
  const float lora_scale = lo ? lo->alpha / (float)lo->rank : 1.f;

  bool fuse_swiglu = false, fuse_rope = false;
  fused_epilogues(c, &fuse_swiglu, &fuse_rope);
  Workspace w;
  memset(&w, 0, sizeof(w));
  carve(w, (unsigned char*)workspace, c, mb_max, fwd_only, r, !fuse_swiglu);
  if (w.bytes > workspace_bytes) return PCM_ERR_WORKSPACE;

  const T* g1 = (const T*)m->g1; const T* g2 = (const T*)m->g2;
  const T* gf = (const T*)m->gf; const T* w_h = (const T*)m->w_h;
  // per projection: base weight [L][out][in], adapters A [L][r][in] and B [L][out][r], and their gradients
  const int p_in[4] = {d, d, d, 4 * d}, p_out[4] = {3 * d, d, 8 * d, d};
  const T* p_w[4] = {(const T*)m->w_qkv, (const T*)m->w_o, (const T*)m->w_gu, (const T*)m->w_d};
  float* p_dw[4] = {nullptr, nullptr, nullptr, nullptr};
  const T* p_a[4] = {nullptr, nullptr, nullptr, nullptr};
  const T* p_b[4] = {nullptr, nullptr, nullptr, nullptr};
  float* p_da[4] = {nullptr, nullptr, nullptr, nullptr};
  float* p_db[4] = {nullptr, nullptr, nullptr, nullptr};
  if (lo) {
    const void* as[4] = {lo->a_qkv, lo->a_o, lo->a_gu, lo->a_d};
    const void* bs[4] = {lo->b_qkv, lo->b_o, lo->b_gu, lo->b_d};
    for (int pj = 0; pj < 4; ++pj) { p_a[pj] = (const T*)as[pj]; p_b[pj] = (const T*)bs[pj]; }
    if (!fwd_only) {
      float* das[4] = {lg->a_qkv, lg->a_o, lg->a_gu, lg->a_d};
      float* dbs[4] = {lg->b_qkv, lg->b_o, lg->b_gu, lg->b_d};
      for (int pj = 0; pj < 4; ++pj) { p_da[pj] = das[pj]; p_db[pj] = dbs[pj]; }
    }
  } else if (!fwd_only) {
    p_dw[PJ_QKV] = gr->w_qkv; p_dw[PJ_O] = gr->w_o; p_dw[PJ_GU] = gr->w_gu; p_dw[PJ_D] = gr->w_d;
  }

  // gradients start from zero unless the caller accumulates
  if (!fwd_only && !(lc->flags & GRPO_ACCUMULATE)) {
    for (int pj = 0; pj < 4; ++pj) {
      const size_t io = (size_t)p_in[pj] * p_out[pj];
      if (p_dw[pj]) PCM_CUDA_TRY(cudaMemsetAsync(p_dw[pj], 0, (size_t)L * io * 4, s));
      if (p_da[pj]) PCM_CUDA_TRY(cudaMemsetAsync(p_da[pj], 0, (size_t)L * r * p_in[pj] * 4, s));
      if (p_db[pj]) PCM_CUDA_TRY(cudaMemsetAsync(p_db[pj], 0, (size_t)L * r * p_out[pj] * 4, s));
    }
    PCM_CUDA_TRY(cudaMemsetAsync(gr->g1, 0, (size_t)L * d * 4, s));
    PCM_CUDA_TRY(cudaMemsetAsync(gr->g2, 0, (size_t)L * d * 4, s));
    PCM_CUDA_TRY(cudaMemsetAsync(gr->gf, 0, (size_t)d * 4, s));
    PCM_CUDA_TRY(cudaMemsetAsync(gr->w_h, 0, (size_t)NB * d * 4, s));
    PCM_CUDA_TRY(cudaMemsetAsync(gr->e_act, 0, (size_t)NB * d * 4, s));
  }
  PCM_CUDA_TRY(cudaMemsetAsync(w.loss_acc, 0, 256, s));
  PCM_CUDA_TRY(cudaMemsetAsync(loss, 0, sizeof(float), s));
  rope_table_kernel<<<ceil_div((long long)S * dh / 2, 256), 256, 0, s>>>(w.rope_tab, S, dh);
  PCM_LAUNCH_CHECK();

  auto GX = [&](const GemmArgs& g) -> int {
    prof_begin(gemm_runs_on_pairs(g) ? PC_GEMM : PC_GEMM_SMALL, s);
    const int rc = gemm(g, s);
    prof_end(s, 2.0 * g.M * (double)g.N * (g.K + g.K2), 0.0);
    return rc;
  };
  auto G = [&](int M_, int N_, int K_, const void* A, long long lda, bool ak, const void* B, long long ldb, bool bk,
               int abdt, void* C, long long ldc, int cdt, const float* R, long long ldr,
               const GemmEpilogue& epi = GemmEpilogue()) -> int {
    GemmArgs g{M_, N_, K_, A, lda, ak, B, ldb, bk, abdt, C, ldc, cdt, R, ldr, epi};
    return GX(g);
  };
#define TRY(expr) do { int rc__ = (expr); if (rc__ != PCM_OK) return rc__; } while (0)
  const double es = (double)sizeof(T);

  // y[rows][out] = x W^T (+ R), with the adapter branch alpha/r (x A^T) B^T entering the same accumulator as a
  // continuation of the contraction: t = alpha/r x A^T is formed first (and kept in t_buf for the backward pass).
  auto lin_fwd = [&](int pj, int l, int rows, const void* x, void* t_buf, void* C, int cdt, const float* R,
                     const GemmEpilogue& epi) -> int {
    const int in = p_in[pj], out = p_out[pj];
    GemmArgs g{rows, out, in, x, in, true, p_w[pj] + (size_t)l * out * in, in, true, dt, C, out, cdt, R, out, epi};
    if (lo) {
      GemmArgs gt{rows, r, in, x, in, true, p_a[pj] + (size_t)l * r * in, in, true, dt, t_buf, r, dt, nullptr, 0};
      gt.alpha = lora_scale;
      TRY(GX(gt));
      g.A2 = t_buf; g.lda2 = r; g.B2 = p_b[pj] + (size_t)l * out * r; g.ldb2 = r; g.K2 = r;
    }
    return GX(g);
  };
  // Backward of the same map: dW += dy^T x (dense), or with adapters u = alpha/r dy B, dA += u^T x, dB += dy^T t
  // (the base weight is frozen); then dX[rows][ldc >= in] = dy W (+ u A), again one contraction.
  auto lin_bwd = [&](int pj, int l, int rows, const void* x, const void* t_buf, const void* dy, void* dX, int ldc, int cdt,
                     const GemmEpilogue& epi) -> int {
    const int in = p_in[pj], out = p_out[pj];
    const T* W = p_w[pj] + (size_t)l * out * in;
    GemmArgs g{rows, in, out, dy, out, true, W, in, false, dt, dX, ldc, cdt, nullptr, 0, epi};
    if (!lo) {
      float* dW = p_dw[pj] + (size_t)l * out * in;
      TRY(G(out, in, rows, dy, out, false, x, in, false, dt, dW, in, DT_F32, dW, in));
    } else {
      GemmArgs gu{rows, r, out, dy, out, true, p_b[pj] + (size_t)l * out * r, r, false, dt, w.lu, r, dt, nullptr, 0};
      gu.alpha = lora_scale;
      TRY(GX(gu));
      float* dA = p_da[pj] + (size_t)l * r * in;
      float* dB = p_db[pj] + (size_t)l * out * r;
      TRY(G(r, in, rows, w.lu, r, false, x, in, false, dt, dA, in, DT_F32, dA, in));
      TRY(G(out, r, rows, dy, out, false, t_buf, r, false, dt, dB, r, DT_F32, dB, r));
      g.A2 = w.lu; g.lda2 = r; g.B2 = p_a[pj] + (size_t)l * r * in; g.ldb2 = in; g.K2 = r;
    }
    return GX(g);
  };

  for (int c0 = 0; c0 < n; c0 += mb_max) {
    const int mb = (n - c0) < mb_max ? (n - c0) : mb_max;
    const long long M = (long long)mb * S, R = (long long)mb * ACT;
    const int Mi = (int)M, Ri = (int)R;
    const T* Xmb = (const T*)pk->X + (long long)c0 * S * d;
    const uint8_t* tgt = pk->tgt + (long long)c0 * ACT;
    const float* lpo = pk->lpo + (long long)c0 * ACT;
    const float* advc = pk->adv_c + c0;

    // ---------------- forward ----------------
    prof_begin(PC_ELEM, s);
    to_residual_kernel<T><<<ceil_div(M * d, 1024), 256, 0, s>>>(Xmb, w.x[0], M * d);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, (double)M * d * (es + 4.0));
    for (int l = 0; l < L; ++l) {
      LayerActs& la = w.la[l];
      const bool last = l == L - 1;
      const float* x_in = w.x[l];
      float* x_out = w.x[l + 1];
      prof_begin(PC_NORM, s);
      rmsnorm_fwd_kernel<T><<<ceil_div(M, 8), 256, 0, s>>>(x_in, g1 + (size_t)l * d, (T*)la.h1, la.rstd1, M, d, 0, 0);
      PCM_LAUNCH_CHECK();
      prof_end(s, 0.0, (double)M * d * (es + 4.0));
      GemmEpilogue e_qkv;
      if (fuse_rope) { e_qkv.kind = EPI_ROPE; e_qkv.rope_tab = w.rope_tab; e_qkv.S = S; e_qkv.dh = dh; e_qkv.d = d; }
      TRY(lin_fwd(PJ_QKV, l, Mi, la.h1, la.lt[PJ_QKV], la.qkv, dt, nullptr, e_qkv));
      if (!fuse_rope) {
        prof_begin(PC_ELEM, s);
        rope_kernel<T><<<ceil_div(M * H * dh / Vec16<T>::N, 256), 256, 0, s>>>((T*)la.qkv, w.rope_tab, M, S, H, dh, 1.f);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)M * 2 * d * es * 2.0);
      }
      prof_begin(PC_ATTN, s);
      TRY(attention_fwd(dt, la.qkv, la.attn, la.lse, mb, S, H, dh, s));
      prof_end(s, 2.0 * S * (double)S * d * mb, (double)M * 4 * d * es);
      // From here on the last layer works on the scored rows only: the head reads nothing else, so the other rows'
      // values would be unread and their gradients exactly zero.
      const long long Mp = last ? R : M;
      const int Mpi = (int)Mp;
      const void* attn_in = la.attn;
      const float* resid = x_in;
      if (last) {
        prof_begin(PC_ELEM, s);
        gather_scored_rows_kernel<T><<<ceil_div(R * (d / 4), 256), 256, 0, s>>>((const T*)la.attn, x_in, (T*)w.attn_s, w.xin_s,
                                                                              R, S, P, d);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)R * d * (es + 4.0) * 2.0);
        attn_in = w.attn_s; resid = w.xin_s;
      }
      TRY(lin_fwd(PJ_O, l, Mpi, attn_in, la.lt[PJ_O], la.x_mid, DT_F32, resid, GemmEpilogue()));
      prof_begin(PC_NORM, s);
      rmsnorm_fwd_kernel<T><<<ceil_div(Mp, 8), 256, 0, s>>>(la.x_mid, g2 + (size_t)l * d, (T*)la.h2, la.rstd2, Mp, d, 0, 0);
      PCM_LAUNCH_CHECK();
      prof_end(s, 0.0, (double)Mp * d * (es + 4.0));
      GemmEpilogue e_gu;
      if (fuse_swiglu) { e_gu.kind = EPI_SWIGLU_FWD; e_gu.out2 = la.act; e_gu.ld_out2 = 4 * d; }
      TRY(lin_fwd(PJ_GU, l, Mpi, la.h2, la.lt[PJ_GU], la.gu, dt, nullptr, e_gu));
      if (!fuse_swiglu) {
        prof_begin(PC_ELEM, s);
        swiglu_fwd_kernel<T><<<ceil_div(Mp * 4 * d / Vec16<T>::N, 256), 256, 0, s>>>((const T*)la.gu, (T*)la.act, Mp, 4 * d);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)Mp * 4 * d * es * 3.0);
      }
      TRY(lin_fwd(PJ_D, l, Mpi, la.act, la.lt[PJ_D], x_out, DT_F32, la.x_mid, GemmEpilogue()));
    }
    // head on the scored rows (x[L] holds exactly those)
    prof_begin(PC_NORM, s);
    rmsnorm_fwd_kernel<T><<<ceil_div(R, 8), 256, 0, s>>>(w.x[L], gf, (T*)w.hs, w.rstdf, R, d, 0, 0);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, (double)R * d * (es + 4.0));
    // Head and loss in one launch: the logits stay in tensor memory (bf16 on the tensor cores) or registers.
    // Returns the number of partial-sum entries the launch wrote (0 when it writes none).
    auto head = [&](int mode, bool want_dz, float* logp_out, float* part, int* n_part) -> int {
      HeadLossArgs h;
      h.tgt = tgt; h.lpo = lpo; h.adv_c = advc; h.coef = w.coef; h.logp = logp_out; h.part = part;
      h.lo = 1.f - lc->eps_low; h.hi = 1.f + lc->eps_high; h.loss_scale = loss_scale; h.ent_scale = ent_scale;
      h.mode = mode; h.want_dz = want_dz ? 1 : 0;
      GemmArgs g{Ri, NB, d, w.hs, d, true, w_h, d, true, dt, w.dz, NB, dt, nullptr, 0};
      g.epi.kind = EPI_HEAD_LOSS; g.epi.hl = h;
      const double bytes = (double)R * (d * es + (want_dz ? NB * es : 0.0) + 9.0) + (double)NB * d * es;
      prof_begin(PC_LOSS, s);
      int rc = PCM_OK;
      if (dt == DT_BF16 && backend_from_env() != GEMM_SIMT && gemm_epilogue_supported(g)) {
        rc = gemm(g, s, GEMM_TCGEN05);
        *n_part = ceil_div(R, 128) * 4;
      } else {
        head_loss_simt_kernel<T><<<ceil_div(R, HL_ROWS), NB, 0, s>>>((const T*)w.hs, w_h, Ri, d, h, (T*)w.dz);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaPeekAtLastError() != cudaSuccess) { cudaGetLastError(); rc = PCM_ERR_CUDA; }
        *n_part = ceil_div(R, HL_ROWS);
      }
      prof_end(s, 2.0 * R * (double)NB * d, bytes);
      return rc;
    };
    int n_part = 0;
    float* lp_out = logp ? logp + (long long)c0 * ACT : w.logp_tmp;
    if (!chunk_ratio) {
      TRY(head(HL_TOKEN, !fwd_only, lp_out, w.loss_part, &n_part));
    } else {
      // the chunk's ratio needs all 56 log-probs first: statistics pass, per-chunk ratio, then (backward only) a
      // second head launch that recomputes the logits and forms their gradient
      TRY(head(HL_STATS, false, lp_out, w.loss_part, &n_part));
      chunk_ratio_kernel<<<ceil_div(mb, 8), 256, 0, s>>>(lp_out, lpo, advc, mb, 1.f - lc->eps_low, 1.f + lc->eps_high, loss_scale,
                                                         w.coef, w.loss_part + (size_t)n_part * 4);
      PCM_LAUNCH_CHECK();
      n_part += mb;
      if (!fwd_only) {
        int unused = 0;
        TRY(head(HL_COEF, true, nullptr, nullptr, &unused));
      }
    }
    loss_reduce_kernel<<<1, 256, 0, s>>>(w.loss_part, n_part, loss_scale, ent_scale, w.loss_acc, loss);
    PCM_LAUNCH_CHECK();
    if (fwd_only) continue;

    // ---------------- backward ----------------
    // head: dW_h += dz^T hs ; dhs = dz W_h
    TRY(G(NB, d, Ri, w.dz, NB, false, w.hs, d, false, dt, gr->w_h, d, DT_F32, gr->w_h, d));
    TRY(G(Ri, d, NB, w.dz, NB, true, w_h, d, false, dt, w.dhs, d, DT_F32, nullptr, 0));
    const size_t nb_smem = (size_t)8 * d * sizeof(float);
    if (nb_smem > 48 * 1024)
    {
      PCM_CUDA_TRY(cudaFuncSetAttribute(rmsnorm_bwd_kernel<T, float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)nb_smem));
      PCM_CUDA_TRY(cudaFuncSetAttribute(rmsnorm_bwd_kernel<T, T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)nb_smem));
      PCM_CUDA_TRY(cudaFuncSetAttribute(rmsnorm_bwd_rows_kernel<T, T, 8, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)nb_smem));
      PCM_CUDA_TRY(cudaFuncSetAttribute(rmsnorm_bwd_rows_kernel<T, T, 8, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)nb_smem));
    }
    // dy_is_t: the incoming gradient is stored in the activation type (the per-layer dh), else in fp32.
    // dx_out = dx_in + (gradient through the norm), in fp32 and in T.
    auto norm_bwd = [&](const void* dy, bool dy_is_t, const float* x, const float* rstd, const T* gamma, const float* dx_in,
                        long long rows, float* dgamma, float* dx_out, T* dx_out_t) -> int {
      const int blocks = (int)(rows / 8 + 1 < NORM_BWD_BLOCKS ? rows / 8 + 1 : NORM_BWD_BLOCKS);
      prof_begin(PC_NORM, s);
      if (dy_is_t && d == 1024)
        rmsnorm_bwd_rows_kernel<T, T, 8, 1><<<blocks, 256, nb_smem, s>>>((const T*)dy, x, rstd, gamma, dx_in, dx_out, dx_out_t,
                                                                          w.norm_part, rows, 0, 0);
      else if (dy_is_t && d == 2048)
        rmsnorm_bwd_rows_kernel<T, T, 8, 2><<<blocks, 256, 8 * 1024 * sizeof(float), s>>>((const T*)dy, x, rstd, gamma, dx_in, dx_out,
                                                                                          dx_out_t, w.norm_part, rows, 0, 0);
      else if (dy_is_t)
        rmsnorm_bwd_kernel<T, T><<<blocks, 256, nb_smem, s>>>((const T*)dy, x, rstd, gamma, dx_in, dx_out, dx_out_t, w.norm_part,
                                                               rows, d, 0, 0);
      else
        rmsnorm_bwd_kernel<T, float><<<blocks, 256, nb_smem, s>>>((const float*)dy, x, rstd, gamma, dx_in, dx_out, dx_out_t,
                                                                   w.norm_part, rows, d, 0, 0);
      PCM_LAUNCH_CHECK();
      prof_end(s, 0.0, (double)rows * d * ((dx_in ? 12.0 : 8.0) + (dy_is_t ? es : 4.0) + es));
      colsum_accumulate_kernel<<<ceil_div(d, 32), 256, 0, s>>>(w.norm_part, blocks, d, dgamma);
      PCM_LAUNCH_CHECK();
      return PCM_OK;
    };
    // final norm: the gradient of the scored rows, kept compact until the last layer's attention block
    TRY(norm_bwd(w.dhs, false, w.x[L], w.rstdf, gf, nullptr, R, gr->gf, w.dxs, (T*)w.dxs_t));

    for (int l = L - 1; l >= 0; --l) {
      LayerActs& la = w.la[l];
      const bool last = l == L - 1;
      const long long Mp = last ? R : M;
      const int Mpi = (int)Mp;
      float* dxp = last ? w.dxs : w.dx;                     // residual gradient of the post-attention rows
      T* dxp_t = last ? (T*)w.dxs_t : (T*)w.dx_t;
      // MLP: x_out = x_mid + act W_d^T
      GemmEpilogue e_d;
      if (fuse_swiglu) { e_d.kind = EPI_SWIGLU_BWD; e_d.aux = la.gu; e_d.ld_aux = 8 * d; }
      TRY(lin_bwd(PJ_D, l, Mpi, la.act, la.lt[PJ_D], dxp_t, fuse_swiglu ? w.dgu : w.dact, fuse_swiglu ? 8 * d : 4 * d, dt, e_d));
      if (!fuse_swiglu) {
        prof_begin(PC_ELEM, s);
        swiglu_bwd_kernel<T><<<ceil_div(Mp * 4 * d / Vec16<T>::N, 256), 256, 0, s>>>((const T*)la.gu, (const T*)w.dact, (T*)w.dgu, Mp, 4 * d);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)Mp * 4 * d * es * 5.0);
      }
      TRY(lin_bwd(PJ_GU, l, Mpi, la.h2, la.lt[PJ_GU], w.dgu, w.dh, d, dt, GemmEpilogue()));
      TRY(norm_bwd(w.dh, true, la.x_mid, la.rstd2, g2 + (size_t)l * d, dxp, Mp, gr->g2 + (size_t)l * d, dxp, dxp_t));
      // attention block: x_mid = x_in + attn W_o^T
      TRY(lin_bwd(PJ_O, l, Mpi, last ? w.attn_s : la.attn, la.lt[PJ_O], dxp_t, last ? w.dattn_s : w.dattn, d, dt, GemmEpilogue()));
      if (last) {
        // back to all rows: the other rows of d(attn) and of the residual gradient are exactly zero
        PCM_CUDA_TRY(cudaMemsetAsync(w.dattn, 0, (size_t)M * d * sizeof(T), s));
        PCM_CUDA_TRY(cudaMemsetAsync(w.dx, 0, (size_t)M * d * 4, s));
        prof_begin(PC_ELEM, s);
        scatter_scored_rows_kernel<T><<<ceil_div(R * (d / 4), 256), 256, 0, s>>>((const T*)w.dattn_s, w.dxs, (T*)w.dattn, w.dx,
                                                                               R, S, P, d);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)M * d * (es + 4.0) + (double)R * d * (es + 4.0) * 2.0);
      }
      prof_begin(PC_ATTN, s);
      TRY(attention_bwd(dt, la.qkv, la.attn, w.dattn, la.lse, w.dsum, w.dqkv, mb, S, H, dh, s,
                        fuse_rope ? w.rope_tab : nullptr));
      prof_end(s, 5.0 * S * (double)S * d * mb, (double)M * 8 * d * es);
      if (!fuse_rope) {
        prof_begin(PC_ELEM, s);
        rope_kernel<T><<<ceil_div(M * H * dh / Vec16<T>::N, 256), 256, 0, s>>>((T*)w.dqkv, w.rope_tab, M, S, H, dh, -1.f);
        PCM_LAUNCH_CHECK();
        prof_end(s, 0.0, (double)M * 2 * d * es * 2.0);
      }
      TRY(lin_bwd(PJ_QKV, l, Mi, la.h1, la.lt[PJ_QKV], w.dqkv, w.dh, d, dt, GemmEpilogue()));
      TRY(norm_bwd(w.dh, true, w.x[l], la.rstd1, g1 + (size_t)l * d, w.dx, M, gr->g1 + (size_t)l * d, w.dx, (T*)w.dx_t));
    }
    prof_begin(PC_EMBED, s);
    embed_grad_kernel<<<dim3(NB, ceil_div(d, 256)), 256, 0, s>>>(w.dx, tgt, mb, S, P, d, gr->e_act);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, (double)mb * ACT * d * 4.0);
  }
#undef TRY

  if (stats) {
    float acc[4] = {0, 0, 0, 0}, l = 0;
    PCM_CUDA_TRY(cudaMemcpyAsync(acc, w.loss_acc, sizeof(acc), cudaMemcpyDeviceToHost, s));
    PCM_CUDA_TRY(cudaMemcpyAsync(&l, loss, sizeof(float), cudaMemcpyDeviceToHost, s));
    PCM_CUDA_TRY(cudaStreamSynchronize(s));
    const float tokens = (float)n * ACT, terms = chunk_ratio ? (float)n : tokens;
    stats->loss = l;
    stats->clip_frac = terms > 0 ? acc[1] / terms : 0.f;
    stats->mean_ratio = terms > 0 ? acc[2] / terms : 0.f;
    stats->entropy = tokens > 0 ? acc[3] / tokens : 0.f;
    stats->reserved = 0;
    stats->n_launches = (int32_t)(g_launches.load() - launches0);
    stats->workspace_high_water = w.bytes;
    const int tcs = tcgen05_poll_status();
    if (tcs != PCM_OK) return tcs;
  }
  return PCM_OK;
}


static GemmBackend backend_from_env() {
  const char* e = getenv("PCM_GEMM_BACKEND");
  if (e && !strcmp(e, "simt")) return GEMM_SIMT;
  if (e && !strcmp(e, "tcgen05")) return GEMM_TCGEN05;
  return GEMM_AUTO;
}

bool gemm_runs_on_pairs(const GemmArgs& g) {
  return backend_from_env() != GEMM_SIMT && gemm_tcgen05_supported(g) && gemm_tcgen05_pair(g);
}

int gemm(const GemmArgs& g, cudaStream_t s, GemmBackend backend) {
  if (backend == GEMM_AUTO) backend = backend_from_env();
  if (backend == GEMM_TCGEN05) {
    if (!gemm_tcgen05_supported(g)) return PCM_ERR_SHAPE;
    return gemm_tcgen05(g, s);
  }
  if (backend == GEMM_AUTO && gemm_tcgen05_supported(g)) return gemm_tcgen05(g, s);
  if (g.epi.kind != EPI_NONE) return PCM_ERR_SHAPE;        // fused epilogues exist on the tensor-core path only
  return gemm_simt(g, s);
}

}  // namespace pcm

using namespace pcm;

static size_t workspace_bytes_for(const grpo_model_cfg* cfg, int rank, int32_t mb_chunks, uint32_t flags) {
  if (check_cfg(cfg) != PCM_OK || mb_chunks < 1) return 0;
  bool fuse_swiglu = false, fuse_rope = false;
  fused_epilogues(*cfg, &fuse_swiglu, &fuse_rope);
  Workspace w;
  memset(&w, 0, sizeof(w));
  carve(w, nullptr, *cfg, mb_chunks, flags & GRPO_FWD_ONLY, rank, !fuse_swiglu);
  return w.bytes;
}

extern "C" size_t grpo_workspace_bytes(const grpo_model_cfg* cfg, int32_t mb_chunks, uint32_t flags) {
  return workspace_bytes_for(cfg, 0, mb_chunks, flags);
}

extern "C" size_t grpo_lora_workspace_bytes(const grpo_model_cfg* cfg, int32_t rank, int32_t mb_chunks, uint32_t flags) {
  if (rank < 8 || rank > 64 || (rank % 8)) return 0;
  return workspace_bytes_for(cfg, rank, mb_chunks, flags);
}

static int actor_entry(const grpo_model* model, const grpo_lora* lora, const grpo_packed* batch, const grpo_loss_cfg* lc,
                       grpo_grads* grads, grpo_lora_grads* lgrads, float* loss, float* logp, grpo_stats* stats,
                       void* workspace, size_t workspace_bytes, pcm_stream stream) {
  if (!model || !batch || !lc || !loss || !workspace) return PCM_ERR_ARG;
  int rc = check_cfg(&model->cfg);
  if (rc) return rc;
  if (!model->w_qkv || !model->w_o || !model->w_gu || !model->w_d || !model->g1 || !model->g2 || !model->gf ||
      !model->w_h || !model->e_act)
    return PCM_ERR_ARG;
  if (batch->n_kept < 0 || lc->mb_chunks < 1 || !(lc->eps_low >= 0.f) || !(lc->eps_high >= 0.f)) return PCM_ERR_ARG;
  if (batch->n_kept > 0 && (!batch->X || !batch->tgt || !batch->lpo || !batch->adv_c)) return PCM_ERR_ARG;
  const bool fwd_only = lc->flags & GRPO_FWD_ONLY;
  if (!fwd_only) {
    if (!grads || !grads->g1 || !grads->g2 || !grads->gf || !grads->w_h || !grads->e_act) return PCM_ERR_ARG;
    if (!lora && (!grads->w_qkv || !grads->w_o || !grads->w_gu || !grads->w_d)) return PCM_ERR_ARG;
    if (lora && (!lgrads || !lgrads->a_qkv || !lgrads->b_qkv || !lgrads->a_o || !lgrads->b_o || !lgrads->a_gu ||
                 !lgrads->b_gu || !lgrads->a_d || !lgrads->b_d))
      return PCM_ERR_ARG;
  }
  if (((uintptr_t)workspace) & 255) return PCM_ERR_WORKSPACE;
  cudaStream_t s = (cudaStream_t)stream;
  if (model->cfg.dtype == GRPO_BF16)
    return run<__nv_bfloat16>(model, lora, batch, lc, grads, lgrads, loss, logp, stats, workspace, workspace_bytes, s);
  return run<float>(model, lora, batch, lc, grads, lgrads, loss, logp, stats, workspace, workspace_bytes, s);
}

extern "C" int grpo_actor_fwd_bwd(const grpo_model* model, const grpo_packed* batch, const grpo_loss_cfg* lc,
                                  grpo_grads* grads, float* loss, float* logp, grpo_stats* stats, void* workspace,
                                  size_t workspace_bytes, pcm_stream stream) {
  return actor_entry(model, nullptr, batch, lc, grads, nullptr, loss, logp, stats, workspace, workspace_bytes, stream);
}

extern "C" int grpo_actor_fwd_bwd_lora(const grpo_model* model, const grpo_lora* lora, const grpo_packed* batch,
                                       const grpo_loss_cfg* lc, grpo_grads* grads, grpo_lora_grads* lora_grads, float* loss,
                                       float* logp, grpo_stats* stats, void* workspace, size_t workspace_bytes,
                                       pcm_stream stream) {
  const int rc = check_lora(lora);
  if (rc) return rc;
  return actor_entry(model, lora, batch, lc, grads, lora_grads, loss, logp, stats, workspace, workspace_bytes, stream);
}

extern "C" int grpo_gemm(int32_t M, int32_t N, int32_t K, const void* A, int64_t lda, int32_t a_kmajor, const void* B,
                         int64_t ldb, int32_t b_kmajor, int32_t ab_dtype, void* C, int64_t ldc, int32_t c_dtype,
                         const float* R, int64_t ldr, int32_t backend, pcm_stream stream) {
  const bool no_sync = (backend & 4) != 0;
  backend &= 3;
  if (!A || !B || !C || M < 1 || N < 1 || K < 1 || backend > 2) return PCM_ERR_ARG;
  if ((ab_dtype != GRPO_F32 && ab_dtype != GRPO_BF16) || (c_dtype != GRPO_F32 && c_dtype != GRPO_BF16)) return PCM_ERR_ARG;
  GemmArgs g{M, N, K, A, lda, a_kmajor != 0, B, ldb, b_kmajor != 0, ab_dtype == GRPO_BF16 ? DT_BF16 : DT_F32,
             C, ldc, c_dtype == GRPO_BF16 ? DT_BF16 : DT_F32, R, ldr};
  cudaStream_t s = (cudaStream_t)stream;
  int rc = gemm(g, s, backend == 1 ? GEMM_SIMT : backend == 2 ? GEMM_TCGEN05 : GEMM_AUTO);
  if (rc != PCM_OK || no_sync) return rc;
  PCM_CUDA_TRY(cudaStreamSynchronize(s));
  return tcgen05_poll_status();
}

namespace pcm { unsigned attention_tc_last_status(); }
extern "C" uint32_t grpo_attention_wait_status(void) { return pcm::attention_tc_last_status(); }

extern "C" int grpo_attention(int32_t dtype, const void* qkv, void* out, float* lse, const void* dout, void* dqkv,
                              float* scratch, int32_t n_seq, int32_t S, int32_t n_heads, int32_t head_dim,
                              pcm_stream stream) {
  if (!qkv || !out || !lse || n_seq < 1 || S < 1 || n_heads < 1) return PCM_ERR_ARG;
  if (dtype != GRPO_F32 && dtype != GRPO_BF16) return PCM_ERR_ARG;
  if (dout && (!dqkv || !scratch)) return PCM_ERR_ARG;
  const int dt = dtype == GRPO_BF16 ? DT_BF16 : DT_F32;
  cudaStream_t s = (cudaStream_t)stream;
  int rc = attention_fwd(dt, qkv, out, lse, n_seq, S, n_heads, head_dim, s);
  if (rc != PCM_OK) return rc;
  if (dout) {
    rc = attention_bwd(dt, qkv, out, dout, lse, scratch, dqkv, n_seq, S, n_heads, head_dim, s);
    if (rc != PCM_OK) return rc;
  }
  PCM_CUDA_TRY(cudaStreamSynchronize(s));
  return tcgen05_poll_status();
}
