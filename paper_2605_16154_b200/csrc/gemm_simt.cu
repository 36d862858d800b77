// Plain tiled SIMT GEMM with fp32 accumulation.  It is the fp32 precision mode of the library and
// the fallback for shapes the tensor-core kernel does not take; operands are addressed through
// (row, column) strides so that every transposition variant is the same kernel.
#include "internal.h"

namespace pcm {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }

constexpr int SG_BM = 64, SG_BN = 64, SG_BK = 16;

// A(m,k) = A[m*sam + k*sak], B(n,k) = B[n*sbn + k*sbk]
template <typename TI, typename TC>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(int M, int N, int K, const TI* __restrict__ A, long long sam, long long sak,
                 const TI* __restrict__ B, long long sbn, long long sbk, TC* C, long long ldc,
                 const float* R, long long ldr, int K2, const TI* __restrict__ A2, long long sam2, long long sak2,
                 const TI* __restrict__ B2, long long sbn2, long long sbk2, float alpha) {
  __shared__ float As[SG_BK][SG_BM + 4];
  __shared__ float Bs[SG_BK][SG_BN + 4];
  const int tid = threadIdx.x;
  const int m0 = blockIdx.y * SG_BM, n0 = blockIdx.x * SG_BN;
  const int tx = tid & 15, ty = tid >> 4;                 // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};
  const bool a_k_fast = (sak == 1), b_k_fast = (sbk == 1);
  for (int seg = 0; seg < 2; ++seg) {                     // the contraction, then its optional continuation
  if (seg == 1) {
    if (K2 <= 0) break;
    A = A2; B = B2; K = K2; sam = sam2; sak = sak2; sbn = sbn2; sbk = sbk2;
  }
  for (int k0 = 0; k0 < K; k0 += SG_BK) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int idx = tid + e * 256;                      // 1024 elements per operand tile
      int m, k;
      if (a_k_fast) { m = idx >> 4; k = idx & 15; } else { k = idx >> 6; m = idx & 63; }
      float v = 0.f;
      if (m0 + m < M && k0 + k < K) v = to_f32(A[(long long)(m0 + m) * sam + (long long)(k0 + k) * sak]);
      As[k][m] = v;
      int n, kb;
      if (b_k_fast) { n = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; n = idx & 63; }
      float w = 0.f;
      if (n0 + n < N && k0 + kb < K) w = to_f32(B[(long long)(n0 + n) * sbn + (long long)(k0 + kb) * sbk]);
      Bs[kb][n] = w;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < SG_BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= N) continue;
      float v = alpha * acc[i][j];
      if (R) v += R[(long long)m * ldr + n];
      if constexpr (sizeof(TC) == 4) C[(long long)m * ldc + n] = v;
      else C[(long long)m * ldc + n] = __float2bfloat16_rn(v);
    }
  }
}

template <typename TI, typename TC>
static int launch_simt(const GemmArgs& g, cudaStream_t s) {
  const long long sam = g.a_kmajor ? g.lda : 1, sak = g.a_kmajor ? 1 : g.lda;
  const long long sbn = g.b_kmajor ? g.ldb : 1, sbk = g.b_kmajor ? 1 : g.ldb;
  dim3 grid(ceil_div(g.N, SG_BN), ceil_div(g.M, SG_BM));
  if (grid.y > 65535) return PCM_ERR_SHAPE;
  gemm_simt_kernel<TI, TC><<<grid, 256, 0, s>>>(g.M, g.N, g.K, (const TI*)g.A, sam, sak, (const TI*)g.B, sbn, sbk,
                                                (TC*)g.C, g.ldc, g.R, g.ldr, g.K2, (const TI*)g.A2,
                                                g.a_kmajor ? g.lda2 : 1, g.a_kmajor ? 1 : g.lda2, (const TI*)g.B2,
                                                g.b_kmajor ? g.ldb2 : 1, g.b_kmajor ? 1 : g.ldb2, g.alpha);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

int gemm_simt(const GemmArgs& g, cudaStream_t s) {
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return PCM_OK;
  if (g.ab_dtype == DT_F32) {
    if (g.c_dtype != DT_F32) return PCM_ERR_ARG;
    return launch_simt<float, float>(g, s);
  }
  if (g.c_dtype == DT_F32) return launch_simt<__nv_bfloat16, float>(g, s);
  return launch_simt<__nv_bfloat16, __nv_bfloat16>(g, s);
}

}  // namespace pcm
