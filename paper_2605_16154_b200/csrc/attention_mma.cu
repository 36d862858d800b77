// bf16 causal attention inside each chunk's sequence on the warp-level tensor-core path
// (mma.sync m16n8k16, fp32 accumulate), flash style: probabilities live in registers only, the
// backward pass rebuilds them from the saved row log-sum-exp.
//
// The operand a CTA sweeps over (keys/values, or queries/dO in the dK/dV pass) streams through two
// shared-memory stages of 64 rows filled with cp.async while the other stage is being consumed:
//   forward / dQ : CTA = 128 (head dim <= 64) or 64 query rows of one (sequence, head); a warp per 16 rows;
//                  loop over 64-key blocks
//   dK / dV      : CTA = 128 or 64 key rows; a warp per 16 keys; loop over 64-query blocks at or below the diagonal
// Shared-memory rows are padded by 16 bytes so that ldmatrix reads are bank-conflict free.
#include "internal.h"

namespace pcm {

// rows per CTA (16 per warp); equal to the inner block so that every warp of a CTA walks the same blocks
template <int DH> struct FaCfg {
  static constexpr int ROWS = 64;
  static constexpr int THREADS = ROWS * 2;
};
constexpr int FA_BLK = 64;                   // columns per inner block
constexpr float LOG2E = 1.4426950408889634f;

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const bf16* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const bf16* p) {
  const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros without touching global memory
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, int src_bytes) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// rows [row0, row0 + nrows) of a [.][DH] matrix (global row stride ld elements) -> shared rows
// [0, nrows) with stride DH + 8; rows at or beyond row_limit are zero.  All copies of a thread are
// in flight together; the caller commits the group and waits with cp_async_wait_group + __syncthreads().
template <int DH>
__device__ __forceinline__ void stage_rows(bf16* dst, const bf16* __restrict__ src, long long ld, int row0, int nrows,
                                           int row_limit) {
  constexpr int RS = DH + 8, VEC = DH / 8;                 // 8 bf16 per 16-byte vector
  for (int idx = threadIdx.x; idx < nrows * VEC; idx += blockDim.x) {
    const int r = idx / VEC, v = idx - r * VEC;
    const bool ok = row0 + r < row_limit;
    const bf16* g = ok ? src + (long long)(row0 + r) * ld + v * 8 : src;
    cp_async16(dst + r * RS + v * 8, g, ok ? 16 : 0);
  }
}

// A fragment: 16 rows x 16 k of a row-major shared tile
template <int RS>
__device__ __forceinline__ void load_a(uint32_t (&a)[4], const bf16* tile, int row0, int k0, int lane) {
  ldsm_x4(a, tile + (row0 + (lane & 15)) * RS + k0 + (lane >> 4) * 8);
}
// B fragments for two adjacent 8-wide n-tiles from a tile stored [n][k]: r0,r1 -> n-tile 0; r2,r3 -> n-tile 1
template <int RS>
__device__ __forceinline__ void load_b_nk(uint32_t (&r)[4], const bf16* tile, int n0, int k0, int lane) {
  const int mi = lane >> 3;
  ldsm_x4(r, tile + (n0 + (mi >> 1) * 8 + (lane & 7)) * RS + k0 + (mi & 1) * 8);
}
// the same from a tile stored [k][n] (transposing load)
template <int RS>
__device__ __forceinline__ void load_b_kn(uint32_t (&r)[4], const bf16* tile, int k0, int n0, int lane) {
  const int mi = lane >> 3;
  ldsm_x4_t(r, tile + (k0 + (mi & 1) * 8 + (lane & 7)) * RS + n0 + (mi >> 1) * 8);
}

__device__ __forceinline__ float quad_max(float v) {
  v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
  return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
}
__device__ __forceinline__ float quad_sum(float v) {
  v += __shfl_xor_sync(0xffffffffu, v, 1);
  return v + __shfl_xor_sync(0xffffffffu, v, 2);
}

// ------------------------------------------------------------------------------------------------
// forward
// ------------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(FaCfg<DH>::THREADS)
fa_fwd_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out, float* __restrict__ lse, int S, int H, float scale) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + 8;
  const int qt = blockIdx.x, h = blockIdx.y, seq = blockIdx.z, d = H * DH;
  const long long ld = 3LL * d;
  const bf16* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  const int q0 = qt * FaCfg<DH>::ROWS;
  const int n_keys = min(S, q0 + FaCfg<DH>::ROWS);                  // causal: keys beyond the tile's last row are never used
  constexpr int STAGE = 2 * FA_BLK * RS;                            // one 64-key block of K followed by the same block of V
  bf16* Qs = reinterpret_cast<bf16*>(smraw);
  bf16* KV = Qs + FaCfg<DH>::ROWS * RS;                              // two stages, refilled while the other one is in use
  auto load_kv = [&](int kb) {
    bf16* st = KV + (kb & 1) * STAGE;
    stage_rows<DH>(st, base + d, ld, kb * FA_BLK, FA_BLK, n_keys);
    stage_rows<DH>(st + FA_BLK * RS, base + 2 * d, ld, kb * FA_BLK, FA_BLK, n_keys);
    cp_async_commit();
  };
  stage_rows<DH>(Qs, base, ld, q0, FaCfg<DH>::ROWS, S);
  load_kv(0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wrow0 = warp * 16;                               // first row of this warp inside the tile
  uint32_t qf[DH / 16][4];

  float o[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;  // rows g and g + 8, log2 domain
  const int row_a = q0 + wrow0 + g, row_b = row_a + 8;
  const float c = scale * LOG2E;
  const int last_blk = (n_keys - 1) / FA_BLK;                 // the same for every warp of the CTA

  for (int kb = 0; kb <= last_blk; ++kb) {
    if (kb < last_blk) { load_kv(kb + 1); cp_async_wait_group<1>(); } else { cp_async_wait_group<0>(); }
    __syncthreads();                                           // block kb has landed for every thread
    if (kb == 0) {
#pragma unroll
      for (int kk = 0; kk < DH / 16; ++kk) load_a<RS>(qf[kk], Qs, wrow0, kk * 16, lane);
    }
    const bf16* Ks = KV + (kb & 1) * STAGE;
    const bf16* Vs = Ks + FA_BLK * RS;
    float s[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b[4];
        load_b_nk<RS>(b, Ks, np * 16, kk * 16, lane);
        mma_bf16(s[2 * np], qf[kk], b[0], b[1]);
        mma_bf16(s[2 * np + 1], qf[kk], b[2], b[3]);
      }
    }
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int col = kb * FA_BLK + nt * 8 + 2 * t;
      s[nt][0] = (col <= row_a) ? s[nt][0] * c : -INFINITY;
      s[nt][1] = (col + 1 <= row_a) ? s[nt][1] * c : -INFINITY;
      s[nt][2] = (col <= row_b) ? s[nt][2] * c : -INFINITY;
      s[nt][3] = (col + 1 <= row_b) ? s[nt][3] * c : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
    }
    mx0 = quad_max(mx0); mx1 = quad_max(mx1);
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);  // finite from block 0 on: column 0 is never masked
    const float al0 = exp2f(m0 - mn0), al1 = exp2f(m1 - mn1);
    float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      s[nt][0] = exp2f(s[nt][0] - mn0); s[nt][1] = exp2f(s[nt][1] - mn0);
      s[nt][2] = exp2f(s[nt][2] - mn1); s[nt][3] = exp2f(s[nt][3] - mn1);
      sum0 += s[nt][0] + s[nt][1];
      sum1 += s[nt][2] + s[nt][3];
    }
    l0 = l0 * al0 + quad_sum(sum0);
    l1 = l1 * al1 + quad_sum(sum1);
    m0 = mn0; m1 = mn1;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) {
      uint32_t pa[4] = {pack_bf16(s[2 * k2][0], s[2 * k2][1]), pack_bf16(s[2 * k2][2], s[2 * k2][3]),
                        pack_bf16(s[2 * k2 + 1][0], s[2 * k2 + 1][1]), pack_bf16(s[2 * k2 + 1][2], s[2 * k2 + 1][3])};
#pragma unroll
      for (int dp = 0; dp < DH / 16; ++dp) {
        uint32_t b[4];
        load_b_kn<RS>(b, Vs, k2 * 16, dp * 16, lane);
        mma_bf16(o[2 * dp], pa, b[0], b[1]);
        mma_bf16(o[2 * dp + 1], pa, b[2], b[3]);
      }
    }
    __syncthreads();                                           // everyone is done with this stage before it is refilled
  }
  const float inv0 = 1.f / l0, inv1 = 1.f / l1;
  if (row_a < S) {
    bf16* op = out + ((long long)seq * S + row_a) * d + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(op + i * 8 + 2 * t) = pack_bf16(o[i][0] * inv0, o[i][1] * inv0);
    if (t == 0) lse[((long long)seq * H + h) * S + row_a] = (m0 + log2f(l0)) * 0.6931471805599453f;
  }
  if (row_b < S) {
    bf16* op = out + ((long long)seq * S + row_b) * d + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i)
      *reinterpret_cast<uint32_t*>(op + i * 8 + 2 * t) = pack_bf16(o[i][2] * inv1, o[i][3] * inv1);
    if (t == 0) lse[((long long)seq * H + h) * S + row_b] = (m1 + log2f(l1)) * 0.6931471805599453f;
  }
}

// Transpose of the rotary embedding applied to an accumulator tile of 16 rows x DH columns: pairs
// (c, c + DH/2) sit in n-tiles i and i + DH/16 of the same thread.  Rows a / b are positions in the sequence.
template <int DH>
__device__ __forceinline__ void unrotate(float (&acc)[DH / 8][4], const float2* __restrict__ tab, int row_a, int row_b,
                                         int S, int t) {
  constexpr int HALF = DH / 2;
  const int pa = min(row_a, S - 1), pb = min(row_b, S - 1);      // rows past the end are never stored
#pragma unroll
  for (int i = 0; i < DH / 16; ++i) {
    const int c = i * 8 + 2 * t;
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const float2 ta = tab[pa * HALF + c + e], tb = tab[pb * HALF + c + e];
      const float la = acc[i][e], ha = acc[i + DH / 16][e];
      acc[i][e] = la * ta.x + ha * ta.y;
      acc[i + DH / 16][e] = ha * ta.x - la * ta.y;
      const float lb = acc[i][2 + e], hb = acc[i + DH / 16][2 + e];
      acc[i][2 + e] = lb * tb.x + hb * tb.y;
      acc[i + DH / 16][2 + e] = hb * tb.x - lb * tb.y;
    }
  }
}

// ------------------------------------------------------------------------------------------------
// dQ: same tiling as the forward pass
// ------------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(FaCfg<DH>::THREADS)
fa_bwd_dq_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ out, const bf16* __restrict__ dout,
                 const float* __restrict__ lse, float* __restrict__ dsum, bf16* __restrict__ dqkv, int S, int H,
                 float scale, const float2* __restrict__ rope_tab) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + 8;
  const int qt = blockIdx.x, h = blockIdx.y, seq = blockIdx.z, d = H * DH;
  const long long ld = 3LL * d;
  const bf16* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  const int q0 = qt * FaCfg<DH>::ROWS;
  const int n_keys = min(S, q0 + FaCfg<DH>::ROWS);
  constexpr int STAGE = 2 * FA_BLK * RS;
  bf16* Qs = reinterpret_cast<bf16*>(smraw);
  bf16* Gs = Qs + FaCfg<DH>::ROWS * RS;                              // dO rows of the tile
  bf16* KV = Gs + FaCfg<DH>::ROWS * RS;                              // two stages of (K block, V block)
  auto load_kv = [&](int kb) {
    bf16* st = KV + (kb & 1) * STAGE;
    stage_rows<DH>(st, base + d, ld, kb * FA_BLK, FA_BLK, n_keys);
    stage_rows<DH>(st + FA_BLK * RS, base + 2 * d, ld, kb * FA_BLK, FA_BLK, n_keys);
    cp_async_commit();
  };
  stage_rows<DH>(Qs, base, ld, q0, FaCfg<DH>::ROWS, S);
  stage_rows<DH>(Gs, dout + (long long)seq * S * d + (long long)h * DH, d, q0, FaCfg<DH>::ROWS, S);
  load_kv(0);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wrow0 = warp * 16;
  const int row_a = q0 + wrow0 + g, row_b = row_a + 8;
  const long long sbase = ((long long)seq * H + h) * S;
  const float c = scale * LOG2E;
  const float la = row_a < S ? lse[sbase + row_a] * LOG2E : 0.f, lb = row_b < S ? lse[sbase + row_b] * LOG2E : 0.f;
  float da = 0.f, db = 0.f;                                  // D = rowsum(dO * O) of rows a and b, computed below

  float dq[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) { dq[i][0] = dq[i][1] = dq[i][2] = dq[i][3] = 0.f; }
  const int last_blk = (n_keys - 1) / FA_BLK;

  for (int kb = 0; kb <= last_blk; ++kb) {
    if (kb < last_blk) { load_kv(kb + 1); cp_async_wait_group<1>(); } else { cp_async_wait_group<0>(); }
    __syncthreads();
    if (kb == 0) {
      // D_i = sum_c dO_i[c] O_i[c] for this warp's 16 rows: two lanes per row, half of the head dimension each.
      // It is also written out for the dK / dV pass.
      const int r = wrow0 + (lane >> 1), hf = lane & 1, grow = q0 + r;
      float acc = 0.f;
      if (grow < S) {
        const bf16* op = out + ((long long)seq * S + grow) * d + (long long)h * DH + hf * (DH / 2);
        const bf16* gp = Gs + r * RS + hf * (DH / 2);
#pragma unroll
        for (int v = 0; v < DH / 16; ++v) {
          const uint4 ov = *reinterpret_cast<const uint4*>(op + v * 8);
          const uint4 gv = *reinterpret_cast<const uint4*>(gp + v * 8);
          const __nv_bfloat162* oh = reinterpret_cast<const __nv_bfloat162*>(&ov);
          const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&gv);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 a = __bfloat1622float2(oh[e]), b = __bfloat1622float2(gh[e]);
            acc = fmaf(a.x, b.x, fmaf(a.y, b.y, acc));
          }
        }
      }
      acc += __shfl_xor_sync(0xffffffffu, acc, 1);
      if (hf == 0 && grow < S) dsum[sbase + grow] = acc;
      da = __shfl_sync(0xffffffffu, acc, 2 * g);
      db = __shfl_sync(0xffffffffu, acc, 2 * (g + 8));
    }
    const bf16* Ks = KV + (kb & 1) * STAGE;
    const bf16* Vs = Ks + FA_BLK * RS;
    float s[8][4], dp[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f;
      dp[i][0] = dp[i][1] = dp[i][2] = dp[i][3] = 0.f;
    }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      uint32_t qa[4], ga[4];
      load_a<RS>(qa, Qs, wrow0, kk * 16, lane);
      load_a<RS>(ga, Gs, wrow0, kk * 16, lane);
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b[4];
        load_b_nk<RS>(b, Ks, np * 16, kk * 16, lane);
        mma_bf16(s[2 * np], qa, b[0], b[1]);
        mma_bf16(s[2 * np + 1], qa, b[2], b[3]);
        load_b_nk<RS>(b, Vs, np * 16, kk * 16, lane);
        mma_bf16(dp[2 * np], ga, b[0], b[1]);
        mma_bf16(dp[2 * np + 1], ga, b[2], b[3]);
      }
    }
    // dS = P * (dP - D) * scale, zero above the diagonal
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int col = kb * FA_BLK + nt * 8 + 2 * t;
      s[nt][0] = (col <= row_a) ? exp2f(s[nt][0] * c - la) * (dp[nt][0] - da) * scale : 0.f;
      s[nt][1] = (col + 1 <= row_a) ? exp2f(s[nt][1] * c - la) * (dp[nt][1] - da) * scale : 0.f;
      s[nt][2] = (col <= row_b) ? exp2f(s[nt][2] * c - lb) * (dp[nt][2] - db) * scale : 0.f;
      s[nt][3] = (col + 1 <= row_b) ? exp2f(s[nt][3] * c - lb) * (dp[nt][3] - db) * scale : 0.f;
    }
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) {
      uint32_t sa[4] = {pack_bf16(s[2 * k2][0], s[2 * k2][1]), pack_bf16(s[2 * k2][2], s[2 * k2][3]),
                        pack_bf16(s[2 * k2 + 1][0], s[2 * k2 + 1][1]), pack_bf16(s[2 * k2 + 1][2], s[2 * k2 + 1][3])};
#pragma unroll
      for (int dpi = 0; dpi < DH / 16; ++dpi) {
        uint32_t b[4];
        load_b_kn<RS>(b, Ks, k2 * 16, dpi * 16, lane);
        mma_bf16(dq[2 * dpi], sa, b[0], b[1]);
        mma_bf16(dq[2 * dpi + 1], sa, b[2], b[3]);
      }
    }
    __syncthreads();
  }
  if (rope_tab) unrotate<DH>(dq, rope_tab, row_a, row_b, S, t);   // gradient w.r.t. q before the rotary embedding
  if (row_a < S) {
    bf16* p = dqkv + ((long long)seq * S + row_a) * ld + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<uint32_t*>(p + i * 8 + 2 * t) = pack_bf16(dq[i][0], dq[i][1]);
  }
  if (row_b < S) {
    bf16* p = dqkv + ((long long)seq * S + row_b) * ld + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) *reinterpret_cast<uint32_t*>(p + i * 8 + 2 * t) = pack_bf16(dq[i][2], dq[i][3]);
  }
}

// ------------------------------------------------------------------------------------------------
// dK, dV: CTA = 64 key rows; transposed score tiles (rows = keys, columns = queries)
// ------------------------------------------------------------------------------------------------
template <int DH>
__global__ void __launch_bounds__(FaCfg<DH>::THREADS)
fa_bwd_dkv_kernel(const bf16* __restrict__ qkv, const bf16* __restrict__ dout, const float* __restrict__ lse,
                  const float* __restrict__ dsum, bf16* __restrict__ dqkv, int S, int H, float scale,
                  const float2* __restrict__ rope_tab) {
  extern __shared__ __align__(16) unsigned char smraw[];
  constexpr int RS = DH + 8;
  const int kt = blockIdx.x, h = blockIdx.y, seq = blockIdx.z, d = H * DH;
  const long long ld = 3LL * d;
  const bf16* base = qkv + (long long)seq * S * ld + (long long)h * DH;
  const int k0 = kt * FaCfg<DH>::ROWS;                               // first key of the tile
  const int q_lo = k0;                                       // queries below the tile's first key never see it
  const int q_rows = (S - q_lo + FA_BLK - 1) / FA_BLK * FA_BLK;
  constexpr int STAGE = 2 * FA_BLK * RS;                      // one 64-query block of Q followed by the same block of dO
  bf16* Ks = reinterpret_cast<bf16*>(smraw);
  bf16* Vs = Ks + FaCfg<DH>::ROWS * RS;
  bf16* QG = Vs + FaCfg<DH>::ROWS * RS;                       // two stages of (Q block, dO block)
  float* Ls = reinterpret_cast<float*>(QG + 2 * STAGE);      // lse * log2(e) for queries q_lo ..
  float* Ds = Ls + q_rows;
  const bf16* gbase = dout + (long long)seq * S * d + (long long)h * DH;
  auto load_qg = [&](int qb) {
    bf16* st = QG + (qb & 1) * STAGE;
    stage_rows<DH>(st, base, ld, q_lo + qb * FA_BLK, FA_BLK, S);
    stage_rows<DH>(st + FA_BLK * RS, gbase, d, q_lo + qb * FA_BLK, FA_BLK, S);
    cp_async_commit();
  };
  stage_rows<DH>(Ks, base + d, ld, k0, FaCfg<DH>::ROWS, S);
  stage_rows<DH>(Vs, base + 2 * d, ld, k0, FaCfg<DH>::ROWS, S);
  load_qg(0);
  const long long sbase = ((long long)seq * H + h) * S;
  for (int i = threadIdx.x; i < q_rows; i += blockDim.x) {
    const bool ok = q_lo + i < S;
    Ls[i] = ok ? lse[sbase + q_lo + i] * LOG2E : 0.f;
    Ds[i] = ok ? dsum[sbase + q_lo + i] : 0.f;
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
  const int wrow0 = warp * 16;
  const int key_a = k0 + wrow0 + g, key_b = key_a + 8;
  const float c = scale * LOG2E;
  float dk[DH / 8][4], dv[DH / 8][4];
#pragma unroll
  for (int i = 0; i < DH / 8; ++i) {
    dk[i][0] = dk[i][1] = dk[i][2] = dk[i][3] = 0.f;
    dv[i][0] = dv[i][1] = dv[i][2] = dv[i][3] = 0.f;
  }
  const int n_blk = q_rows / FA_BLK;
  for (int qb = 0; qb < n_blk; ++qb) {
    if (qb + 1 < n_blk) { load_qg(qb + 1); cp_async_wait_group<1>(); } else { cp_async_wait_group<0>(); }
    __syncthreads();                                           // also publishes Ls / Ds on the first pass
    const bf16* Qs = QG + (qb & 1) * STAGE;
    const bf16* Gs = Qs + FA_BLK * RS;
    float st[8][4], dpt[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      st[i][0] = st[i][1] = st[i][2] = st[i][3] = 0.f;
      dpt[i][0] = dpt[i][1] = dpt[i][2] = dpt[i][3] = 0.f;
    }
#pragma unroll
    for (int kk = 0; kk < DH / 16; ++kk) {
      uint32_t ka[4], va[4];
      load_a<RS>(ka, Ks, wrow0, kk * 16, lane);
      load_a<RS>(va, Vs, wrow0, kk * 16, lane);
#pragma unroll
      for (int np = 0; np < 4; ++np) {
        uint32_t b[4];
        load_b_nk<RS>(b, Qs, np * 16, kk * 16, lane);
        mma_bf16(st[2 * np], ka, b[0], b[1]);
        mma_bf16(st[2 * np + 1], ka, b[2], b[3]);
        load_b_nk<RS>(b, Gs, np * 16, kk * 16, lane);
        mma_bf16(dpt[2 * np], va, b[0], b[1]);
        mma_bf16(dpt[2 * np + 1], va, b[2], b[3]);
      }
    }
    // P^T and dS^T; a query column is live when key <= query < S
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
      const int ql = qb * FA_BLK + nt * 8 + 2 * t;           // local query index (relative to q_lo)
      const int q = q_lo + ql;
      const float l0 = Ls[ql], l1 = Ls[ql + 1], d0 = Ds[ql], d1 = Ds[ql + 1];
      const bool v0 = q < S, v1 = q + 1 < S;
      const float p0 = (v0 && q >= key_a) ? exp2f(st[nt][0] * c - l0) : 0.f;
      const float p1 = (v1 && q + 1 >= key_a) ? exp2f(st[nt][1] * c - l1) : 0.f;
      const float p2 = (v0 && q >= key_b) ? exp2f(st[nt][2] * c - l0) : 0.f;
      const float p3 = (v1 && q + 1 >= key_b) ? exp2f(st[nt][3] * c - l1) : 0.f;
      st[nt][0] = p0; st[nt][1] = p1; st[nt][2] = p2; st[nt][3] = p3;
      dpt[nt][0] = p0 * (dpt[nt][0] - d0) * scale;
      dpt[nt][1] = p1 * (dpt[nt][1] - d1) * scale;
      dpt[nt][2] = p2 * (dpt[nt][2] - d0) * scale;
      dpt[nt][3] = p3 * (dpt[nt][3] - d1) * scale;
    }
#pragma unroll
    for (int k2 = 0; k2 < 4; ++k2) {
      uint32_t pa[4] = {pack_bf16(st[2 * k2][0], st[2 * k2][1]), pack_bf16(st[2 * k2][2], st[2 * k2][3]),
                        pack_bf16(st[2 * k2 + 1][0], st[2 * k2 + 1][1]), pack_bf16(st[2 * k2 + 1][2], st[2 * k2 + 1][3])};
      uint32_t sa[4] = {pack_bf16(dpt[2 * k2][0], dpt[2 * k2][1]), pack_bf16(dpt[2 * k2][2], dpt[2 * k2][3]),
                        pack_bf16(dpt[2 * k2 + 1][0], dpt[2 * k2 + 1][1]), pack_bf16(dpt[2 * k2 + 1][2], dpt[2 * k2 + 1][3])};
#pragma unroll
      for (int dpi = 0; dpi < DH / 16; ++dpi) {
        uint32_t b[4];
        load_b_kn<RS>(b, Gs, k2 * 16, dpi * 16, lane);
        mma_bf16(dv[2 * dpi], pa, b[0], b[1]);
        mma_bf16(dv[2 * dpi + 1], pa, b[2], b[3]);
        load_b_kn<RS>(b, Qs, k2 * 16, dpi * 16, lane);
        mma_bf16(dk[2 * dpi], sa, b[0], b[1]);
        mma_bf16(dk[2 * dpi + 1], sa, b[2], b[3]);
      }
    }
    __syncthreads();
  }
  if (rope_tab) unrotate<DH>(dk, rope_tab, key_a, key_b, S, t);   // gradient w.r.t. k before the rotary embedding
  if (key_a < S) {
    bf16* pk = dqkv + ((long long)seq * S + key_a) * ld + d + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      *reinterpret_cast<uint32_t*>(pk + i * 8 + 2 * t) = pack_bf16(dk[i][0], dk[i][1]);
      *reinterpret_cast<uint32_t*>(pk + d + i * 8 + 2 * t) = pack_bf16(dv[i][0], dv[i][1]);
    }
  }
  if (key_b < S) {
    bf16* pk = dqkv + ((long long)seq * S + key_b) * ld + d + (long long)h * DH;
#pragma unroll
    for (int i = 0; i < DH / 8; ++i) {
      *reinterpret_cast<uint32_t*>(pk + i * 8 + 2 * t) = pack_bf16(dk[i][2], dk[i][3]);
      *reinterpret_cast<uint32_t*>(pk + d + i * 8 + 2 * t) = pack_bf16(dv[i][2], dv[i][3]);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
template <int DH>
static int fa_fwd_launch(const void* qkv, void* out, float* lse, int n_seq, int S, int H, cudaStream_t s) {
  const int tiles = (S + FaCfg<DH>::ROWS - 1) / FaCfg<DH>::ROWS;
  const size_t smem = (size_t)(FaCfg<DH>::ROWS + 4 * FA_BLK) * (DH + 8) * sizeof(bf16);     // Q tile + 2 stages of (K, V)
  if (smem > 227 * 1024) return PCM_ERR_SHAPE;
  PCM_CUDA_TRY(cudaFuncSetAttribute(fa_fwd_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  fa_fwd_kernel<DH><<<dim3(tiles, H, n_seq), FaCfg<DH>::THREADS, smem, s>>>((const bf16*)qkv, (bf16*)out, lse, S, H,
                                                                    1.0f / sqrtf((float)DH));
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

template <int DH>
static int fa_bwd_launch(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                         int n_seq, int S, int H, const float2* rope_tab, cudaStream_t s) {
  const int tiles = (S + FaCfg<DH>::ROWS - 1) / FaCfg<DH>::ROWS;
  const int key_rows = (S + FA_BLK - 1) / FA_BLK * FA_BLK;
  const size_t smem_dq = (size_t)(2 * FaCfg<DH>::ROWS + 4 * FA_BLK) * (DH + 8) * sizeof(bf16);   // 2 tiles + 2 stages of 2 blocks
  const size_t smem_dkv = smem_dq + (size_t)2 * key_rows * sizeof(float);
  if (smem_dkv > 227 * 1024) return PCM_ERR_SHAPE;
  const float scale = 1.0f / sqrtf((float)DH);
  PCM_CUDA_TRY(cudaFuncSetAttribute(fa_bwd_dq_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dq));
  fa_bwd_dq_kernel<DH><<<dim3(tiles, H, n_seq), FaCfg<DH>::THREADS, smem_dq, s>>>((const bf16*)qkv, (const bf16*)out, (const bf16*)dout, lse, dsum,
                                                                         (bf16*)dqkv, S, H, scale, rope_tab);
  PCM_LAUNCH_CHECK();
  PCM_CUDA_TRY(cudaFuncSetAttribute(fa_bwd_dkv_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dkv));
  fa_bwd_dkv_kernel<DH><<<dim3(tiles, H, n_seq), FaCfg<DH>::THREADS, smem_dkv, s>>>((const bf16*)qkv, (const bf16*)dout, lse,
                                                                           dsum, (bf16*)dqkv, S, H, scale, rope_tab);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

int attention_fwd_bf16(const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh, cudaStream_t s) {
  if (n_seq > 65535 || H > 65535) return PCM_ERR_SHAPE;
  if (dh == 32) return fa_fwd_launch<32>(qkv, out, lse, n_seq, S, H, s);
  if (dh == 64) return fa_fwd_launch<64>(qkv, out, lse, n_seq, S, H, s);
  if (dh == 128) return fa_fwd_launch<128>(qkv, out, lse, n_seq, S, H, s);
  return PCM_ERR_SHAPE;
}

int attention_bwd_bf16(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                       int n_seq, int S, int H, int dh, const float2* rope_tab, cudaStream_t s) {
  if (n_seq > 65535 || H > 65535) return PCM_ERR_SHAPE;
  if (dh == 32) return fa_bwd_launch<32>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s);
  if (dh == 64) return fa_bwd_launch<64>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s);
  if (dh == 128) return fa_bwd_launch<128>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s);
  return PCM_ERR_SHAPE;
}

}  // namespace pcm
