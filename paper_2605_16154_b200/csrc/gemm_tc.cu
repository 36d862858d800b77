// bf16 GEMM on the 5th-generation tensor cores: TMA (cp.async.bulk.tensor) fills a shared-memory
// ring with 128-byte-swizzled operand tiles, one thread issues tcgen05.mma with the fp32
// accumulator in tensor memory, and four epilogue warps read it back with tcgen05.ld.
//
//   C[m][n] = sum_k A(m,k) B(n,k) (+ R[m][n])      store as bf16 / fp32, or
//   C[m][n] += sum_k A(m,k) B(n,k)                  fp32 reduction (weight gradients, split along k)
//
// Either operand may be K-major (contraction index contiguous in memory) or MN-major (the other
// index contiguous); the layout enters through the tensor map, the shared-memory descriptor and
// one bit of the instruction descriptor, so forward, input-gradient and weight-gradient GEMMs
// are the same kernel.
//
// Persistent: one CTA per SM walks a static list of output tiles; the shared-memory ring keeps
// flowing across tile boundaries and the accumulator is double-buffered in tensor memory, so the
// epilogue of one tile overlaps the MMAs of the next.
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = tensor-memory allocation + MMA issue,
// warps 2..9 = epilogue (two per tensor-memory lane quadrant, splitting the tile's columns).  Every mbarrier wait is bounded; when one runs out the CTA sets a status
// flag, all roles leave their loops, tensor memory is released and the kernel returns.
#include <cuda.h>

#include <cstdlib>

#include "async_ptx.cuh"
#include "internal.h"

namespace pcm {

constexpr int TC_BM = 128;
constexpr int TC_BK = 64;                     // 64 bf16 = one 128-byte swizzle row
// Ring depth of the single-CTA kernel: as deep as shared memory allows.  Its launches are the narrow or short GEMMs
// (adapter products, the head), which are bound by getting their A operand out of HBM: bytes in flight, not MMAs.
template <int BN> constexpr int tc_stages() { return BN == 128 ? 5 : 3; }
constexpr int TC_EPI_WARPS = 8;                // two per tensor-memory lane quadrant, each takes half of the columns
constexpr int EPI_STAGE_STRIDE = 36;            // floats per staged epilogue row (32 + 4 of padding: conflict free)
constexpr int EPI_STAGE_FLOATS = 32 * EPI_STAGE_STRIDE;   // per epilogue warp
constexpr int EPI_STAGE_BYTES = TC_EPI_WARPS * EPI_STAGE_FLOATS * 4;
constexpr int TC_THREADS = 320;               // producer warp, MMA warp, 8 epilogue warps
constexpr unsigned long long TC_WAIT_LIMIT_NS = 2000000000ull;   // 2 s per mbarrier wait

__device__ unsigned g_tc_status = 0;          // bit 0: a bounded wait expired

struct TcParams {
  int M, N, K;
  int kb_per_split;                           // k-blocks of 64 handled by one split of the contraction
  int tiles_m, tiles_n, splits;
  void* C; long long ldc; int c_dtype;        // DT_BF16 / DT_F32
  const float* R; long long ldr;
  int reduce;                                 // 1: fp32 reduction into C
  int a_kmajor, b_kmajor;
  // fused epilogues (see GemmEpilogue)
  const __nv_bfloat16* aux; long long ld_aux;
  __nv_bfloat16* out2; long long ld_out2;
  const float2* rope_tab; int S, dh, d;
  int up_row0;                                // EPI_SWIGLU_FWD: first "up" row of B (= F)
  HeadLossArgs hl;                            // EPI_HEAD_LOSS
  int kb_main;                                // k-blocks taken from the first operand pair; later ones come from the second
  int kb_total;                               // all k-blocks of the contraction (first pair + continuation)
  int ext_ksteps;                             // MMAs of 16 k-columns in a k-block of the continuation (K2 / 16)
  float alpha;                                // scale of the product in the plain store epilogue
};

__device__ __forceinline__ void store_bf16x32(__nv_bfloat16* dst, const float (&v)[32]) {
  uint4* d4 = reinterpret_cast<uint4*>(dst);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    __nv_bfloat162 h0 = __floats2bfloat162_rn(v[8 * e], v[8 * e + 1]);
    __nv_bfloat162 h1 = __floats2bfloat162_rn(v[8 * e + 2], v[8 * e + 3]);
    __nv_bfloat162 h2 = __floats2bfloat162_rn(v[8 * e + 4], v[8 * e + 5]);
    __nv_bfloat162 h3 = __floats2bfloat162_rn(v[8 * e + 6], v[8 * e + 7]);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
    o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
    d4[e] = o;
  }
}
__device__ __forceinline__ void fetch_bf16x32(const __nv_bfloat16* src, uint4 (&raw)[4]) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int e = 0; e < 4; ++e) raw[e] = s4[e];
}
__device__ __forceinline__ void unpack_bf16x32(const uint4 (&raw)[4], float (&v)[32]) {
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw[e]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h[j]);
      v[8 * e + 2 * j] = f.x; v[8 * e + 2 * j + 1] = f.y;
    }
  }
}
__device__ __forceinline__ void load_bf16x32(const __nv_bfloat16* src, float (&v)[32]) {
  const uint4* s4 = reinterpret_cast<const uint4*>(src);
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const uint4 raw = s4[e];
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h[j]);
      v[8 * e + 2 * j] = f.x; v[8 * e + 2 * j + 1] = f.y;
    }
  }
}

// Shared-memory matrix descriptor (tcgen05): start address, leading / stride byte offsets in
// 16-byte units, descriptor version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;                     // version
  d |= (uint64_t)2 << 61;                     // SWIZZLE_128B
  return d;
}

// Instruction descriptor for kind::f16: fp32 accumulator, bf16 A and B, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

template <int BN>
struct TcSmem {
  static constexpr int A_BYTES = TC_BM * TC_BK * 2;           // 16 KB
  static constexpr int B_BYTES = BN * TC_BK * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int STAGES = tc_stages<BN>();
  static constexpr int TOTAL = STAGES * STAGE_BYTES + 1024 /* alignment slack */ + 256 /* barriers */ + EPI_STAGE_BYTES;
  static_assert(TOTAL <= 227 * 1024, "shared-memory plan does not fit");
};

// The plain epilogue stores through a per-warp shared-memory buffer: tcgen05.ld hands every thread one row
// of 32 columns, the buffer turns that into "a quarter warp per row" so that each global access of a warp
// covers whole 128-byte (fp32) or 64-byte (bf16) row segments instead of 32 scattered rows.

// fp32 output: pass i covers rows 4i .. 4i+3, lane -> (row 4i + lane/8, columns 4 (lane%8) ..)
// bf16 output: pass i covers rows 8i .. 8i+7, lane -> (row 8i + lane/4, columns 8 (lane%4) ..)
__device__ __forceinline__ void fetch_residual(const TcParams& p, int row_base, int col, int lane, float4 (&r)[8]) {
  if (p.c_dtype == DT_F32) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int gr = row_base + i * 4 + (lane >> 3);
      if (gr < p.M) r[i] = *reinterpret_cast<const float4*>(p.R + (long long)gr * p.ldr + col + (lane & 7) * 4);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int gr = row_base + i * 8 + (lane >> 2);
      if (gr < p.M) {
        const float4* q = reinterpret_cast<const float4*>(p.R + (long long)gr * p.ldr + col + (lane & 3) * 8);
        r[2 * i] = q[0];
        r[2 * i + 1] = q[1];
      }
    }
  }
}

// Row layout (thread = row, 32 fp32 columns) -> bf16 rows in global memory, an eighth of a warp per row.
__device__ __forceinline__ void staged_store_bf16(float* stage, int lane, const float (&v)[32], __nv_bfloat16* C,
                                                  long long ldc, int row_base, int M, int col) {
  float* srow = stage + lane * EPI_STAGE_STRIDE;
#pragma unroll
  for (int e = 0; e < 8; ++e) *reinterpret_cast<float4*>(srow + 4 * e) = make_float4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = i * 8 + (lane >> 2), gr = row_base + r;
    const float* sp = stage + r * EPI_STAGE_STRIDE + (lane & 3) * 8;
    const float4 a = *reinterpret_cast<const float4*>(sp), b = *reinterpret_cast<const float4*>(sp + 4);
    __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
    __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
    uint4 o;
    o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
    o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
    if (gr < M) *reinterpret_cast<uint4*>(C + (long long)gr * ldc + col + (lane & 3) * 8) = o;
  }
  __syncwarp();
}
// 32 rows x 32 bf16 columns fetched with an eighth of a warp per row (kept in that layout until used)
__device__ __forceinline__ void fetch_bf16_rows(const __nv_bfloat16* A, long long ld, int row_base, int M, int col, int lane,
                                                uint4 (&o)[4]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gr = row_base + i * 8 + (lane >> 2);
    o[i] = gr < M ? *reinterpret_cast<const uint4*>(A + (long long)gr * ld + col + (lane & 3) * 8) : make_uint4(0, 0, 0, 0);
  }
}
// ... and turned into the row layout (thread = row) through the staging buffer
__device__ __forceinline__ void unstage_bf16_rows(float* stage, int lane, const uint4 (&o)[4], float (&v)[32]) {
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float* sp = stage + (i * 8 + (lane >> 2)) * EPI_STAGE_STRIDE + (lane & 3) * 8;
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&o[i]);
    const float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
    const float2 f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
    *reinterpret_cast<float4*>(sp) = make_float4(f0.x, f0.y, f1.x, f1.y);
    *reinterpret_cast<float4*>(sp + 4) = make_float4(f2.x, f2.y, f3.x, f3.y);
  }
  __syncwarp();
  const float* srow = stage + lane * EPI_STAGE_STRIDE;
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float4 t = *reinterpret_cast<const float4*>(srow + 4 * e);
    v[4 * e] = t.x; v[4 * e + 1] = t.y; v[4 * e + 2] = t.z; v[4 * e + 3] = t.w;
  }
  __syncwarp();
}

// Row layout (thread = row, 32 fp32 columns, raw tcgen05.ld registers) into the staging buffer ...
__device__ __forceinline__ void stage_put_rows(float* stage, int lane, const uint32_t (&r)[32]) {
  float* srow = stage + lane * EPI_STAGE_STRIDE;
#pragma unroll
  for (int e = 0; e < 8; ++e) *reinterpret_cast<uint4*>(srow + 4 * e) = make_uint4(r[4 * e], r[4 * e + 1], r[4 * e + 2], r[4 * e + 3]);
}
// ... and back out as 8 consecutive columns of row 8 i + lane / 4 (the layout of fetch_bf16_rows / bf16 stores)
__device__ __forceinline__ void stage_get8(const float* stage, int lane, int i, float (&v)[8]) {
  const float* sp = stage + (i * 8 + (lane >> 2)) * EPI_STAGE_STRIDE + (lane & 3) * 8;
  const float4 a = *reinterpret_cast<const float4*>(sp), b = *reinterpret_cast<const float4*>(sp + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ uint4 pack8_bf16(const float (&v)[8]) {
  __nv_bfloat162 h0 = __floats2bfloat162_rn(v[0], v[1]), h1 = __floats2bfloat162_rn(v[2], v[3]);
  __nv_bfloat162 h2 = __floats2bfloat162_rn(v[4], v[5]), h3 = __floats2bfloat162_rn(v[6], v[7]);
  uint4 o;
  o.x = *reinterpret_cast<uint32_t*>(&h0); o.y = *reinterpret_cast<uint32_t*>(&h1);
  o.z = *reinterpret_cast<uint32_t*>(&h2); o.w = *reinterpret_cast<uint32_t*>(&h3);
  return o;
}
__device__ __forceinline__ void unpack8_bf16(const uint4& raw, float (&v)[8]) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __bfloat1622float2(h[j]);
    v[2 * j] = f.x; v[2 * j + 1] = f.y;
  }
}

// Operands of the epilogue that are fetched one 32-column slice ahead of their use.
struct EpiRegs {
  uint4 g[4], u[4];                           // EPI_SWIGLU_BWD: gate / up
  float4 r[8];                                // fp32 residual
};

// Issued before the wait for the accumulator, so that the first slice's loads overlap it.
template <int BN, int EPI>
__device__ __forceinline__ void epi_prefetch(const TcParams& p, int row, int n0, int chalf, EpiRegs& pre) {
  const int lane_ = threadIdx.x & 31;
      if constexpr (EPI == EPI_SWIGLU_BWD) {
        const int col0 = n0 + chalf * (BN / 2);
        if (col0 < p.N) {                     // issued before waiting for the accumulator
          fetch_bf16_rows(p.aux, p.ld_aux, row - lane_, p.M, col0, lane_, pre.g);
          fetch_bf16_rows(p.aux + p.N, p.ld_aux, row - lane_, p.M, col0, lane_, pre.u);
        }
      }
      if constexpr (EPI == EPI_NONE) {
        const int col0 = n0 + chalf * (BN / 2);
        if (p.R && !p.reduce && col0 < p.N) fetch_residual(p, row - lane_, col0, lane_, pre.r);
      }
}

// One epilogue warp's share of a tile: rows = this warp's 32 tensor-memory lanes, columns = its half of the tile.
template <int BN, int EPI>
__device__ __forceinline__ void epi_tile(const TcParams& p, uint32_t tmem_acc, int row, int n0, int chalf, EpiRegs& pre,
                                         float* stage) {
  const int lane_ = threadIdx.x & 31;
      if constexpr (EPI == EPI_HEAD_LOSS) {
        // The tile is 128 scored rows x the whole 256-bin vocabulary.  One thread owns one row (the warps of the
        // first column half take all 256 columns, so no statistics cross warps) and reads it from tensor memory
        // three times: maximum; sum of exponentials, entropy sum and the target's logit; gradient.
        static_assert(BN == 256, "a row's vocabulary is one accumulator tile");
        if (chalf != 0) return;
        const HeadLossArgs& h = p.hl;
        const bool valid = row < p.M;
        const int t = valid ? (int)h.tgt[row] : -1;
        uint32_t r[32];
        float mx = -3.0e38f;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          tmem_ld_32x32(tmem_acc + (uint32_t)c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) mx = fmaxf(mx, __uint_as_float(r[e]));
        }
        RowStats st{mx, 0.f, 0.f};
        float zt = 0.f;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          tmem_ld_32x32(tmem_acc + (uint32_t)c0, r);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float z = __uint_as_float(r[e]);
            const float ex = expf(z - mx);
            st.se += ex;
            st.sz += ex * (z - mx);
            zt = (c0 + e == t) ? z : zt;
          }
        }
        const float lse = hl_lse(st), ent = hl_entropy(st), logp = zt - lse;
        RowTerms tm{0.f, 0.f, 0.f, 0.f};
        if (valid) {
          if (h.mode == HL_TOKEN) tm = hl_token_terms(logp, h.lpo[row], h.adv_c[row / PCM_ACT_DIM], h.lo, h.hi, h.loss_scale);
          else if (h.mode == HL_COEF) tm.dlogp = h.coef[row];
          if (h.logp && h.mode != HL_COEF) h.logp[row] = logp;
        }
        if (h.part) {
          float s0 = tm.surrogate, s1 = tm.clipped, s2 = tm.ratio, s3 = valid ? ent : 0.f;
#pragma unroll
          for (int off = 16; off; off >>= 1) {
            s0 += __shfl_xor_sync(0xffffffffu, s0, off); s1 += __shfl_xor_sync(0xffffffffu, s1, off);
            s2 += __shfl_xor_sync(0xffffffffu, s2, off); s3 += __shfl_xor_sync(0xffffffffu, s3, off);
          }
          if (lane_ == 0)
            *reinterpret_cast<float4*>(h.part + ((long long)(row >> 5)) * 4) = make_float4(s0, s1, s2, s3);   // one entry per 32 rows
        }
        if (h.want_dz) {
          __nv_bfloat16* dz = reinterpret_cast<__nv_bfloat16*>(p.C);
#pragma unroll 1
          for (int c0 = 0; c0 < BN; c0 += 32) {
            tmem_ld_32x32(tmem_acc + (uint32_t)c0, r);
            tmem_ld_wait();
            float v[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) v[e] = hl_dz(__uint_as_float(r[e]), lse, ent, tm.dlogp, h.ent_scale, c0 + e == t);
            staged_store_bf16(stage, lane_, v, dz, p.ldc, row - lane_, p.M, n0 + c0);
          }
        }
      } else if constexpr (EPI == EPI_SWIGLU_FWD) {
        // accumulator columns [0,128) = gate, [128,256) = up, for hidden units hid0 .. hid0+127
        const int hid0 = n0 / 2, F = p.up_row0;
#pragma unroll 1
        for (int c0 = chalf * 64; c0 < chalf * 64 + 64; c0 += 32) {
          if (hid0 + c0 >= F) break;
          uint32_t rg[32], ru[32];
          tmem_ld_32x32(tmem_acc + (uint32_t)c0, rg);
          tmem_ld_32x32(tmem_acc + (uint32_t)(128 + c0), ru);
          tmem_ld_wait();
          {
            // gate and up go through the staging buffer one after the other; the activation is formed and all
            // three tensors are stored in the "eighth of a warp per row" layout
            const int row_base = row - lane_;
            float gq[4][8];
            stage_put_rows(stage, lane_, rg);
            __syncwarp();
#pragma unroll
            for (int i = 0; i < 4; ++i) stage_get8(stage, lane_, i, gq[i]);
            __syncwarp();
            stage_put_rows(stage, lane_, ru);
            __syncwarp();
            __nv_bfloat16* gu = reinterpret_cast<__nv_bfloat16*>(p.C);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              float u[8];
              stage_get8(stage, lane_, i, u);
              const int gr = row_base + i * 8 + (lane_ >> 2);
              const uint4 pg = pack8_bf16(gq[i]), pu = pack8_bf16(u);
#pragma unroll
              for (int e = 0; e < 8; ++e) u[e] = __fdividef(gq[i][e], 1.f + __expf(-gq[i][e])) * u[e];
              if (gr < p.M) {
                __nv_bfloat16* dst = gu + (long long)gr * p.ldc + hid0 + c0 + (lane_ & 3) * 8;
                *reinterpret_cast<uint4*>(dst) = pg;
                *reinterpret_cast<uint4*>(dst + F) = pu;
                *reinterpret_cast<uint4*>(p.out2 + (long long)gr * p.ld_out2 + hid0 + c0 + (lane_ & 3) * 8) = pack8_bf16(u);
              }
            }
            __syncwarp();
          }
        }
      } else if constexpr (EPI == EPI_ROPE) {
        // every head of a row uses the same (cos, sin) values: load them once per 32-pair slice and
        // reuse them for all heads of this warp's half of the tile
        const int half = p.dh / 2;
        const int pos = row % p.S;
#pragma unroll 1
        for (int ic = 0; ic < half; ic += 32) {
          float2 cs[32];
          {
            const float4* tp = reinterpret_cast<const float4*>(p.rope_tab + (long long)pos * half + ic);
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float4 t4 = tp[e];
              cs[2 * e] = make_float2(t4.x, t4.y);
              cs[2 * e + 1] = make_float2(t4.z, t4.w);
            }
          }
#pragma unroll 1
          for (int h0 = chalf * (BN / 2); h0 < (chalf + 1) * (BN / 2); h0 += p.dh) {   // heads inside this warp's half
            if (n0 + h0 >= p.N) break;
            const bool rotate = n0 + h0 < 2 * p.d;        // q and k regions; v passes through
            uint32_t rl[32], rh[32];
            tmem_ld_32x32(tmem_acc + (uint32_t)(h0 + ic), rl);
            tmem_ld_32x32(tmem_acc + (uint32_t)(h0 + half + ic), rh);
            tmem_ld_wait();
            {
              float lo[32], hi[32];
#pragma unroll
              for (int e = 0; e < 32; ++e) { lo[e] = __uint_as_float(rl[e]); hi[e] = __uint_as_float(rh[e]); }
              if (rotate) {
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  const float x = lo[e], y = hi[e];
                  lo[e] = x * cs[e].x - y * cs[e].y;
                  hi[e] = y * cs[e].x + x * cs[e].y;
                }
              }
              __nv_bfloat16* Cb = reinterpret_cast<__nv_bfloat16*>(p.C);
              staged_store_bf16(stage, lane_, lo, Cb, p.ldc, row - lane_, p.M, n0 + h0 + ic);
              staged_store_bf16(stage, lane_, hi, Cb, p.ldc, row - lane_, p.M, n0 + h0 + ic + half);
            }
          }
        }
      } else {
#pragma unroll 1
      for (int c0 = chalf * (BN / 2); c0 < (chalf + 1) * (BN / 2); c0 += 32) {
        const int col = n0 + c0;
        if (col >= p.N) break;                // warp-uniform: N is a multiple of 32 on this path
        uint32_t r[32];
        tmem_ld_32x32(tmem_acc + (uint32_t)c0, r);
        tmem_ld_wait();
        if constexpr (EPI == EPI_SWIGLU_BWD) {
          // r = d(act) in fp32 goes through the staging buffer into the "eighth of a warp per row" layout, where
          // gate | up (fetched one slice ahead in that layout) are combined with it and d(gate) | d(up) are stored
          const int F = p.N, row_base = row - lane_;
          stage_put_rows(stage, lane_, r);
          __syncwarp();
          uint4 og[4], ou[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            float da[8], g[8], u[8];
            stage_get8(stage, lane_, i, da);
            unpack8_bf16(pre.g[i], g);
            unpack8_bf16(pre.u[i], u);
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const float sg = __fdividef(1.f, 1.f + __expf(-g[e]));
              const float dg = da[e] * u[e] * sg * (1.f + g[e] * (1.f - sg));
              u[e] = da[e] * g[e] * sg;
              g[e] = dg;
            }
            og[i] = pack8_bf16(g);
            ou[i] = pack8_bf16(u);
          }
          __syncwarp();
          if (c0 + 32 < (chalf + 1) * (BN / 2) && col + 32 < p.N) {
            fetch_bf16_rows(p.aux, p.ld_aux, row_base, p.M, col + 32, lane_, pre.g);
            fetch_bf16_rows(p.aux + F, p.ld_aux, row_base, p.M, col + 32, lane_, pre.u);
          }
          __nv_bfloat16* Cb = reinterpret_cast<__nv_bfloat16*>(p.C);
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int gr = row_base + i * 8 + (lane_ >> 2);
            if (gr < p.M) {
              __nv_bfloat16* dst = Cb + (long long)gr * p.ldc + col + (lane_ & 3) * 8;
              *reinterpret_cast<uint4*>(dst) = og[i];
              *reinterpret_cast<uint4*>(dst + F) = ou[i];
            }
          }
        } else if (p.reduce) {
          if (row < p.M) {
            float* dst = reinterpret_cast<float*>(p.C) + (long long)row * p.ldc + col;
#pragma unroll
            for (int e = 0; e < 32; e += 4)
              red_add_v4(dst + e, __uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                         __uint_as_float(r[e + 3]));
          }
        } else {
          // stage the 32 x 32 slice (thread = row), then store it with a quarter (or eighth) warp per row
          float* srow = stage + lane_ * EPI_STAGE_STRIDE;
#pragma unroll
          for (int e = 0; e < 8; ++e)
            *reinterpret_cast<uint4*>(srow + 4 * e) = make_uint4(r[4 * e], r[4 * e + 1], r[4 * e + 2], r[4 * e + 3]);
          __syncwarp();
          const int row_base = row - lane_;
          const bool more = c0 + 32 < (chalf + 1) * (BN / 2) && col + 32 < p.N;
          if (p.c_dtype == DT_F32) {
            float4 v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              v[i] = *reinterpret_cast<const float4*>(stage + (i * 4 + (lane_ >> 3)) * EPI_STAGE_STRIDE + (lane_ & 7) * 4);
              if (p.alpha != 1.f) { v[i].x *= p.alpha; v[i].y *= p.alpha; v[i].z *= p.alpha; v[i].w *= p.alpha; }
              if (p.R) { v[i].x += pre.r[i].x; v[i].y += pre.r[i].y; v[i].z += pre.r[i].z; v[i].w += pre.r[i].w; }
            }
            if (p.R && more) fetch_residual(p, row_base, col + 32, lane_, pre.r);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int gr = row_base + i * 4 + (lane_ >> 3);
              if (gr < p.M)
                *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.C) + (long long)gr * p.ldc + col + (lane_ & 7) * 4) = v[i];
            }
          } else {
            uint4 o[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float* sp = stage + (i * 8 + (lane_ >> 2)) * EPI_STAGE_STRIDE + (lane_ & 3) * 8;
              float4 a = *reinterpret_cast<const float4*>(sp), b = *reinterpret_cast<const float4*>(sp + 4);
              if (p.alpha != 1.f) {
                a.x *= p.alpha; a.y *= p.alpha; a.z *= p.alpha; a.w *= p.alpha;
                b.x *= p.alpha; b.y *= p.alpha; b.z *= p.alpha; b.w *= p.alpha;
              }
              if (p.R) {
                a.x += pre.r[2 * i].x; a.y += pre.r[2 * i].y; a.z += pre.r[2 * i].z; a.w += pre.r[2 * i].w;
                b.x += pre.r[2 * i + 1].x; b.y += pre.r[2 * i + 1].y; b.z += pre.r[2 * i + 1].z; b.w += pre.r[2 * i + 1].w;
              }
              __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
              __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
              o[i].x = *reinterpret_cast<uint32_t*>(&h0); o[i].y = *reinterpret_cast<uint32_t*>(&h1);
              o[i].z = *reinterpret_cast<uint32_t*>(&h2); o[i].w = *reinterpret_cast<uint32_t*>(&h3);
            }
            if (p.R && more) fetch_residual(p, row_base, col + 32, lane_, pre.r);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int gr = row_base + i * 8 + (lane_ >> 2);
              if (gr < p.M)
                *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.C) + (long long)gr * p.ldc + col + (lane_ & 3) * 8) = o[i];
            }
          }
          __syncwarp();                       // the buffer is free again for the next slice
        }
      }
      }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  using SM = TcSmem<BN>;
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* tiles = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);       // swizzle atoms need 1024-byte alignment
  constexpr int TC_STAGES = SM::STAGES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + TC_STAGES * SM::STAGE_BYTES);
  uint64_t* full = bars;                      // [TC_STAGES] producer -> MMA
  uint64_t* empty = bars + TC_STAGES;         // [TC_STAGES] MMA -> producer
  uint64_t* acc_full = bars + 2 * TC_STAGES;  // [2] MMA -> epilogue, one per accumulator buffer
  uint64_t* acc_empty = acc_full + 2;         // [2] epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* epi_stage = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int num_kb_total = p.kb_total;
  const int tiles_mn = p.tiles_m * p.tiles_n;
  const int total_tiles = tiles_mn * p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < TC_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], TC_EPI_WARPS); }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 2 * BN);            // two accumulator buffers: the epilogue of one tile overlaps the next tile's MMAs
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Tiles are walked in the same order by every role: tile -> (split, m, n) with n fastest, so that
  // CTAs running at the same time share A row-tiles and the whole B operand stays in L2.
  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------ TMA producer ------------------------------
      unsigned it = 0;                        // k-blocks issued so far, across tiles
      for (int tile = blockIdx.x; tile < total_tiles && !*abort_flag; tile += gridDim.x) {
        const int split = tile / tiles_mn, mn = tile - split * tiles_mn;
        const int m0 = (mn / p.tiles_n) * TC_BM, n0 = (mn % p.tiles_n) * BN;
        const int kb_lo = split * p.kb_per_split, kb_hi = min(kb_lo + p.kb_per_split, num_kb_total);
        for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
          const int st = it % TC_STAGES;
          const unsigned ph = (it / TC_STAGES) & 1u;
          if (!mbar_wait_bounded(&empty[st], ph ^ 1u, TC_WAIT_LIMIT_NS)) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); break; }
          uint8_t* sa = tiles + st * SM::STAGE_BYTES;
          uint8_t* sb = sa + SM::A_BYTES;
          mbar_expect_tx(&full[st], SM::STAGE_BYTES);
          const bool ext = kb >= p.kb_main;                               // continuation: second operand pair
          const CUtensorMap* mA = ext ? &tmA2 : &tmA;
          const CUtensorMap* mB = ext ? &tmB2 : &tmB;
          const int k0 = (ext ? kb - p.kb_main : kb) * TC_BK;
          if (p.a_kmajor) {
            tma_load_2d(sa, mA, k0, m0, &full[st]);                       // box {64 k, 128 m}
          } else {
#pragma unroll
            for (int b = 0; b < TC_BM / 64; ++b) tma_load_2d(sa + b * 8192, mA, m0 + b * 64, k0, &full[st]);  // box {64 m, 64 k}
          }
          if (EPI == EPI_SWIGLU_FWD) {
            // n0 counts accumulator columns (256 per tile = 128 hidden units): gate rows, then the matching up rows
            tma_load_2d(sb, mB, k0, n0 / 2, &full[st]);                   // box {64 k, 128 n}
            tma_load_2d(sb + 128 * 128, mB, k0, p.up_row0 + n0 / 2, &full[st]);
          } else if (p.b_kmajor) {
            tma_load_2d(sb, mB, k0, n0, &full[st]);                       // box {64 k, BN n}
          } else {
#pragma unroll
            for (int b = 0; b < BN / 64; ++b) tma_load_2d(sb + b * 8192, mB, n0 + b * 64, k0, &full[st]);
          }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------ MMA issuer ------------------------------
      const uint32_t idesc = make_idesc(BN, p.a_kmajor ? 0 : 1, p.b_kmajor ? 0 : 1);
      // K-major tile: rows of 128 B, 8-row groups 1024 B apart; a k-step of 16 elements is 32 B along the row.
      // MN-major tile: boxes of 64 (mn) x 64 (k): k-rows of 128 B, 8-row groups 1024 B apart, next 64 mn 8192 B on;
      //                a k-step of 16 rows is 2048 B.
      const uint32_t a_lbo = p.a_kmajor ? 16u : 8192u, b_lbo = p.b_kmajor ? 16u : 8192u;
      const uint32_t a_step = p.a_kmajor ? 32u : 2048u, b_step = p.b_kmajor ? 32u : 2048u;
      unsigned it = 0, tcount = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
        const int split = tile / tiles_mn;
        const int kb_lo = split * p.kb_per_split, kb_hi = min(kb_lo + p.kb_per_split, num_kb_total);
        const unsigned ab = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (*abort_flag || !mbar_wait_bounded(&acc_empty[ab], aph ^ 1u, TC_WAIT_LIMIT_NS)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + ab * BN;
        for (int kb = kb_lo; kb < kb_hi; ++kb, ++it) {
          const int st = it % TC_STAGES;
          const unsigned ph = (it / TC_STAGES) & 1u;
          if (*abort_flag || !mbar_wait_bounded(&full[st], ph, TC_WAIT_LIMIT_NS)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(tiles + st * SM::STAGE_BYTES);
          const uint32_t sb = sa + SM::A_BYTES;
          const int ksteps = kb >= p.kb_main ? p.ext_ksteps : TC_BK / 16;   // the continuation may be narrower than 64
#pragma unroll
          for (int k = 0; k < TC_BK / 16; ++k) {
            if (k >= ksteps) break;
            const uint64_t da = make_smem_desc(sa + k * a_step, a_lbo, 1024u);
            const uint64_t db = make_smem_desc(sb + k * b_step, b_lbo, 1024u);
            umma_bf16(tmem_acc, da, db, idesc, (kb > kb_lo || k > 0) ? 1u : 0u);
          }
          umma_commit(&empty[st]);            // frees the stage once the MMAs above have read it
        }
        if (ok) umma_commit(&acc_full[ab]);
      }
      if (!ok) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); }
    }
  } else {
    // ------------------------------ epilogue: warps 2..9 ------------------------------
    const int quad = warp & 3;                // tensor-memory lane quadrant this warp may access
    const int chalf = (warp - 2) >> 2;        // which half of the tile's columns this warp handles
    unsigned tcount = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tcount) {
      const int split = tile / tiles_mn, mn = tile - split * tiles_mn;
      const int m0 = (mn / p.tiles_n) * TC_BM, n0 = (mn % p.tiles_n) * BN;
      const int row = m0 + quad * 32 + lane;
      const unsigned ab = tcount & 1u, aph = (tcount >> 1) & 1u;
      EpiRegs pre;
      epi_prefetch<BN, EPI>(p, row, n0, chalf, pre);
      int ok = 1;
      if (lane == 0) {
        ok = (!*abort_flag && mbar_wait_bounded(&acc_full[ab], aph, TC_WAIT_LIMIT_NS * 2ull)) ? 1 : 0;
        if (!ok) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tmem_acc = tmem_base + ab * BN + ((uint32_t)(quad * 32) << 16);
      epi_tile<BN, EPI>(p, tmem_acc, row, n0, chalf, pre, epi_stage + (warp - 2) * EPI_STAGE_FLOATS);
      // hand the accumulator buffer back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[ab]);
    }
  }

  // teardown: on the abort path give copies still in flight time to land before shared memory is released
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant: two CTAs of a cluster share one 256 x 256 output tile.  Each CTA stages its own
// 128 rows of A and one half (128 of the 256 columns) of B, so every byte of B is read into shared
// memory once per pair instead of once per CTA; the leader CTA issues tcgen05.mma.cta_group::2 and
// each CTA's tensor memory receives the accumulator rows of its half of the tile.
//   full[s]      (leader)  <- both producers' TMA bytes + the leader producer's arrival
//   empty[s]     (each)    <- multicast commit from the leader's MMA thread
//   acc_full[b]  (each)    <- multicast commit from the leader's MMA thread
//   acc_empty[b] (leader)  <- the epilogue warps of both CTAs
// ------------------------------------------------------------------------------------------------
// Position of a CTA pair's current tile in the (split, m, n) grid, n fastest, advanced by a fixed stride without
// divisions: the stride is decomposed once.
struct TileWalk {
  int split, m, n, d_split, d_m, d_n;
  __device__ void init(int first, int stride, int tiles_m, int tiles_n) {
    const int tiles_mn = tiles_m * tiles_n;
    split = first / tiles_mn;
    int r = first - split * tiles_mn;
    m = r / tiles_n; n = r - m * tiles_n;
    d_split = stride / tiles_mn;
    r = stride - d_split * tiles_mn;
    d_m = r / tiles_n; d_n = r - d_m * tiles_n;
  }
  __device__ void next(int tiles_m, int tiles_n) {
    n += d_n;
    if (n >= tiles_n) { n -= tiles_n; ++m; }
    m += d_m;
    if (m >= tiles_m) { m -= tiles_m; ++split; }
    split += d_split;
  }
};

constexpr int T2_BN = 256;
constexpr int T2_STAGES = 5;
constexpr int T2_A_BYTES = TC_BM * TC_BK * 2;          // 16 KB: this CTA's 128 rows of A
constexpr int T2_B_BYTES = (T2_BN / 2) * TC_BK * 2;    // 16 KB: this CTA's 128 columns of B
constexpr int T2_STAGE_BYTES = T2_A_BYTES + T2_B_BYTES;
constexpr int T2_PRODUCER_B_WARP = 10;               // after the eight epilogue warps 2..9
constexpr int T2_THREADS = TC_THREADS + 32;
constexpr int T2_SMEM_TOTAL = T2_STAGES * T2_STAGE_BYTES + 1024 + 256 + EPI_STAGE_BYTES;   // ring + slack + barriers + epilogue staging

template <int EPI>
__global__ void __launch_bounds__(T2_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2, const TcParams p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int BN = T2_BN;
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* tiles = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + T2_STAGES * T2_STAGE_BYTES);
  uint64_t* full = bars;                       // [T2_STAGES]
  uint64_t* empty = bars + T2_STAGES;          // [T2_STAGES]
  uint64_t* acc_full = bars + 2 * T2_STAGES;   // [2]
  uint64_t* acc_empty = acc_full + 2;          // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* epi_stage = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(bars) + 256);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int num_kb_total = p.kb_total;
  const int tiles_mn = p.tiles_m * p.tiles_n;  // tiles of 256 x 256
  const int total_tiles = tiles_mn * p.splits;

  if (threadIdx.x == 0) {
    for (int s = 0; s < T2_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 2 * TC_EPI_WARPS); }
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc_pair(tmem_slot, 2 * BN);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                          // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == T2_PRODUCER_B_WARP) {
    if (lane == 0) {
      // ------------------------------ TMA producers (both CTAs) ------------------------------
      // Two threads per CTA, one per operand (warp 0: A, warp 10: B): a TMA issue costs its thread about a hundred
      // cycles, and a k-block must cost each producer well under the 512 tensor-core cycles it feeds.  Ring positions
      // and the tile walk are counters (no division or modulo per k-block).
      const bool load_a = warp == 0;
      const uint32_t bar0 = mapa_shared(smem_u32(&full[0]), 0);               // the leader's barriers count both CTAs' bytes
      TileWalk tw;
      tw.init(pair, n_pairs, p.tiles_m, p.tiles_n);
      int st = 0;
      unsigned ph = 0;
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok && !*abort_flag; tile += n_pairs, tw.next(p.tiles_m, p.tiles_n)) {
        const int m0 = tw.m * (2 * TC_BM) + (int)rank * TC_BM;                  // this CTA's rows
        const int n0 = tw.n * BN;
        const int nb0 = n0 + (int)rank * (BN / 2);                              // this CTA's columns of B
        const int kb_lo = tw.split * p.kb_per_split, kb_hi = min(kb_lo + p.kb_per_split, num_kb_total);
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          if (!mbar_wait_bounded(&empty[st], ph ^ 1u, TC_WAIT_LIMIT_NS)) { ok = false; break; }
          uint8_t* sa = tiles + st * T2_STAGE_BYTES;
          uint8_t* sb = sa + T2_A_BYTES;
          const uint32_t bar = bar0 + (uint32_t)st * 8u;
          const bool ext = kb >= p.kb_main;                                     // continuation: second operand pair
          const CUtensorMap* mA = ext ? &tmA2 : &tmA;
          const CUtensorMap* mB = ext ? &tmB2 : &tmB;
          const int k0 = (ext ? kb - p.kb_main : kb) * TC_BK;
          if (load_a) {
            if (leader) mbar_expect_tx(&full[st], 2 * T2_STAGE_BYTES);
            if (p.a_kmajor) {
              tma_load_2d_pair(sa, mA, k0, m0, bar);                            // box {64 k, 128 m}
            } else {
#pragma unroll
              for (int b = 0; b < 2; ++b) tma_load_2d_pair(sa + b * 8192, mA, m0 + b * 64, k0, bar);   // box {64 m, 64 k}
            }
          } else if (EPI == EPI_SWIGLU_FWD) {
            // accumulator columns [0,128) = gate (leader's half of B), [128,256) = up (the peer's half)
            tma_load_2d_pair(sb, mB, k0, (leader ? 0 : p.up_row0) + n0 / 2, bar);                   // box {64 k, 128 n}
          } else if (p.b_kmajor) {
            tma_load_2d_pair(sb, mB, k0, nb0, bar);                             // box {64 k, 128 n}
          } else {
#pragma unroll
            for (int b = 0; b < 2; ++b) tma_load_2d_pair(sb + b * 8192, mB, nb0 + b * 64, k0, bar);
          }
          if (++st == T2_STAGES) { st = 0; ph ^= 1u; }
        }
      }
      if (!ok) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // ------------------------------ MMA issuer (leader CTA only) ------------------------------
      // The four MMAs of a k-block take 512 tensor-core cycles; this thread must spend less than that per k-block
      // (a poll of an already completed barrier alone costs about 125 cycles).  Descriptors are therefore built once
      // and advanced by adding constants to their low word, and the ring position is a counter.
      constexpr uint32_t idesc_base = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) |
                                      ((uint32_t)((2 * TC_BM) >> 4) << 24);
      const uint32_t idesc = idesc_base | ((p.a_kmajor ? 0u : 1u) << 15) | ((p.b_kmajor ? 0u : 1u) << 16);
      const uint32_t a_lbo = p.a_kmajor ? 16u : 8192u, b_lbo = p.b_kmajor ? 16u : 8192u;
      const uint32_t a_step16 = (p.a_kmajor ? 32u : 2048u) >> 4, b_step16 = (p.b_kmajor ? 32u : 2048u) >> 4;
      const uint64_t da0 = make_smem_desc(smem_u32(tiles), a_lbo, 1024u);
      const uint64_t db0 = make_smem_desc(smem_u32(tiles) + T2_A_BYTES, b_lbo, 1024u);
      const uint32_t da_hi = (uint32_t)(da0 >> 32), db_hi = (uint32_t)(db0 >> 32);
      const uint32_t da_lo = (uint32_t)da0, db_lo = (uint32_t)db0;
      auto desc = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; };
      TileWalk tw;
      tw.init(pair, n_pairs, p.tiles_m, p.tiles_n);
      unsigned tcount = 0, ph = 0;
      int st = 0;
      uint32_t st_off = 0;                       // st * stage bytes, in descriptor units of 16 bytes
      bool ok = true;
      for (int tile = pair; tile < total_tiles && ok; tile += n_pairs, ++tcount, tw.next(p.tiles_m, p.tiles_n)) {
        const int kb_lo = tw.split * p.kb_per_split, kb_hi = min(kb_lo + p.kb_per_split, num_kb_total);
        const unsigned ab = tcount & 1u, aph = (tcount >> 1) & 1u;
        if (*abort_flag || !mbar_wait_bounded(&acc_empty[ab], aph ^ 1u, TC_WAIT_LIMIT_NS)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_acc = tmem_base + ab * BN;
        for (int kb = kb_lo; kb < kb_hi; ++kb) {
          if (!mbar_wait_bounded(&full[st], ph, TC_WAIT_LIMIT_NS)) { ok = false; break; }
          tc_fence_after();
          const uint32_t alo = da_lo + st_off, blo = db_lo + st_off;
          umma_bf16_pair(tmem_acc, desc(alo, da_hi), desc(blo, db_hi), idesc, kb > kb_lo ? 1u : 0u);
          if (kb < p.kb_main) {
#pragma unroll
            for (int k = 1; k < TC_BK / 16; ++k)
              umma_bf16_pair(tmem_acc, desc(alo + k * a_step16, da_hi), desc(blo + k * b_step16, db_hi), idesc, 1u);
          } else {                               // continuation block: K2 / 16 MMAs, the rest of the tile is zero fill
#pragma unroll 1
            for (int k = 1; k < p.ext_ksteps; ++k)
              umma_bf16_pair(tmem_acc, desc(alo + k * a_step16, da_hi), desc(blo + k * b_step16, db_hi), idesc, 1u);
          }
          umma_commit_pair(&empty[st], 3);     // both CTAs may refill the stage
          st_off += T2_STAGE_BYTES >> 4;
          if (++st == T2_STAGES) { st = 0; st_off = 0; ph ^= 1u; }
        }
        if (ok) umma_commit_pair(&acc_full[ab], 3);
      }
      if (!ok) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); }
    }
  } else {
    // ------------------------------ epilogue: warps 2..9 of both CTAs ------------------------------
    const int quad = warp & 3;
    const int chalf = (warp - 2) >> 2;
    unsigned tcount = 0;
    for (int tile = pair; tile < total_tiles; tile += n_pairs, ++tcount) {
      const int split = tile / tiles_mn, mn = tile - split * tiles_mn;
      const int m0 = (mn / p.tiles_n) * (2 * TC_BM) + (int)rank * TC_BM, n0 = (mn % p.tiles_n) * BN;
      const int row = m0 + quad * 32 + lane;
      const unsigned ab = tcount & 1u, aph = (tcount >> 1) & 1u;
      EpiRegs pre;
      epi_prefetch<BN, EPI>(p, row, n0, chalf, pre);
      int ok = 1;
      if (lane == 0) {
        ok = (!*abort_flag && mbar_wait_bounded(&acc_full[ab], aph, TC_WAIT_LIMIT_NS * 2ull)) ? 1 : 0;
        if (!ok) { *abort_flag = 1; atomicOr(&g_tc_status, 1u); }
      }
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) break;
      tc_fence_after();
      const uint32_t tmem_acc = tmem_base + ab * BN + ((uint32_t)(quad * 32) << 16);
      epi_tile<BN, EPI>(p, tmem_acc, row, n0, chalf, pre, epi_stage + (warp - 2) * EPI_STAGE_FLOATS);
      // hand the accumulator buffer back to the leader's MMA thread
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_shared(smem_u32(&acc_empty[ab]), 0));
    }
  }

  // teardown: neither CTA may leave while its peer can still touch its shared memory or barriers
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  cluster_sync_all();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 2 * BN);
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  }
  return fn;
}

// 2-D bf16 tensor [rows][cols] with row stride ld (elements); box {box_cols, box_rows}, 128-byte swizzle,
// out-of-range elements read as zero.
static bool make_tmap(CUtensorMap* tm, const void* base, long long rows, long long cols, long long ld, int box_cols,
                      int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_tcgen05_supported(const GemmArgs& g) {
  if (g.ab_dtype != DT_BF16) return false;
  if (g.M < 1 || g.N < 32 || g.K < 1 || (g.N % 32)) return false;
  if ((g.lda % 8) || (g.ldb % 8)) return false;
  if (((uintptr_t)g.A | (uintptr_t)g.B | (uintptr_t)g.C) & 15) return false;
  if (g.c_dtype == DT_BF16 && (g.ldc % 8)) return false;
  if (g.c_dtype == DT_F32 && (g.ldc % 4)) return false;
  if (g.R && (((uintptr_t)g.R & 15) || (g.ldr % 4))) return false;
  if (g.R && (const void*)g.R == (const void*)g.C && g.c_dtype != DT_F32) return false;
  if (g.K2 < 0 || g.K2 > TC_BK || (g.K2 % 16)) return false;
  if (g.K2 > 0 && (!g.A2 || !g.B2 || (g.lda2 % 8) || (g.ldb2 % 8) || (((uintptr_t)g.A2 | (uintptr_t)g.B2) & 15))) return false;
  if (g.alpha != 1.f && (g.epi.kind != EPI_NONE || (g.R && (const void*)g.R == (const void*)g.C))) return false;
    return encode_fn() != nullptr;
}

static void fill_params(TcParams& p, const GemmArgs& g) {
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.C = g.C; p.ldc = g.ldc; p.c_dtype = g.c_dtype;
  p.reduce = (g.R && (const void*)g.R == (const void*)g.C) ? 1 : 0;
  p.R = p.reduce ? nullptr : g.R; p.ldr = g.ldr;
  p.a_kmajor = g.a_kmajor; p.b_kmajor = g.b_kmajor;
  p.aux = (const __nv_bfloat16*)g.epi.aux; p.ld_aux = g.epi.ld_aux;
  p.out2 = (__nv_bfloat16*)g.epi.out2; p.ld_out2 = g.epi.ld_out2;
  p.rope_tab = g.epi.rope_tab; p.S = g.epi.S; p.dh = g.epi.dh; p.d = g.epi.d;
  p.up_row0 = g.N / 2;
  p.hl = g.epi.hl;
  p.kb_main = (g.K + TC_BK - 1) / TC_BK;
  p.kb_total = p.kb_main + (g.K2 > 0 ? 1 : 0);
  p.ext_ksteps = g.K2 / 16;
  p.alpha = g.alpha;
  p.kb_per_split = 1; p.tiles_m = p.tiles_n = p.splits = 1;
}

template <int BN, int EPI>
static int launch_tc(const GemmArgs& g, cudaStream_t s) {
  CUtensorMap tmA, tmB;
  constexpr int B_BOX_ROWS = (EPI == EPI_SWIGLU_FWD) ? 128 : BN;
  // K-major operand: tensor [MN][K] -> box {64 k, rows}.  MN-major operand: tensor [K][MN] -> box {64 mn, 64 k}.
  const bool okA = g.a_kmajor ? make_tmap(&tmA, g.A, g.M, g.K, g.lda, TC_BK, TC_BM)
                              : make_tmap(&tmA, g.A, g.K, g.M, g.lda, 64, TC_BK);
  const bool okB = g.b_kmajor ? make_tmap(&tmB, g.B, g.N, g.K, g.ldb, TC_BK, B_BOX_ROWS)
                              : make_tmap(&tmB, g.B, g.K, g.N, g.ldb, 64, TC_BK);
  if (!okA || !okB) return PCM_ERR_CUDA;
  CUtensorMap tmA2 = tmA, tmB2 = tmB;                      // continuation of the contraction, laid out like A / B
  if (g.K2 > 0) {
    const bool okA2 = g.a_kmajor ? make_tmap(&tmA2, g.A2, g.M, g.K2, g.lda2, TC_BK, TC_BM)
                                 : make_tmap(&tmA2, g.A2, g.K2, g.M, g.lda2, 64, TC_BK);
    const bool okB2 = g.b_kmajor ? make_tmap(&tmB2, g.B2, g.N, g.K2, g.ldb2, TC_BK, B_BOX_ROWS)
                                 : make_tmap(&tmB2, g.B2, g.K2, g.N, g.ldb2, 64, TC_BK);
    if (!okA2 || !okB2) return PCM_ERR_CUDA;
  }
  TcParams p;
  fill_params(p, g);
  const int tiles_m = (g.M + TC_BM - 1) / TC_BM, tiles_n = (g.N + BN - 1) / BN;
  const int num_kb = p.kb_total;
  int splits = 1;
  if (p.reduce) {
    // split the contraction until there are about two waves of CTAs, keeping >= 8 k-blocks per split
    const long long tiles = (long long)tiles_m * tiles_n;
    long long want = (2 * 148 + tiles - 1) / tiles;
    long long cap = num_kb / 8 > 0 ? num_kb / 8 : 1;
    splits = (int)(want < cap ? want : cap);
    if (splits < 1) splits = 1;
  }
  p.kb_per_split = (num_kb + splits - 1) / splits;
  splits = (num_kb + p.kb_per_split - 1) / p.kb_per_split;          // no empty split
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, TcSmem<BN>::TOTAL));
  p.tiles_m = tiles_m; p.tiles_n = tiles_n; p.splits = splits;
  const long long total = (long long)tiles_m * tiles_n * splits;
  const int grid = (int)(total < sm_count() ? total : sm_count());      // persistent: one CTA per SM walks the tile list
  gemm_tc_kernel<BN, EPI><<<grid, TC_THREADS, TcSmem<BN>::TOTAL, s>>>(tmA, tmB, tmA2, tmB2, p);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

static bool pair_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("PCM_GEMM_PAIR");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v == 1;
}

// CTA-pair launch: 256 x 256 tiles, clusters of two CTAs, one pair per two SMs.
template <int EPI>
static int launch_tc2(const GemmArgs& g, cudaStream_t s) {
  CUtensorMap tmA, tmB;
  const bool okA = g.a_kmajor ? make_tmap(&tmA, g.A, g.M, g.K, g.lda, TC_BK, TC_BM)
                              : make_tmap(&tmA, g.A, g.K, g.M, g.lda, 64, TC_BK);
  const bool okB = g.b_kmajor ? make_tmap(&tmB, g.B, g.N, g.K, g.ldb, TC_BK, T2_BN / 2)
                              : make_tmap(&tmB, g.B, g.K, g.N, g.ldb, 64, TC_BK);
  if (!okA || !okB) return PCM_ERR_CUDA;
  CUtensorMap tmA2 = tmA, tmB2 = tmB;
  if (g.K2 > 0) {
    const bool okA2 = g.a_kmajor ? make_tmap(&tmA2, g.A2, g.M, g.K2, g.lda2, TC_BK, TC_BM)
                                 : make_tmap(&tmA2, g.A2, g.K2, g.M, g.lda2, 64, TC_BK);
    const bool okB2 = g.b_kmajor ? make_tmap(&tmB2, g.B2, g.N, g.K2, g.ldb2, TC_BK, T2_BN / 2)
                                 : make_tmap(&tmB2, g.B2, g.K2, g.N, g.ldb2, 64, TC_BK);
    if (!okA2 || !okB2) return PCM_ERR_CUDA;
  }
  TcParams p;
  fill_params(p, g);
  const int tiles_m = (g.M + 2 * TC_BM - 1) / (2 * TC_BM), tiles_n = (g.N + T2_BN - 1) / T2_BN;
  const int num_kb = p.kb_total;
  const int n_pairs_max = sm_count() / 2;
  int splits = 1;
  if (p.reduce) {
    // Split the contraction so that the work items fill whole waves of CTA pairs: with tiles x splits items on
    // n_pairs_max pairs, ceil(items / pairs) waves run and the last one is as long as the others.  Among the
    // candidates (at least 8 k-blocks per split) take the fullest waves, charging each extra split a little for its
    // fp32 reduction traffic.
    const long long tiles = (long long)tiles_m * tiles_n;
    const int cap = num_kb / 8 > 0 ? (num_kb / 8 < 32 ? num_kb / 8 : 32) : 1;
    double best = -1.0;
    for (int cand = 1; cand <= cap; ++cand) {
      const int per = (num_kb + cand - 1) / cand;
      const int actual = (num_kb + per - 1) / per;                 // no empty split
      const long long items = tiles * actual;
      const long long waves = (items + n_pairs_max - 1) / n_pairs_max;
      const double score = (double)items / (double)(waves * n_pairs_max) - 0.004 * actual;
      if (score > best) { best = score; splits = actual; }
    }
  }
  p.kb_per_split = (num_kb + splits - 1) / splits;
  splits = (num_kb + p.kb_per_split - 1) / p.kb_per_split;
  p.tiles_m = tiles_m; p.tiles_n = tiles_n; p.splits = splits;
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, T2_SMEM_TOTAL));
  const long long total = (long long)tiles_m * tiles_n * splits;
  const int pairs = (int)(total < n_pairs_max ? total : n_pairs_max);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(T2_THREADS);
  cfg.dynamicSmemBytes = T2_SMEM_TOTAL;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI>, tmA, tmB, tmA2, tmB2, p) != cudaSuccess) {
    cudaGetLastError();
    return PCM_ERR_CUDA;
  }
  pcm::g_launches.fetch_add(1, std::memory_order_relaxed);
  return PCM_OK;
}

bool gemm_epilogue_supported(const GemmArgs& g) {
  if (!gemm_tcgen05_supported(g) || g.c_dtype != DT_BF16 || g.R) return false;
  const GemmEpilogue& e = g.epi;
  switch (e.kind) {
    case EPI_NONE: return true;
    case EPI_SWIGLU_FWD:   // N = 2F accumulator columns; tiles of 128 hidden units
      return g.b_kmajor && (g.N % 256 == 0) && e.out2 && (e.ld_out2 % 8 == 0) && !(((uintptr_t)e.out2) & 15);
    case EPI_SWIGLU_BWD:   // N = F
      return e.aux && (e.ld_aux % 8 == 0) && !(((uintptr_t)e.aux) & 15) && (g.N % 32 == 0);
    case EPI_ROPE:
      return e.rope_tab && (e.dh == 64 || e.dh == 128) && e.S > 0 && e.d > 0 && (e.d % 256 == 0) && g.N == 3 * e.d;
    case EPI_HEAD_LOSS:    // one 256-column tile holds a row's whole vocabulary
      return g.N == 256 && g.a_kmajor && g.b_kmajor && e.hl.tgt && (!e.hl.want_dz || (g.C && g.ldc == 256)) &&
             (e.hl.mode == HL_COEF ? e.hl.coef != nullptr : true) &&
             (e.hl.mode == HL_TOKEN ? (e.hl.lpo && e.hl.adv_c) : true) && !(((uintptr_t)e.hl.part) & 15);
  }
  return false;
}

// CTA pairs whenever the output is at least one 256-wide tile; single CTAs otherwise (or with PCM_GEMM_PAIR=0)
static bool wants_pair(const GemmArgs& g) {
  return pair_enabled() && g.N >= 256 && g.M > TC_BM && g.epi.kind != EPI_HEAD_LOSS;
}
bool gemm_tcgen05_pair(const GemmArgs& g) { return wants_pair(g); }

int gemm_tcgen05(const GemmArgs& g, cudaStream_t s) {
  const bool pair = wants_pair(g);
  switch (g.epi.kind) {
    case EPI_SWIGLU_FWD:
      if (!gemm_epilogue_supported(g)) return PCM_ERR_SHAPE;
      return pair ? launch_tc2<EPI_SWIGLU_FWD>(g, s) : launch_tc<256, EPI_SWIGLU_FWD>(g, s);
    case EPI_SWIGLU_BWD:
      if (!gemm_epilogue_supported(g)) return PCM_ERR_SHAPE;
      return pair ? launch_tc2<EPI_SWIGLU_BWD>(g, s) : launch_tc<256, EPI_SWIGLU_BWD>(g, s);
    case EPI_ROPE:
      if (!gemm_epilogue_supported(g)) return PCM_ERR_SHAPE;
      return pair ? launch_tc2<EPI_ROPE>(g, s) : launch_tc<256, EPI_ROPE>(g, s);
    case EPI_HEAD_LOSS:
      if (!gemm_epilogue_supported(g)) return PCM_ERR_SHAPE;
      return launch_tc<256, EPI_HEAD_LOSS>(g, s);
    default: break;
  }
  if (pair) return launch_tc2<EPI_NONE>(g, s);
  if (g.N % 256 == 0 || g.N > 256) return launch_tc<256, EPI_NONE>(g, s);
  return launch_tc<128, EPI_NONE>(g, s);
}

int attention_tc_poll_status();

int tcgen05_poll_status() {
  const int arc = attention_tc_poll_status();
  if (arc != PCM_OK) return arc;
  unsigned h = 0;
  if (cudaMemcpyFromSymbol(&h, g_tc_status, sizeof(h)) != cudaSuccess) return PCM_ERR_CUDA;
  if (h) {
    unsigned z = 0;
    cudaMemcpyToSymbol(g_tc_status, &z, sizeof(z));
    return PCM_ERR_DEVICE_TIMEOUT;
  }
  return PCM_OK;
}

}  // namespace pcm
