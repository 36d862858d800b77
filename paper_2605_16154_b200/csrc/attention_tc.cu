// bf16 causal attention inside each chunk's sequence on the 5th-generation tensor cores (forward).
//
// One persistent CTA per SM walks (sequence, head) items.  The whole K and V of an item (S <= 384 rows)
// sit in shared memory (TMA, 128-byte swizzle); query tiles of 128 rows stream through a small ring.
// For a query tile the full score row block S = Q K^T (128 x n, n <= 384 columns, causal: only the
// columns at or left of the tile's last row) is produced by tcgen05.mma into tensor memory, so the
// softmax is a plain two-pass softmax over tensor memory (no running rescale): pass 1 takes the row
// maximum, pass 2 writes P = exp(.) as packed bf16 back into tensor memory over the scores it has
// consumed, and O = P V runs with P as the tensor-memory A operand and V as an MN-major shared-memory
// B operand.  Probabilities never touch shared or global memory.
//
// Warp roles (320 threads): warp 0 = TMA producer, warp 1 = tensor-memory allocation + MMA issue,
// warps 2..9 = softmax and output (two per tensor-memory lane quadrant; the two split a tile's columns).
// Every mbarrier wait is bounded; when one runs out the CTA latches a status bit, all roles leave at the
// next tile boundary, tensor memory is released and the kernel returns.
#include <cuda.h>

#include "async_ptx.cuh"
#include "internal.h"

namespace pcm {

__device__ unsigned g_fa_status = 0;          // bit 0: a bounded wait expired

namespace fatc {

constexpr int BM = 128;                        // query rows per tile = tensor-memory lanes
constexpr int THREADS = 320;
constexpr int SM_WARPS = 8;                    // softmax warps
constexpr unsigned long long WAIT_NS = 2000000000ull;
constexpr int TMEM_COLS = 512;
constexpr int S_COLS = 384;                    // score columns (fp32); P (packed bf16) overwrites consumed scores
constexpr int O_COL = 384;                     // output accumulator: columns [384, 384 + DH)
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

struct Params {
  int n_seq, S, H, d;
  int n_items;                                 // n_seq * H
  int nq;                                      // query tiles per item
  int kv_rows;                                 // rows of K / V staged per item (multiple of 64)
  int n_total;                                 // S rounded up to 16: columns of the widest score block
  int kv_stages, q_stages;
  float scale_log2;                            // log2(e) / sqrt(dh)
  __nv_bfloat16* out;
  float* lse;
};

__device__ __forceinline__ void tma_load_3d(void* smem_dst, const void* tmap, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(smem_dst)),
      "l"(tmap), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]: A is read from tensor memory (lane = row, 16-bit elements packed two per column)
__device__ __forceinline__ void umma_bf16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
      "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Shared-memory matrix descriptor (tcgen05), 128-byte swizzle: start address, leading / stride byte offsets.
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// kind::f16 instruction descriptor: fp32 accumulator, bf16 A and B, M = 128, K-major A
__device__ __forceinline__ uint32_t idesc_bf16(int n, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
         ((uint32_t)(BM >> 4) << 24);
}

// Shared-memory plan (bytes, after 1024-byte alignment):
//   K ring   kv_stages x DH/64 slabs x kv_rows x 128 B     slab = 64 head-dim columns of every staged row
//   V ring   the same
//   Q ring   q_stages x DH/64 slabs x 128 rows x 128 B
//   barriers, row statistics exchanged between the two warps of a lane quadrant
struct Plan {
  uint32_t k_off, v_off, q_off, bar_off, red_off, total;
};
__host__ __device__ inline Plan make_plan(int dh, int kv_rows, int kv_stages, int q_stages) {
  Plan p;
  const uint32_t kv_bytes = (uint32_t)(dh / 64) * kv_rows * 128u;
  const uint32_t q_bytes = (uint32_t)(dh / 64) * BM * 128u;
  p.k_off = 0;
  p.v_off = p.k_off + kv_stages * kv_bytes;
  p.q_off = p.v_off + kv_stages * kv_bytes;
  p.bar_off = p.q_off + q_stages * q_bytes;
  p.red_off = p.bar_off + 256;
  p.total = p.red_off + 2 * 2 * BM * 4 + 1024 /* alignment slack */;
  return p;
}


template <int DH>
__global__ void __launch_bounds__(THREADS, 1)
fa_tc_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int NSLAB = DH / 64;
  constexpr uint32_t Q_SLAB = BM * 128u, Q_BYTES = NSLAB * Q_SLAB;
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* base = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
  const Plan pl = make_plan(DH, p.kv_rows, p.kv_stages, p.q_stages);
  const uint32_t kv_slab = (uint32_t)p.kv_rows * 128u, kv_bytes = NSLAB * kv_slab;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + pl.bar_off);
  uint64_t* kv_full = bars;                    // [2] producer -> MMA, K and V of one item
  uint64_t* kv_empty = bars + 2;               // [2] MMA -> producer
  uint64_t* q_full = bars + 4;                 // [2]
  uint64_t* q_empty = bars + 6;                // [2]
  uint64_t* s_full = bars + 8;                 // MMA -> softmax: scores of a tile are in tensor memory
  uint64_t* p_full = bars + 9;                 // softmax -> MMA: probabilities are in tensor memory (8 warp arrivals)
  uint64_t* o_full = bars + 10;                // MMA -> softmax: the tile's output is in tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 11);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* red_max = reinterpret_cast<float*>(base + pl.red_off);   // [2][128]
  float* red_sum = red_max + 2 * BM;                              // [2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_local = ((int)blockIdx.x < p.n_items) ? (p.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int n_tiles = n_local * p.nq;

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1);
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1);
    }
    mbar_init(s_full, 1); mbar_init(p_full, SM_WARPS); mbar_init(o_full, 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmKV);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------ TMA producer ------------------------------
      bool ok = true;
      for (int k = 0; k < n_local && ok && !*abort_flag; ++k) {
        const int item = blockIdx.x + k * gridDim.x, seq = item / p.H, h = item - seq * p.H;
        const int st = k % p.kv_stages;
        const unsigned ph = (unsigned)(k / p.kv_stages) & 1u;
        if (!mbar_wait_bounded(&kv_empty[st], ph ^ 1u, WAIT_NS)) { ok = false; break; }
        mbar_expect_tx(&kv_full[st], 2 * kv_bytes);
        uint8_t* ks = base + pl.k_off + st * kv_bytes;
        uint8_t* vs = base + pl.v_off + st * kv_bytes;
        for (int sl = 0; sl < NSLAB; ++sl)
          for (int rb = 0; rb < p.kv_rows / 64; ++rb) {
            tma_load_3d(ks + sl * kv_slab + rb * 8192, &tmKV, p.d + h * DH + sl * 64, rb * 64, seq, &kv_full[st]);
            tma_load_3d(vs + sl * kv_slab + rb * 8192, &tmKV, 2 * p.d + h * DH + sl * 64, rb * 64, seq, &kv_full[st]);
          }
        for (int t = 0; t < p.nq; ++t) {
          const int g = k * p.nq + t, qs = g % p.q_stages;
          const unsigned qph = (unsigned)(g / p.q_stages) & 1u;
          if (*abort_flag || !mbar_wait_bounded(&q_empty[qs], qph ^ 1u, WAIT_NS)) { ok = false; break; }
          mbar_expect_tx(&q_full[qs], Q_BYTES);
          uint8_t* qd = base + pl.q_off + qs * Q_BYTES;
          for (int sl = 0; sl < NSLAB; ++sl)
            tma_load_3d(qd + sl * Q_SLAB, &tmQ, h * DH + sl * 64, t * BM, seq, &q_full[qs]);
        }
      }
      if (!ok) { *abort_flag = 1; atomicOr(&g_fa_status, 1u); }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------ MMA issuer ------------------------------
      bool ok = true;
      const uint32_t k_base = smem_u32(base + pl.k_off), v_base = smem_u32(base + pl.v_off);
      const uint32_t q_base = smem_u32(base + pl.q_off);
      // S(g) = Q K^T for local tile g: columns 0 .. n-1 of the score block
      auto issue_scores = [&](int g) {
        const int k = g / p.nq, t = g - k * p.nq, st = k % p.kv_stages, qs = g % p.q_stages;
        if (t == 0 && !mbar_wait_bounded(&kv_full[st], (unsigned)(k / p.kv_stages) & 1u, WAIT_NS)) { ok = false; return; }
        if (!mbar_wait_bounded(&q_full[qs], (unsigned)(g / p.q_stages) & 1u, WAIT_NS)) { ok = false; return; }
        tc_fence_after();
        const int n = min(p.n_total, (t + 1) * BM);
        const uint32_t qa = q_base + qs * Q_BYTES, ka = k_base + st * kv_bytes;
        for (int c0 = 0; c0 < n; c0 += 128) {
          const int nn = min(128, n - c0);
          const uint32_t idesc = idesc_bf16(nn, 0);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks) {
            const uint64_t da = smem_desc(qa + (ks >> 2) * Q_SLAB + (ks & 3) * 32, 16u, 1024u);
            const uint64_t db = smem_desc(ka + (ks >> 2) * kv_slab + c0 * 128 + (ks & 3) * 32, 16u, 1024u);
            umma_bf16(tmem_base + (uint32_t)c0, da, db, idesc, ks > 0 ? 1u : 0u);
          }
        }
        umma_commit(s_full);
        umma_commit(&q_empty[qs]);             // the query tile may be replaced once these MMAs have read it
      };
      if (n_tiles > 0) issue_scores(0);
      for (int g = 0; g < n_tiles && ok; ++g) {
        const int k = g / p.nq, t = g - k * p.nq, st = k % p.kv_stages;
        if (*abort_flag || !mbar_wait_bounded(p_full, (unsigned)g & 1u, WAIT_NS)) { ok = false; break; }
        tc_fence_after();
        // O = P V: P from tensor memory in two segments (one per softmax warp of a quadrant), V MN-major from shared memory
        const int n = min(p.n_total, (t + 1) * BM);
        const int nsl = (n + 31) >> 5, seg_a = ((nsl + 1) >> 1) * 32;
        const uint32_t idesc = idesc_bf16(DH, 1);
        const uint32_t va = v_base + st * kv_bytes;
        for (int kv0 = 0; kv0 < n; kv0 += 16) {
          const uint32_t a_col = kv0 < seg_a ? (uint32_t)(kv0 >> 1) : (uint32_t)(seg_a + ((kv0 - seg_a) >> 1));
          const uint64_t db = smem_desc(va + kv0 * 128, kv_slab, 1024u);
          umma_bf16_ts(tmem_base + O_COL, tmem_base + a_col, db, idesc, kv0 > 0 ? 1u : 0u);
        }
        umma_commit(o_full);
        if (t == p.nq - 1) umma_commit(&kv_empty[st]);   // last use of this item's K and V
        if (g + 1 < n_tiles) issue_scores(g + 1);
      }
      if (!ok) { *abort_flag = 1; atomicOr(&g_fa_status, 1u); }
    }
  } else {
    // ------------------------------ softmax + output: warps 2..9 ------------------------------
    const int quad = warp & 3, half = (warp - 2) >> 2;
    const int row = quad * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c2 = p.scale_log2;
    bool dead = false;
    for (int g = 0; g < n_tiles; ++g) {
      named_bar_sync(1, SM_WARPS * 32);
      if (*abort_flag) break;                  // read after the barrier: the same answer in all softmax warps
      const int k = g / p.nq, t = g - k * p.nq;
      const int item = blockIdx.x + k * gridDim.x, seq = item / p.H, h = item - seq * p.H;
      const int n = min(p.n_total, (t + 1) * BM);
      const int nsl = (n + 31) >> 5, sl_a = (nsl + 1) >> 1;
      const int sl_lo = half ? sl_a : 0, sl_hi = half ? nsl : sl_a;
      const int qi = t * BM + row, qc = min(qi, p.S - 1);             // rows past the sequence are computed but not stored
      const int q_warp_min = min(t * BM + quad * 32, p.S - 1);
      auto wait_all = [&](uint64_t* bar, unsigned parity) {
        int ok = 1;
        if (lane == 0) {
          ok = (!dead && !*abort_flag && mbar_wait_bounded(bar, parity, WAIT_NS * 2ull)) ? 1 : 0;
          if (!ok) { *abort_flag = 1; atomicOr(&g_fa_status, 1u); }
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      };
      wait_all(s_full, (unsigned)g & 1u);
      tc_fence_after();
      // pass 1: row maximum over this warp's slices of 32 columns
      float m = -INFINITY;
      if (!dead) {
        for (int sl = sl_lo; sl < sl_hi; ++sl) {
          uint32_t r[32];
          tmem_ld_32x32(lane_addr + (uint32_t)(sl * 32), r);
          tmem_ld_wait();
          if (sl * 32 + 31 <= q_warp_min) {
#pragma unroll
            for (int e = 0; e < 32; ++e) m = fmaxf(m, __uint_as_float(r[e]));
          } else {
#pragma unroll
            for (int e = 0; e < 32; ++e) m = (sl * 32 + e <= qc) ? fmaxf(m, __uint_as_float(r[e])) : m;
          }
        }
      }
      red_max[half * BM + row] = m;
      named_bar_sync(2, SM_WARPS * 32);
      m = fmaxf(m, red_max[(half ^ 1) * BM + row]);                    // column 0 is never masked: finite
      const float mc = m * c2;
      // pass 2: P = exp2(s c - m c), packed bf16 written over scores this warp has already consumed
      float sum = 0.f;
      if (!dead) {
        for (int sl = sl_lo; sl < sl_hi; ++sl) {
          uint32_t r[32], pk[16];
          tmem_ld_32x32(lane_addr + (uint32_t)(sl * 32), r);
          tmem_ld_wait();
          if (sl * 32 + 31 <= q_warp_min) {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(r[e]), c2, -mc));
              const float p1 = ex2_approx(fmaf(__uint_as_float(r[e + 1]), c2, -mc));
              sum += p0 + p1;
              pk[e >> 1] = pack_bf16x2(p0, p1);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float p0 = (sl * 32 + e <= qc) ? ex2_approx(fmaf(__uint_as_float(r[e]), c2, -mc)) : 0.f;
              const float p1 = (sl * 32 + e + 1 <= qc) ? ex2_approx(fmaf(__uint_as_float(r[e + 1]), c2, -mc)) : 0.f;
              sum += p0 + p1;
              pk[e >> 1] = pack_bf16x2(p0, p1);
            }
          }
          const int pcol = half ? sl_a * 32 + (sl - sl_a) * 16 : sl * 16;
          tmem_st_32x16(lane_addr + (uint32_t)pcol, pk);
        }
        tmem_st_wait();
      }
      red_sum[half * BM + row] = sum;
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(p_full);
      named_bar_sync(2, SM_WARPS * 32);
      const float tot = sum + red_sum[(half ^ 1) * BM + row];
      wait_all(o_full, (unsigned)g & 1u);
      tc_fence_after();
      if (!dead) {
        const float inv = 1.f / tot;
        __nv_bfloat16* op = p.out + ((long long)seq * p.S + qi) * p.d + h * DH + half * (DH / 2);
#pragma unroll
        for (int cc = 0; cc < DH / 2; cc += 32) {
          uint32_t r[32];
          tmem_ld_32x32(lane_addr + (uint32_t)(O_COL + half * (DH / 2) + cc), r);
          tmem_ld_wait();
          if (qi < p.S) {
#pragma unroll
            for (int e = 0; e < 32; e += 8) {
              uint4 o;
              o.x = pack_bf16x2(__uint_as_float(r[e]) * inv, __uint_as_float(r[e + 1]) * inv);
              o.y = pack_bf16x2(__uint_as_float(r[e + 2]) * inv, __uint_as_float(r[e + 3]) * inv);
              o.z = pack_bf16x2(__uint_as_float(r[e + 4]) * inv, __uint_as_float(r[e + 5]) * inv);
              o.w = pack_bf16x2(__uint_as_float(r[e + 6]) * inv, __uint_as_float(r[e + 7]) * inv);
              *reinterpret_cast<uint4*>(op + cc + e) = o;
            }
          }
        }
        if (half == 0 && qi < p.S) p.lse[((long long)seq * p.H + h) * p.S + qi] = (mc + log2f(tot)) * LN2;
      }
      tc_fence_before();                       // the next tile's P V overwrites the accumulator only after these reads
    }
  }

  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);   // let copies still in flight land before shared memory goes away
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn attn_encode_fn() {
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

// bf16 tensor [n_seq][S][cols] (row stride ld elements, sequences S rows apart), box {64 columns, box_rows, 1},
// 128-byte swizzle.  Rows past the end of a sequence read as zero, so a tile never sees its neighbour's rows.
static bool make_seq_tmap(CUtensorMap* tm, const void* base, int n_seq, int S, long long cols, long long ld, int box_rows) {
  EncodeTiledFn fn = attn_encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)S, (cuuint64_t)n_seq};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)ld * 2 * (cuuint64_t)S};
  cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, 1u};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int attn_sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1)
      n = 148;
  }
  return n;
}

constexpr uint32_t SMEM_LIMIT = 227u * 1024u;
constexpr uint32_t SMEM_FLOOR = 120u * 1024u;  // more than half of an SM's shared memory: one CTA per SM, which owns all of tensor memory

template <int DH>
static int fwd_launch(const void* qkv, void* out, float* lse, int n_seq, int S, int H, cudaStream_t s) {
  const int d = H * DH;
  Params p;
  p.n_seq = n_seq; p.S = S; p.H = H; p.d = d;
  p.n_items = n_seq * H;
  p.nq = (S + BM - 1) / BM;
  p.kv_rows = ((S + 63) / 64) * 64;
  p.n_total = ((S + 15) / 16) * 16;
  p.scale_log2 = LOG2E / sqrtf((float)DH);
  p.out = (__nv_bfloat16*)out;
  p.lse = lse;
  // deepest rings that fit: two items' K and V when possible, so the next item loads while this one computes
  p.kv_stages = 2; p.q_stages = 2;
  if (make_plan(DH, p.kv_rows, p.kv_stages, p.q_stages).total > SMEM_LIMIT) p.kv_stages = 1;
  if (make_plan(DH, p.kv_rows, p.kv_stages, p.q_stages).total > SMEM_LIMIT) p.q_stages = 1;
  const Plan pl = make_plan(DH, p.kv_rows, p.kv_stages, p.q_stages);
  if (pl.total > SMEM_LIMIT) return PCM_ERR_SHAPE;
  const uint32_t smem = pl.total < SMEM_FLOOR ? SMEM_FLOOR : pl.total;
  CUtensorMap tmQ, tmKV;
  if (!make_seq_tmap(&tmQ, qkv, n_seq, S, 3LL * d, 3LL * d, BM) || !make_seq_tmap(&tmKV, qkv, n_seq, S, 3LL * d, 3LL * d, 64))
    return PCM_ERR_CUDA;
  static bool attr_done = false;
  if (!attr_done) {
    PCM_CUDA_TRY(cudaFuncSetAttribute(fa_tc_fwd_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT));
    attr_done = true;
  }
  const int grid = p.n_items < attn_sm_count() ? p.n_items : attn_sm_count();
  fa_tc_fwd_kernel<DH><<<grid, THREADS, smem, s>>>(tmQ, tmKV, p);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

}  // namespace fatc

bool attention_tc_supported(const void* qkv, const void* out, int S, int H, int dh) {
  if (dh != 64 && dh != 128) return false;
  if (S < 1 || S > fatc::S_COLS) return false;
  if ((((uintptr_t)qkv) | ((uintptr_t)out)) & 15) return false;
  (void)H;
  return fatc::attn_encode_fn() != nullptr;
}

int attention_fwd_bf16_tc(const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh, cudaStream_t s) {
  if (!attention_tc_supported(qkv, out, S, H, dh)) return PCM_ERR_SHAPE;
  if (n_seq < 1) return PCM_OK;
  return dh == 64 ? fatc::fwd_launch<64>(qkv, out, lse, n_seq, S, H, s) : fatc::fwd_launch<128>(qkv, out, lse, n_seq, S, H, s);
}

// Reads and clears this file's device status word (synchronous copy).
int attention_tc_poll_status() {
  unsigned h = 0;
  if (cudaMemcpyFromSymbol(&h, g_fa_status, sizeof(h)) != cudaSuccess) return PCM_ERR_CUDA;
  if (h) {
    unsigned z = 0;
    cudaMemcpyToSymbol(g_fa_status, &z, sizeof(z));
    return PCM_ERR_DEVICE_TIMEOUT;
  }
  return PCM_OK;
}

}  // namespace pcm
