// bf16 causal attention inside each chunk's sequence on the 5th-generation tensor cores: the forward pass
// (described here) and, further down, the backward pass: one kernel template launched for dQ and for dK / dV (head
// dim 128, and head dim 64 on request), and the one-pass kernel of attention_tc_bwd1.cuh (head dim 64).
//
// Forward.  One persistent CTA per SM walks (sequence, head) items.  The whole K and V of an item (S <= 384 rows)
// sit in shared memory (TMA, 128-byte swizzle); query tiles of 128 rows stream through a small ring.
// A query tile is processed as independent blocks of 128 keys (causal: the blocks at or left of the
// diagonal).  For block j, tcgen05.mma puts S_j = Q K_j^T (128 x 128, fp32) into one of the score
// buffers in tensor memory; the softmax warps take the block's own row maximum m_j, write
// P_j = exp(S_j - m_j) as packed bf16 over the scores they have consumed and keep the row sums l_j;
// O_j = P_j V_j then runs with P_j as the tensor-memory A operand and V_j as an MN-major shared-memory
// B operand into its own accumulator slot.  Blocks never wait for one another (no running rescale);
// the output warps combine the slots at the end of the tile:
//   m = max_j m_j,  w_j = exp(m_j - m),  O = sum_j w_j O_j / sum_j w_j l_j,  lse = m + log(sum_j w_j l_j).
// With two score buffers the tensor core works on one block while the softmax warps work on the other.
// Probabilities never touch shared or global memory.
//
// Warp roles: warp 0 = TMA producer, warp 1 = tensor-memory allocation + MMA issue, warps 2..5 = output
// (one per tensor-memory lane quadrant), then 8 softmax warps per score buffer (two per lane quadrant,
// splitting the block's columns).  Every mbarrier wait is bounded; when one runs out the CTA latches a
// status bit, all roles leave at their next block boundary, tensor memory is released and the kernel returns.
#include <cuda.h>

#include "async_ptx.cuh"
#include "internal.h"

namespace pcm {

__device__ unsigned g_fa_status = 0;          // bit 0: a bounded wait expired; bit 8 + site: which wait it was
__device__ __forceinline__ void fa_timeout(int site) { atomicOr(&g_fa_status, 1u | (1u << (8 + site))); }
enum { SITE_KV_EMPTY = 0, SITE_Q_EMPTY = 1, SITE_KV_FULL = 2, SITE_Q_FULL = 3, SITE_P_FULL = 4, SITE_O_EMPTY = 5, SITE_O_FULL = 6, SITE_S_FULL = 7, SITE_PLAN = 8 };

namespace fatc {

constexpr int BM = 128;                        // query rows per tile = tensor-memory lanes
constexpr int BN = 128;                        // keys per block
constexpr int MAX_SLOTS = 3;                   // blocks per tile at most: S <= 384
constexpr int S_MAX = BN * MAX_SLOTS;
constexpr int SM_WARPS_PER_BUF = 8;
constexpr unsigned long long WAIT_NS = 2000000000ull;
constexpr int TMEM_COLS = 512;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;
constexpr int OUT_BAR = 9;                     // named barrier of the four output warps (1..8: softmax warp pairs)
constexpr int STAT_RING = 3;                   // tiles whose row statistics may be live at once

template <int DH> struct Cfg {
  static constexpr int NBUF = DH == 64 ? 2 : 1;                       // score buffers that fit beside the output slots
  static constexpr int O_COL = NBUF * BN;                             // accumulator slot s: columns [O_COL + s DH, +DH)
  static constexpr int NSLOT = (TMEM_COLS - O_COL) / DH;              // slots form a ring over all blocks of the CTA
  static constexpr int THREADS = (2 + 4 + NBUF * SM_WARPS_PER_BUF) * 32;
  static_assert(NSLOT >= MAX_SLOTS, "tensor memory plan does not fit");
};

struct Params {
  int n_seq, S, H, d;
  int n_items;                                 // n_seq * H
  int nq;                                      // query tiles per item
  int kv_rows;                                 // rows of K / V staged per item (multiple of 64)
  int n_total;                                 // S rounded up to 16: keys that take part in the MMAs
  int kv_stages, q_stages;
  float scale_log2;                            // log2(e) / sqrt(dh)
  __nv_bfloat16* out;
  float* lse;
};

// Walks the blocks of this CTA's items in issue order: item k, query tile t, key block j <= t.
struct BlockIter {
  int nq, k, t, j, tile;                       // tile = running count of query tiles (all items)
  __device__ void init(int nq_) { nq = nq_; k = t = j = tile = 0; }
  __device__ void next() {
    if (j < t) { ++j; return; }
    j = 0; ++tile;
    if (t + 1 < nq) { ++t; } else { t = 0; ++k; }
  }
  __device__ void advance(int n) { for (int i = 0; i < n; ++i) next(); }
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
__device__ __forceinline__ void tma_store_3d(const void* tmap, const void* smem_src, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(tmap),
               "r"(smem_u32(smem_src)), "r"(x), "r"(y), "r"(z)
               : "memory");
}
// makes this thread's shared-memory writes visible to the asynchronous proxy (TMA)
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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
//   output staging for the TMA store
//   barriers; row statistics (m_j, l_j per tile of the ring, block and row); the maxima the two warps of a
//   lane quadrant exchange
struct Plan {
  uint32_t k_off, v_off, q_off, ostage_off, bar_off, stat_m_off, stat_l_off, red_off, total;
};
__host__ __device__ inline Plan make_plan(int dh, int kv_rows, int kv_stages, int q_stages) {
  Plan p;
  const uint32_t kv_bytes = (uint32_t)(dh / 64) * kv_rows * 128u;
  const uint32_t q_bytes = (uint32_t)(dh / 64) * BM * 128u;
  p.k_off = 0;
  p.v_off = p.k_off + kv_stages * kv_bytes;
  p.q_off = p.v_off + kv_stages * kv_bytes;
  p.ostage_off = p.q_off + q_stages * q_bytes;                       // 128 rows x 64 bf16 columns, swizzled
  p.bar_off = p.ostage_off + BM * 128;
  p.stat_m_off = p.bar_off + 256;
  p.stat_l_off = p.stat_m_off + STAT_RING * MAX_SLOTS * BM * 4;
  p.red_off = p.stat_l_off + STAT_RING * MAX_SLOTS * 2 * BM * 4;
  p.total = p.red_off + 2 * 2 * BM * 4 + 1024 /* alignment slack */;
  return p;
}

template <int DH>
__global__ void __launch_bounds__(Cfg<DH>::THREADS, 1)
fa_tc_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmKV,
                 const __grid_constant__ CUtensorMap tmO, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  constexpr int NSLAB = DH / 64;
  constexpr int NBUF = Cfg<DH>::NBUF;
  constexpr int O_COL = Cfg<DH>::O_COL;
  constexpr int NSLOT = Cfg<DH>::NSLOT;
  constexpr uint32_t Q_SLAB = BM * 128u, Q_BYTES = NSLAB * Q_SLAB;
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* base = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
  const Plan pl = make_plan(DH, p.kv_rows, p.kv_stages, p.q_stages);
  const uint32_t kv_slab = (uint32_t)p.kv_rows * 128u, kv_bytes = NSLAB * kv_slab;
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + pl.bar_off);
  uint64_t* kv_full = bars;                    // [2] producer -> MMA: K and V of one item
  uint64_t* kv_empty = bars + 2;               // [2] MMA -> producer
  uint64_t* q_full = bars + 4;                 // [2]
  uint64_t* q_empty = bars + 6;                // [2]
  uint64_t* s_full = bars + 8;                 // [2] MMA -> softmax: a block's scores are in the buffer
  uint64_t* p_full = bars + 10;                // [2] softmax -> MMA: the block's probabilities are in the buffer (8 warp arrivals)
  uint64_t* o_full = bars + 12;                // [2] MMA -> output warps: every slot of the tile is complete
  uint64_t* o_empty = bars + 14;               // [2] output warps -> MMA: the tile's slots may be overwritten (4 warp
                                               //     arrivals); tiles alternate between the two barriers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 16);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* stat_m = reinterpret_cast<float*>(base + pl.stat_m_off);   // [STAT_RING][MAX_SLOTS][128]
  float* stat_l = reinterpret_cast<float*>(base + pl.stat_l_off);   // [STAT_RING][MAX_SLOTS][2][128]: one partial sum per softmax warp of a quadrant
  float* red_max = reinterpret_cast<float*>(base + pl.red_off);     // [2][2][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_local = ((int)blockIdx.x < p.n_items) ? (p.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  const int n_tiles = n_local * p.nq;
  const int n_blocks = n_local * (p.nq * (p.nq + 1) / 2);

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) {
      mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1);
      mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 1);
      mbar_init(&s_full[s], 1); mbar_init(&p_full[s], SM_WARPS_PER_BUF);
    }
    mbar_init(&o_full[0], 1); mbar_init(&o_full[1], 1); mbar_init(&o_empty[0], 4); mbar_init(&o_empty[1], 4);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmKV);
    prefetch_tmap(&tmO);
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
        const int st = k & (p.kv_stages - 1);                          // stages are 1 or 2
        const unsigned ph = (unsigned)(k >> (p.kv_stages - 1)) & 1u;
        if (!mbar_wait_bounded(&kv_empty[st], ph ^ 1u, WAIT_NS)) { fa_timeout(SITE_KV_EMPTY); ok = false; break; }
        mbar_expect_tx(&kv_full[st], 2 * kv_bytes);
        uint8_t* ks = base + pl.k_off + st * kv_bytes;
        uint8_t* vs = base + pl.v_off + st * kv_bytes;
        for (int sl = 0; sl < NSLAB; ++sl)
          for (int rb = 0; rb < p.kv_rows / 64; ++rb) {
            tma_load_3d(ks + sl * kv_slab + rb * 8192, &tmKV, p.d + h * DH + sl * 64, rb * 64, seq, &kv_full[st]);
            tma_load_3d(vs + sl * kv_slab + rb * 8192, &tmKV, 2 * p.d + h * DH + sl * 64, rb * 64, seq, &kv_full[st]);
          }
        for (int t = 0; t < p.nq; ++t) {
          const int g = k * p.nq + t, qs = g & (p.q_stages - 1);
          const unsigned qph = (unsigned)(g >> (p.q_stages - 1)) & 1u;
          if (*abort_flag) { ok = false; break; }
          if (!mbar_wait_bounded(&q_empty[qs], qph ^ 1u, WAIT_NS)) { fa_timeout(SITE_Q_EMPTY); ok = false; break; }
          mbar_expect_tx(&q_full[qs], Q_BYTES);
          uint8_t* qd = base + pl.q_off + qs * Q_BYTES;
          for (int sl = 0; sl < NSLAB; ++sl)
            tma_load_3d(qd + sl * Q_SLAB, &tmQ, h * DH + sl * 64, t * BM, seq, &q_full[qs]);
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------ MMA issuer ------------------------------
      // One thread issues every MMA, so its instruction count per MMA matters (the MMAs are short: 32-64
      // tensor-core cycles): descriptors are built once and advanced by adding constants to their low word,
      // the block loops are unrolled, and ring positions are kept as counters instead of being divided out.
      bool ok = true;
      const uint32_t kslab16 = kv_slab >> 4;                           // descriptor units (16 bytes)
      const uint64_t dq0 = smem_desc(smem_u32(base + pl.q_off), 16u, 1024u);
      const uint64_t dk0 = smem_desc(smem_u32(base + pl.k_off), 16u, 1024u);
      const uint64_t dv0 = smem_desc(smem_u32(base + pl.v_off), kv_slab, 1024u);
      const uint32_t dq_hi = (uint32_t)(dq0 >> 32), dk_hi = (uint32_t)(dk0 >> 32), dv_hi = (uint32_t)(dv0 >> 32);
      const uint32_t dq_lo = (uint32_t)dq0, dk_lo = (uint32_t)dk0, dv_lo = (uint32_t)dv0;
      const int kv_mask = p.kv_stages - 1, kv_shift = p.kv_stages - 1;  // stages are 1 or 2
      const int q_mask = p.q_stages - 1, q_shift = p.q_stages - 1;
      const int nb_tail = p.n_total - (p.nq - 1) * BN;                  // keys in an item's last block (multiple of 16)
      const uint32_t idesc_s_full = idesc_bf16(BN, 0), idesc_s_tail = idesc_bf16(nb_tail, 0);
      const uint32_t idesc_pv = idesc_bf16(DH, 1);
      auto desc = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; };
      int released = 0;                          // tiles whose slots and statistics the output warps have handed back
      // S_j = Q K_j^T for the block `it` points at, into score buffer `buf`
      auto issue_scores = [&](const BlockIter& it, int buf) {
        const int st = it.k & kv_mask, qs = it.tile & q_mask;
        if (it.t == 0 && it.j == 0 && !mbar_wait_bounded(&kv_full[st], (unsigned)(it.k >> kv_shift) & 1u, WAIT_NS)) {
          fa_timeout(SITE_KV_FULL); ok = false; return;
        }
        if (it.j == 0 && !mbar_wait_bounded(&q_full[qs], (unsigned)(it.tile >> q_shift) & 1u, WAIT_NS)) {
          fa_timeout(SITE_Q_FULL); ok = false; return;
        }
        // the statistics ring holds STAT_RING tiles: this tile's softmax overwrites those of tile - STAT_RING
        while (it.j == 0 && released <= it.tile - STAT_RING && ok) {
          if (!mbar_wait_bounded(&o_empty[released & 1], (unsigned)(released >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_O_EMPTY); ok = false; }
          ++released;
        }
        if (!ok) return;
        tc_fence_after();
        const uint32_t qa = dq_lo + (uint32_t)qs * (Q_BYTES >> 4);
        const uint32_t ka = dk_lo + (uint32_t)st * (kv_bytes >> 4) + (uint32_t)it.j * (BN * 128 >> 4);
        const uint32_t idesc = (it.j == p.nq - 1) ? idesc_s_tail : idesc_s_full;
        const uint32_t d_col = tmem_base + (uint32_t)(buf * BN);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks) {
          const uint32_t qo = (uint32_t)((ks >> 2) * (Q_SLAB >> 4) + (ks & 3) * 2);
          const uint32_t ko = (uint32_t)(ks >> 2) * kslab16 + (uint32_t)((ks & 3) * 2);
          if (ks == 0) umma_bf16(d_col, desc(qa + qo, dq_hi), desc(ka + ko, dk_hi), idesc, 0u);
          else umma_bf16(d_col, desc(qa + qo, dq_hi), desc(ka + ko, dk_hi), idesc, 1u);
        }
        umma_commit(&s_full[buf]);
        if (it.j == it.t) umma_commit(&q_empty[qs]);    // the tile's last block: its queries may be replaced
      };
      BlockIter ahead, cur;
      ahead.init(p.nq); cur.init(p.nq);
      int b_ahead = 0;
      int hist[NSLOT];                           // tile of the last NSLOT blocks, oldest first: hist[0] used this block's slot
#pragma unroll
      for (int i = 0; i < NSLOT; ++i) hist[i] = -1;
      for (; b_ahead < NBUF && b_ahead < n_blocks && ok; ++b_ahead) { issue_scores(ahead, b_ahead); ahead.next(); }
      int buf = 0, slot = 0, buf_phase = 0;
      for (int b = 0; b < n_blocks && ok; ++b) {
        const int st = cur.k & kv_mask;
        if (*abort_flag) { ok = false; break; }
        if (!mbar_wait_bounded(&p_full[buf], (unsigned)buf_phase, WAIT_NS)) { fa_timeout(SITE_P_FULL); ok = false; break; }
        // the accumulator slot must have been read by the output warps of the tile that used it last.  Releases are
        // consumed in tile order and at least up to tile - 2: with the tiles alternating between two barriers, the
        // phase waited for is then never a whole lap behind its barrier
        const int need = max(hist[0], cur.tile - 2);
        while (released <= need && ok) {
          if (!mbar_wait_bounded(&o_empty[released & 1], (unsigned)(released >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_O_EMPTY); ok = false; }
          ++released;
        }
        if (!ok) break;
#pragma unroll
        for (int i = 0; i + 1 < NSLOT; ++i) hist[i] = hist[i + 1];
        hist[NSLOT - 1] = cur.tile;
        tc_fence_after();
        // O_j = P_j V_j: P from the score buffer in two segments (one per softmax warp of a quadrant)
        const uint32_t va = dv_lo + (uint32_t)st * (kv_bytes >> 4) + (uint32_t)cur.j * (BN * 128 >> 4);
        const uint32_t d_col = tmem_base + (uint32_t)(O_COL + slot * DH);
        const uint32_t a_base = tmem_base + (uint32_t)(buf * BN);
        if (cur.j < p.nq - 1 || nb_tail == BN) {
          // full block: keys 0..63 packed in columns 0..31, keys 64..127 in columns 64..95
#pragma unroll
          for (int i = 0; i < BN / 16; ++i) {
            const uint32_t a_col = a_base + (uint32_t)(i < 4 ? i * 8 : 64 + (i - 4) * 8);
            if (i == 0) umma_bf16_ts(d_col, a_col, desc(va + (uint32_t)(i * 128), dv_hi), idesc_pv, 0u);
            else umma_bf16_ts(d_col, a_col, desc(va + (uint32_t)(i * 128), dv_hi), idesc_pv, 1u);
          }
        } else {
          const int nsl = (nb_tail + 31) >> 5, seg_a = ((nsl + 1) >> 1) * 32;
          for (int kv0 = 0; kv0 < nb_tail; kv0 += 16) {
            const uint32_t a_col = a_base + (kv0 < seg_a ? (uint32_t)(kv0 >> 1) : (uint32_t)(seg_a + ((kv0 - seg_a) >> 1)));
            umma_bf16_ts(d_col, a_col, desc(va + (uint32_t)(kv0 * 8), dv_hi), idesc_pv, kv0 > 0 ? 1u : 0u);
          }
        }
        if (cur.j == cur.t) {
          umma_commit(&o_full[cur.tile & 1]);
          if (cur.t == p.nq - 1) umma_commit(&kv_empty[st]);          // last use of this item's K and V
        }
        cur.next();
        // the buffer's next scores: issued after the MMAs above, which read P from it
        if (b_ahead < n_blocks) { issue_scores(ahead, buf); ahead.next(); ++b_ahead; }
        if (++buf == NBUF) { buf = 0; buf_phase ^= 1; }
        if (++slot == NSLOT) slot = 0;
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp < 6) {
    // ------------------------------ output: warps 2..5 ------------------------------
    // Combines the tile's accumulator slots, stages the bf16 result in shared memory in the 128-byte-swizzled
    // layout of the output tensor map (64 columns at a time) and lets one TMA store write it: rows past the end
    // of the sequence are clipped by the tensor map.
    const int quad = warp & 3, row = quad * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c2 = p.scale_log2;
    uint8_t* stage_row = base + pl.ostage_off + row * 128;
    const bool storer = warp == 2 && lane == 0;
    bool dead = false;
    int b0 = 0;                                // index of the tile's first block among this CTA's blocks
    for (int g = 0; g < n_tiles; ++g) {
      named_bar_sync(OUT_BAR, 128);
      if (*abort_flag) break;                  // read after the barrier: the same answer in all four warps
      const int k = g / p.nq, t = g - k * p.nq;
      const int item = blockIdx.x + k * gridDim.x, seq = item / p.H, h = item - seq * p.H;
      {
        int ok = 1;
        if (lane == 0) {
          ok = *abort_flag ? 0 : 1;
          if (ok && !mbar_wait_bounded(&o_full[g & 1], (unsigned)(g >> 1) & 1u, WAIT_NS * 2ull)) { fa_timeout(SITE_O_FULL); ok = 0; }
          if (!ok) *abort_flag = 1;
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      }
      tc_fence_after();
      const int nj = t + 1, ring = g % STAT_RING;
      const int qi = t * BM + row;
      float mj[MAX_SLOTS], w[MAX_SLOTS];
      float m = -INFINITY;
#pragma unroll
      for (int j = 0; j < MAX_SLOTS; ++j) {
        mj[j] = j < nj ? stat_m[(ring * MAX_SLOTS + j) * BM + row] : -INFINITY;
        m = fmaxf(m, mj[j]);
      }
      float L = 0.f;
#pragma unroll
      for (int j = 0; j < MAX_SLOTS; ++j) {
        w[j] = j < nj ? ex2_approx((mj[j] - m) * c2) : 0.f;
        if (j < nj) {
          const float* lp = stat_l + ((ring * MAX_SLOTS + j) * 2) * BM + row;
          L = fmaf(w[j], lp[0] + lp[BM], L);
        }
      }
      const float inv = 1.f / L;
#pragma unroll
      for (int j = 0; j < MAX_SLOTS; ++j) w[j] *= inv;
#pragma unroll 1
      for (int cb = 0; cb < DH; cb += 64) {
        if (storer) bulk_wait_read_all();      // the previous store has finished reading the staging buffer
        named_bar_sync(OUT_BAR, 128);
#pragma unroll 1
        for (int cc = 0; cc < 64; cc += 32) {
          float acc[32];
#pragma unroll
          for (int e = 0; e < 32; ++e) acc[e] = 0.f;
          if (!dead) {
#pragma unroll
            for (int j = 0; j < MAX_SLOTS; ++j) {
              if (j < nj) {
                int sl = b0 + j;
                sl -= (sl / NSLOT) * NSLOT;
                uint32_t r[32];
                tmem_ld_32x32(lane_addr + (uint32_t)(O_COL + sl * DH + cb + cc), r);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) acc[e] = fmaf(w[j], __uint_as_float(r[e]), acc[e]);
              }
            }
          }
#pragma unroll
          for (int e = 0; e < 32; e += 8) {
            uint4 o;
            o.x = pack_bf16x2(acc[e], acc[e + 1]); o.y = pack_bf16x2(acc[e + 2], acc[e + 3]);
            o.z = pack_bf16x2(acc[e + 4], acc[e + 5]); o.w = pack_bf16x2(acc[e + 6], acc[e + 7]);
            const int chunk = (cc + e) >> 3;                            // 16-byte chunk of the 128-byte row
            *reinterpret_cast<uint4*>(stage_row + ((chunk ^ (row & 7)) << 4)) = o;
          }
        }
        fence_proxy_async_smem();
        named_bar_sync(OUT_BAR, 128);
        if (storer && !dead) {
          tma_store_3d(&tmO, base + pl.ostage_off, h * DH + cb, t * BM, seq);
          bulk_commit();
        }
      }
      if (!dead && qi < p.S) p.lse[((long long)seq * p.H + h) * p.S + qi] = (m * c2 + log2f(L)) * LN2;
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(&o_empty[g & 1]);
      b0 += nj;
    }
    if (storer) bulk_wait_read_all();
  } else {
    // ------------------------------ softmax: 8 warps per score buffer ------------------------------
    const int sw = warp - 6, buf = sw / SM_WARPS_PER_BUF, wq = sw % SM_WARPS_PER_BUF;
    const int quad = warp & 3, half = wq >> 2;                        // warps 6..9 -> quadrants 2,3,0,1
    const int row = quad * 32 + lane;
    const int pair_bar = 1 + buf * 4 + quad;                          // named barrier of the two warps sharing these rows
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * BN);
    float* my_red = red_max + (buf * 2 + half) * BM + row;
    const float* other_red = red_max + (buf * 2 + (half ^ 1)) * BM + row;
    const float c2 = p.scale_log2;
    bool dead = false;
    BlockIter it;
    it.init(p.nq);
    it.advance(buf);
    for (int b = buf; b < n_blocks; b += NBUF, it.advance(NBUF)) {
      named_bar_sync(pair_bar, 64);
      if (*abort_flag) break;                  // read after the barrier: the same answer in both warps of the pair
      const int nb = min(BN, p.n_total - it.j * BN);
      const int nsl = (nb + 31) >> 5, sl_a = (nsl + 1) >> 1;
      const int sl_lo = half ? sl_a : 0, sl_hi = half ? nsl : sl_a;
      const bool diag = it.j == it.t;
      // last valid column of this row inside a diagonal block (rows past the sequence are computed, never stored)
      const int lim = min(it.t * BM + row, p.S - 1) - it.j * BN;
      const int lim_warp = min(it.t * BM + quad * 32, p.S - 1) - it.j * BN;
      {
        int ok = 1;
        if (lane == 0) {
          ok = *abort_flag ? 0 : 1;
          if (ok && !mbar_wait_bounded(&s_full[buf], (unsigned)(b / NBUF) & 1u, WAIT_NS * 2ull)) { fa_timeout(SITE_S_FULL); ok = 0; }
          if (!ok) *abort_flag = 1;
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      }
      tc_fence_after();
      // pass 1: row maximum over this warp's slices of 32 columns
      float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
      if (!dead) {
        for (int sl = sl_lo; sl < sl_hi; ++sl) {
          uint32_t r[32];
          tmem_ld_32x32(lane_addr + (uint32_t)(sl * 32), r);
          tmem_ld_wait();
          if (!diag || sl * 32 + 31 <= lim_warp) {
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              m0 = fmaxf(m0, __uint_as_float(r[e])); m1 = fmaxf(m1, __uint_as_float(r[e + 1]));
              m2 = fmaxf(m2, __uint_as_float(r[e + 2])); m3 = fmaxf(m3, __uint_as_float(r[e + 3]));
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; e += 4) {
              m0 = (sl * 32 + e <= lim) ? fmaxf(m0, __uint_as_float(r[e])) : m0;
              m1 = (sl * 32 + e + 1 <= lim) ? fmaxf(m1, __uint_as_float(r[e + 1])) : m1;
              m2 = (sl * 32 + e + 2 <= lim) ? fmaxf(m2, __uint_as_float(r[e + 2])) : m2;
              m3 = (sl * 32 + e + 3 <= lim) ? fmaxf(m3, __uint_as_float(r[e + 3])) : m3;
            }
          }
        }
      }
      float m = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
      *my_red = m;
      named_bar_sync(pair_bar, 64);
      m = fmaxf(m, *other_red);                                        // column 0 of a block is never masked: finite
      const float mc = m * c2;
      // pass 2: P = exp2(s c - m c) as packed bf16 over scores this warp has already consumed
      float sum0 = 0.f, sum1 = 0.f;
      if (!dead) {
        for (int sl = sl_lo; sl < sl_hi; ++sl) {
          uint32_t r[32], pk[16];
          tmem_ld_32x32(lane_addr + (uint32_t)(sl * 32), r);
          tmem_ld_wait();
          if (!diag || sl * 32 + 31 <= lim_warp) {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float p0 = ex2_approx(fmaf(__uint_as_float(r[e]), c2, -mc));
              const float p1 = ex2_approx(fmaf(__uint_as_float(r[e + 1]), c2, -mc));
              sum0 += p0; sum1 += p1;
              pk[e >> 1] = pack_bf16x2(p0, p1);
            }
          } else {
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float p0 = (sl * 32 + e <= lim) ? ex2_approx(fmaf(__uint_as_float(r[e]), c2, -mc)) : 0.f;
              const float p1 = (sl * 32 + e + 1 <= lim) ? ex2_approx(fmaf(__uint_as_float(r[e + 1]), c2, -mc)) : 0.f;
              sum0 += p0; sum1 += p1;
              pk[e >> 1] = pack_bf16x2(p0, p1);
            }
          }
          const int pcol = half ? sl_a * 32 + (sl - sl_a) * 16 : sl * 16;
          tmem_st_32x16(lane_addr + (uint32_t)pcol, pk);
        }
        tmem_st_wait();
      }
      {
        const int ring = it.tile % STAT_RING;
        stat_l[((ring * MAX_SLOTS + it.j) * 2 + half) * BM + row] = sum0 + sum1;
        if (half == 0) stat_m[(ring * MAX_SLOTS + it.j) * BM + row] = m;
      }
      __threadfence_block();
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(&p_full[buf]);
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
// backward
// ------------------------------------------------------------------------------------------------
// Two launches of one kernel template, both built like the forward pass (TMA producer, MMA issue - here by two
// threads -, compute warps on tensor memory, output warps with a TMA store), both recomputing the probabilities
// from the saved log-sum-exp:
//   BW_DQ   item = (sequence, head, query tile i): the tile's Q_i and dO_i stay in shared memory, the key
//           blocks j <= i stream by.  Per block: S = Q_i K_j^T and dP = dO_i V_j^T into tensor memory;
//           the compute warps form dS = P o (dP - rowsum(dO o O)) with P = exp(S / sqrt(dh) - lse) and write
//           it as packed bf16 over the scores; dQ_i += dS K_j with dS as the tensor-memory A operand.
//           This launch also writes rowsum(dO o O) for the second one.
//   BW_DKV  item = (sequence, head, key block j): K_j and V_j stay, the query tiles i >= j stream by.
//           Per block: S^T = K_j Q_i^T and dP^T = V_j dO_i^T (rows = keys); P^T and dS^T are written over S^T,
//           side by side; dV_j += P^T dO_i and dK_j += dS^T Q_i.
// The streamed tile is the B operand twice: K-major for the first two products, MN-major (same bytes,
// another descriptor) for the accumulating ones.  Scores are double-buffered for head dim 64, so the
// tensor core forms the next block's scores while the compute warps work.  The output warps scale by
// 1 / sqrt(dh), rotate dQ and dK back through the rotary embedding when a table is given, and store.
enum { BW_DQ = 0, BW_DKV = 1 };
constexpr int BW_COMPUTE_WARPS = 16;            // four per tensor-memory lane quadrant: one 32-column slice each
constexpr int BW_ACC_WARP = 2 + 4 + BW_COMPUTE_WARPS;   // the warp whose lane 0 issues the accumulating products
constexpr int BW_THREADS = (BW_ACC_WARP + 1) * 32;
constexpr int BW_COMPUTE_BAR = 10;              // named barrier of the compute warps
constexpr int BW_OUT_BAR = 11;                  // named barrier of the output warps

template <int DH> struct BwCfg {
  static constexpr int NSBUF = DH == 64 ? 2 : 1;                      // score buffers
  static constexpr int DP_COL = NSBUF * BN;                           // dP buffer
  static constexpr int ACC_COL = DP_COL + BN;                         // two accumulators of DH columns
  // resident operand pairs: an item's pair can only be requested once the item FIX_STAGES back has ended, and items
  // are as short as one block, so three stages are needed to request it a whole item ahead of its use
  static constexpr int FIX_STAGES = DH == 64 ? 3 : 1;
  // streamed operand pairs in flight: a pair is held from its load until the block's last product has read it
  // (two blocks after its scores were issued), and its successor's load takes about a block and a half to land
  static constexpr int STR_STAGES = DH == 64 ? 3 : 2;
  static constexpr uint32_t TILE_BYTES = (DH / 64) * BM * 128u;       // one 128-row operand tile: DH/64 slabs of 16 KB
  static constexpr bool O_IN_SMEM = false;                            // BW_DQ could keep O_i resident too; the shared memory goes to the streamed ring instead
  static_assert(ACC_COL + 2 * DH <= TMEM_COLS, "tensor memory plan does not fit");
};

struct BwParams {
  int n_seq, S, H, d;
  int n_items;                                  // n_seq * H * nq
  int nq;                                       // 128-row tiles per sequence
  int n_total;                                  // S rounded up to 16
  float scale, scale_log2;                      // 1 / sqrt(dh), log2(e) / sqrt(dh)
  const float* lse;                             // [n_seq][H][S]
  float* dsum;                                  // [n_seq][H][S]: written by BW_DQ, read by BW_DKV
  const __nv_bfloat16* out;                     // [n_seq*S][d]
  const __nv_bfloat16* dout;                    // [n_seq*S][d]
  const float2* rope_tab;                       // [S][dh/2] (cos, sin) or nullptr
  __nv_bfloat16* dqkv;                          // [n_seq*S][3d]: the one-pass kernel stores rows itself
};

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x8(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
               "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}

// Walks this CTA's items and their blocks in issue order.  Item = ((sequence * H + head) * nq + tile); a BW_DQ
// item streams the key blocks 0 .. tile, a BW_DKV item the query tiles tile .. nq - 1.
struct BwShape { int nq, mode, grid, n_items, gmod; };   // gmod = grid % nq: how the tile index moves from item to item
struct BwIter {
  int k, item, tt, u, cnt, b;                   // k = local item count, b = local block count
  __device__ void setup(const BwShape& sh) {
    cnt = sh.mode == BW_DQ ? tt + 1 : sh.nq - tt;
    u = 0;
  }
  __device__ void init(const BwShape& sh) {
    k = 0; b = 0; item = blockIdx.x;
    tt = item % sh.nq;
    setup(sh);
  }
  __device__ bool valid(const BwShape& sh) const { return item < sh.n_items; }
  __device__ bool first() const { return u == 0; }
  __device__ bool last() const { return u == cnt - 1; }
  __device__ int stile(const BwShape& sh) const { return sh.mode == BW_DQ ? u : tt + u; }   // index of the streamed tile in its sequence
  __device__ bool diag(const BwShape& sh) const { return stile(sh) == tt; }
  __device__ void next(const BwShape& sh) {
    ++b;
    if (++u == cnt) {
      ++k; item += sh.grid;
      tt += sh.gmod;
      if (tt >= sh.nq) tt -= sh.nq;
      setup(sh);
    }
  }
};

// Shared-memory plan of the backward kernel (bytes, after 1024-byte alignment): resident pairs, streamed
// pairs, output staging, barriers, per-column or per-row statistics.
struct BwPlan {
  uint32_t fix_off, str_off, ostage_off, bar_off, stat_off, total;
};
template <int DH, int MODE>
__host__ __device__ inline BwPlan bw_make_plan() {
  BwPlan p;
  constexpr int n_fix = (MODE == BW_DQ && BwCfg<DH>::O_IN_SMEM) ? 3 : 2;     // tiles per resident group
  p.fix_off = 0;
  p.str_off = p.fix_off + BwCfg<DH>::FIX_STAGES * n_fix * BwCfg<DH>::TILE_BYTES;
  p.ostage_off = p.str_off + BwCfg<DH>::STR_STAGES * 2 * BwCfg<DH>::TILE_BYTES;
  p.bar_off = p.ostage_off + BM * 128;
  p.stat_off = p.bar_off + 256;
  p.total = p.stat_off + 2 * 2 * BM * 4 + 1024 /* alignment slack */;
  return p;
}

template <int DH, int MODE>
__global__ void __launch_bounds__(BW_THREADS, 1)
fa_tc_bwd_kernel(const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmDO,
                 const __grid_constant__ CUtensorMap tmOUT, const __grid_constant__ CUtensorMap tmDQKV, const BwParams p) {
  extern __shared__ uint8_t smem_raw[];
  using C = BwCfg<DH>;
  constexpr int NSLAB = DH / 64;
  constexpr int NSBUF = C::NSBUF;
  constexpr uint32_t TILE = C::TILE_BYTES, PAIR = 2 * TILE;
  const uint32_t raw_addr = smem_u32(smem_raw);
  uint8_t* base = smem_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
  const BwPlan pl = bw_make_plan<DH, MODE>();
  constexpr bool O_SMEM = MODE == BW_DQ && C::O_IN_SMEM;
  constexpr uint32_t FIXB = (O_SMEM ? 3u : 2u) * TILE;              // bytes of a resident group
  uint64_t* bars = reinterpret_cast<uint64_t*>(base + pl.bar_off);
  uint64_t* fix_full = bars;                   // [3] producer -> MMA: an item's resident pair has landed
  uint64_t* fix_empty = bars + 3;              // [3] MMA -> producer
  uint64_t* str_full = bars + 6;               // [4] producer -> MMA: a block's streamed pair has landed
  uint64_t* str_empty = bars + 10;             // [4] MMA -> producer
  uint64_t* sdp_full = bars + 20;              // MMA -> compute: S and dP of a block are in tensor memory
  // compute -> MMA threads: P / dS of the block are in tensor memory (16 warp arrivals).  Two barriers, used by
  // alternate blocks: the accumulating threads may still be on their way to block b's phase when block b + 1
  // completes, and a parity wait cannot tell a phase from the one two later on the same barrier; block b + 2, the
  // next one on this barrier, cannot complete before every accumulating thread has seen block b (its scores need
  // the score buffer those threads release).
  uint64_t* p_ready0 = bars + 21;
  uint64_t* acc_full = bars + 14;              // [2] MMA -> output warps: the item's accumulators are complete
  uint64_t* acc_empty = bars + 16;             // [2] output warps -> MMA (4 warp arrivals): dQ / dK accumulator read; items alternate
  uint64_t* accv_empty = bars + 18;            // [2] the same for the dV accumulator
  uint64_t* s_free = bars + 22;                // [2] accumulating MMAs -> score MMAs: P / dS of the block that used the score buffer have been read
  uint64_t* p_ready1 = bars + 24;
  auto p_ready = [&](int block) { return (block & 1) ? p_ready1 : p_ready0; };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
  volatile uint32_t* abort_flag = tmem_slot + 1;
  float* stat = reinterpret_cast<float*>(base + pl.stat_off);        // BW_DKV: [2][2][128] column statistics; BW_DQ: [4][128] partial row sums

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nb_tail = p.n_total - (p.nq - 1) * BN;                  // rows of a sequence's last tile that take part (multiple of 16)
  const BwShape shp = {p.nq, MODE, (int)gridDim.x, p.n_items, (int)(gridDim.x % p.nq)};

  if (threadIdx.x == 0) {
    for (int s = 0; s < 3; ++s) { mbar_init(&fix_full[s], 1); mbar_init(&fix_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { mbar_init(&acc_full[s], 1); mbar_init(&acc_empty[s], 4); mbar_init(&accv_empty[s], 4); }
    for (int s = 0; s < 4; ++s) { mbar_init(&str_full[s], 1); mbar_init(&str_empty[s], 1); }
    mbar_init(sdp_full, 1); mbar_init(p_ready0, BW_COMPUTE_WARPS); mbar_init(p_ready1, BW_COMPUTE_WARPS);
    mbar_init(&s_free[0], 1); mbar_init(&s_free[1], 1);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmQKV);
    prefetch_tmap(&tmDO);
    prefetch_tmap(&tmOUT);
    prefetch_tmap(&tmDQKV);
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
      // BW_DQ: resident = (Q_i, dO_i), streamed = (K_j, V_j).  BW_DKV: resident = (K_j, V_j), streamed = (Q_i, dO_i).
      bool ok = true;
      BwIter it;
      it.init(shp);
      int fs = 0, fph = 0, ss = 0, sph = 0;
      auto load_pair = [&](uint8_t* dst, bool qdo, int h, int tile, int seq, uint64_t* bar) {
        for (int sl = 0; sl < NSLAB; ++sl) {
          if (qdo) {
            tma_load_3d(dst + sl * 16384, &tmQKV, h * DH + sl * 64, tile * BM, seq, bar);
            tma_load_3d(dst + TILE + sl * 16384, &tmDO, h * DH + sl * 64, tile * BM, seq, bar);
          } else {
            tma_load_3d(dst + sl * 16384, &tmQKV, p.d + h * DH + sl * 64, tile * BM, seq, bar);
            tma_load_3d(dst + TILE + sl * 16384, &tmQKV, 2 * p.d + h * DH + sl * 64, tile * BM, seq, bar);
          }
        }
      };
      int fix_issued = 0;                         // items whose resident group has been requested
      auto load_resident = [&](int item) {
        const int sh = item / p.nq, h = sh % p.H, seq = sh / p.H, tile = item - sh * p.nq;
        if (!mbar_wait_bounded(&fix_empty[fs], (unsigned)fph ^ 1u, WAIT_NS)) { fa_timeout(SITE_KV_EMPTY); ok = false; return; }
        mbar_expect_tx(&fix_full[fs], FIXB);
        uint8_t* dst = base + pl.fix_off + fs * FIXB;
        load_pair(dst, MODE == BW_DQ, h, tile, seq, &fix_full[fs]);
        if (O_SMEM)
          for (int sl = 0; sl < NSLAB; ++sl) tma_load_3d(dst + 2 * TILE + sl * 16384, &tmOUT, h * DH + sl * 64, tile * BM, seq, &fix_full[fs]);
        if (++fs == C::FIX_STAGES) { fs = 0; fph ^= 1; }
        ++fix_issued;
      };
      while (it.valid(shp) && ok && !*abort_flag) {
        const int sh = it.item / p.nq, h = sh % p.H, seq = sh / p.H;
        const bool first = it.first();
        if (first && fix_issued <= it.k) load_resident(it.item);
        if (!ok) break;
        if (!mbar_wait_bounded(&str_empty[ss], (unsigned)sph ^ 1u, WAIT_NS)) { fa_timeout(SITE_Q_EMPTY); ok = false; break; }
        mbar_expect_tx(&str_full[ss], PAIR);
        load_pair(base + pl.str_off + ss * PAIR, MODE == BW_DKV, h, it.stile(shp), seq, &str_full[ss]);
        if (++ss == C::STR_STAGES) { ss = 0; sph ^= 1; }
        // Resident groups of the following items are requested as far ahead as there are free stages, so that their
        // loads overlap this item's blocks.  Only a stage that is free right now is taken (one poll per block): this
        // thread also feeds the streamed ring and must not sit in a wait for an item to end.
        while (ok && fix_issued < it.k + C::FIX_STAGES && blockIdx.x + (long long)fix_issued * gridDim.x < p.n_items &&
               mbar_try_wait(&fix_empty[fs], (unsigned)fph ^ 1u))
          load_resident(blockIdx.x + fix_issued * gridDim.x);
        if (!ok) break;
        it.next(shp);
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == 1 || warp == BW_ACC_WARP) {
    if (lane == 0) {
      // ------------------------------ MMA issuers ------------------------------
      // Two threads: a tcgen05.mma costs its issuing thread 70 to 140 cycles (most with the A operand in tensor
      // memory) and a block needs 16 (dQ pass) or 24 (dK / dV pass) of them.  Warp 1 issues the products that open a
      // block (scores, then dP) as far ahead as the buffers allow; the last warp issues the accumulating products
      // once the compute warps have written P / dS, and releases operands and accumulators.  What one thread's
      // products must wait for in the other's travels through barriers: p_ready (dP buffer consumed; P / dS written)
      // and s_free (a score buffer's P / dS have been read by the accumulating products).  (A third thread, one per
      // accumulator in the dK / dV pass, measured no faster.)
      bool ok = true;
      auto desc = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; };
      const uint64_t dfk = smem_desc(smem_u32(base + pl.fix_off), 16u, 1024u);        // resident tiles: K-major A operands
      const uint64_t dsk = smem_desc(smem_u32(base + pl.str_off), 16u, 1024u);        // streamed tiles, K-major B
      const uint64_t dsm = smem_desc(smem_u32(base + pl.str_off), 16384u, 1024u);     // streamed tiles, MN-major B
      const uint32_t dfk_lo = (uint32_t)dfk, dfk_hi = (uint32_t)(dfk >> 32);
      const uint32_t dsk_lo = (uint32_t)dsk, dsk_hi = (uint32_t)(dsk >> 32);
      const uint32_t dsm_lo = (uint32_t)dsm, dsm_hi = (uint32_t)(dsm >> 32);
      const uint32_t idesc_full = idesc_bf16(BN, 0), idesc_tail = idesc_bf16(nb_tail, 0), idesc_acc = idesc_bf16(DH, 1);
      // position of an issue stream in the operand rings
      struct Pos { BwIter it; int fs, ss, sph, fph; };
      auto pos_init = [&](Pos& q) { q.it.init(shp); q.fs = q.ss = q.sph = q.fph = 0; };
      auto pos_next = [&](Pos& q) {
        const bool item_end = q.it.last();
        q.it.next(shp);
        if (++q.ss == C::STR_STAGES) { q.ss = 0; q.sph ^= 1; }
        if (item_end && ++q.fs == C::FIX_STAGES) { q.fs = 0; q.fph ^= 1; }
      };
      if (warp == 1) {
        // ---- opening products: S (or S^T) into score buffer n % NSBUF, dP (dP^T) into the dP buffer ----
        Pos pa;
        pos_init(pa);
        for (int n = 0; pa.it.valid(shp) && ok; ++n) {
          if (*abort_flag) { ok = false; break; }
          const int sb = NSBUF == 2 ? (n & 1) : 0;
          // operands of the block (first use of both pairs)
          if (pa.it.first() && !mbar_wait_bounded(&fix_full[pa.fs], (unsigned)pa.fph, WAIT_NS)) { fa_timeout(SITE_KV_FULL); ok = false; break; }
          if (!mbar_wait_bounded(&str_full[pa.ss], (unsigned)pa.sph, WAIT_NS)) { fa_timeout(SITE_Q_FULL); ok = false; break; }
          // the score buffer: block n - NSBUF left P / dS in it until its accumulating products had read them
          if (n >= NSBUF && !mbar_wait_bounded(&s_free[sb], (unsigned)(n / NSBUF - 1) & 1u, WAIT_NS)) { fa_timeout(SITE_S_FULL); ok = false; break; }
          tc_fence_after();
          const uint32_t idesc = (pa.it.stile(shp) == p.nq - 1) ? idesc_tail : idesc_full;
          {
            const uint32_t a = dfk_lo + (uint32_t)pa.fs * (FIXB >> 4), bq = dsk_lo + (uint32_t)pa.ss * (PAIR >> 4);
            const uint32_t d_col = tmem_base + (uint32_t)(sb * BN);
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
              const uint32_t o = (uint32_t)((ks >> 2) * 1024 + (ks & 3) * 2);
              if (ks == 0) umma_bf16(d_col, desc(a + o, dfk_hi), desc(bq + o, dsk_hi), idesc, 0u);
              else umma_bf16(d_col, desc(a + o, dfk_hi), desc(bq + o, dsk_hi), idesc, 1u);
            }
          }
          // the dP buffer: free once the compute warps have read the previous block's dP
          if (n >= 1 && !mbar_wait_bounded(p_ready(n - 1), (unsigned)((n - 1) >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_P_FULL); ok = false; break; }
          tc_fence_after();
          {
            const uint32_t a = dfk_lo + (uint32_t)pa.fs * (FIXB >> 4) + (TILE >> 4), bq = dsk_lo + (uint32_t)pa.ss * (PAIR >> 4) + (TILE >> 4);
            const uint32_t d_col = tmem_base + (uint32_t)C::DP_COL;
#pragma unroll
            for (int ks = 0; ks < DH / 16; ++ks) {
              const uint32_t o = (uint32_t)((ks >> 2) * 1024 + (ks & 3) * 2);
              if (ks == 0) umma_bf16(d_col, desc(a + o, dfk_hi), desc(bq + o, dsk_hi), idesc, 0u);
              else umma_bf16(d_col, desc(a + o, dfk_hi), desc(bq + o, dsk_hi), idesc, 1u);
            }
          }
          umma_commit(sdp_full);                                       // this thread's S and dP of block n are complete
          pos_next(pa);
        }
      } else {
        // ---- accumulating products: D (+)= A[tensor memory, packed bf16 at a_col0] * streamed tile read MN-major ----
        Pos pc;
        pos_init(pc);
        auto issue_acc = [&](const Pos& q, uint32_t d_col, uint32_t a_col0, int which, bool fresh) {
          const uint32_t bq = dsm_lo + (uint32_t)q.ss * (PAIR >> 4) + (uint32_t)which * (TILE >> 4);
          const int nk = (q.it.stile(shp) == p.nq - 1 ? nb_tail : BN) >> 4;          // 16-row steps of the streamed tile
#pragma unroll
          for (int kk = 0; kk < BN / 16; ++kk) {
            if (kk < nk) {
              const uint32_t a_col = a_col0 + (uint32_t)((kk >> 1) * 32 + (kk & 1) * 8);   // slice kk/2, half kk%2
              umma_bf16_ts(d_col, a_col, desc(bq + (uint32_t)(kk * 128), dsm_hi), idesc_acc, (kk > 0 || !fresh) ? 1u : 0u);
            }
          }
        };
        int sb = 0;                               // score buffer of the current block
        for (int b = 0; pc.it.valid(shp) && ok; ++b) {
          if (*abort_flag) { ok = false; break; }
          if (!mbar_wait_bounded(p_ready(b), (unsigned)(b >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_P_FULL); ok = false; break; }
          const int k = pc.it.k;
          if (pc.it.first()) {
            // BW_DQ alternates between two accumulators: the one of item k was last read for item k - 2;
            // BW_DKV uses both accumulators for every item: wait for item k - 1
            const int prev = MODE == BW_DQ ? k - 2 : k - 1;
            if (prev >= 0 && !mbar_wait_bounded(&acc_empty[prev & 1], (unsigned)(prev >> 1) & 1u, WAIT_NS)) {
              fa_timeout(SITE_O_EMPTY); ok = false; break;
            }
          }
          tc_fence_after();
          const uint32_t s_col = tmem_base + (uint32_t)(sb * BN);
          const uint32_t acc0 = tmem_base + (uint32_t)C::ACC_COL, acc1 = acc0 + DH;
          const bool fresh = pc.it.first();
          if (MODE == BW_DKV) {
            issue_acc(pc, acc0, s_col + 16u, 0, fresh);                // dK += dS^T Q_i (dS^T sits beside P^T in the score buffer)
            if (fresh && k >= 1 && !mbar_wait_bounded(&accv_empty[(k - 1) & 1], (unsigned)((k - 1) >> 1) & 1u, WAIT_NS)) {
              fa_timeout(SITE_O_EMPTY); ok = false; break;
            }
            issue_acc(pc, acc1, s_col, 1, fresh);                      // dV += P^T dO_i
          } else {
            issue_acc(pc, (k & 1) ? acc1 : acc0, s_col, 0, fresh);     // dQ += dS K_j
          }
          umma_commit(&s_free[sb]);                                    // the score buffer may take the scores of block b + NSBUF
          umma_commit(&str_empty[pc.ss]);                              // the streamed pair has been read for the last time
          if (pc.it.last()) {
            umma_commit(&acc_full[k & 1]);
            umma_commit(&fix_empty[pc.fs]);
          }
          pos_next(pc);
          if (++sb == NSBUF) sb = 0;
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp < 6) {
    // ------------------------------ output: warps 2..5 ------------------------------
    // Scale by 1 / sqrt(dh) (dQ, dK), rotate back through the rotary embedding, stage 64 columns at a time in
    // the swizzled layout of the gradient tensor map, TMA store (rows past the sequence are clipped).  An
    // accumulator is handed back to the MMA thread as soon as it has been read into registers.
    const int quad = warp & 3, row = quad * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    uint8_t* stage_row = base + pl.ostage_off + row * 128;
    const bool storer = warp == 2 && lane == 0;
    constexpr int HALF = DH / 2;
    bool dead = false;
    BwIter it;
    it.init(shp);
    // a staged box = 64 bf16 columns of every row: begin, two chunks of 32 columns, end (which issues the TMA store)
    auto stage_begin = [&]() {
      if (storer) bulk_wait_read_all();        // the previous store has finished reading the staging buffer
      named_bar_sync(BW_OUT_BAR, 128);
    };
    auto stage_chunk = [&](const float* v, int cc) {
#pragma unroll
      for (int e = 0; e < 32; e += 8) {
        uint4 ov;
        ov.x = pack_bf16x2(v[e], v[e + 1]); ov.y = pack_bf16x2(v[e + 2], v[e + 3]);
        ov.z = pack_bf16x2(v[e + 4], v[e + 5]); ov.w = pack_bf16x2(v[e + 6], v[e + 7]);
        *reinterpret_cast<uint4*>(stage_row + ((((cc + e) >> 3) ^ (row & 7)) << 4)) = ov;
      }
    };
    auto stage_end = [&](int x, int tile, int seq) {
      fence_proxy_async_smem();
      named_bar_sync(BW_OUT_BAR, 128);
      if (storer && !dead) {
        tma_store_3d(&tmDQKV, base + pl.ostage_off, x, tile * BM, seq);
        bulk_commit();
      }
    };
    while (it.valid(shp)) {
      named_bar_sync(BW_OUT_BAR, 128);
      if (*abort_flag) break;                  // read after the barrier: the same answer in all four warps
      const int k = it.k, tile = it.tt;
      const int sh = it.item / p.nq, h = sh % p.H, seq = sh / p.H;
      {
        int ok = 1;
        if (lane == 0) {
          ok = *abort_flag ? 0 : 1;
          if (ok && !mbar_wait_bounded(&acc_full[k & 1], (unsigned)(k >> 1) & 1u, WAIT_NS * 2ull)) { fa_timeout(SITE_O_FULL); ok = 0; }
          if (!ok) *abort_flag = 1;
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      }
      tc_fence_after();
      const int pos = min(tile * BM + row, p.S - 1);                  // position of this row in its sequence
      constexpr int N_OUT = MODE == BW_DQ ? 1 : 2;                     // dQ | dK, dV
#pragma unroll 1
      for (int o = 0; o < N_OUT; ++o) {
        const uint32_t acc = lane_addr + (uint32_t)(C::ACC_COL + (MODE == BW_DQ ? (k & 1) : o) * DH);
        const bool rotate = p.rope_tab != nullptr && !(MODE == BW_DKV && o == 1);   // dV is not rotated
        const float sc = (MODE == BW_DKV && o == 1) ? 1.f : p.scale;
        const int x0 = (MODE == BW_DQ ? 0 : (o == 0 ? p.d : 2 * p.d)) + h * DH;
        uint64_t* release = (MODE == BW_DKV && o == 1) ? &accv_empty[k & 1] : &acc_empty[k & 1];
        if constexpr (DH == 64) {
          float v[64];
          if (!dead) {
            uint32_t r0[32], r1[32];
            tmem_ld_32x32(acc, r0);
            tmem_ld_32x32(acc + 32u, r1);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 32; ++e) { v[e] = __uint_as_float(r0[e]) * sc; v[32 + e] = __uint_as_float(r1[e]) * sc; }
          } else {
#pragma unroll
            for (int e = 0; e < 64; ++e) v[e] = 0.f;
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0 && !dead) mbar_arrive(release);                // the accumulator is in registers
          if (rotate) {
            // pair (c, c + 32): lo' = lo cos + hi sin, hi' = hi cos - lo sin
            const float2* tab = p.rope_tab + (long long)pos * HALF;
#pragma unroll
            for (int e = 0; e < 32; e += 2) {
              const float4 cs = *reinterpret_cast<const float4*>(tab + e);      // (cos, sin) of two pairs
              const float l0 = v[e], h0 = v[32 + e], l1 = v[e + 1], h1 = v[33 + e];
              v[e] = l0 * cs.x + h0 * cs.y; v[32 + e] = h0 * cs.x - l0 * cs.y;
              v[e + 1] = l1 * cs.z + h1 * cs.w; v[33 + e] = h1 * cs.z - l1 * cs.w;
            }
          }
          stage_begin();
          stage_chunk(v, 0);
          stage_chunk(v + 32, 32);
          stage_end(x0, tile, seq);
        } else {
#pragma unroll 1
          for (int cb = 0; cb < DH; cb += 64) {
            stage_begin();
#pragma unroll 1
            for (int cc = 0; cc < 64; cc += 32) {
              const int c0 = cb + cc;                                   // first output column of this chunk
              float v[32];
              if (!dead) {
                uint32_t r[32];
                tmem_ld_32x32(acc + (uint32_t)c0, r);
                tmem_ld_wait();
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = __uint_as_float(r[e]) * sc;
                if (rotate) {
                  const bool is_lo = c0 < HALF;
                  tmem_ld_32x32(acc + (uint32_t)(is_lo ? c0 + HALF : c0 - HALF), r);
                  tmem_ld_wait();
                  const float2* tab = p.rope_tab + (long long)pos * HALF + (is_lo ? c0 : c0 - HALF);
#pragma unroll
                  for (int e = 0; e < 32; e += 2) {
                    const float4 cs = *reinterpret_cast<const float4*>(tab + e);
                    const float o0 = __uint_as_float(r[e]) * sc, o1 = __uint_as_float(r[e + 1]) * sc;
                    v[e] = is_lo ? v[e] * cs.x + o0 * cs.y : v[e] * cs.x - o0 * cs.y;
                    v[e + 1] = is_lo ? v[e + 1] * cs.z + o1 * cs.w : v[e + 1] * cs.z - o1 * cs.w;
                  }
                }
              } else {
#pragma unroll
                for (int e = 0; e < 32; ++e) v[e] = 0.f;
              }
              if (c0 + 32 == DH) {                                      // last read of this accumulator
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && !dead) mbar_arrive(release);
              }
              stage_chunk(v, cc);
            }
            stage_end(x0 + cb, tile, seq);
          }
        }
      }
      // advance to the next item
      const int cnt = it.cnt;
      for (int i = 0; i < cnt; ++i) it.next(shp);
    }
    if (storer) bulk_wait_read_all();
  } else {
    // ------------------------------ compute: 16 warps, one 32-column slice each ------------------------------
    const int cw = warp - 6, quad = warp & 3, slice = cw >> 2;        // warps 6..9 -> quadrants 2,3,0,1
    const int row = quad * 32 + lane;
    const int ct = threadIdx.x - 6 * 32;                              // 0..511 within the compute warps
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c2 = p.scale_log2;
    bool dead = false;
    float lse2_row = INFINITY, dsum_row = 0.f;                         // BW_DQ: this row's statistics
    int cfs = 0;                                                       // BW_DQ: resident stage of the current item
    BwIter it;
    it.init(shp);
    // BW_DKV: lse * log2(e) (threads 0..127) and rowsum(dO o O) (threads 128..255) of one streamed query tile
    auto load_col_stat = [&](const BwIter& q) -> float {
      const int sh = q.item / p.nq, h = sh % p.H, seq = sh / p.H;
      const long long sb0 = ((long long)seq * p.H + h) * p.S;
      const int qi = q.stile(shp) * BM + (ct & (BM - 1));
      // raw values: the scaling by log2(e) happens where the value is stored, so that the load has a block to land
      if (ct < BM) return qi < p.S ? p.lse[sb0 + qi] : INFINITY;          // +inf: probability 0 past the sequence
      return qi < p.S ? p.dsum[sb0 + qi] : 0.f;
    };
    if (MODE == BW_DKV && it.valid(shp) && ct < 2 * BM) stat[ct] = load_col_stat(it) * (ct < BM ? LOG2E : 1.f);
    // BW_DQ: this row's quarter (DH/4 columns) of the item's forward output, zero past the sequence
    uint4 o_pref[DH / 32];
    float lse_pref = INFINITY;                                         // BW_DQ: this row's log-sum-exp (+inf past the sequence)
    auto load_o_quarter = [&](int item) {
      const int sh = item / p.nq, h = sh % p.H, seq = sh / p.H, qi = (item - sh * p.nq) * BM + row;
      lse_pref = qi < p.S ? p.lse[((long long)seq * p.H + h) * p.S + qi] : INFINITY;
      const __nv_bfloat16* src = p.out + ((long long)seq * p.S + qi) * p.d + h * DH + slice * (DH / 4);
#pragma unroll
      for (int cix = 0; cix < DH / 32; ++cix)
        o_pref[cix] = qi < p.S ? *reinterpret_cast<const uint4*>(src + cix * 8) : make_uint4(0u, 0u, 0u, 0u);
    };
    if (MODE == BW_DQ && it.valid(shp)) load_o_quarter(it.item);
    for (int b = 0; it.valid(shp); ++b, it.next(shp)) {
      const int sh = it.item / p.nq, h = sh % p.H, seq = sh / p.H;
      const long long stat_base = ((long long)seq * p.H + h) * p.S;
      float* cstat = stat + (b & 1) * 2 * BM;                          // BW_DKV: statistics of this block's queries
      named_bar_sync(BW_COMPUTE_BAR, BW_COMPUTE_WARPS * 32);           // statistics visible; also the block boundary for leaving
      if (*abort_flag) break;
      // BW_DKV: the next block's statistics are fetched now and stored at the end of this block
      float next_stat = 0.f;
      BwIter nx = it;
      nx.next(shp);
      const bool have_next = MODE == BW_DKV && nx.valid(shp) && ct < 2 * BM;
      if (have_next) next_stat = load_col_stat(nx);
      if (MODE == BW_DQ && it.first()) lse2_row = lse_pref * LOG2E;     // fetched one item ahead
      {
        int ok = 1;
        if (lane == 0) {
          ok = (dead || *abort_flag) ? 0 : 1;
          if (ok && !mbar_wait_bounded(sdp_full, (unsigned)b & 1u, WAIT_NS * 2ull)) { fa_timeout(SITE_S_FULL); ok = 0; }
          if (!ok) *abort_flag = 1;
        }
        if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      }
      if (MODE == BW_DQ && it.first()) {
        // rowsum(dO o O) of this query row: each of the quadrant's four warps takes a quarter of the columns.  The
        // item's tiles have landed (the scores above were formed from them).
        const int qi = it.tt * BM + row;
        float part = 0.f;
        {
          // dO_i sits in the resident group (128-byte-swizzled rows, DH/64 slabs); this row's quarter of O_i was
          // fetched from global memory one item ahead
          const int c0 = slice * (DH / 4);                              // first column of this warp's quarter
          const uint8_t* g_row = base + pl.fix_off + cfs * FIXB + TILE + (c0 >> 6) * 16384 + row * 128;
#pragma unroll
          for (int cix = 0; cix < DH / 32; ++cix) {
            const int chunk = ((((c0 & 63) >> 3) + cix) ^ (row & 7)) << 4;
            const uint4 a = o_pref[cix];
            const uint4 g = *reinterpret_cast<const uint4*>(g_row + chunk);
            const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
            const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&g);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 af = __bfloat1622float2(ah[i]), gf = __bfloat1622float2(gh[i]);
              part = fmaf(af.x, gf.x, part);
              part = fmaf(af.y, gf.y, part);
            }
          }
          if (it.item + (long long)gridDim.x < p.n_items) load_o_quarter(it.item + gridDim.x);   // the next item's
        }
        stat[slice * BM + row] = part;
        named_bar_sync(BW_COMPUTE_BAR, BW_COMPUTE_WARPS * 32);
        dsum_row = (stat[row] + stat[BM + row]) + (stat[2 * BM + row] + stat[3 * BM + row]);
        if (slice == 0 && qi < p.S) p.dsum[stat_base + qi] = dsum_row;
        if (++cfs == C::FIX_STAGES) cfs = 0;
      }
      tc_fence_after();
      const int nbc = it.stile(shp) == p.nq - 1 ? nb_tail : BN;           // columns of this block
      if (!dead && slice * 32 < nbc) {
        const uint32_t s_addr = lane_addr + (uint32_t)((b % NSBUF) * BN + slice * 32);
        const uint32_t dp_addr = lane_addr + (uint32_t)(C::DP_COL + slice * 32);
        // causal mask on the diagonal block.  BW_DQ: column (key) <= row (query).  BW_DKV: column (query) >= row (key).
        // 0 = every element of this warp's slice is kept, 1 = mixed, 2 = every element is masked
        int mode_mask = 0;
        if (it.diag(shp)) mode_mask = slice == quad ? 1 : ((MODE == BW_DQ ? slice > quad : slice < quad) ? 2 : 0);
        uint32_t ds_first[8];                                       // BW_DKV: dS^T of the first half, stored after the second half's scores are read
#pragma unroll 1
        for (int hc = 0; hc < 32; hc += 16) {
          uint32_t pp[8], pd8[8];
          if (mode_mask == 2) {
#pragma unroll
            for (int e = 0; e < 8; ++e) { pp[e] = 0u; pd8[e] = 0u; }
          } else {
            uint32_t rs[16], rd[16];
            tmem_ld_32x16(s_addr + (uint32_t)hc, rs);
            tmem_ld_32x16(dp_addr + (uint32_t)hc, rd);
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 16; e += 2) {
              float pr[2], ds[2];
#pragma unroll
              for (int u = 0; u < 2; ++u) {
                const int c = slice * 32 + hc + e + u;                  // column inside the block
                const float l2 = MODE == BW_DQ ? lse2_row : cstat[c];
                const float dsm = MODE == BW_DQ ? dsum_row : cstat[BM + c];
                float pv = ex2_approx(fmaf(__uint_as_float(rs[e + u]), c2, -l2));
                if (mode_mask == 1) {
                  const bool keep = MODE == BW_DQ ? (c <= row) : (c >= row);
                  pv = keep ? pv : 0.f;
                }
                pr[u] = pv;
                ds[u] = pv * (__uint_as_float(rd[e + u]) - dsm);
              }
              pp[e >> 1] = pack_bf16x2(pr[0], pr[1]);
              pd8[e >> 1] = pack_bf16x2(ds[0], ds[1]);
            }
          }
          // packed results go over this warp's own 32 score columns, each column only after it has been read:
          // P^T (BW_DQ: dS) into columns 0..15 (0..7 consumed in the first half, 8..15 in the second); BW_DKV keeps
          // dS^T beside it in columns 16..31, which are free once the second half has been read.  Nothing is
          // written into the dP buffer, so the next block's dP may be formed as soon as this block's has been read.
          if (MODE == BW_DQ) {
            tmem_st_32x8(s_addr + (uint32_t)(hc >> 1), pd8);           // dS over the scores
          } else {
            tmem_st_32x8(s_addr + (uint32_t)(hc >> 1), pp);            // P^T over S^T
            if (hc == 0) {
#pragma unroll
              for (int e = 0; e < 8; ++e) ds_first[e] = pd8[e];
            } else {
              tmem_st_32x8(s_addr + 16u, ds_first);                    // dS^T, first half
              tmem_st_32x8(s_addr + 24u, pd8);                         // dS^T, second half
            }
          }
        }
        tmem_st_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(p_ready(b));
      if (have_next) stat[((b + 1) & 1) * 2 * BM + ct] = next_stat * (ct < BM ? LOG2E : 1.f);
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

#include "attention_tc_bwd1.cuh"

// rowsum(dO o O) per (token, head) for head dim 64, written as dsum[sequence][head][position]: 16-byte chunks, eight
// consecutive lanes per head, fully coalesced; HBM-bound (reads O and dO once).
__global__ void __launch_bounds__(256)
fa_rowsum64_kernel(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout, float* __restrict__ dsum,
                   long long n_tokens, int S, int H) {
  const int cpr = H * 8;                                              // 16-byte chunks per token row
  const long long total = n_tokens * cpr;
  const long long stride = (long long)gridDim.x * blockDim.x;        // a multiple of 32: a head's 8 chunks stay in one lane group
  for (long long c0 = (long long)blockIdx.x * blockDim.x + threadIdx.x; c0 - (threadIdx.x & 31) < total; c0 += stride) {   // warp-uniform
    float part = 0.f;
    if (c0 < total) {
      const uint4 a = reinterpret_cast<const uint4*>(out)[c0], g = reinterpret_cast<const uint4*>(dout)[c0];
      const __nv_bfloat162* ah = reinterpret_cast<const __nv_bfloat162*>(&a);
      const __nv_bfloat162* gh = reinterpret_cast<const __nv_bfloat162*>(&g);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float2 af = __bfloat1622float2(ah[e]), gf = __bfloat1622float2(gh[e]);
        part = fmaf(af.x, gf.x, part);
        part = fmaf(af.y, gf.y, part);
      }
    }
    part += __shfl_xor_sync(0xffffffffu, part, 1);
    part += __shfl_xor_sync(0xffffffffu, part, 2);
    part += __shfl_xor_sync(0xffffffffu, part, 4);
    if ((threadIdx.x & 7) == 0 && c0 < total) {
      const long long tok = c0 / cpr;
      const int h = (int)(c0 - tok * cpr) >> 3;
      const long long seq = tok / S;
      dsum[(seq * H + h) * S + (tok - seq * S)] = part;
    }
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
  CUtensorMap tmO;
  if (!make_seq_tmap(&tmO, out, n_seq, S, d, d, BM)) return PCM_ERR_CUDA;
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(fa_tc_fwd_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT));
  const int grid = p.n_items < sm_count() ? p.n_items : sm_count();
  fa_tc_fwd_kernel<DH><<<grid, Cfg<DH>::THREADS, smem, s>>>(tmQ, tmKV, tmO, p);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}


template <int DH, int MODE>
static int bwd_launch_one(const CUtensorMap& tmQKV, const CUtensorMap& tmDO, const CUtensorMap& tmOUT, const CUtensorMap& tmDQKV, const BwParams& p,
                          cudaStream_t s) {
  const BwPlan pl = bw_make_plan<DH, MODE>();
  if (pl.total > SMEM_LIMIT) return PCM_ERR_SHAPE;
  const uint32_t smem = pl.total < SMEM_FLOOR ? SMEM_FLOOR : pl.total;
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(fa_tc_bwd_kernel<DH, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_LIMIT));
  const int grid = p.n_items < sm_count() ? p.n_items : sm_count();
  fa_tc_bwd_kernel<DH, MODE><<<grid, BW_THREADS, smem, s>>>(tmQKV, tmDO, tmOUT, tmDQKV, p);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

template <int DH>
static int bwd_launch(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                      int n_seq, int S, int H, const float2* rope_tab, cudaStream_t s) {
  const int d = H * DH;
  BwParams p;
  p.n_seq = n_seq; p.S = S; p.H = H; p.d = d;
  p.nq = (S + BM - 1) / BM;
  p.n_items = n_seq * H * p.nq;
  p.n_total = ((S + 15) / 16) * 16;
  p.scale = 1.f / sqrtf((float)DH);
  p.scale_log2 = LOG2E / sqrtf((float)DH);
  p.lse = lse; p.dsum = dsum;
  p.out = (const __nv_bfloat16*)out; p.dout = (const __nv_bfloat16*)dout;
  p.rope_tab = rope_tab;
  p.dqkv = (__nv_bfloat16*)dqkv;
  CUtensorMap tmQKV, tmDO, tmOUT, tmDQKV;
  if (!make_seq_tmap(&tmQKV, qkv, n_seq, S, 3LL * d, 3LL * d, BM) || !make_seq_tmap(&tmDO, dout, n_seq, S, d, d, BM) ||
      !make_seq_tmap(&tmOUT, out, n_seq, S, d, d, BM) ||
      !make_seq_tmap(&tmDQKV, dqkv, n_seq, S, 3LL * d, 3LL * d, BM))
    return PCM_ERR_CUDA;
  const int rc = bwd_launch_one<DH, BW_DQ>(tmQKV, tmDO, tmOUT, tmDQKV, p, s);     // also writes rowsum(dO o O) for the second launch
  if (rc != PCM_OK) return rc;
  return bwd_launch_one<DH, BW_DKV>(tmQKV, tmDO, tmOUT, tmDQKV, p, s);
}

// PCM_ATTN_BWD=2 keeps head dim 64 on the two-launch backward (dQ, then dK / dV), for comparison runs.
static bool one_pass_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("PCM_ATTN_BWD");
    v = (e && e[0] == '2') ? 0 : 1;
  }
  return v == 1;
}

static int bwd1_launch(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                       int n_seq, int S, int H, const float2* rope_tab, cudaStream_t s) {
  constexpr int DH = 64;
  const int d = H * DH;
  BwParams p;
  p.n_seq = n_seq; p.S = S; p.H = H; p.d = d;
  p.nq = (S + BM - 1) / BM;
  p.n_items = n_seq * H;
  p.n_total = ((S + 15) / 16) * 16;
  p.scale = 1.f / sqrtf((float)DH);
  p.scale_log2 = LOG2E / sqrtf((float)DH);
  p.lse = lse; p.dsum = dsum;
  p.out = (const __nv_bfloat16*)out; p.dout = (const __nv_bfloat16*)dout;
  p.rope_tab = rope_tab;
  p.dqkv = (__nv_bfloat16*)dqkv;
  CUtensorMap tmQKV, tmDO, tmDQKV;
  if (!make_seq_tmap(&tmQKV, qkv, n_seq, S, 3LL * d, 3LL * d, BM) || !make_seq_tmap(&tmDO, dout, n_seq, S, d, d, BM) ||
      !make_seq_tmap(&tmDQKV, dqkv, n_seq, S, 3LL * d, 3LL * d, BM))
    return PCM_ERR_CUDA;
  fa_rowsum64_kernel<<<sm_count() * 8, 256, 0, s>>>(p.out, p.dout, dsum, (long long)n_seq * S, S, H);
  PCM_LAUNCH_CHECK();
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(fa_tc_bwd1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)b1::SMEM_BYTES));
  const int grid = p.n_items < sm_count() ? p.n_items : sm_count();
  fa_tc_bwd1_kernel<<<grid, b1::THREADS, b1::SMEM_BYTES, s>>>(tmQKV, tmDO, tmDQKV, p);
  PCM_LAUNCH_CHECK();
  return PCM_OK;
}

}  // namespace fatc

bool attention_tc_supported(const void* qkv, const void* out, int S, int H, int dh) {
  if (dh != 64 && dh != 128) return false;
  if (S < 1 || S > fatc::S_MAX) return false;
  // the forward kernel keeps a whole sequence's K and V in shared memory: head dim 128 fits up to 320 rows
  if (fatc::make_plan(dh, ((S + 63) / 64) * 64, 1, 1).total > fatc::SMEM_LIMIT) return false;
  if ((((uintptr_t)qkv) | ((uintptr_t)out)) & 15) return false;
  (void)H;
  return fatc::attn_encode_fn() != nullptr;
}

int attention_bwd_bf16_tc(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                          int n_seq, int S, int H, int dh, const float2* rope_tab, cudaStream_t s) {
  if (!attention_tc_supported(qkv, out, S, H, dh) || ((((uintptr_t)dout) | ((uintptr_t)dqkv)) & 15)) return PCM_ERR_SHAPE;
  if (n_seq < 1) return PCM_OK;
  if (dh == 64 && fatc::one_pass_enabled()) return fatc::bwd1_launch(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s);
  return dh == 64 ? fatc::bwd_launch<64>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s)
                  : fatc::bwd_launch<128>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, rope_tab, s);
}

int attention_fwd_bf16_tc(const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh, cudaStream_t s) {
  if (!attention_tc_supported(qkv, out, S, H, dh)) return PCM_ERR_SHAPE;
  if (n_seq < 1) return PCM_OK;
  return dh == 64 ? fatc::fwd_launch<64>(qkv, out, lse, n_seq, S, H, s) : fatc::fwd_launch<128>(qkv, out, lse, n_seq, S, H, s);
}

static unsigned g_fa_last_status = 0;
// The raw status word of the last expired wait (bit 8 + site says which barrier): for diagnostics.
unsigned attention_tc_last_status() { return g_fa_last_status; }

// Reads and clears this file's device status word (synchronous copy).
int attention_tc_poll_status() {
  unsigned h = 0;
  if (cudaMemcpyFromSymbol(&h, g_fa_status, sizeof(h)) != cudaSuccess) return PCM_ERR_CUDA;
  if (h) {
    unsigned z = 0;
    cudaMemcpyToSymbol(g_fa_status, &z, sizeof(z));
    g_fa_last_status = h;
    return PCM_ERR_DEVICE_TIMEOUT;
  }
  return PCM_OK;
}

}  // namespace pcm
