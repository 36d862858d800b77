// Backward attention in one pass for head dim 64; included by attention_tc.cu inside namespace pcm::fatc.
//
// Item = (sequence, head).  Its key tiles j are taken one after the other; for key tile j the query tiles
// i = j .. nq-1 stream by (causal: the blocks at or below the diagonal).  Per block, with rows = keys:
//   S^T = K_j Q_i^T and dP^T = V_j dO_i^T go into tensor memory (two products with N = 128 queries);
//   the compute warps form P^T = exp(S^T / sqrt(dh) - lse) and dS^T = P^T o (dP^T - rowsum(dO o O)) and write both
//   as bf16 into shared memory, row per key, in the 128-byte-swizzled layout of a K-major operand;
//   dV_j += P^T dO_i and dK_j += dS^T Q_i read them as K-major A operands, dQ_i += dS K_j reads the same dS bytes
//   as an MN-major A operand (rows = queries).  S and P are formed once for all three gradients.
// Tensor memory (512 columns): S^T 128 | dP^T 128 | dK 64 | dV 64 | two dQ accumulators of 64.  With j ascending
// and i ascending inside it, at most two dQ tiles are live at once for S <= 384 (dQ_0 ends with the item's first
// block); the running count of dQ tiles picks the accumulator.
// Shared memory: K_j | V_j in two stages (the next key tile loads while this one is used), the item's query tiles
// Q_i | dO_i in three resident slots (each loaded once per item and released after its diagonal block), one P^T and
// one dS^T buffer.  The compute warps hold a block's results in registers until the previous block's products have
// read the buffers, so single buffers do not stall the tensor pipe.
// Roles: warp 0 TMA producer; warp 1 allocates tensor memory and issues the opening products; the last two warps issue
// the accumulating products (dV and dK; dQ); warps 2..5 read finished accumulators, scale, rotate dQ / dK back through the rotary
// embedding and store each tile with one TMA store, staged in an operand tile that has just been read for the last
// time; 16 compute warps (one 32-query slice of one lane quadrant each).  rowsum(dO o O) comes from a small kernel
// that runs before this one.

namespace b1 {
constexpr uint32_t TILE = BM * 128u;                     // 16 KB: 128 rows x 64 bf16
constexpr uint32_t PAIR = 2u * TILE;
constexpr int KV_STAGES = 2;
constexpr uint32_t HEAD = 256u + 2u * 2u * BM * 4u;      // barriers; (lse, rowsum(dO o O)) of a block's queries, two buffers
constexpr int THREADS = BW_THREADS + 32;                 // one more issuing warp than the two-launch kernel
constexpr int ACC_Q_WARP = BW_ACC_WARP + 1;
constexpr uint32_t KV_OFF = 0u;
constexpr uint32_t Q_OFF = KV_OFF + KV_STAGES * PAIR;
constexpr uint32_t P_OFF = Q_OFF + MAX_SLOTS * PAIR;
constexpr uint32_t DS_OFF = P_OFF + 2u * TILE;
constexpr uint32_t TILES = DS_OFF + 2u * TILE;           // 224 KB
constexpr uint32_t SMEM_BYTES = 227u * 1024u;            // everything an SM has; the tiles start at the first 1024-byte boundary after HEAD
static_assert(HEAD + 768u + TILES == SMEM_BYTES, "plan is sized for a 1024-byte-aligned dynamic shared memory base");
constexpr int COL_S = 0, COL_DP = BN, COL_DK = 2 * BN, COL_DV = COL_DK + 64, COL_DQ = COL_DV + 64;
static_assert(COL_DQ + 2 * 64 == TMEM_COLS, "tensor memory plan");
}  // namespace b1

// Walks this CTA's blocks in issue order: item k = (sequence, head) sh, key tile j, query tile i >= j.
struct B1Iter {
  int k, sh, j, i, b, g;                        // b = local block count, g = local count of key tiles (groups)
  __device__ void init() { k = 0; sh = blockIdx.x; j = 0; i = 0; b = 0; g = 0; }
  __device__ bool valid(int n_sh) const { return sh < n_sh; }
  __device__ bool group_first() const { return i == j; }          // also the diagonal block: dQ_i ends here
  __device__ bool group_last(int nq) const { return i == nq - 1; }
  __device__ void next(int nq) {
    ++b;
    if (i + 1 < nq) { ++i; return; }
    ++g;
    if (++j == nq) { j = 0; ++k; sh += gridDim.x; }
    i = j;
  }
};

// Asks for a tile of a 3-D tensor map to be brought into L2 (no shared-memory destination, nothing to wait for).
__device__ __forceinline__ void tma_prefetch_3d(const void* tmap, int x, int y, int z) {
  asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(tmap), "r"(x), "r"(y), "r"(z)
               : "memory");
}

// Named barrier that also ORs a flag over its participants: every thread gets the same answer, so a group of warps
// leaves a loop together and none is left waiting at the barrier.
__device__ __forceinline__ bool named_bar_or(int id, int nthreads, bool flag) {
  unsigned out;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %1, 0;\n\t"
      "barrier.cta.red.or.pred p, %2, %3, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(out)
      : "r"((unsigned)flag), "r"(id), "r"(nthreads)
      : "memory");
  return out != 0;
}

__global__ void __launch_bounds__(b1::THREADS, 1)
fa_tc_bwd1_kernel(const __grid_constant__ CUtensorMap tmQKV, const __grid_constant__ CUtensorMap tmDO,
                  const __grid_constant__ CUtensorMap tmDQKV, const BwParams p) {
  extern __shared__ uint8_t smem_raw[];
  using namespace b1;
  constexpr int DH = 64;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_raw);
  float* cstat = reinterpret_cast<float*>(smem_raw + 256);           // [2][lse * log2(e) of the block's 128 queries | rowsum(dO o O)]
  const uint32_t head_end = smem_u32(smem_raw) + HEAD;
  const uint32_t tiles_at = HEAD + ((1024u - (head_end & 1023u)) & 1023u);
  if (tiles_at + TILES > SMEM_BYTES) {                               // base not 1024-byte aligned: the plan does not fit
    if (threadIdx.x == 0) fa_timeout(SITE_PLAN);
    return;
  }
  uint8_t* base = smem_raw + tiles_at;
  uint64_t* kv_full = bars;                    // [2] producer -> opening MMAs: K_j | V_j landed
  uint64_t* kv_empty = bars + 2;               // [2] dQ's MMAs (the key tile's last readers) -> producer
  uint64_t* q_full = bars + 4;                 // [3] producer -> opening MMAs, compute warps: Q_i | dO_i landed
  uint64_t* q_empty = bars + 7;                // [3] dK / dV's MMAs of the tile's diagonal block and the storing thread (dQ_i, dK_i, dV_i were staged there) -> producer
  uint64_t* sdp_full = bars + 10;              // opening MMAs -> compute: S^T and dP^T of a block are in tensor memory
  uint64_t* sdp_read = bars + 11;              // compute (16 warps) -> opening MMAs: both have been read
  uint64_t* pds_ready = bars + 12;             // [2] compute (16 warps) -> accumulating MMAs: P^T and dS^T are in shared memory
  uint64_t* ds_free = bars + 15;               // accumulating MMAs (two threads) -> compute: the block's products have read P^T and dS^T
  uint64_t* dq_full = bars + 16;               // [2] accumulating MMAs -> output warps
  uint64_t* dq_empty = bars + 18;              // [2] output warps (4) -> accumulating MMAs
  uint64_t* dkv_full = bars + 20;
  uint64_t* dkv_empty = bars + 21;             // output warps (4): dK and dV have been read
  uint64_t* qi_done = bars + 22;               // dK / dV's MMAs -> output warps: a diagonal block's products have read Q_i | dO_i
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 25);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nq = p.nq, n_sh = p.n_seq * p.H;
  const int nb_tail = p.n_total - (nq - 1) * BN;                      // rows of a sequence's last tile that take part (multiple of 16)

  if (threadIdx.x == 0) {
    for (int s = 0; s < 2; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
    for (int s = 0; s < 3; ++s) { mbar_init(&q_full[s], 1); mbar_init(&q_empty[s], 2); }
    mbar_init(sdp_full, 1); mbar_init(sdp_read, BW_COMPUTE_WARPS);
    mbar_init(&pds_ready[0], BW_COMPUTE_WARPS); mbar_init(&pds_ready[1], BW_COMPUTE_WARPS);
    mbar_init(ds_free, 2);                                            // dS^T is read by both accumulating threads
    mbar_init(qi_done, 1);
    for (int s = 0; s < 2; ++s) { mbar_init(&dq_full[s], 1); mbar_init(&dq_empty[s], 4); }
    mbar_init(dkv_full, 1); mbar_init(dkv_empty, 4);
    *abort_flag = 0;
    fence_mbar_init();
    prefetch_tmap(&tmQKV);
    prefetch_tmap(&tmDO);
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
  auto desc = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | lo; };

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------ TMA producer ------------------------------
      // Two independent request streams, each in the order its consumers free the space: key tiles (K_j | V_j) into the
      // two stages, query tiles (Q_i | dO_i, once per item) into their slots.  Whichever has room goes next, so the next
      // item's query tiles load as soon as their diagonal blocks have ended and are not held up behind a key tile
      // whose stage is still in use.
      int kv_sh = blockIdx.x, kv_j = 0, kv_g = 0;           // next key tile: (sequence, head), tile, running count
      int q_sh = blockIdx.x, q_i = 0, q_k = 0;              // next query tile: (sequence, head), tile, item count
      unsigned long long t_idle = 0;
      while ((kv_sh < n_sh || q_sh < n_sh) && !*abort_flag) {
        bool moved = false;
        if (kv_sh < n_sh && mbar_test_wait(&kv_empty[kv_g & 1], ((unsigned)(kv_g >> 1) & 1u) ^ 1u)) {
          const int h = kv_sh % p.H, seq = kv_sh / p.H, st = kv_g & 1;
          if (kv_j == 0 && kv_sh + (int)gridDim.x < n_sh) {
            // an item's first request: ask L2 for the whole next item, so that its loads, which can only be issued
            // a block or two before they are needed, do not wait for DRAM
            const int nsh = kv_sh + gridDim.x, nh = nsh % p.H, nseq = nsh / p.H;
            for (int t = 0; t < nq; ++t) {
              tma_prefetch_3d(&tmQKV, nh * DH, t * BM, nseq);
              tma_prefetch_3d(&tmDO, nh * DH, t * BM, nseq);
              tma_prefetch_3d(&tmQKV, p.d + nh * DH, t * BM, nseq);
              tma_prefetch_3d(&tmQKV, 2 * p.d + nh * DH, t * BM, nseq);
            }
          }
          mbar_expect_tx(&kv_full[st], PAIR);
          uint8_t* dst = base + KV_OFF + st * PAIR;
          tma_load_3d(dst, &tmQKV, p.d + h * DH, kv_j * BM, seq, &kv_full[st]);
          tma_load_3d(dst + TILE, &tmQKV, 2 * p.d + h * DH, kv_j * BM, seq, &kv_full[st]);
          ++kv_g;
          if (++kv_j == nq) { kv_j = 0; kv_sh += gridDim.x; }
          moved = true;
        }
        if (q_sh < n_sh && mbar_test_wait(&q_empty[q_i], ((unsigned)q_k & 1u) ^ 1u)) {
          const int h = q_sh % p.H, seq = q_sh / p.H;
          mbar_expect_tx(&q_full[q_i], PAIR);
          uint8_t* dst = base + Q_OFF + q_i * PAIR;
          tma_load_3d(dst, &tmQKV, h * DH, q_i * BM, seq, &q_full[q_i]);
          tma_load_3d(dst + TILE, &tmDO, h * DH, q_i * BM, seq, &q_full[q_i]);
          if (++q_i == nq) { q_i = 0; ++q_k; q_sh += gridDim.x; }
          moved = true;
        }
        if (moved) {
          t_idle = 0;
        } else {                                            // nothing free: bounded like every other wait
          const unsigned long long now = global_timer_ns();
          if (t_idle == 0) t_idle = now;
          else if (now - t_idle > WAIT_NS) { fa_timeout(SITE_KV_EMPTY); *abort_flag = 1; break; }
          __nanosleep(100);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------ opening products: S^T, dP^T ------------------------------
      bool ok = true;
      const uint64_t dkv = smem_desc(smem_u32(base + KV_OFF), 16u, 1024u);       // K_j, V_j: K-major A
      const uint64_t dq = smem_desc(smem_u32(base + Q_OFF), 16u, 1024u);         // Q_i, dO_i: K-major B
      const uint32_t dkv_lo = (uint32_t)dkv, dkv_hi = (uint32_t)(dkv >> 32), dq_lo = (uint32_t)dq, dq_hi = (uint32_t)(dq >> 32);
      const uint32_t idesc_full = idesc_bf16(BN, 0), idesc_tail = idesc_bf16(nb_tail, 0);
      B1Iter it;
      for (it.init(); it.valid(n_sh) && ok; it.next(nq)) {
        if (*abort_flag) { ok = false; break; }
        if (it.group_first() && !mbar_wait_bounded(&kv_full[it.g & 1], (unsigned)(it.g >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_KV_FULL); ok = false; break; }
        if (it.j == 0 && !mbar_wait_bounded(&q_full[it.i], (unsigned)it.k & 1u, WAIT_NS)) { fa_timeout(SITE_Q_FULL); ok = false; break; }
        if (it.b >= 1 && !mbar_wait_bounded(sdp_read, (unsigned)(it.b - 1) & 1u, WAIT_NS)) { fa_timeout(SITE_S_FULL); ok = false; break; }
        tc_fence_after();
        const uint32_t idesc = it.i == nq - 1 ? idesc_tail : idesc_full;         // N = queries of tile i
        uint32_t a = dkv_lo + (uint32_t)(it.g & 1) * (PAIR >> 4), bq = dq_lo + (uint32_t)it.i * (PAIR >> 4);
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
          umma_bf16(tmem_base + COL_S, desc(a + ks * 2, dkv_hi), desc(bq + ks * 2, dq_hi), idesc, ks > 0 ? 1u : 0u);
        a += TILE >> 4; bq += TILE >> 4;
#pragma unroll
        for (int ks = 0; ks < DH / 16; ++ks)
          umma_bf16(tmem_base + COL_DP, desc(a + ks * 2, dkv_hi), desc(bq + ks * 2, dq_hi), idesc, ks > 0 ? 1u : 0u);
        umma_commit(sdp_full);
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp == BW_ACC_WARP || warp == ACC_Q_WARP) {
    if (lane == 0) {
      // ------------------------------ accumulating products ------------------------------
      // Two threads, each behind the same pds_ready barrier: one issues dV += P^T dO_i and dK += dS^T Q_i (16 products a
      // block), the other dQ_i += dS K_j (8).  An issue costs its thread 65 cycles or more, so one thread for all 24
      // would need longer than the tensor pipe does.
      bool ok = true;
      const uint64_t dpk = smem_desc(smem_u32(base + P_OFF), 16u, 1024u);        // P^T: K-major A (rows = keys)
      const uint64_t dsk = smem_desc(smem_u32(base + DS_OFF), 16u, 1024u);       // dS^T: K-major A
      const uint64_t dsm = smem_desc(smem_u32(base + DS_OFF), 16384u, 1024u);    // dS: the same bytes, MN-major A (rows = queries)
      const uint64_t dqm = smem_desc(smem_u32(base + Q_OFF), 16384u, 1024u);     // Q_i, dO_i: MN-major B
      const uint64_t dkm = smem_desc(smem_u32(base + KV_OFF), 16384u, 1024u);    // K_j: MN-major B
      const uint32_t dpk_lo = (uint32_t)dpk, dsk_lo = (uint32_t)dsk, dsm_lo = (uint32_t)dsm, dqm_lo = (uint32_t)dqm, dkm_lo = (uint32_t)dkm;
      const uint32_t hi_k = (uint32_t)(dpk >> 32), hi_m = (uint32_t)(dsm >> 32);
      const uint32_t idesc_kk = idesc_bf16(DH, 1), idesc_mm = idesc_kk | (1u << 15);
      B1Iter it;
      if (warp == BW_ACC_WARP) {
        for (it.init(); it.valid(n_sh) && ok; it.next(nq)) {
          if (*abort_flag) { ok = false; break; }
          if (!mbar_wait_bounded(&pds_ready[it.b & 1], (unsigned)(it.b >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_P_FULL); ok = false; break; }
          const bool first = it.group_first(), last = it.group_last(nq);
          // the output warps have read the previous key tile's dK and dV
          if (first && it.g >= 1 && !mbar_wait_bounded(dkv_empty, (unsigned)(it.g - 1) & 1u, WAIT_NS)) { fa_timeout(SITE_O_EMPTY); ok = false; break; }
          tc_fence_after();
          const int nkq = (it.i == nq - 1 ? nb_tail : BN) >> 4;                  // 16-query steps
          const uint32_t q_lo = dqm_lo + (uint32_t)it.i * (PAIR >> 4);
          const uint32_t acc = first ? 0u : 1u;
          umma_bf16(tmem_base + COL_DV, desc(dpk_lo, hi_k), desc(q_lo + (TILE >> 4), hi_m), idesc_kk, acc);
#pragma unroll
          for (int ks = 1; ks < BN / 16; ++ks)
            if (ks < nkq)
              umma_bf16(tmem_base + COL_DV, desc(dpk_lo + (uint32_t)((ks >> 2) * 1024 + (ks & 3) * 2), hi_k),
                        desc(q_lo + (TILE >> 4) + (uint32_t)(ks * 128), hi_m), idesc_kk, 1u);
          umma_bf16(tmem_base + COL_DK, desc(dsk_lo, hi_k), desc(q_lo, hi_m), idesc_kk, acc);
#pragma unroll
          for (int ks = 1; ks < BN / 16; ++ks)
            if (ks < nkq)
              umma_bf16(tmem_base + COL_DK, desc(dsk_lo + (uint32_t)((ks >> 2) * 1024 + (ks & 3) * 2), hi_k),
                        desc(q_lo + (uint32_t)(ks * 128), hi_m), idesc_kk, 1u);
          umma_commit(ds_free);
          if (last) umma_commit(dkv_full);
          if (first) { umma_commit(qi_done); umma_commit(&q_empty[it.i]); }      // tile i's last block in this item
        }
      } else {
        for (it.init(); it.valid(n_sh) && ok; it.next(nq)) {
          if (*abort_flag) { ok = false; break; }
          if (!mbar_wait_bounded(&pds_ready[it.b & 1], (unsigned)(it.b >> 1) & 1u, WAIT_NS)) { fa_timeout(SITE_P_FULL); ok = false; break; }
          const int cnt = it.k * nq + it.i, slot = cnt & 1;                      // running count of dQ tiles picks the accumulator
          if (it.j == 0 && cnt >= 2 && !mbar_wait_bounded(&dq_empty[slot], (unsigned)((cnt >> 1) - 1) & 1u, WAIT_NS)) {
            fa_timeout(SITE_O_EMPTY); ok = false; break;
          }
          tc_fence_after();
          const int nkk = (it.j == nq - 1 ? nb_tail : BN) >> 4;                  // 16-key steps
          const uint32_t k_lo = dkm_lo + (uint32_t)(it.g & 1) * (PAIR >> 4);
          const uint32_t d_col = tmem_base + (uint32_t)(COL_DQ + slot * DH);
          umma_bf16(d_col, desc(dsm_lo, hi_m), desc(k_lo, hi_m), idesc_mm, it.j > 0 ? 1u : 0u);
#pragma unroll
          for (int kk = 1; kk < BN / 16; ++kk)
            if (kk < nkk)
              umma_bf16(d_col, desc(dsm_lo + (uint32_t)(kk * 128), hi_m), desc(k_lo + (uint32_t)(kk * 128), hi_m), idesc_mm, 1u);
          umma_commit(ds_free);
          if (it.group_first()) umma_commit(&dq_full[slot]);                     // the diagonal block is dQ_i's last
          if (it.group_last(nq)) umma_commit(&kv_empty[it.g & 1]);
        }
      }
      if (!ok) *abort_flag = 1;
    }
  } else if (warp < 6) {
    // ------------------------------ output: warps 2..5, one lane quadrant each ------------------------------
    // A thread owns one row of an accumulator: 64 fp32 columns -> scale, inverse rotary embedding (dQ, dK) -> bf16 into
    // a staging tile in the swizzled layout of the gradient tensor map -> one TMA store (rows past the sequence are
    // clipped).  The staging tiles are the slot of query tile t, which no product reads after t's diagonal block: dQ_t
    // right after that block, dK_t and dV_t (both halves of the slot) after key tile t's last block; then the storing
    // thread hands the slot to the producer for the next item.  Accumulators are released as soon as they are in
    // registers.
    const int quad = warp & 3, row = quad * 32 + lane;
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const bool storer = warp == 2 && lane == 0;
    bool dead = false;
    auto wait_warp = [&](uint64_t* bar, unsigned parity) {
      int ok = 1;
      if (lane == 0) {
        ok = (dead || *abort_flag) ? 0 : 1;
        if (ok && !mbar_wait_bounded(bar, parity, WAIT_NS * 2ull)) { fa_timeout(SITE_O_FULL); ok = 0; }
        if (!ok) *abort_flag = 1;
      }
      if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
      tc_fence_after();
    };
    // which: 0 = dQ, 1 = dK, 2 = dV.  `release`: accumulator barrier (may be null); `operand_done` / parity: the barrier
    // after which `stage` may be overwritten.
    auto emit = [&](uint32_t col, uint64_t* release, int which, int tile, int seq, int h, uint64_t* operand_done,
                    unsigned od_parity, uint8_t* stage) {
      float v[64];
      if (!dead) {
        uint32_t r0[32], r1[32];
        tmem_ld_32x32(lane_addr + col, r0);
        tmem_ld_32x32(lane_addr + col + 32u, r1);
        tmem_ld_wait();
        const float sc = which == 2 ? 1.f : p.scale;
#pragma unroll
        for (int e = 0; e < 32; ++e) { v[e] = __uint_as_float(r0[e]) * sc; v[32 + e] = __uint_as_float(r1[e]) * sc; }
      } else {
#pragma unroll
        for (int e = 0; e < 64; ++e) v[e] = 0.f;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0 && release && !dead) mbar_arrive(release);
      if (which != 2 && p.rope_tab != nullptr) {
        // pair (c, c + 32): lo' = lo cos + hi sin, hi' = hi cos - lo sin
        const int pos = min(tile * BM + row, p.S - 1);
        const float2* tab = p.rope_tab + (long long)pos * (DH / 2);
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const float4 cs = *reinterpret_cast<const float4*>(tab + e);
          const float l0 = v[e], h0 = v[32 + e], l1 = v[e + 1], h1 = v[33 + e];
          v[e] = l0 * cs.x + h0 * cs.y; v[32 + e] = h0 * cs.x - l0 * cs.y;
          v[e + 1] = l1 * cs.z + h1 * cs.w; v[33 + e] = h1 * cs.z - l1 * cs.w;
        }
      }
      if (operand_done) wait_warp(operand_done, od_parity);
      uint8_t* stage_row = stage + row * 128;
#pragma unroll
      for (int e = 0; e < 64; e += 8) {
        uint4 ov;
        ov.x = pack_bf16x2(v[e], v[e + 1]); ov.y = pack_bf16x2(v[e + 2], v[e + 3]);
        ov.z = pack_bf16x2(v[e + 4], v[e + 5]); ov.w = pack_bf16x2(v[e + 6], v[e + 7]);
        *reinterpret_cast<uint4*>(stage_row + (((e >> 3) ^ (row & 7)) << 4)) = ov;
      }
      fence_proxy_async_smem();
      named_bar_sync(BW_OUT_BAR, 128);
      if (storer && !dead && !*abort_flag) {
        tma_store_3d(&tmDQKV, stage, which * p.d + h * DH, tile * BM, seq);
        bulk_commit();
      }
    };
    B1Iter it;
    for (it.init(); it.valid(n_sh); it.next(nq)) {
      if (named_bar_or(BW_OUT_BAR, 128, dead || *abort_flag)) break;     // all four warps leave together
      const int h = it.sh % p.H, seq = it.sh / p.H;
      if (it.group_first()) {
        const int cnt = it.k * nq + it.i, slot = cnt & 1;
        wait_warp(&dq_full[slot], (unsigned)(cnt >> 1) & 1u);
        emit((uint32_t)(COL_DQ + slot * DH), &dq_empty[slot], 0, it.i, seq, h, qi_done, (unsigned)it.g & 1u,
             base + Q_OFF + it.i * PAIR);
        if (storer) bulk_wait_read_all();                                 // dK_i will be staged over it
      }
      if (it.group_last(nq)) {
        wait_warp(dkv_full, (unsigned)it.g & 1u);
        named_bar_sync(BW_OUT_BAR, 128);                                  // the store of dQ_j has read its staging tile
        uint8_t* slot_j = base + Q_OFF + it.j * PAIR;
        // the two accumulators are released together: one arrival per warp, after dV has been read as well
        emit((uint32_t)COL_DK, nullptr, 1, it.j, seq, h, nullptr, 0u, slot_j);
        emit((uint32_t)COL_DV, dkv_empty, 2, it.j, seq, h, nullptr, 0u, slot_j + TILE);
        if (storer) {
          bulk_wait_read_all();
          if (!dead) mbar_arrive(&q_empty[it.j]);                         // query tile j's slot goes back to the producer
        }
      }
    }
    if (storer) bulk_wait_read_all();
  } else {
    // ------------------------------ compute: 16 warps, one 32-query slice of one lane quadrant each ------------------------------
    const int cw = warp - 6, quad = warp & 3, slice = cw >> 2;
    const int row = quad * 32 + lane;                                  // key inside tile j
    const int ct = threadIdx.x - 6 * 32;                               // 0..511
    const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c2 = p.scale_log2;
    bool dead = false;
    auto wait_warp = [&](uint64_t* bar, unsigned parity, int site) {
      int ok = 1;
      if (lane == 0) {
        ok = (dead || *abort_flag) ? 0 : 1;
        if (ok && !mbar_wait_bounded(bar, parity, WAIT_NS * 2ull)) { fa_timeout(site); ok = 0; }
        if (!ok) *abort_flag = 1;
      }
      if (!__shfl_sync(0xffffffffu, ok, 0)) dead = true;
    };
    // statistics of a block's 128 queries: lse (threads 0..127; +inf past the sequence gives probability 0) and
    // rowsum(dO o O) (threads 128..255), both from global memory.  Raw values: the scaling by log2(e) happens where the
    // value is stored, a block later, so that the load has that block to land.
    auto stat_of = [&](const B1Iter& q) -> float {
      const int qi = q.i * BM + (ct & (BM - 1));
      if (ct >= 2 * BM) return 0.f;
      const long long at = ((long long)(q.sh / p.H) * p.H + q.sh % p.H) * p.S + qi;
      if (ct < BM) return qi < p.S ? p.lse[at] : INFINITY;
      return qi < p.S ? p.dsum[at] : 0.f;
    };
    const float stat_scale = ct < BM ? LOG2E : 1.f;
    B1Iter it;
    it.init();
    if (it.valid(n_sh) && ct < 2 * BM) cstat[ct] = stat_of(it) * stat_scale;
    for (; it.valid(n_sh); it.next(nq)) {
      const int b = it.b;
      const float* cst = cstat + (b & 1) * 2 * BM;
      // statistics visible; also the block boundary at which all compute warps leave together
      if (named_bar_or(BW_COMPUTE_BAR, BW_COMPUTE_WARPS * 32, dead || *abort_flag)) break;
      B1Iter nx = it;
      nx.next(nq);
      const bool have_next = nx.valid(n_sh);
      const float stat_next = have_next ? stat_of(nx) : 0.f;
      wait_warp(sdp_full, (unsigned)b & 1u, SITE_S_FULL);
      tc_fence_after();
      const int nbc = it.i == nq - 1 ? nb_tail : BN;                   // query columns of this block
      const bool active = !dead && slice * 32 < nbc;
      // causal mask on the diagonal block: column (query) >= row (key).  0 = slice kept, 1 = mixed, 2 = slice masked
      int mode_mask = 0;
      if (it.group_first()) mode_mask = slice == quad ? 1 : (slice < quad ? 2 : 0);
      uint32_t pp[16], pd[16];                                         // P^T and dS^T of this thread's 32 columns, packed bf16
#pragma unroll
      for (int e = 0; e < 16; ++e) { pp[e] = 0u; pd[e] = 0u; }
      if (active && mode_mask != 2) {
        const uint32_t s_addr = lane_addr + (uint32_t)(COL_S + slice * 32);
        const uint32_t dp_addr = lane_addr + (uint32_t)(COL_DP + slice * 32);
#pragma unroll
        for (int hc = 0; hc < 32; hc += 16) {
          uint32_t rs[16], rd[16];
          tmem_ld_32x16(s_addr + (uint32_t)hc, rs);
          tmem_ld_32x16(dp_addr + (uint32_t)hc, rd);
          tmem_ld_wait();
          if (hc == 16) {                                              // both buffers are in registers: the next block's products may overwrite them
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(sdp_read);
          }
#pragma unroll
          for (int e = 0; e < 16; e += 4) {
            const int c0 = slice * 32 + hc + e;                        // statistics of four queries per 16-byte load
            const float4 l4 = *reinterpret_cast<const float4*>(cst + c0);
            const float4 d4 = *reinterpret_cast<const float4*>(cst + BM + c0);
            const float lv[4] = {l4.x, l4.y, l4.z, l4.w}, dv[4] = {d4.x, d4.y, d4.z, d4.w};
            float pr[4], ds[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              float pv = ex2_approx(fmaf(__uint_as_float(rs[e + u]), c2, -lv[u]));
              if (mode_mask == 1) pv = c0 + u >= row ? pv : 0.f;
              pr[u] = pv;
              ds[u] = pv * (__uint_as_float(rd[e + u]) - dv[u]);
            }
            pp[(hc + e) >> 1] = pack_bf16x2(pr[0], pr[1]);
            pp[((hc + e) >> 1) + 1] = pack_bf16x2(pr[2], pr[3]);
            pd[(hc + e) >> 1] = pack_bf16x2(ds[0], ds[1]);
            pd[((hc + e) >> 1) + 1] = pack_bf16x2(ds[2], ds[3]);
          }
        }
      } else {
        tc_fence_before();
        __syncwarp();
        if (lane == 0 && !dead) mbar_arrive(sdp_read);
      }
      // the buffers are single: the previous block's products must have read them
      uint8_t* prow = base + P_OFF + (slice >> 1) * TILE + row * 128;
      uint8_t* drow = base + DS_OFF + (slice >> 1) * TILE + row * 128;
      // (ds_free counts the commit that follows dK's products, which the same thread issues after dV's: it covers P^T too)
      if (b >= 1) wait_warp(ds_free, (unsigned)(b - 1) & 1u, SITE_P_FULL);
      if (active) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          *reinterpret_cast<uint4*>(prow + (((((slice & 1) << 2) + c) ^ (row & 7)) << 4)) =
              make_uint4(pp[4 * c], pp[4 * c + 1], pp[4 * c + 2], pp[4 * c + 3]);
      }
      if (active) {
#pragma unroll
        for (int c = 0; c < 4; ++c)
          *reinterpret_cast<uint4*>(drow + (((((slice & 1) << 2) + c) ^ (row & 7)) << 4)) =
              make_uint4(pd[4 * c], pd[4 * c + 1], pd[4 * c + 2], pd[4 * c + 3]);
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0 && !dead) mbar_arrive(&pds_ready[b & 1]);
      if (have_next && ct < 2 * BM) cstat[((b + 1) & 1) * 2 * BM + ct] = stat_next * stat_scale;
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
