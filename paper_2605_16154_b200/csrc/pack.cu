// Physical shrinking (Sec. 4.5): gather the kept chunks into a dense batch with bulk asynchronous
// copies (global -> shared -> global through the TMA engine); no thread touches the payload.
#include "async_ptx.cuh"
#include "internal.h"

struct pcm_ctx;   // opaque here; only the status word is needed
namespace pcm { unsigned* ctx_status(pcm_ctx*); }

namespace pcm {

constexpr int PK_STAGE_BYTES = 32 * 1024;
constexpr int PK_STAGES = 2;
constexpr int PK_PIECE_BYTES = 128 * 1024;        // prefix bytes handled by one CTA
constexpr unsigned long long PK_WAIT_LIMIT_NS = 2000000000ull;   // 2 s per mbarrier wait

// grid = (pieces_per_chunk + 1, n_kept).  blockIdx.x < pieces: a slice of the chunk's observation
// prefix (one contiguous span in both source and destination).  blockIdx.x == pieces: the 56
// action-token embedding rows (gathered rows -> one contiguous span) and the per-chunk metadata.
__global__ void __launch_bounds__(64)
pack_chunks_kernel(const uint8_t* __restrict__ obs, const uint8_t* __restrict__ e_act,
                   const uint8_t* __restrict__ tok, const float* __restrict__ logp_old,
                   const float* __restrict__ adv, const int32_t* __restrict__ kept_idx,
                   const int32_t* __restrict__ kept_off, int n_traj, int n_chunks, int n_kept,
                   long long prefix_bytes, int row_bytes, int pieces, uint8_t* __restrict__ X,
                   uint8_t* __restrict__ tgt, float* __restrict__ lpo, float* __restrict__ adv_c,
                   int32_t* __restrict__ src, unsigned* __restrict__ status) {
  extern __shared__ __align__(128) uint8_t stage_mem[];
  __shared__ __align__(8) uint64_t bars[PK_STAGES];
  const int j = blockIdx.y;
  const int c = kept_idx[j];
  if (c < 0 || c >= n_chunks) {
    if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_OFFSETS);
    return;
  }
  const long long chunk_out_bytes = prefix_bytes + (long long)PCM_ACT_DIM * row_bytes;
  uint8_t* dst_chunk = X + (long long)j * chunk_out_bytes;
  const bool emb = (int)blockIdx.x == pieces;

  if (emb) {
    for (int t = threadIdx.x; t < PCM_ACT_DIM; t += blockDim.x) {
      tgt[(size_t)j * PCM_ACT_DIM + t] = tok[(size_t)c * PCM_ACT_DIM + t];
      lpo[(size_t)j * PCM_ACT_DIM + t] = logp_old[(size_t)c * PCM_ACT_DIM + t];
    }
    if (threadIdx.x == 32) {
      int lo = 0, hi = n_traj;                           // last i with kept_off[i] <= j
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (kept_off[mid] <= j) lo = mid; else hi = mid;
      }
      adv_c[j] = adv[lo];
      src[j] = c;
    }
  }
  if (threadIdx.x != 0) return;

  for (int s = 0; s < PK_STAGES; ++s) mbar_init(&bars[s], 1);
  fence_mbar_init();

  // tile list: prefix slice -> spans of PK_STAGE_BYTES; embedding piece -> groups of whole rows
  long long span_lo = 0, span_hi = 0;
  int rows_per_tile = 0, n_tiles = 0;
  if (!emb) {
    span_lo = (long long)blockIdx.x * PK_PIECE_BYTES;
    span_hi = span_lo + PK_PIECE_BYTES < prefix_bytes ? span_lo + PK_PIECE_BYTES : prefix_bytes;
    n_tiles = (int)((span_hi - span_lo + PK_STAGE_BYTES - 1) / PK_STAGE_BYTES);
  } else {
    rows_per_tile = PK_STAGE_BYTES / row_bytes;
    n_tiles = (PCM_ACT_DIM + rows_per_tile - 1) / rows_per_tile;
  }
  const uint8_t* src_chunk = obs + (long long)c * prefix_bytes;

  auto issue = [&](int k) {
    const int st = k % PK_STAGES;
    uint8_t* buf = stage_mem + (size_t)st * PK_STAGE_BYTES;
    if (!emb) {
      const long long lo = span_lo + (long long)k * PK_STAGE_BYTES;
      const unsigned bytes = (unsigned)((span_hi - lo) < PK_STAGE_BYTES ? (span_hi - lo) : PK_STAGE_BYTES);
      mbar_expect_tx(&bars[st], bytes);
      bulk_g2s(buf, src_chunk + lo, bytes, &bars[st]);
    } else {
      const int r0 = k * rows_per_tile;
      const int nr = (PCM_ACT_DIM - r0) < rows_per_tile ? (PCM_ACT_DIM - r0) : rows_per_tile;
      mbar_expect_tx(&bars[st], (unsigned)(nr * row_bytes));
      for (int r = 0; r < nr; ++r) {
        const unsigned t = tok[(size_t)c * PCM_ACT_DIM + r0 + r];
        bulk_g2s(buf + (size_t)r * row_bytes, e_act + (size_t)t * row_bytes, (unsigned)row_bytes, &bars[st]);
      }
    }
  };
  auto drain = [&](int k) {
    const int st = k % PK_STAGES;
    const uint8_t* buf = stage_mem + (size_t)st * PK_STAGE_BYTES;
    if (!emb) {
      const long long lo = span_lo + (long long)k * PK_STAGE_BYTES;
      const unsigned bytes = (unsigned)((span_hi - lo) < PK_STAGE_BYTES ? (span_hi - lo) : PK_STAGE_BYTES);
      bulk_s2g(dst_chunk + lo, buf, bytes);
    } else {
      const int r0 = k * rows_per_tile;
      const int nr = (PCM_ACT_DIM - r0) < rows_per_tile ? (PCM_ACT_DIM - r0) : rows_per_tile;
      bulk_s2g(dst_chunk + prefix_bytes + (long long)r0 * row_bytes, buf, (unsigned)(nr * row_bytes));
    }
    bulk_commit();
  };

  for (int k = 0; k < n_tiles && k < PK_STAGES; ++k) issue(k);
  for (int k = 0; k < n_tiles; ++k) {
    const int st = k % PK_STAGES;
    if (!mbar_wait_bounded(&bars[st], (unsigned)((k / PK_STAGES) & 1), PK_WAIT_LIMIT_NS)) {
      atomicOr(status, STATUS_TIMEOUT);
      break;
    }
    drain(k);
    if (k + PK_STAGES < n_tiles) {
      bulk_wait_read_all();                              // the stage's store has finished reading shared memory
      issue(k + PK_STAGES);
    }
  }
  bulk_wait_read_all();
}

}  // namespace pcm

using namespace pcm;

extern "C" int grpo_pack_chunks(pcm_ctx* ctx, const pcm_batch* b, const grpo_model_cfg* cfg, const int32_t* kept_idx,
                                const int32_t* kept_off, const void* e_act, const float* adv, grpo_packed* out,
                                pcm_stream stream) {
  if (!ctx || !b || !cfg || !kept_idx || !kept_off || !e_act || !adv || !out) return PCM_ERR_ARG;
  if (!b->obs || !b->tok || !b->logp_old || !out->X || !out->tgt || !out->lpo || !out->adv_c || !out->src)
    return PCM_ERR_ARG;
  if (out->n_kept < 0 || b->n_traj <= 0 || cfg->prefix_len < 1 || cfg->d < 1) return PCM_ERR_ARG;
  if (cfg->dtype != GRPO_F32 && cfg->dtype != GRPO_BF16) return PCM_ERR_ARG;
  const int es = cfg->dtype == GRPO_BF16 ? 2 : 4;
  const long long row_bytes = (long long)cfg->d * es;
  if (row_bytes % 16 || row_bytes > PK_STAGE_BYTES) return PCM_ERR_SHAPE;
  if (((uintptr_t)b->obs | (uintptr_t)e_act | (uintptr_t)out->X) & 15) return PCM_ERR_ARG;
  if (out->n_kept == 0) return PCM_OK;
  if (out->n_kept > 65535) return PCM_ERR_SHAPE;
  const long long prefix_bytes = (long long)cfg->prefix_len * row_bytes;
  const int pieces = (int)((prefix_bytes + PK_PIECE_BYTES - 1) / PK_PIECE_BYTES);
  const size_t smem = (size_t)PK_STAGES * PK_STAGE_BYTES;
  static unsigned long long attr_devices = 0;
  if (attr_needed(&attr_devices))
    PCM_CUDA_TRY(cudaFuncSetAttribute(pack_chunks_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid(pieces + 1, out->n_kept);
  prof_begin(PC_PACK, (cudaStream_t)stream);
  pack_chunks_kernel<<<grid, 64, smem, (cudaStream_t)stream>>>(
      (const uint8_t*)b->obs, (const uint8_t*)e_act, b->tok, b->logp_old, adv, kept_idx, kept_off, b->n_traj,
      b->n_chunks, out->n_kept, prefix_bytes, (int)row_bytes, pieces, (uint8_t*)out->X, out->tgt, out->lpo,
      out->adv_c, out->src, ctx_status(ctx));
  PCM_LAUNCH_CHECK();
  prof_end((cudaStream_t)stream, 0.0, (double)out->n_kept * (2.0 * prefix_bytes + 2.0 * PCM_ACT_DIM * row_bytes));
  return PCM_OK;
}
