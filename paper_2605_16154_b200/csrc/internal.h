// Internal interfaces between the translation units of the library (not part of the C ABI).
#pragma once
#include "common.cuh"
#include "head_loss.cuh"

namespace pcm {

enum { DT_F32 = 0, DT_BF16 = 1 };

// C[m][n] = sum_k A(m,k) * B(n,k)  (+ R[m][n] when R != nullptr; R may alias C to accumulate).
// An operand is "K-major" when its contraction index is contiguous in memory:
//   a_kmajor: A stored [M][K] with row stride lda;   otherwise A stored [K][M] with row stride lda.
//   b_kmajor: B stored [N][K] with row stride ldb;   otherwise B stored [K][N] with row stride ldb.
// Work fused into the tensor-core GEMM's epilogue (ignored by the SIMT kernel: callers use it only
// when gemm_tcgen05_supported() holds).
enum { EPI_NONE = 0, EPI_SWIGLU_FWD = 1, EPI_SWIGLU_BWD = 2, EPI_ROPE = 3, EPI_HEAD_LOSS = 4 };
struct GemmEpilogue {
  int kind = EPI_NONE;
  // EPI_SWIGLU_FWD: B is [2F][K] (gate rows, then up rows); C receives gate | up as [M][2F] and
  //                 out2 [M][F] receives silu(gate) * up, both from the fp32 accumulators.
  // EPI_SWIGLU_BWD: the product is d(act) [M][F]; aux = gate | up [M][2F]; C [M][2F] receives
  //                 d(gate) | d(up); d(act) itself is never stored.
  // EPI_ROPE:       C = q | k | v [M][3d]; columns below 2d are rotated (pairs (i, i + dh/2) of each
  //                 head, position = row % S) with the (cos, sin) table before the bf16 store.
  const void* aux = nullptr; long long ld_aux = 0;
  void* out2 = nullptr; long long ld_out2 = 0;
  // EPI_HEAD_LOSS:  the product is the logits z [M][256] of the scored rows (N = 256: a row's whole vocabulary is
  //                 one accumulator tile); the epilogue turns them into log-probs, loss terms and, with
  //                 hl.want_dz, C = d loss / d z [M][256] bf16.  z is never stored.
  const float2* rope_tab = nullptr; int S = 0, dh = 0, d = 0;
  HeadLossArgs hl;
};

struct GemmArgs {
  int M, N, K;
  const void* A; long long lda; bool a_kmajor;
  const void* B; long long ldb; bool b_kmajor;
  int ab_dtype;                 // DT_F32 or DT_BF16 (both operands)
  void* C; long long ldc; int c_dtype;
  const float* R; long long ldr;
  GemmEpilogue epi;
  // Optional continuation of the contraction: sum_k A(m,k) B(n,k) + sum_k2 A2(m,k2) B2(n,k2), with A2 / B2 laid out
  // like A / B (same major-ness, own row strides) and K2 <= 64 a multiple of 16.  This is how a low-rank adapter
  // branch enters the accumulator before any fused epilogue: [x | x A^T] [W | B]^T.
  const void* A2 = nullptr; long long lda2 = 0;
  const void* B2 = nullptr; long long ldb2 = 0;
  int K2 = 0;
  float alpha = 1.f;            // the product is scaled by alpha before R is added (plain epilogue, no reduction)
};

enum GemmBackend { GEMM_AUTO = 0, GEMM_SIMT = 1, GEMM_TCGEN05 = 2 };

int gemm(const GemmArgs& g, cudaStream_t s, GemmBackend backend = GEMM_AUTO);
int gemm_simt(const GemmArgs& g, cudaStream_t s);
int gemm_tcgen05(const GemmArgs& g, cudaStream_t s);
bool gemm_tcgen05_supported(const GemmArgs& g);
// True when gemm() would run g on the CTA-pair kernel (256 x 256 tiles) rather than on a single-CTA or SIMT kernel.
bool gemm_runs_on_pairs(const GemmArgs& g);
bool gemm_tcgen05_pair(const GemmArgs& g);      // the tensor-core path's own choice, given that it takes g
// True when the tensor-core kernel can run g including its fused epilogue.
bool gemm_epilogue_supported(const GemmArgs& g);
// Reads and clears the tensor-core kernels' device status word (synchronous copy).
int tcgen05_poll_status();

// Causal attention within each sequence of S tokens.  qkv [n_seq*S][3d] (q | k | v, heads of dh
// inside each), out [n_seq*S][d], lse [n_seq][H][S].
int attention_fwd(int dtype, const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh,
                  cudaStream_t s);
// dqkv [n_seq*S][3d] receives dq | dk | dv.  dsum [n_seq][H][S] is scratch.  With rope_tab (bf16 only:
// the [S][dh/2] table of (cos, sin)) dq and dk are rotated back, i.e. they are the gradients with
// respect to q and k before the rotary embedding.
int attention_bwd(int dtype, const void* qkv, const void* out, const void* dout, const float* lse, float* dsum,
                  void* dqkv, int n_seq, int S, int H, int dh, cudaStream_t s, const float2* rope_tab = nullptr);

// Event-pair profiling (profile.cu).  prof_begin/prof_end nest like a stack and cost nothing when off.
enum { PC_GEMM = 0, PC_ATTN = 1, PC_NORM = 2, PC_ELEM = 3, PC_LOSS = 4, PC_EMBED = 5, PC_PACK = 6, PC_SCORE = 7, PC_SAMPLE = 8,
       PC_GEMM_SMALL = 9 };
bool prof_enabled();
void prof_begin(int cls, cudaStream_t s);
void prof_end(cudaStream_t s, double flops, double bytes);

}  // namespace pcm
