// Dispatch of the attention entry points on the activation dtype: fp32 runs the SIMT kernels
// (attention_f32.cu); bf16 runs the tcgen05 kernels (attention_tc.cu) when they take the shape (head dim 64 or
// 128, S <= 384, 16-byte aligned tensors), else the warp-level mma.sync kernels (attention_mma.cu: head dim 32).
#include <cstdlib>

#include "internal.h"

namespace pcm {

int attention_fwd_f32(const void*, void*, float*, int, int, int, int, cudaStream_t);
int attention_fwd_bf16(const void*, void*, float*, int, int, int, int, cudaStream_t);
int attention_bwd_f32(const void*, const void*, const void*, const float*, float*, void*, int, int, int, int, cudaStream_t);
int attention_bwd_bf16(const void*, const void*, const void*, const float*, float*, void*, int, int, int, int, const float2*,
                       cudaStream_t);

bool attention_tc_supported(const void* qkv, const void* out, int S, int H, int dh);
int attention_fwd_bf16_tc(const void*, void*, float*, int, int, int, int, cudaStream_t);
int attention_bwd_bf16_tc(const void*, const void*, const void*, const float*, float*, void*, int, int, int, int, const float2*,
                          cudaStream_t);

// PCM_ATTN_TC=0 keeps bf16 attention on the warp-level (mma.sync) kernels, for comparison runs.
static bool attn_tc_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("PCM_ATTN_TC");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v == 1;
}

int attention_fwd(int dtype, const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh,
                  cudaStream_t s) {
  if (S > 384 || n_seq > 65535) return PCM_ERR_SHAPE;
  if (dtype == DT_F32) return attention_fwd_f32(qkv, out, lse, n_seq, S, H, dh, s);
  if (attn_tc_enabled() && attention_tc_supported(qkv, out, S, H, dh))
    return attention_fwd_bf16_tc(qkv, out, lse, n_seq, S, H, dh, s);
  return attention_fwd_bf16(qkv, out, lse, n_seq, S, H, dh, s);
}

int attention_bwd(int dtype, const void* qkv, const void* out, const void* dout, const float* lse, float* dsum,
                  void* dqkv, int n_seq, int S, int H, int dh, cudaStream_t s, const float2* rope_tab) {
  if (S > 384 || n_seq > 65535) return PCM_ERR_SHAPE;
  if (dtype == DT_F32) return rope_tab ? PCM_ERR_ARG : attention_bwd_f32(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, s);
  if (attn_tc_enabled() && attention_tc_supported(qkv, out, S, H, dh) && !((((uintptr_t)dout) | ((uintptr_t)dqkv)) & 15))
    return attention_bwd_bf16_tc(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, rope_tab, s);
  return attention_bwd_bf16(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, rope_tab, s);
}

}  // namespace pcm
