// Dispatch of the attention entry points on the activation dtype: fp32 runs the SIMT kernels
// (attention_f32.cu), bf16 the tensor-core kernels (attention_mma.cu).
#include "internal.h"

namespace pcm {

int attention_fwd_f32(const void*, void*, float*, int, int, int, int, cudaStream_t);
int attention_fwd_bf16(const void*, void*, float*, int, int, int, int, cudaStream_t);
int attention_bwd_f32(const void*, const void*, const void*, const float*, float*, void*, int, int, int, int, cudaStream_t);
int attention_bwd_bf16(const void*, const void*, const void*, const float*, float*, void*, int, int, int, int, const float2*,
                       cudaStream_t);

int attention_fwd(int dtype, const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh,
                  cudaStream_t s) {
  if (S > 384 || n_seq > 65535) return PCM_ERR_SHAPE;
  return dtype == DT_F32 ? attention_fwd_f32(qkv, out, lse, n_seq, S, H, dh, s)
                         : attention_fwd_bf16(qkv, out, lse, n_seq, S, H, dh, s);
}

int attention_bwd(int dtype, const void* qkv, const void* out, const void* dout, const float* lse, float* dsum,
                  void* dqkv, int n_seq, int S, int H, int dh, cudaStream_t s, const float2* rope_tab) {
  if (S > 384 || n_seq > 65535) return PCM_ERR_SHAPE;
  if (dtype == DT_F32) return rope_tab ? PCM_ERR_ARG : attention_bwd_f32(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, s);
  return attention_bwd_bf16(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, rope_tab, s);
}

}  // namespace pcm
