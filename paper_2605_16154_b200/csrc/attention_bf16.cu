// Attention kernels instantiated for __nv_bfloat16 activations.
#include "attention_impl.cuh"

namespace pcm {
int attention_fwd_bf16(const void* qkv, void* out, float* lse, int n_seq, int S, int H, int dh, cudaStream_t s) {
  return attention_fwd_t<__nv_bfloat16>(qkv, out, lse, n_seq, S, H, dh, s);
}
int attention_bwd_bf16(const void* qkv, const void* out, const void* dout, const float* lse, float* dsum, void* dqkv,
                       int n_seq, int S, int H, int dh, cudaStream_t s) {
  return attention_bwd_t<__nv_bfloat16>(qkv, out, dout, lse, dsum, dqkv, n_seq, S, H, dh, s);
}
}  // namespace pcm
