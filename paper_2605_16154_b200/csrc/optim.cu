// Optimizer step after the actor update (App. E): global-norm gradient clipping and AdamW on fp32 master
// weights, with the model-dtype copy of every weight rewritten in the same pass.  HBM bound: 16 B read and
// 12 + sizeof(T) B written per parameter.
#include <cmath>

#include "internal.h"

namespace pcm {

constexpr int OPT_NORM_BLOCKS = 296;          // 2 CTAs per SM
constexpr int OPT_MAX_TENSORS = 9;

__global__ void __launch_bounds__(256)
sumsq_kernel(const float* __restrict__ g, long long n, double* __restrict__ partial) {
  __shared__ double red[256];
  double acc = 0.0;
  const long long n4 = n >> 2;
  const float4* g4 = reinterpret_cast<const float4*>(g);
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
    const float4 v = g4[i];
    acc += (double)v.x * v.x + (double)v.y * v.y + (double)v.z * v.z + (double)v.w * v.w;
  }
  if (blockIdx.x == 0)
    for (long long i = (n4 << 2) + threadIdx.x; i < n; i += blockDim.x) acc += (double)g[i] * g[i];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int off = 128; off; off >>= 1) {
    if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) partial[blockIdx.x] = red[0];
}

// out[0] = global norm, out[1] = clip coefficient min(1, max_norm / (norm + 1e-6)); fixed summation order
__global__ void norm_finalize_kernel(const double* __restrict__ partial, int n_partial, float max_norm,
                                     float* __restrict__ out, float* __restrict__ grad_norm) {
  __shared__ double red[256];
  double acc = 0.0;
  for (int i = threadIdx.x; i < n_partial; i += blockDim.x) acc += partial[i];
  red[threadIdx.x] = acc;
  __syncthreads();
  for (int off = 128; off; off >>= 1) {
    if (threadIdx.x < off) red[threadIdx.x] += red[threadIdx.x + off];
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double norm = sqrt(red[0]);
    double coef = 1.0;
    if (max_norm > 0.f) coef = fmin(1.0, (double)max_norm / (norm + 1e-6));
    out[0] = (float)norm;
    out[1] = (float)coef;
    if (grad_norm) grad_norm[0] = (float)norm;
  }
}

template <typename T> __device__ __forceinline__ void store_weight(T* p, float v);
template <> __device__ __forceinline__ void store_weight<float>(float* p, float v) { *p = v; }
template <> __device__ __forceinline__ void store_weight<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T>
__global__ void __launch_bounds__(256)
adamw_kernel(float* __restrict__ master, T* __restrict__ weight, const float* __restrict__ grad, float* __restrict__ m,
             float* __restrict__ v, long long n, const float* __restrict__ norm_coef, float lr, float beta1, float beta2,
             float eps, float wd, float inv_bc1, float inv_bc2) {
  const float coef = norm_coef[1];
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const float g = grad[i] * coef;
    const float mi = beta1 * m[i] + (1.f - beta1) * g;
    const float vi = beta2 * v[i] + (1.f - beta2) * g * g;
    m[i] = mi;
    v[i] = vi;
    const float p = master[i];
    const float np_ = p - lr * ((mi * inv_bc1) / (sqrtf(vi * inv_bc2) + eps) + wd * p);
    master[i] = np_;
    store_weight<T>(weight + i, np_);
  }
}

}  // namespace pcm

using namespace pcm;

extern "C" size_t grpo_adamw_scratch_bytes(void) {
  return (size_t)OPT_MAX_TENSORS * OPT_NORM_BLOCKS * sizeof(double) + 256;
}

extern "C" int grpo_adamw_step(const grpo_model_cfg* cfg, const grpo_adamw_cfg* opt, int64_t step, grpo_model* model,
                               grpo_grads* master, const grpo_grads* grads, grpo_grads* m, grpo_grads* v,
                               float* grad_norm, void* scratch, size_t scratch_bytes, pcm_stream stream) {
  if (!cfg || !opt || !model || !master || !grads || !m || !v || !scratch) return PCM_ERR_ARG;
  if (step < 1 || !(opt->lr >= 0.f) || !(opt->beta1 >= 0.f && opt->beta1 < 1.f) || !(opt->beta2 >= 0.f && opt->beta2 < 1.f) ||
      !(opt->eps > 0.f) || !(opt->weight_decay >= 0.f) || !(opt->max_grad_norm >= 0.f))
    return PCM_ERR_ARG;
  if (cfg->dtype != GRPO_F32 && cfg->dtype != GRPO_BF16) return PCM_ERR_ARG;
  if (cfg->d < 1 || cfg->n_layers < 1) return PCM_ERR_ARG;
  if (scratch_bytes < grpo_adamw_scratch_bytes() || (((uintptr_t)scratch) & 255)) return PCM_ERR_WORKSPACE;
  const long long d = cfg->d, L = cfg->n_layers, dd = d * d;
  const long long numel[OPT_MAX_TENSORS] = {L * 3 * dd, L * dd, L * 8 * dd, L * 4 * dd, L * d, L * d, d, PCM_N_BINS * d, PCM_N_BINS * d};
  float* P[OPT_MAX_TENSORS] = {master->w_qkv, master->w_o, master->w_gu, master->w_d, master->g1, master->g2, master->gf, master->w_h, master->e_act};
  const float* Gd[OPT_MAX_TENSORS] = {grads->w_qkv, grads->w_o, grads->w_gu, grads->w_d, grads->g1, grads->g2, grads->gf, grads->w_h, grads->e_act};
  float* Mo[OPT_MAX_TENSORS] = {m->w_qkv, m->w_o, m->w_gu, m->w_d, m->g1, m->g2, m->gf, m->w_h, m->e_act};
  float* Vo[OPT_MAX_TENSORS] = {v->w_qkv, v->w_o, v->w_gu, v->w_d, v->g1, v->g2, v->gf, v->w_h, v->e_act};
  void* Wt[OPT_MAX_TENSORS] = {(void*)model->w_qkv, (void*)model->w_o, (void*)model->w_gu, (void*)model->w_d, (void*)model->g1,
                               (void*)model->g2, (void*)model->gf, (void*)model->w_h, (void*)model->e_act};
  for (int t = 0; t < OPT_MAX_TENSORS; ++t)
    if (!P[t] || !Gd[t] || !Mo[t] || !Vo[t] || !Wt[t] || (((uintptr_t)Gd[t]) & 15)) return PCM_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  double* partial = (double*)scratch;
  float* norm_coef = (float*)((unsigned char*)scratch + (size_t)OPT_MAX_TENSORS * OPT_NORM_BLOCKS * sizeof(double));
  for (int t = 0; t < OPT_MAX_TENSORS; ++t) {
    prof_begin(PC_NORM, s);           // accounted with the norm class: a bandwidth-bound reduction
    sumsq_kernel<<<OPT_NORM_BLOCKS, 256, 0, s>>>(Gd[t], numel[t], partial + (size_t)t * OPT_NORM_BLOCKS);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, 4.0 * numel[t]);
  }
  norm_finalize_kernel<<<1, 256, 0, s>>>(partial, OPT_MAX_TENSORS * OPT_NORM_BLOCKS, opt->max_grad_norm, norm_coef, grad_norm);
  PCM_LAUNCH_CHECK();
  const float inv_bc1 = (float)(1.0 / (1.0 - pow((double)opt->beta1, (double)step)));
  const float inv_bc2 = (float)(1.0 / (1.0 - pow((double)opt->beta2, (double)step)));
  for (int t = 0; t < OPT_MAX_TENSORS; ++t) {
    const int blocks = (int)((numel[t] + 255) / 256 < 148 * 8 ? (numel[t] + 255) / 256 : 148 * 8);
    prof_begin(PC_ELEM, s);
    if (cfg->dtype == GRPO_BF16)
      adamw_kernel<__nv_bfloat16><<<blocks, 256, 0, s>>>(P[t], (__nv_bfloat16*)Wt[t], Gd[t], Mo[t], Vo[t], numel[t], norm_coef,
                                                         opt->lr, opt->beta1, opt->beta2, opt->eps, opt->weight_decay, inv_bc1, inv_bc2);
    else
      adamw_kernel<float><<<blocks, 256, 0, s>>>(P[t], (float*)Wt[t], Gd[t], Mo[t], Vo[t], numel[t], norm_coef, opt->lr,
                                                 opt->beta1, opt->beta2, opt->eps, opt->weight_decay, inv_bc1, inv_bc2);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, (28.0 + (cfg->dtype == GRPO_BF16 ? 2.0 : 4.0)) * numel[t]);
  }
  return PCM_OK;
}
