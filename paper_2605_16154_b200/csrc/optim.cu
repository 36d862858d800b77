// Optimizer step after the actor update (App. E): global-norm gradient clipping and AdamW on fp32 master
// weights, with the model-dtype copy of every weight rewritten in the same pass.  HBM bound: 16 B read and
// 12 + sizeof(T) B written per parameter.
#include <cmath>

#include "internal.h"

namespace pcm {

constexpr int OPT_NORM_BLOCKS = 296;          // 2 CTAs per SM
constexpr int OPT_MAX_TENSORS = 13;         // 8 adapter tensors + norm gains, head and embedding

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

__device__ __forceinline__ void store_weight4(float* p, const float4& v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store_weight4(__nv_bfloat16* p, const float4& v) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<const uint32_t*>(&lo);
  u.y = *reinterpret_cast<const uint32_t*>(&hi);
  *reinterpret_cast<uint2*>(p) = u;
}

struct AdamScalars {
  float lr, beta1, beta2, eps, wd, inv_bc1, inv_bc2;
};

__device__ __forceinline__ float adamw_one(float g, float coef, float& m, float& v, float p, const AdamScalars& a) {
  g *= coef;
  m = a.beta1 * m + (1.f - a.beta1) * g;
  v = a.beta2 * v + (1.f - a.beta2) * g * g;
  return p - a.lr * ((m * a.inv_bc1) / (sqrtf(v * a.inv_bc2) + a.eps) + a.wd * p);
}

// VEC = 4: every pointer is 16-byte aligned (the weight copy 4 * sizeof(T)); the last n % 4 elements go one by one.
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
adamw_kernel(float* __restrict__ master, T* __restrict__ weight, const float* __restrict__ grad, float* __restrict__ m,
             float* __restrict__ v, long long n, const float* __restrict__ norm_coef, AdamScalars a) {
  const float coef = norm_coef[1];
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x, nthr = (long long)gridDim.x * blockDim.x;
  long long done = 0;
  if constexpr (VEC == 4) {
    const long long n4 = n >> 2;
    for (long long i = tid; i < n4; i += nthr) {
      const float4 g = reinterpret_cast<const float4*>(grad)[i];
      float4 mi = reinterpret_cast<float4*>(m)[i], vi = reinterpret_cast<float4*>(v)[i];
      const float4 p = reinterpret_cast<float4*>(master)[i];
      float4 q;
      q.x = adamw_one(g.x, coef, mi.x, vi.x, p.x, a);
      q.y = adamw_one(g.y, coef, mi.y, vi.y, p.y, a);
      q.z = adamw_one(g.z, coef, mi.z, vi.z, p.z, a);
      q.w = adamw_one(g.w, coef, mi.w, vi.w, p.w, a);
      reinterpret_cast<float4*>(m)[i] = mi;
      reinterpret_cast<float4*>(v)[i] = vi;
      reinterpret_cast<float4*>(master)[i] = q;
      store_weight4(weight + (i << 2), q);
    }
    done = n4 << 2;
  }
  for (long long i = done + tid; i < n; i += nthr) {
    float mi = m[i], vi = v[i];
    const float q = adamw_one(grad[i], coef, mi, vi, master[i], a);
    m[i] = mi;
    v[i] = vi;
    master[i] = q;
    store_weight<T>(weight + i, q);
  }
}

struct OptTensor {
  float* master;
  void* weight;
  const float* grad;
  float *m, *v;
  long long n;
};

// Clip by the global norm over `t[0..nt)`, then AdamW on each of them.
static int adamw_run(const OptTensor* t, int nt, int dtype, const grpo_adamw_cfg* opt, int64_t step, float* grad_norm,
                     void* scratch, size_t scratch_bytes, cudaStream_t s) {
  if (step < 1 || !(opt->lr >= 0.f) || !(opt->beta1 >= 0.f && opt->beta1 < 1.f) || !(opt->beta2 >= 0.f && opt->beta2 < 1.f) ||
      !(opt->eps > 0.f) || !(opt->weight_decay >= 0.f) || !(opt->max_grad_norm >= 0.f))
    return PCM_ERR_ARG;
  if (dtype != GRPO_F32 && dtype != GRPO_BF16) return PCM_ERR_ARG;
  if (nt < 1 || nt > OPT_MAX_TENSORS) return PCM_ERR_ARG;
  if (scratch_bytes < grpo_adamw_scratch_bytes() || (((uintptr_t)scratch) & 255)) return PCM_ERR_WORKSPACE;
  for (int i = 0; i < nt; ++i)
    if (!t[i].master || !t[i].weight || !t[i].grad || !t[i].m || !t[i].v || t[i].n < 1 || (((uintptr_t)t[i].grad) & 15))
      return PCM_ERR_ARG;
  double* partial = (double*)scratch;
  float* norm_coef = (float*)((unsigned char*)scratch + (size_t)OPT_MAX_TENSORS * OPT_NORM_BLOCKS * sizeof(double));
  for (int i = 0; i < nt; ++i) {
    prof_begin(PC_NORM, s);           // accounted with the norm class: a bandwidth-bound reduction
    sumsq_kernel<<<OPT_NORM_BLOCKS, 256, 0, s>>>(t[i].grad, t[i].n, partial + (size_t)i * OPT_NORM_BLOCKS);
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, 4.0 * t[i].n);
  }
  norm_finalize_kernel<<<1, 256, 0, s>>>(partial, nt * OPT_NORM_BLOCKS, opt->max_grad_norm, norm_coef, grad_norm);
  PCM_LAUNCH_CHECK();
  AdamScalars a;
  a.lr = opt->lr; a.beta1 = opt->beta1; a.beta2 = opt->beta2; a.eps = opt->eps; a.wd = opt->weight_decay;
  a.inv_bc1 = (float)(1.0 / (1.0 - pow((double)opt->beta1, (double)step)));
  a.inv_bc2 = (float)(1.0 / (1.0 - pow((double)opt->beta2, (double)step)));
  const int wsize = dtype == GRPO_BF16 ? 2 : 4;
  for (int i = 0; i < nt; ++i) {
    const uintptr_t f32_ptrs = (uintptr_t)t[i].master | (uintptr_t)t[i].grad | (uintptr_t)t[i].m | (uintptr_t)t[i].v;
    const bool vec = !(f32_ptrs & 15) && !(((uintptr_t)t[i].weight) & (uintptr_t)(4 * wsize - 1));
    const long long work = vec ? (t[i].n + 3) / 4 : t[i].n;
    const int blocks = (int)((work + 255) / 256 < 148 * 8 ? (work + 255) / 256 : 148 * 8);
    prof_begin(PC_ELEM, s);
    if (dtype == GRPO_BF16) {
      auto* wt = (__nv_bfloat16*)t[i].weight;
      if (vec) adamw_kernel<__nv_bfloat16, 4><<<blocks, 256, 0, s>>>(t[i].master, wt, t[i].grad, t[i].m, t[i].v, t[i].n, norm_coef, a);
      else adamw_kernel<__nv_bfloat16, 1><<<blocks, 256, 0, s>>>(t[i].master, wt, t[i].grad, t[i].m, t[i].v, t[i].n, norm_coef, a);
    } else {
      auto* wt = (float*)t[i].weight;
      if (vec) adamw_kernel<float, 4><<<blocks, 256, 0, s>>>(t[i].master, wt, t[i].grad, t[i].m, t[i].v, t[i].n, norm_coef, a);
      else adamw_kernel<float, 1><<<blocks, 256, 0, s>>>(t[i].master, wt, t[i].grad, t[i].m, t[i].v, t[i].n, norm_coef, a);
    }
    PCM_LAUNCH_CHECK();
    prof_end(s, 0.0, (28.0 + wsize) * t[i].n);
  }
  return PCM_OK;
}

// g1, g2, gf, w_h, e_act of a parameter set; returns how many were appended (0 when the set is absent)
static int small_tensors(const grpo_model_cfg* cfg, grpo_model* model, grpo_grads* master, const grpo_grads* grads,
                         grpo_grads* m, grpo_grads* v, OptTensor* out) {
  const long long d = cfg->d, L = cfg->n_layers;
  const long long numel[5] = {L * d, L * d, d, PCM_N_BINS * d, PCM_N_BINS * d};
  float* P[5] = {master->g1, master->g2, master->gf, master->w_h, master->e_act};
  const float* G[5] = {grads->g1, grads->g2, grads->gf, grads->w_h, grads->e_act};
  float* Mo[5] = {m->g1, m->g2, m->gf, m->w_h, m->e_act};
  float* Vo[5] = {v->g1, v->g2, v->gf, v->w_h, v->e_act};
  void* W[5] = {(void*)model->g1, (void*)model->g2, (void*)model->gf, (void*)model->w_h, (void*)model->e_act};
  for (int i = 0; i < 5; ++i) out[i] = OptTensor{P[i], W[i], G[i], Mo[i], Vo[i], numel[i]};
  return 5;
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
  if (cfg->d < 1 || cfg->n_layers < 1) return PCM_ERR_ARG;
  const long long d = cfg->d, L = cfg->n_layers, dd = d * d;
  OptTensor t[OPT_MAX_TENSORS];
  t[0] = OptTensor{master->w_qkv, (void*)model->w_qkv, grads->w_qkv, m->w_qkv, v->w_qkv, L * 3 * dd};
  t[1] = OptTensor{master->w_o, (void*)model->w_o, grads->w_o, m->w_o, v->w_o, L * dd};
  t[2] = OptTensor{master->w_gu, (void*)model->w_gu, grads->w_gu, m->w_gu, v->w_gu, L * 8 * dd};
  t[3] = OptTensor{master->w_d, (void*)model->w_d, grads->w_d, m->w_d, v->w_d, L * 4 * dd};
  const int nt = 4 + small_tensors(cfg, model, master, grads, m, v, t + 4);
  return adamw_run(t, nt, cfg->dtype, opt, step, grad_norm, scratch, scratch_bytes, (cudaStream_t)stream);
}

extern "C" int grpo_adamw_step_lora(const grpo_model_cfg* cfg, const grpo_adamw_cfg* opt, int64_t step, grpo_lora* lora,
                                    grpo_lora_grads* lora_master, const grpo_lora_grads* lora_grads, grpo_lora_grads* lora_m,
                                    grpo_lora_grads* lora_v, grpo_model* model, grpo_grads* master, const grpo_grads* grads,
                                    grpo_grads* m, grpo_grads* v, float* grad_norm, void* scratch, size_t scratch_bytes,
                                    pcm_stream stream) {
  if (!cfg || !opt || !lora || !lora_master || !lora_grads || !lora_m || !lora_v || !scratch) return PCM_ERR_ARG;
  if (cfg->d < 1 || cfg->n_layers < 1 || lora->rank < 1) return PCM_ERR_ARG;
  const bool with_small = model || master || grads || m || v;
  if (with_small && !(model && master && grads && m && v)) return PCM_ERR_ARG;
  const long long d = cfg->d, L = cfg->n_layers, r = lora->rank;
  OptTensor t[OPT_MAX_TENSORS];
  t[0] = OptTensor{lora_master->a_qkv, (void*)lora->a_qkv, lora_grads->a_qkv, lora_m->a_qkv, lora_v->a_qkv, L * r * d};
  t[1] = OptTensor{lora_master->b_qkv, (void*)lora->b_qkv, lora_grads->b_qkv, lora_m->b_qkv, lora_v->b_qkv, L * 3 * d * r};
  t[2] = OptTensor{lora_master->a_o, (void*)lora->a_o, lora_grads->a_o, lora_m->a_o, lora_v->a_o, L * r * d};
  t[3] = OptTensor{lora_master->b_o, (void*)lora->b_o, lora_grads->b_o, lora_m->b_o, lora_v->b_o, L * d * r};
  t[4] = OptTensor{lora_master->a_gu, (void*)lora->a_gu, lora_grads->a_gu, lora_m->a_gu, lora_v->a_gu, L * r * d};
  t[5] = OptTensor{lora_master->b_gu, (void*)lora->b_gu, lora_grads->b_gu, lora_m->b_gu, lora_v->b_gu, L * 8 * d * r};
  t[6] = OptTensor{lora_master->a_d, (void*)lora->a_d, lora_grads->a_d, lora_m->a_d, lora_v->a_d, L * r * 4 * d};
  t[7] = OptTensor{lora_master->b_d, (void*)lora->b_d, lora_grads->b_d, lora_m->b_d, lora_v->b_d, L * d * r};
  int nt = 8;
  if (with_small) nt += small_tensors(cfg, model, master, grads, m, v, t + 8);
  return adamw_run(t, nt, cfg->dtype, opt, step, grad_norm, scratch, scratch_bytes, (cudaStream_t)stream);
}
