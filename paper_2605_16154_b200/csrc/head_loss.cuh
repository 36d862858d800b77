// The loss over the 256-bin action head, as device functions shared by the kernels that hold a row of logits in
// registers (the tensor-core head GEMM's epilogue and the SIMT head kernel): log-softmax, the clipped
// importance-ratio surrogate of Eq. 11 with the clip of App. E, the entropy bonus, and the logit gradient.
// The logits themselves are never stored.
#pragma once
#include <stdint.h>

namespace pcm {

// What a head launch computes per scored row.
//   HL_TOKEN  one clipped ratio per row (token level): log-prob, surrogate terms and d loss / d logits in one pass.
//   HL_STATS  log-prob and entropy only (first pass of the chunk-level ratio, which needs all 56 rows of a chunk
//             before any gradient exists).
//   HL_COEF   d loss / d logits from a given d loss / d logp per row (second pass of the chunk-level ratio).
enum { HL_TOKEN = 0, HL_STATS = 1, HL_COEF = 2 };

struct HeadLossArgs {
  const uint8_t* tgt = nullptr;   // [rows] action token each row has to predict
  const float* lpo = nullptr;     // [rows] behaviour-policy log-prob
  const float* adv_c = nullptr;   // [rows / 56] advantage of the row's chunk
  const float* coef = nullptr;    // HL_COEF: [rows] d loss / d logp
  float* logp = nullptr;          // [rows] out (HL_TOKEN, HL_STATS; may be null)
  float* part = nullptr;          // [blocks][4] out: {surrogate, clipped terms, ratio, entropy} summed per block
  float lo = 0.f, hi = 0.f;       // clip range [1 - eps_low, 1 + eps_high]
  float loss_scale = 0.f, ent_scale = 0.f;
  int mode = HL_TOKEN;
  int want_dz = 0;                // store d loss / d logits (C of the GEMM, [rows][256])
};

// Softmax statistics of a set of logits against a reference value m >= all of them:
// se = sum e^(z - m), sz = sum e^(z - m) (z - m).
struct RowStats { float m, se, sz; };

__device__ __forceinline__ float hl_lse(const RowStats& s) { return s.m + logf(s.se); }
// entropy of softmax(z): lse - sum p z = log se - sz / se
__device__ __forceinline__ float hl_entropy(const RowStats& s) { return logf(s.se) - s.sz / s.se; }

struct RowTerms { float dlogp, surrogate, clipped, ratio; };

// Token-level clipped surrogate of one row: the term min(r A, clip(r) A), whether its gradient is clipped away,
// and d loss / d logp = -loss_scale * A * r where the term is active.
__device__ __forceinline__ RowTerms hl_token_terms(float logp, float lpo, float A, float lo, float hi, float loss_scale) {
  const float ratio = expf(logp - lpo);
  const float cl = fminf(fmaxf(ratio, lo), hi);
  const bool active = (A >= 0.f && ratio <= hi) || (A < 0.f && ratio >= lo);
  RowTerms t;
  t.dlogp = active ? -loss_scale * A * ratio : 0.f;
  t.surrogate = fminf(ratio * A, cl * A);
  t.clipped = active ? 0.f : 1.f;
  t.ratio = ratio;
  return t;
}

// d loss / d z_v = dlogp (1[v = target] - p_v) + ent_scale p_v (log p_v + H)
__device__ __forceinline__ float hl_dz(float z, float lse, float ent, float dlogp, float ent_scale, bool is_target) {
  const float lp = z - lse;
  const float p = expf(lp);
  return dlogp * ((is_target ? 1.f : 0.f) - p) + ent_scale * p * (lp + ent);
}

}  // namespace pcm
