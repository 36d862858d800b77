/*
 * pcm_b200.h - C ABI of the B200 (sm_100a) GRPO actor update with Probabilistic Chunk Masking.
 *
 * One training iteration of Algorithm 1 maps onto five calls, in this order:
 *
 *   pcm_score_phases       Eq. 1 (advantages) and Eq. 5 (success-failure action variance per phase)
 *   pcm_update_keep_probs  Eq. 7-9 (score buffer, share / max normalisation, floor p_min)
 *   pcm_sample_chunks      Eq. 10 (fixed-budget weighted sampling without replacement)
 *   grpo_pack_chunks       Sec. 4.5 "physical shrinking": dense batch of the kept chunks only
 *   grpo_actor_fwd_bwd     Eq. 11 (masked GRPO objective, with the PPO clip of App. E): loss + gradients
 *
 * Conventions
 *   - Every pointer named "device" is device memory owned by the caller; the library neither frees
 *     nor reallocates it.  Host pointers are marked "host".  `stream` is a cudaStream_t.
 *   - All device work is enqueued on `stream`; calls return without synchronising unless stated.
 *   - Return value: PCM_OK (0) or a negative pcm_status.  Nothing is printed; no exception crosses
 *     the boundary.  Bad arguments are rejected on the host before anything is launched.
 *     Device-side problems (a phase label >= n_phases, a trajectory longer than max_len, a bounded
 *     wait that ran out) are latched in a status word read by pcm_poll_status().
 *   - Trajectories g*G .. g*G+G-1 form rollout group g (G = group_size).
 *   - Chunks are stored CSR style: trajectory i owns chunks traj_off[i] .. traj_off[i+1]-1.
 *   - A chunk is 56 action tokens (8 actions x 7 degrees of freedom, Sec. 5.1) over 256 bins.
 *   - Every linear weight is stored row-major [out_features][in_features] (y = x W^T).
 *   - Four environment variables, read once per process, exist for comparison runs and are not part of the
 *     interface: PCM_GEMM_BACKEND=simt|tcgen05 forces the GEMM kernel family, PCM_GEMM_PAIR=0 keeps the tensor-core
 *     GEMM on single CTAs, PCM_ATTN_TC=0 keeps bf16 attention on the warp-level kernels, PCM_ATTN_BWD=2 keeps the
 *     head-dim-64 attention backward on the two-launch kernels.
 */
#ifndef PCM_B200_H
#define PCM_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PCM_ACT_DIM 56
#define PCM_N_BINS 256
#define PCM_MAX_PHASES 32
#define PCM_MAX_TRC 16

typedef enum {
  PCM_OK = 0,
  PCM_ERR_ARG = -1,            /* null pointer, value out of range                                */
  PCM_ERR_SHAPE = -2,          /* sizes the kernels do not support (see each call)                */
  PCM_ERR_WORKSPACE = -3,      /* workspace too small or misaligned                               */
  PCM_ERR_CUDA = -4,           /* a CUDA runtime / driver call failed                             */
  PCM_ERR_DEVICE_TIMEOUT = -5, /* a bounded device-side wait expired                              */
  PCM_ERR_STATE = -6,          /* state blob of the wrong size / version                          */
  PCM_ERR_DEVICE_DATA = -7     /* device-side data check failed, e.g. phase label >= n_phases     */
} pcm_status;

typedef void* pcm_stream;      /* cudaStream_t */
typedef struct pcm_ctx pcm_ctx;

typedef struct {
  int32_t n_phases;            /* the paper's K, 1..PCM_MAX_PHASES                                */
  int32_t budget;              /* the paper's B: chunks kept per trajectory, >= 1                 */
  int32_t group_size;          /* G rollouts per group, >= 1                                      */
  int32_t t_rc;                /* refresh window T_rc, 1..PCM_MAX_TRC                             */
  double p_min;                /* keep-probability floor, in (0, 1]                               */
  double adv_eps;              /* epsilon of Eq. 1                                                */
  uint64_t seed;               /* Philox key of the sampler                                       */
  int32_t mode;                /* pcm_mask_mode: how keep-probabilities are formed                */
  int32_t reserved;
} pcm_config;

/* PCM_MASK_PCM: Eq. 8-9.  The other two are the ablations of RQ4: PCM_MASK_RANDOM keeps every phase at
 * weight 1 (B chunks uniformly at random per trajectory); PCM_MASK_FULL gives weight 1 to the single
 * highest-S_c phase (first one on ties) and 0 to all others, so only chunks of that phase are kept and a
 * trajectory keeps min(B, its chunks in that phase). */
typedef enum { PCM_MASK_PCM = 0, PCM_MASK_RANDOM = 1, PCM_MASK_FULL = 2 } pcm_mask_mode;

typedef struct {
  int32_t n_traj;              /* multiple of group_size                                          */
  int32_t n_chunks;            /* traj_off[n_traj]                                                */
  int32_t max_len;             /* upper bound on chunks per trajectory (sizes shared memory)      */
  int32_t reserved;
  const int32_t* traj_off;     /* device [n_traj+1]                                               */
  const uint8_t* tok;          /* device [n_chunks][56], 16-byte aligned                          */
  const uint8_t* phase;        /* device [n_chunks], labels < n_phases, any order                 */
  const uint8_t* reward;       /* device [n_traj], 0 or 1                                         */
  const void* obs;             /* device [n_chunks][P][d] in the model dtype; pack only           */
  const float* logp_old;       /* device [n_chunks][56]; pack only                                */
} pcm_batch;

/* ---- context: configuration, persistent keep-probability state, small scratch ---------------- */

/* Creates a context on the current device.  Allocates device memory for the keep-probability
 * state, the status word and per-group score scratch: about 9 * n_phases bytes per group for
 * max_traj / group_size groups, plus a few KB.  Batches passed later may hold at most max_traj
 * trajectories. */
int pcm_create(pcm_ctx** out, const pcm_config* cfg, int32_t max_traj);
int pcm_destroy(pcm_ctx* ctx);

/* Reads and clears the device status word (synchronises `stream`).  Returns PCM_OK,
 * PCM_ERR_DEVICE_TIMEOUT or PCM_ERR_DEVICE_DATA. */
int pcm_poll_status(pcm_ctx* ctx, pcm_stream stream);

/* Keep-probability state (buffers B_c, step counter, p_c) as a flat host blob, so that a chain of
 * iterations can be stopped and resumed bit-exactly.  Both calls synchronise the device.
 * pcm_state_export: *bytes in = capacity of host_buf, out = bytes needed / written; with
 * host_buf == NULL only the size is reported. */
int pcm_state_export(pcm_ctx* ctx, void* host_buf, size_t* bytes);
int pcm_state_import(pcm_ctx* ctx, const void* host_buf, size_t bytes);

/* ---- Eq. 1 + Eq. 5 ---------------------------------------------------------------------------
 * For every group with both outcomes present and every phase c that has chunks from a successful
 * and from a failed rollout of that group:
 *     C_{c,g} = || mean_{success chunks in c} a - mean_{failure chunks in c} a ||_2
 * with a the 56-vector of bin-centre values a = -1 + (tok + 1/2) * 2/256.  C[c] is the mean of
 * C_{c,g} over the groups where it is defined (ascending g); valid[c] = 0 and C[c] = 0 when there
 * is none (uniform-reward groups are ignored, a phase missing from one outcome is skipped).
 * Token sums are exact integers; the remaining fp64 operations are individually rounded IEEE
 * operations in a fixed order, so the result does not depend on the launch shape.
 * adv (may be NULL) receives Eq. 1 with population variance: A_i = (r_i - mu) / (sigma + adv_eps).
 * Outputs: device C[n_phases] f64, valid[n_phases] u8, n_valid_groups[n_phases] i32 (may be NULL),
 * adv[n_traj] f32. */
int pcm_score_phases(pcm_ctx* ctx, const pcm_batch* batch, double* C, uint8_t* valid,
                     int32_t* n_valid_groups, float* adv, pcm_stream stream);

/* ---- Eq. 5 on continuous actions -----------------------------------------------------------------
 * pcm_score_phases for policies whose chunk action is a float vector: act is device float32
 * [n_chunks][56] (16-byte aligned), batch->tok is not read.  Groups, skip rules, reductions and outputs
 * are those of pcm_score_phases with a = act.  To make the sums over chunks independent of their order
 * every value is read as the integer round-half-even(a * 2^32) (exact for |a| >= 2^-9, off by at most
 * 2^-33 below) and summed in 64-bit integers; the rest is the same chain of individually rounded fp64
 * operations, with the unit 2^-32 applied once at the end.  Limits: |a| <= 4096 and finite (another value
 * counts as 0 and raises the context's status word: PCM_ERR_DEVICE_DATA from pcm_poll_status);
 * group_size * max_len <= 262144 chunks (PCM_ERR_SHAPE), so that no sum can overflow. */
int pcm_score_phases_f32(pcm_ctx* ctx, const pcm_batch* batch, const float* act, double* C, uint8_t* valid,
                         int32_t* n_valid_groups, float* adv, pcm_stream stream);

/* ---- allocation-free variant of pcm_score_phases (the paper has no counterpart) -----------------
 * Same computation and outputs as pcm_score_phases, for callers that are not allowed to allocate
 * device memory: code that runs inside a region where the allocator is off limits (a serving or
 * training loop with a frozen memory plan, a real-time control thread next to the robot, a plugin
 * that only gets pointers from its host program), where a cudaMalloc would synchronise the device,
 * fragment the plan or simply be forbidden.  It needs no pcm_ctx (pcm_create allocates): the
 * per-group scratch (C_{c,g} and its validity flag) lives in a fixed array inside the library,
 * PCM_STATIC_SCRATCH_BYTES of device memory that every GPU which loads the library holds until the
 * process exits.  Limits: n_traj / group_size <= PCM_STATIC_MAX_GROUPS; larger batches are rejected
 * with PCM_ERR_SHAPE before anything is launched.
 * The first call on each device looks up the array's device address (no allocation, but a
 * synchronous runtime query): make that first call before any stream capture.
 * All calls share the one array, which keeps whatever the previous call left in it; every entry a
 * call reads is rewritten by that call first, and the status word is cleared at the start of each
 * call.  Two calls whose kernels overlap on the GPU (different streams, no dependency) race on the
 * array: order them.
 * device_status (device [1], may be NULL) receives 0, or a non-zero bit mask when a phase label
 * >= n_phases was met (that chunk is ignored), once the stream reaches that point.
 * Calls no cudaMalloc / cudaFree and no allocating library routine. */
#define PCM_STATIC_MAX_GROUPS 4096
#define PCM_STATIC_SCRATCH_BYTES (PCM_STATIC_MAX_GROUPS * PCM_MAX_PHASES * 9 + 256)
int pcm_score_phases_static(int32_t n_phases, int32_t group_size, double adv_eps, const pcm_batch* batch,
                            double* C, uint8_t* valid, int32_t* n_valid_groups, float* adv,
                            uint32_t* device_status, pcm_stream stream);

/* ---- phase labelling (Sec. 5.1 "Phase Labeling", App. E.2; Algorithm 1, the step before scoring) -------
 * Labels every chunk with one of five phases from the per-timestep gripper-close command:
 * 0 approach, 1 pre-grasp, 2 active-grip, 3 release-ramp, 4 tail.  g_f = fraction of the chunk's timesteps
 * with the command active (the last chunk of a trajectory may be shorter than chunk_len).  A sustained-close
 * interval is a maximal run of chunks with g_f >= 0.75.  active-grip: g_f >= 0.5.  pre-grasp: the three chunk
 * positions before a sustained interval, where 0.1 <= g_f < 0.5.  release-ramp: the three positions after
 * it, where g_f < 0.5.  Overlaps resolve by active-grip > pre-grasp > release-ramp > approach > tail.  Chunks
 * left over: approach when a sustained interval starts later; tail when after the last one with g_f < 0.1;
 * approach otherwise.  Fractions are compared through integer counts.
 * Inputs (device): traj_off[n_traj+1] in chunks, step_off[n_traj+1] in timesteps with
 * N_i = ceil(T_i / chunk_len) (a mismatch is latched in the status word), grip_close[total timesteps]
 * (non-zero = close).  Output: device phase[n_chunks]. */
int pcm_label_phases(pcm_ctx* ctx, int32_t n_traj, const int32_t* traj_off, const int32_t* step_off,
                     const uint8_t* grip_close, int32_t chunk_len, uint8_t* phase, pcm_stream stream);

/* ---- Eq. 7-9, Algorithm 1 ---------------------------------------------------------------------
 * Appends C (0 where valid[c] == 0) to the phase buffers.  On the first call, or when the buffers
 * hold t_rc entries: S_c = sum of buffer, rho_c = S_c / sum S, rho~_c = rho_c / max rho,
 * p_c = max(p_min, rho~_c); buffers cleared.  If every S_c is 0 the previous p_c is kept.
 * Otherwise p_c is unchanged.  The state lives in the context (device memory).
 * Outputs: device p[n_phases] f32 and q[n_phases] u32 = round-half-even(p_c * 2^24), the integer
 * chunk weight used by pcm_sample_chunks. */
int pcm_update_keep_probs(pcm_ctx* ctx, const double* C, const uint8_t* valid, float* p, uint32_t* q,
                          pcm_stream stream);

/* ---- Eq. 10 -----------------------------------------------------------------------------------
 * For every trajectory draws m_i = min(budget, N_i) chunks by successive sampling without
 * replacement (Plackett-Luce) with integer weights w_ik = q[phase(i,k)]; chunks of weight 0 (only with
 * PCM_MASK_FULL) are never kept and N_i then counts the chunks of positive weight.  Draw r of trajectory i
 * takes 64 bits from Philox4x32-10 with key (seed lo, seed hi) and counter (iter lo, i, r, iter hi),
 * maps them to x = floor(bits * W_remaining / 2^64) and selects the first remaining chunk, in index
 * order, whose running weight sum exceeds x.  When m_i = N_i every chunk is kept and no random
 * numbers are consumed.  max_len <= 12000.  Uses n_traj ints of context scratch.
 * Outputs: device kept_idx[sum m_i] i32 global chunk ids, trajectory-major and ascending within a
 * trajectory (capacity n_traj*budget is always enough); kept_off[n_traj+1] i32;
 * kept_per_phase[n_phases] i32 (may be NULL). */
int pcm_sample_chunks(pcm_ctx* ctx, const pcm_batch* batch, const uint32_t* q, uint64_t iter,
                      int32_t* kept_idx, int32_t* kept_off, int32_t* kept_per_phase, pcm_stream stream);

/* ---- model ----------------------------------------------------------------------------------- */
typedef enum { GRPO_F32 = 0, GRPO_BF16 = 1 } grpo_dtype;

typedef struct {
  int32_t d;                   /* model width, multiple of 8                                      */
  int32_t n_layers;            /* 1..128                                                          */
  int32_t n_heads;             /* head dim d / n_heads in {32, 64, 128}                           */
  int32_t prefix_len;          /* P observation-prefix tokens per chunk, >= 1; S = P + 56 <= 384  */
  int32_t dtype;               /* grpo_dtype of weights, observations and activations             */
  int32_t reserved;
} grpo_model_cfg;

/* Decoder-only policy: per layer RMSNorm(g1) -> fused QKV -> rotary embedding (base 10000, pairs
 * (i, i + dh/2)) -> causal attention within the chunk -> W_o + residual -> RMSNorm(g2) -> SwiGLU
 * (gate rows first, then up rows, hidden 4d) -> W_d + residual; then RMSNorm(gf) and the 256-bin
 * head.  RMSNorm epsilon 1e-5.  All tensors device, in cfg.dtype. */
typedef struct {
  grpo_model_cfg cfg;
  const void* w_qkv;           /* [L][3d][d]                                                      */
  const void* w_o;             /* [L][d][d]                                                       */
  const void* w_gu;            /* [L][8d][d]                                                      */
  const void* w_d;             /* [L][d][4d]                                                      */
  const void* g1;              /* [L][d]                                                          */
  const void* g2;              /* [L][d]                                                          */
  const void* gf;              /* [d]                                                             */
  const void* w_h;             /* [256][d]                                                        */
  const void* e_act;           /* [256][d]                                                        */
} grpo_model;

/* fp32 gradients with the shapes of grpo_model (device). */
typedef struct {
  float* w_qkv; float* w_o; float* w_gu; float* w_d; float* g1; float* g2; float* gf; float* w_h; float* e_act;
} grpo_grads;

/* Dense batch of kept chunks, caller-allocated device views. */
typedef struct {
  int32_t n_kept;
  int32_t reserved;
  void* X;                     /* [n_kept][S][d] model dtype: prefix rows then E_act[token] rows  */
  uint8_t* tgt;                /* [n_kept][56] action tokens                                      */
  float* lpo;                  /* [n_kept][56] behaviour-policy log-probs                         */
  float* adv_c;                /* [n_kept] advantage of the owning trajectory                     */
  int32_t* src;                /* [n_kept] global chunk id                                        */
} grpo_packed;

/* ---- Sec. 4.5 physical shrinking ----------------------------------------------------------------
 * Copies the kept chunks, in kept_idx order, into the dense batch: X[j] = [obs[kept_idx[j]] ;
 * E_act[tok[kept_idx[j]][0..55]]], plus targets, old log-probs, advantage and source id.  A pure
 * byte copy (bit-exact).  Requires d * sizeof(dtype) to be a multiple of 16 and at most 32768, and
 * 16-byte aligned obs, E_act and X.  n_kept = out->n_kept must equal kept_off[n_traj] (<= 65535). */
int grpo_pack_chunks(pcm_ctx* ctx, const pcm_batch* batch, const grpo_model_cfg* cfg,
                     const int32_t* kept_idx, const int32_t* kept_off, const void* e_act,
                     const float* adv, grpo_packed* out, pcm_stream stream);

/* ---- Eq. 11 ------------------------------------------------------------------------------------ */
#define GRPO_FWD_ONLY 1u       /* forward only: writes logp (and loss), touches no gradient       */
#define GRPO_ACCUMULATE 2u     /* add into grads instead of overwriting them                      */
#define GRPO_CHUNK_RATIO 4u    /* one importance ratio per chunk (joint of its 56 tokens) instead of per token */

typedef struct {
  float eps_low;               /* clip range [1 - eps_low, 1 + eps_high]                          */
  float eps_high;
  float loss_scale;            /* <= 0: mean over the surrogate's terms, 1 / (56 * n_kept) per token,
                                  1 / n_kept with GRPO_CHUNK_RATIO                                */
  int32_t mb_chunks;           /* chunks per micro-batch, >= 1                                    */
  uint32_t flags;
  float entropy_coef;          /* App. E: 1e-3; the loss subtracts entropy_coef * mean entropy    */
} grpo_loss_cfg;

typedef struct {
  float loss;
  float clip_frac;             /* fraction of ratios (tokens, or chunks with GRPO_CHUNK_RATIO) whose gradient is clipped */
  float mean_ratio;
  float entropy;               /* mean over the scored positions of H(pi(. | s)), in nats          */
  int32_t n_launches;          /* kernels launched by this call                                   */
  int32_t reserved;
  uint64_t workspace_high_water;
} grpo_stats;

/* Bytes of workspace grpo_actor_fwd_bwd needs for micro-batches of mb_chunks chunks (activations
 * are kept, not recomputed).  0 when cfg is not supported. */
size_t grpo_workspace_bytes(const grpo_model_cfg* cfg, int32_t mb_chunks, uint32_t flags);

/* Forward and backward of the policy on the packed batch under
 *     loss = -loss_scale * sum_{kept chunks} sum_{j<56} min(r_j A, clip(r_j, 1-eps_low, 1+eps_high) A),
 *     r_j = exp(logp_j - lpo_j), logp_j = log softmax(z_j)[tgt_j], z_j = head(position P-1+j).
 * A term's gradient is r_j A when (A >= 0 and r_j <= 1+eps_high) or (A < 0 and r_j >= 1-eps_low),
 * else 0.  With GRPO_CHUNK_RATIO the inner sum is one term per chunk with r = exp(sum_j (logp_j - lpo_j)).
 * The entropy bonus of App. E subtracts entropy_coef * (1 / (56 n_kept)) * sum over the scored positions of
 * H(softmax(z_j)) from the loss (entropy_coef = 0: none).  The batch is processed in micro-batches of mb_chunks chunks; gradients accumulate in
 * fp32, so the micro-batch size only changes the rounding order.  No gradient reaches the
 * observation prefix.
 * Outputs: device loss[1] f32; device logp[n_kept][56] f32 (may be NULL); grads (ignored with
 * GRPO_FWD_ONLY); host stats (may be NULL; when given the call synchronises `stream` and returns
 * PCM_ERR_DEVICE_TIMEOUT if a bounded device-side wait expired).
 * workspace: device, 256-byte aligned, >= grpo_workspace_bytes(). */
int grpo_actor_fwd_bwd(const grpo_model* model, const grpo_packed* batch, const grpo_loss_cfg* loss_cfg,
                       grpo_grads* grads, float* loss, float* logp, grpo_stats* stats,
                       void* workspace, size_t workspace_bytes, pcm_stream stream);

/* ---- LoRA fine-tuning (App. E "Training": LoRA rank r = 32, alpha = 32) -----------------------------------
 * The regime the paper trains in: the four weight matrices of every decoder layer stay frozen and each gets a
 * low-rank adapter, y = x W^T + (alpha / rank) (x A^T) B^T.  The adapter branch is evaluated as written (never
 * merged into W, which would round a small update away in bf16): t = (alpha / rank) x A^T is formed first and enters
 * the same tensor-core accumulator as x W^T through a continuation of the contraction, before the fused rotary /
 * SwiGLU epilogues; backward likewise with u = (alpha / rank) dy B, dx = dy W + u A, dA += u^T x, dB += dy^T t.
 * No gradient of W_qkv, W_o, W_gu, W_d is formed (a third of the dense update's linear flops).
 * Adapter tensors are device, in cfg.dtype; rank a multiple of 8, 8..64 (32 or 64 run entirely on the tensor-core
 * kernels; other ranks send the adapters' own small products through the SIMT kernel). */
typedef struct {
  int32_t rank;
  float alpha;                 /* scale = alpha / rank, > 0                                         */
  const void* a_qkv;           /* [L][rank][d]                                                      */
  const void* b_qkv;           /* [L][3d][rank]                                                     */
  const void* a_o;             /* [L][rank][d]                                                      */
  const void* b_o;             /* [L][d][rank]                                                      */
  const void* a_gu;            /* [L][rank][d]                                                      */
  const void* b_gu;            /* [L][8d][rank]                                                     */
  const void* a_d;             /* [L][rank][4d]                                                     */
  const void* b_d;             /* [L][d][rank]                                                      */
} grpo_lora;

/* fp32 gradients with the shapes of the adapter tensors (device). */
typedef struct {
  float* a_qkv; float* b_qkv; float* a_o; float* b_o; float* a_gu; float* b_gu; float* a_d; float* b_d;
} grpo_lora_grads;

/* Workspace of grpo_actor_fwd_bwd_lora (0 when cfg or rank is not supported). */
size_t grpo_lora_workspace_bytes(const grpo_model_cfg* cfg, int32_t rank, int32_t mb_chunks, uint32_t flags);

/* grpo_actor_fwd_bwd with adapters.  Same batch, loss configuration, outputs and error behaviour.  grads receives
 * g1, g2, gf, w_h, e_act (its w_qkv, w_o, w_gu, w_d are ignored and may be NULL); lora_grads receives the adapter
 * gradients (both ignored with GRPO_FWD_ONLY; GRPO_ACCUMULATE adds into both). */
int grpo_actor_fwd_bwd_lora(const grpo_model* model, const grpo_lora* lora, const grpo_packed* batch,
                            const grpo_loss_cfg* loss_cfg, grpo_grads* grads, grpo_lora_grads* lora_grads, float* loss,
                            float* logp, grpo_stats* stats, void* workspace, size_t workspace_bytes, pcm_stream stream);

/* ---- optimizer step (App. E: AdamW, lr 1e-5, betas (0.9, 0.999), weight decay 0, clipping at 2.0) -----
 * The step that follows grpo_actor_fwd_bwd.  Global L2 norm of all gradients (fp64 partial sums in a fixed
 * order), clip coefficient min(1, max_grad_norm / (norm + 1e-6)) (max_grad_norm = 0: no clipping), then per
 * parameter, with g the clipped gradient and t = step (counted from 1):
 *     m = beta1 m + (1 - beta1) g;  v = beta2 v + (1 - beta2) g^2;
 *     w = w - lr * ( (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps) + weight_decay * w )
 * on fp32 master weights; the weights of `model` (cfg.dtype, device, WRITTEN by this call) receive the
 * rounded masters.  master, m, v, grads: fp32 tensors with the shapes of grpo_model.  grad_norm (device
 * [1], may be NULL) receives the norm before clipping.  scratch: device, 256-byte aligned,
 * >= grpo_adamw_scratch_bytes(). */
typedef struct {
  float lr, beta1, beta2, eps, weight_decay, max_grad_norm;
} grpo_adamw_cfg;
size_t grpo_adamw_scratch_bytes(void);
int grpo_adamw_step(const grpo_model_cfg* cfg, const grpo_adamw_cfg* opt, int64_t step, grpo_model* model,
                    grpo_grads* master, const grpo_grads* grads, grpo_grads* m, grpo_grads* v, float* grad_norm,
                    void* scratch, size_t scratch_bytes, pcm_stream stream);

/* The same step for LoRA fine-tuning (App. E: the adapters are what is trained), after grpo_actor_fwd_bwd_lora.
 * The eight adapter tensors of `lora` (cfg.dtype, device, WRITTEN by this call although the struct types them
 * const) receive the rounded fp32 masters lora_master; lora_grads / lora_m / lora_v have the same shapes.
 * The norm gains, head and action embedding, for which grpo_actor_fwd_bwd_lora also returns gradients, are
 * trained along when model / master / grads / m / v are given (their g1, g2, gf, w_h, e_act; the four projection
 * members are ignored), and stay frozen when all five are NULL (some but not all NULL: PCM_ERR_ARG).  One global
 * norm and one clip coefficient over everything that is trained.  Arguments otherwise as grpo_adamw_step. */
int grpo_adamw_step_lora(const grpo_model_cfg* cfg, const grpo_adamw_cfg* opt, int64_t step, grpo_lora* lora,
                         grpo_lora_grads* lora_master, const grpo_lora_grads* lora_grads, grpo_lora_grads* lora_m,
                         grpo_lora_grads* lora_v, grpo_model* model, grpo_grads* master, const grpo_grads* grads,
                         grpo_grads* m, grpo_grads* v, float* grad_norm, void* scratch, size_t scratch_bytes,
                         pcm_stream stream);

/* ---- diagnostic entry points (per-kernel tests and measurements; not part of Algorithm 1) -------
 * grpo_gemm: C[m][n] = sum_k A(m,k) B(n,k) (+ R[m][n]) with the GEMM kernels the actor update uses.
 * a_kmajor != 0: A is stored [M][K] with row stride lda, else [K][M]; likewise B ([N][K] / [K][N]).
 * ab_dtype / c_dtype are grpo_dtype values; R (fp32, may be NULL) may alias C to accumulate (C fp32).
 * backend: 0 = automatic, 1 = SIMT kernel, 2 = tcgen05 kernel (PCM_ERR_SHAPE when it cannot take the
 * problem); adding 4 skips the synchronisation.  Otherwise synchronises `stream` and returns
 * PCM_ERR_DEVICE_TIMEOUT when a bounded wait expired. */
int grpo_gemm(int32_t M, int32_t N, int32_t K, const void* A, int64_t lda, int32_t a_kmajor, const void* B,
              int64_t ldb, int32_t b_kmajor, int32_t ab_dtype, void* C, int64_t ldc, int32_t c_dtype,
              const float* R, int64_t ldr, int32_t backend, pcm_stream stream);

/* grpo_attention: causal attention inside each of n_seq sequences of S tokens, as used by the actor
 * update.  qkv [n_seq*S][3d] holds q | k | v (rotary embedding already applied), out [n_seq*S][d],
 * lse [n_seq][H][S] fp32.  With dout != NULL also runs the backward pass: dqkv [n_seq*S][3d],
 * scratch [n_seq][H][S] fp32.  Synchronises `stream`. */
int grpo_attention(int32_t dtype, const void* qkv, void* out, float* lse, const void* dout, void* dqkv,
                   float* scratch, int32_t n_seq, int32_t S, int32_t n_heads, int32_t head_dim, pcm_stream stream);

/* Which bounded wait of the tensor-core attention kernels expired last (0 = none since the library was
 * loaded): bit 0 set, bit 8 + k names the barrier (k = 0 K/V buffer free, 1 query buffer free, 2 K/V landed,
 * 3 queries landed, 4 probabilities ready, 5 accumulator slot free, 6 output ready, 7 scores ready).
 * Updated when a call returns PCM_ERR_DEVICE_TIMEOUT.  Host value, no GPU work. */
uint32_t grpo_attention_wait_status(void);

/* Per-kernel-class timing.  While enabled, every launch of the classes below is bracketed by a
 * pair of CUDA events on its stream; pcm_profile_read() synchronises the device, adds up elapsed
 * milliseconds, the algorithmic flops / bytes of the launches and their count since the last read,
 * and clears the records.  Classes: 0 GEMMs on the CTA-pair tensor-core kernel (the linear layers at
 * training sizes), 1 attention, 2 RMSNorm, 3 element-wise (rotary, SwiGLU, residual cast), 4 loss rows,
 * 5 embedding gradient, 6 pack, 7 phase-score reduction (the per-group kernel of pcm_score_phases),
 * 8 chunk sampling, 9 GEMMs on the single-CTA or SIMT kernels (narrow outputs, the head, fp32 mode). */
#define PCM_PROFILE_CLASSES 10
typedef struct {
  double ms[PCM_PROFILE_CLASSES];
  double flops[PCM_PROFILE_CLASSES];
  double bytes[PCM_PROFILE_CLASSES];
  int64_t launches[PCM_PROFILE_CLASSES];
} pcm_profile;
int pcm_profile_enable(int32_t on);
int pcm_profile_read(pcm_profile* out);

/* Number of kernels this library has launched in the calling process (for accounting). */
int64_t pcm_launch_count(void);

/* Host-only helper behind the library's per-device set-up (kernel attributes such as the dynamic shared-memory
 * limit belong to one device, so each launcher keeps a bit mask of the devices it has prepared): returns 1 and
 * sets bit `device` of *seen_mask on the first call for that device, 0 afterwards; devices outside 0..63 always
 * return 1.  No GPU work. */
int32_t pcm_first_use_on_device(uint64_t* seen_mask, int32_t device);

#ifdef __cplusplus
}
#endif
#endif /* PCM_B200_H */
