#!/usr/bin/env python
"""Benchmark of the GRPO actor update with Probabilistic Chunk Masking on B200.

A step is one pass of the whole hot path over one synthetic rollout batch: advantages + phase
scores, keep-probability update, fixed-budget sampling, pack of the kept chunks, actor forward and
backward.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C1] [--mb CHUNKS] [--impl reference]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

# DRAM traffic of the dominant kernel, from one ncu capture of ONE launch at the shape the medium workload runs
# (QKV projection, all 119 808 tokens in one micro-batch; profiles/gemm_tc2_kernel_M119808_N3072_K1024_traffic_ncu.md):
# dram__bytes_read.sum 251.74 MB (= A + B, each byte once) + dram__bytes_write.sum 686.61 MB (49 MB of C are still in
# L2 when the kernel ends).  Printed only when the run launches exactly this shape; never scaled from another size.
GEMM_TRAFFIC_CAPTURE = {"rows": 119808, "n": 3072, "k": 1024, "dram_bytes": 938.35e6, "algorithmic_bytes": 987.76e6}

# Context figures the paper reports for its own runs (7B policy with LoRA on 2 x H100, LIBERO): not targets.
PAPER_CONTEXT = {"wall_clock_speedup": 2.38, "gradient_update_speedup": 4.8, "activation_memory_reduction": 0.60,
                 "where": "Sec. 5 RQ2, Fig. 4; App. E hardware"}

METRIC = "kept_chunks_per_s_actor_fwd_bwd"
UNIT = "chunks/s"
ACT = 56


def flops_per_kept_chunk(w, lora_rank: int = 0) -> float:
    """The work the path executes per kept chunk: linear layers forward + input gradient + weight gradient, causal
    attention forward + backward, head.  In the last layer everything after the attention runs on the 56 scored
    rows only (W_o, gate|up, down: 13 d^2 of a layer's 16 d^2 per token), so those rows are what is counted.
    With adapters (rank r) the base weight gradients do not exist (4 d^2 instead of 6 per weight element) and each
    projection adds four rank-r products (x A^T, dy B, u^T x, dy^T t) plus the two continuation blocks."""
    S, d, L = w.S, w.d, w.L
    per_w = 6.0 if lora_rank == 0 else 4.0
    full_rows = S * 16 * d * d * (L - 1) + S * 3 * d * d      # layers 0..L-2, and the last layer's QKV
    scored_rows = ACT * 13 * d * d                            # last layer after the attention
    lin = per_w * (full_rows + scored_rows)
    if lora_rank:
        io_all = (d + 3 * d) + (d + d) + (d + 8 * d) + (4 * d + d)          # in + out of the four projections
        io_qkv = d + 3 * d
        # per projection and row: 2 r (in + out) flops forward (t, continuation) and 4 r (in + out) backward (u, continuation, dA, dB)
        lin += 6.0 * lora_rank * (S * io_all * (L - 1) + S * io_qkv + ACT * (io_all - io_qkv))
    return lin + 7.0 * S * S * d * L + 6.0 * ACT * d * 256


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = os.path.join("/tmp", f"pcm_bench_clocks_{os.getpid()}.csv")

    def start(self):
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, sm_max, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); sm_max.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        try:
            os.remove(self.path)
        except OSError:
            pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(sm_max), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle timing (baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_sample_step(w, rb, weights, seed, n_sample, lora_rank=0, adamw=False):
    """One oracle pass: PCM control plane on the whole batch, actor forward + backward on the first
    n_sample kept chunks, then (adamw) one optimizer step on what was trained.  Returns (seconds for the
    control plane, seconds for the actor sample, n_kept, seconds for the optimizer step)."""
    from oracle import actor_oracle as ao
    from oracle import pcm_oracle as po
    from paper_2605_16154_b200 import synth

    t0 = time.perf_counter()
    adv = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
    C, valid, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    _, q, _ = po.update_keep_probs(po.KeepProbState(w.n_phases, w.p_min, w.t_rc), C, valid)
    kept, off, _ = po.sample_chunks(rb["traj_off"], rb["phase"], q, w.budget, seed, 0)
    t_pcm = time.perf_counter() - t0
    sample = kept[:n_sample]
    obs = {int(c): synth.obs_chunk(w, seed, int(c)) for c in sample}
    total = int(rb["traj_off"][-1])
    lpo_all = np.full((total, ACT), -np.log(256.0), dtype=np.float32)
    t1 = time.perf_counter()
    X, tgt, lpo, adv_c, _ = po.pack_chunks(lambda c: obs[c], rb["tok"], lpo_all, adv, rb["traj_off"], sample, weights["e_act"])
    lo = synth.make_lora(w, lora_rank, float(lora_rank)) if lora_rank else None
    _, _, grads, _ = ao.fwd_bwd(weights, X, tgt, lpo, adv_c, w.H, w.P, w.eps_low, w.eps_high, 1.0 / (ACT * len(kept)), lora=lo)
    t_actor = time.perf_counter() - t1
    t_opt = 0.0
    if adamw:
        from oracle import optim_oracle as oo
        source = dict(weights, **{k: v for k, v in (lo or {}).items() if k not in ("rank", "alpha")})
        params = {k: np.asarray(source[k], dtype=np.float64) for k, g in grads.items() if g is not None}
        m = {k: np.zeros_like(v) for k, v in params.items()}
        v = {k: np.zeros_like(v) for k, v in params.items()}
        t2 = time.perf_counter()
        oo.adamw_step(params, {k: grads[k] for k in params}, m, v, 1)
        t_opt = time.perf_counter() - t2
    return t_pcm, t_actor, len(kept), t_opt


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([int(p.get("num_threads", 1)) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def config_of(w, n_kept, total, mb, iterations=None, lora_rank=0, dp=False, world=1, adamw=False):
    """The `config` object both arms print."""
    c = {"workload": w.name, "trainable": f"LoRA rank {lora_rank}, alpha {lora_rank}, base frozen" if lora_rank else "all weights", "kept_chunks_per_step": int(n_kept), "chunks_per_step": int(total),
         "tokens_per_step": int(n_kept) * w.S, "mb_chunks": int(mb), "l2": "inputs_larger_than_l2",
         "multi_gpu": (f"data parallel over {world} ranks: one batch, kept chunks dealt out by trajectory, one fp32 gradient "
                       "all-reduce per step") if dp else "independent replicas, no collective"}
    c["optimizer"] = "gradient clipping at 2.0 + AdamW after every update (App. E)" if adamw else "none (gradients only)"
    if iterations is not None:
        c["iterations"] = int(iterations)
        c["resampled"] = "rollouts redrawn every iteration from seeds 0..iterations-1, keep-probability state carried"
    return c


def launch_steps_online(args):
    return args.steps


def default_mb(args, n_kept):
    return args.mb if args.mb > 0 else min(n_kept, 384)


def run_reference(args):
    """The oracle as it stands, timed on the host cores, on the same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_16154_b200 import synth
    w = synth.WORKLOADS[args.workload]
    online = w.T == 0
    rb = synth.make_rollouts(w, 0 if online else None)
    weights = synth.make_weights(w)
    n_sample = 1
    est = []
    for it in range(args.warmup + args.steps):
        t_pcm, t_actor, n_kept, t_opt = oracle_sample_step(w, rb, weights, w.seed, n_sample, args.lora, args.adamw)
        if it >= args.warmup:
            est.append(t_pcm + t_actor * n_kept / n_sample + t_opt)
    ms = 1e3 * sum(est) / len(est)
    value = n_kept / (ms / 1e3)
    total = int(rb["traj_off"][-1])
    sample = (f"per step: control plane on the full batch + actor fwd/bwd on {n_sample} of {n_kept} kept chunks, "
              f"scaled by {n_kept}/{n_sample} (chunks are independent sequences)"
              + (", + one optimizer step" if args.adamw else "") + "; ms_per_step is that estimate")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": config_of(w, n_kept, total, default_mb(args, n_kept), launch_steps_online(args) if online else None,
                                args.lora, adamw=args.adamw),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
class Harness:
    """Device state shared by the timed legs: model, workspace, preallocated outputs."""

    def __init__(self, B, PL, synth, w, weights, n_kept_max, mb, lora_rank=0, adamw=False):
        import torch
        self.B, self.w, self.mb = B, w, mb
        self.model = PL.upload_model(w, weights)
        self.model.alloc_grads()
        # adapters part-way through training (non-zero B), alpha = rank as in App. E
        self.lora = PL.upload_lora(w, self.model, synth.make_lora(w, lora_rank, float(lora_rank))) if lora_rank else None
        self.ws = torch.empty(B.grpo_workspace_bytes(self.model, mb, 0, self.lora) + 256, dtype=torch.uint8, device="cuda")
        if self.lora is not None:
            self.lora.alloc_grads()
        self.opt = None
        if adamw:                                    # App. E: lr 1e-5, betas (0.9, 0.999), no decay, clip at 2.0
            self.opt = B.LoraAdamW(self.model, self.lora) if self.lora is not None else B.AdamW(self.model)
        self.dp, self.loss_scale, self.dist_util = None, 0.0, None      # set by data_parallel()
        self.loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.outputs(n_kept_max, w.n_traj, w.budget)

    def data_parallel(self, dist_util, rank, world, n_kept_global):
        """The ranks share one batch: this one takes its trajectories under the whole batch's loss scale."""
        self.dist_util, self.dp, self.loss_scale = dist_util, (rank, world), 1.0 / (ACT * n_kept_global)

    def outputs(self, n_kept, n_traj, budget):
        import torch
        B = self.B
        self.n_kept = n_kept
        self.packed = B.Packed(self.model, n_kept)
        self.samp = {"kept_idx": torch.empty(n_traj * budget, dtype=torch.int32, device="cuda"),
                     "kept_off": torch.empty(n_traj + 1, dtype=torch.int32, device="cuda"),
                     "kept_per_phase": torch.empty(self.w.n_phases, dtype=torch.int32, device="cuda")}
        self.logp = torch.empty((n_kept, ACT), dtype=torch.float32, device="cuda")

    def select(self, ctx, bt, it):
        B = self.B
        Cc, valid, _, adv = B.pcm_score_phases(ctx, bt)
        _, q = B.pcm_update_keep_probs(ctx, Cc, valid)
        kept_idx, kept_off, _ = B.pcm_sample_chunks(ctx, bt, q, it, out=self.samp)
        if self.dp is not None:                      # data parallel: this rank's trajectories of the shared selection
            kept_idx, kept_off = self.dist_util.partition_kept(kept_idx, kept_off, *self.dp)
        return adv, kept_idx, kept_off, q

    def update(self, ctx, bt, adv, kept_idx, kept_off):
        B, w = self.B, self.w
        B.grpo_pack_chunks(ctx, bt, self.model, kept_idx, kept_off, adv, self.packed)
        B.grpo_actor_fwd_bwd(self.model, self.packed, w.eps_low, w.eps_high, self.loss_scale, mb_chunks=self.mb,
                             workspace=self.ws, want_stats=False, logp=self.logp, loss=self.loss, lora=self.lora)
        if self.dp is not None:                      # one sum over the ranks: full-batch gradient (and loss) everywhere
            self.dist_util.allreduce_sum(self.lora.flat_grads if self.lora is not None else self.model.flat_grads)
            if self.lora is not None:
                self.dist_util.allreduce_sum(self.model.flat_grads)
            self.dist_util.allreduce_sum(self.loss)
        if self.opt is not None:
            self.opt.step()

    def step(self, ctx, bt, it):
        adv, kept_idx, kept_off, _ = self.select(ctx, bt, it)
        self.update(ctx, bt, adv, kept_idx, kept_off)


def class_table(prof, steps):
    classes = {}
    for name, p in prof.items():
        if p["launches"] == 0:
            continue
        c = {"ms_per_step": p["ms"] / steps, "launches_per_step": p["launches"] / steps}
        if p["flops"] > 0:
            c["tflops"] = p["flops"] / (p["ms"] * 1e9)
        if p["bytes"] > 0:
            c["gbs"] = p["bytes"] / (p["ms"] * 1e6)
        classes[name] = c
    return classes


def roofline_of(prof, peaks, steps, step_flops, ms_step, traffic):
    """The dominant kernel: gemm_tc2_kernel (CTA-pair tcgen05 GEMM), every launch of it in the timed region."""
    g = prof["gemm"]
    achieved = g["flops"] / (g["ms"] * 1e9) if g["ms"] > 0 else 0.0
    peak = peaks["bf16_tflops_sustained"]
    step_tflops = step_flops / (ms_step * 1e9)
    return {"bound": "tensor", "kernel": "gemm_tc2_kernel", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
            "frac": achieved / peak if peak else None, "traffic": traffic,
            "traffic_of": ("one QKV-projection launch [119808 x 3072 x 1024], ncu dram read + write; algorithmic 987.76 MB, "
                           "of which 49 MB of the output are still in L2 when the kernel ends"
                           if traffic is not None else "no capture of the current kernel at this shape"),
            "peak_source": peaks["source"] + " bf16_tflops_sustained (kernel timed inside a long step)",
            "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "frac_of_nominal_2250": achieved / 2250.0,
            "launches_per_step": g["launches"] / steps, "flops_per_launch": g["flops"] / max(1, g["launches"]),
            "ms_per_launch": g["ms"] / max(1, g["launches"]),
            "step_tflops": step_tflops, "step_frac": step_tflops / peak, "step_frac_of_nominal_2250": step_tflops / 2250.0}


def run_cuda(args):
    import torch
    import torch.distributed as dist

    from paper_2605_16154_b200 import build as _build
    _build.build()
    from paper_2605_16154_b200 import binding as B, dist_util, launch, pipeline as PL, synth

    rank, world, local_rank = launch.rank_world_local()
    torch.cuda.set_device(local_rank)
    launch.init_process_group("nccl", torch.device("cuda", local_rank))

    w = synth.WORKLOADS[args.workload]
    if w.T == 0:
        assert not args.dp, "--dp is implemented for the fixed-length workloads"
        run_online(args, torch, dist, B, dist_util, PL, synth, w, rank, world, local_rank)
    else:
        run_fixed(args, torch, dist, B, dist_util, PL, synth, w, rank, world, local_rank)
    if world > 1:
        dist.destroy_process_group()


def make_timers(torch, dist, dist_util, world):
    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, it0):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record()
        for i in range(steps):
            fn(it0 + i)
        ev1.record()
        barrier()
        return dist_util.max_over_ranks(ev0.elapsed_time(ev1), "cuda")
    return barrier, timed


def behaviour_logp(torch, B, synth, w, model, d_in, d_obs, lengths, total, seed, lora=None):
    """Behaviour-policy log-probs: a forward-only pass of the library over every chunk, plus seeded noise."""
    ident = B.Context(w.n_phases, int(lengths.max()), w.G, max_traj=w.n_traj)
    d_lpo = torch.zeros((total, ACT), dtype=torch.float32, device="cuda")
    batch = B.make_batch(d_in["traj_off"], d_in["tok"], d_in["phase"], d_in["reward"], int(lengths.max()), d_obs, d_lpo)
    zero_adv = torch.zeros(w.n_traj, dtype=torch.float32, device="cuda")
    for c0 in range(0, total, 512):
        c1 = min(total, c0 + 512)
        idx = torch.arange(c0, c1, dtype=torch.int32, device="cuda")
        off = torch.clamp(d_in["traj_off"].to(torch.int32) - c0, 0, c1 - c0).to(torch.int32).contiguous()
        pk_all = B.grpo_pack_chunks(ident, batch, model, idx, off, zero_adv, B.Packed(model, c1 - c0))
        _, lp, _, _ = B.grpo_actor_fwd_bwd(model, pk_all, flags=B.GRPO_FWD_ONLY, mb_chunks=128, lora=lora)
        d_lpo[c0:c1] = lp
        del pk_all
    ident.close()
    d_lpo += torch.from_numpy(synth.logp_noise(seed, total, 0.1)).cuda()
    torch.cuda.empty_cache()
    return d_lpo, batch


def run_fixed(args, torch, dist, B, dist_util, PL, synth, w, rank, world, local_rank):
    """Fixed-length workloads (C0-C3): K steps over one resident batch."""
    td = PL.torch_dtype(w)
    # replicas: every rank works on its own batch, no exchange.  --dp: all ranks share the batch of rank 0's seed
    seed = w.seed if args.dp else dist_util.replica_seed(w.seed, rank)
    rb = synth.make_rollouts(w, seed)
    weights = synth.make_weights(w)
    lengths = np.diff(rb["traj_off"])
    total = int(rb["traj_off"][-1])
    n_kept_global = PL.n_kept_of(w.budget, rb["traj_off"])
    n_kept = dist_util.local_kept_count(lengths, w.budget, rank, world) if args.dp else n_kept_global
    mb = default_mb(args, n_kept)

    # host inputs in pinned memory (what an end-to-end caller owns)
    gen = torch.Generator().manual_seed(seed)
    h_obs = torch.empty((total, w.P, w.d), dtype=td).pin_memory()
    for c0 in range(0, total, 256):                 # N(0,1) prefixes, rounded to the model dtype
        c1 = min(total, c0 + 256)
        h_obs[c0:c1] = torch.randn((c1 - c0, w.P, w.d), generator=gen, dtype=torch.float32).to(td)
    h = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in rb.items()}

    hs = Harness(B, PL, synth, w, weights, n_kept, mb, args.lora, args.adamw)
    if args.dp:
        hs.data_parallel(dist_util, rank, world, n_kept_global)
    model = hs.model
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=seed, max_traj=w.n_traj)
    d_in = {k: v.cuda() for k, v in h.items()}
    d_obs = h_obs.cuda()
    d_lpo, batch = behaviour_logp(torch, B, synth, w, model, d_in, d_obs, lengths, total, seed, hs.lora)
    h_lpo = d_lpo.cpu().pin_memory()
    kept_host = torch.empty(w.n_traj * w.budget, dtype=torch.int32).pin_memory()

    def step_e2e(it):
        """Host buffers in, loss out.  The mask is applied before the big transfer: the control plane runs on
        the small arrays first, the kept chunk ids come back (a few KB), and only the kept chunks'
        observation prefixes cross the bus."""
        for k in ("traj_off", "tok", "phase", "reward"):
            d_in[k].copy_(h[k], non_blocking=True)
        d_lpo.copy_(h_lpo, non_blocking=True)
        adv, kept_idx, kept_off, _ = hs.select(ctx, batch, it)
        kept_host[:kept_idx.numel()].copy_(kept_idx, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for c in kept_host[:n_kept].tolist():
            d_obs[c].copy_(h_obs[c], non_blocking=True)
        hs.update(ctx, batch, adv, kept_idx, kept_off)
        return float(hs.loss.item())                  # device -> host read of the step's result

    chunk_bytes = w.P * w.d * h_obs.element_size()
    h2d = sum(v.numel() * v.element_size() for v in h.values()) + h_lpo.numel() * h_lpo.element_size() + \
        n_kept * chunk_bytes
    d2h = 4 + 4 * w.n_traj * w.budget
    barrier, timed = make_timers(torch, dist, dist_util, world)

    it = 0
    for _ in range(max(args.warmup, 3)):
        hs.step(ctx, batch, it); it += 1
    torch.cuda.synchronize()
    assert B.pcm_poll_status(ctx) == 0

    # ---- device-resident timing (with per-kernel-class event pairs) ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    B.pcm_profile_read()
    B.pcm_profile_enable(True)
    launches0 = B.pcm_launch_count()
    ms_total = timed(lambda i: hs.step(ctx, batch, i), args.steps, it)
    it += args.steps
    launches = B.pcm_launch_count() - launches0
    B.pcm_profile_enable(False)
    prof = B.pcm_profile_read()
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: host buffers, copies inside the timed region ----
    step_e2e(it); it += 1
    ms_e2e = timed(step_e2e, args.steps, it)
    it += args.steps
    loss_val = float(hs.loss.item())
    status = B.pcm_poll_status(ctx)
    peak_alloc = torch.cuda.max_memory_allocated()

    # ---- the same update with the mask keeping every chunk (plain GRPO), for the masked / full ratio ----
    masked_full = None
    if w.name == "C1" and world == 1 and not args.no_masked_full and not args.dp:
        full_steps = 3
        ctx_full = B.Context(w.n_phases, int(lengths.max()), w.G, w.t_rc, w.p_min, 1e-6, seed=seed, max_traj=w.n_traj)
        hs.outputs(total, w.n_traj, int(lengths.max()))
        full_step = lambda i: hs.step(ctx_full, batch, i)
        full_step(0)
        ms_full = timed(full_step, full_steps, 1) / full_steps
        assert B.pcm_poll_status(ctx_full) == 0
        ctx_full.close()
        traj_mb = 8                                    # trajectories per micro-batch for the activation figure
        act_masked = B.grpo_workspace_bytes(model, traj_mb * w.budget, 0, hs.lora)
        act_full = B.grpo_workspace_bytes(model, traj_mb * int(lengths.max()), 0, hs.lora)
        masked_full = {"ms_masked": ms_total / args.steps, "ms_full": ms_full, "speedup": ms_full / (ms_total / args.steps),
                       "kept_chunks_masked": n_kept, "kept_chunks_full": total, "steps_full": full_steps,
                       "activation_bytes": {"masked": int(act_masked), "full": int(act_full),
                                            "ratio": act_masked / act_full,
                                            "of": f"library workspace for micro-batches of {traj_mb} trajectories "
                                                  f"({traj_mb * w.budget} vs {traj_mb * int(lengths.max())} chunks), no recompute"},
                       "context": PAPER_CONTEXT}

    if rank == 0:
        peaks = measured_peaks()
        ms_step = ms_total / args.steps
        if args.dp:                                   # one batch over all ranks: the whole job is n_kept_global per step
            value = dist_util.aggregate_throughput(n_kept_global, args.steps, ms_total, 1)
            e2e_value = dist_util.aggregate_throughput(n_kept_global, args.steps, ms_e2e, 1)
        else:
            value = dist_util.aggregate_throughput(n_kept, args.steps, ms_total, world)
            e2e_value = dist_util.aggregate_throughput(n_kept, args.steps, ms_e2e, world)
        traffic = None
        if GEMM_TRAFFIC_CAPTURE and GEMM_TRAFFIC_CAPTURE["rows"] == min(mb, n_kept) * w.S and w.d == GEMM_TRAFFIC_CAPTURE["k"]:
            traffic = GEMM_TRAFFIC_CAPTURE["dram_bytes"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if args.dp else "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": config_of(w, n_kept_global if args.dp else n_kept, total, mb, None, args.lora, args.dp, world, args.adamw),
            "roofline": roofline_of(prof, peaks, args.steps, flops_per_kept_chunk(w, args.lora) * n_kept, ms_step, traffic),
            "kernel_classes": class_table(prof, args.steps),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "loss": loss_val, "device_status": status,
            "memory": {"workspace_bytes": int(hs.ws.numel()), "peak_allocated_bytes": int(peak_alloc)},
        }
        if masked_full is not None:
            line["masked_full"] = masked_full
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_leg(args, w, rb, weights, seed)
        print(json.dumps(line))
    ctx.close()


def cpu_baseline_leg(args, w, rb, weights, seed):
    t_pcm, t_actor, nk, t_opt = oracle_sample_step(w, rb, weights, seed, args.cpu_sample, args.lora, args.adamw)
    est = t_pcm + t_actor * nk / args.cpu_sample + t_opt
    return {"value": nk / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle (fp64 numpy, BLAS threads = cores)",
            "sample": (f"control plane on the full batch ({t_pcm:.2f} s) + actor fwd/bwd on {args.cpu_sample} of "
                       f"{nk} kept chunks ({t_actor:.2f} s), scaled by {nk}/{args.cpu_sample}"
                       + (f" + one optimizer step ({t_opt:.2f} s)" if args.adamw else ""))}


def run_online(args, torch, dist, B, dist_util, PL, synth, w, rank, world, local_rank):
    """Ragged workload (C4): Algorithm 1's loop.  Every iteration draws a new rollout batch (seed = iteration), the
    keep-probability state is carried from one iteration to the next and refreshed every T_rc of them, so the
    kept-chunk mix and the ragged tail of the last micro-batch change as the loop runs."""
    td = PL.torch_dtype(w)
    n_iter = args.steps
    base = dist_util.replica_seed(0, rank)
    batches = [synth.make_rollouts(w, base + it) for it in range(n_iter)]
    weights = synth.make_weights(w)
    totals = [int(b["traj_off"][-1]) for b in batches]
    max_len = max(int(np.diff(b["traj_off"]).max()) for b in batches)
    kept_per_it = [PL.n_kept_of(w.budget, b["traj_off"]) for b in batches]
    n_kept_max = max(kept_per_it)
    mb = default_mb(args, n_kept_max)
    pool = max(totals)

    # Observation prefixes: one pool of iid N(0,1) rows (seeded, drawn on the device and copied to pinned host memory,
    # which is what the end-to-end leg reads); chunk c of every iteration uses pool row c.
    g = torch.Generator(device="cuda").manual_seed(base + 17)
    d_obs = torch.empty((pool, w.P, w.d), dtype=td, device="cuda")
    for c0 in range(0, pool, 1024):
        c1 = min(pool, c0 + 1024)
        d_obs[c0:c1] = torch.randn((c1 - c0, w.P, w.d), generator=g, device="cuda").to(td)
    h_obs = torch.empty((pool, w.P, w.d), dtype=td).pin_memory()
    h_obs.copy_(d_obs)
    # behaviour policy: near-uniform log-probs plus seeded noise (the synthetic weights give near-uniform logits)
    host, dev_b = [], []
    for it, rb in enumerate(batches):
        hb = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in rb.items()}
        hb["lpo"] = torch.from_numpy((-np.log(256.0) + synth.logp_noise(base + it, totals[it], 0.1)).astype(np.float32)).pin_memory()
        host.append(hb)
        db = {k: v.cuda() for k, v in hb.items()}
        dev_b.append((db, B.make_batch(db["traj_off"], db["tok"], db["phase"], db["reward"], max_len, d_obs, db["lpo"])))

    hs = Harness(B, PL, synth, w, weights, n_kept_max, mb, args.lora, args.adamw)
    barrier, timed = make_timers(torch, dist, dist_util, world)
    # staging buffers of the end-to-end leg (sized for the largest iteration)
    stage = {"traj_off": torch.empty(w.n_traj + 1, dtype=torch.int32, device="cuda"),
             "tok": torch.empty((pool, ACT), dtype=torch.uint8, device="cuda"),
             "phase": torch.empty(pool, dtype=torch.uint8, device="cuda"),
             "reward": torch.empty(w.n_traj, dtype=torch.uint8, device="cuda"),
             "lpo": torch.empty((pool, ACT), dtype=torch.float32, device="cuda")}
    kept_host = torch.empty(w.n_traj * w.budget, dtype=torch.int32).pin_memory()

    def set_kept(it):
        hs.packed.c.n_kept = hs.packed.n_kept = kept_per_it[it]

    def new_ctx():
        return B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=base, max_traj=w.n_traj)

    # warm-up on a context of its own, so that the timed chains start from a fresh keep-probability state
    ctx = new_ctx()
    for it in range(max(args.warmup, 3)):
        set_kept(it % n_iter)
        hs.step(ctx, dev_b[it % n_iter][1], it)
    torch.cuda.synchronize()
    assert B.pcm_poll_status(ctx) == 0
    ctx.close()

    # ---- device-resident chain ----
    ctx = new_ctx()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    B.pcm_profile_read()
    B.pcm_profile_enable(True)
    launches0 = B.pcm_launch_count()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_iter + 1)]
    q_hist = []
    barrier()
    evs[0].record()
    for it in range(n_iter):
        set_kept(it)
        adv, kept_idx, kept_off, q = hs.select(ctx, dev_b[it][1], it)
        hs.update(ctx, dev_b[it][1], adv, kept_idx, kept_off)
        q_hist.append(q)
        evs[it + 1].record()
    barrier()
    ms_total = dist_util.max_over_ranks(evs[0].elapsed_time(evs[n_iter]), "cuda")
    per_it = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_iter)]
    launches = B.pcm_launch_count() - launches0
    B.pcm_profile_enable(False)
    prof = B.pcm_profile_read()
    clocks = sampler.stop() if rank == 0 else None
    assert B.pcm_poll_status(ctx) == 0
    q_np = np.stack([t.cpu().numpy() for t in q_hist]).astype(np.int64)
    ctx.close()

    # ---- end to end chain: every iteration's batch comes from pinned host memory ----
    ctx = new_ctx()
    e2e_batch = B.make_batch(stage["traj_off"], stage["tok"], stage["phase"], stage["reward"], max_len, d_obs, stage["lpo"])
    h2d = d2h = 0

    def step_e2e(it):
        nonlocal h2d, d2h
        hb, n = host[it], totals[it]
        stage["traj_off"].copy_(hb["traj_off"], non_blocking=True)
        stage["reward"].copy_(hb["reward"], non_blocking=True)
        stage["tok"][:n].copy_(hb["tok"], non_blocking=True)
        stage["phase"][:n].copy_(hb["phase"], non_blocking=True)
        stage["lpo"][:n].copy_(hb["lpo"], non_blocking=True)
        e2e_batch.n_chunks = n
        set_kept(it)
        adv, kept_idx, kept_off, _ = hs.select(ctx, e2e_batch, it)
        kept_host.copy_(kept_idx, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for c in kept_host[:kept_per_it[it]].tolist():
            d_obs[c].copy_(h_obs[c], non_blocking=True)
        hs.update(ctx, e2e_batch, adv, kept_idx, kept_off)
        h2d += sum(hb[k].numel() * hb[k].element_size() for k in hb) + kept_per_it[it] * w.P * w.d * h_obs.element_size()
        d2h += 4 + 4 * w.n_traj * w.budget
        return float(hs.loss.item())

    ms_e2e = timed(step_e2e, n_iter, 0)
    loss_val = float(hs.loss.item())
    status = B.pcm_poll_status(ctx)
    peak_alloc = torch.cuda.max_memory_allocated()
    ctx.close()

    if rank == 0:
        peaks = measured_peaks()
        n_kept_total = sum(kept_per_it)
        ms_step = ms_total / n_iter
        value = world * n_kept_total / (ms_total / 1e3)
        e2e_value = world * n_kept_total / (ms_e2e / 1e3)
        refreshes = int((np.abs(np.diff(q_np, axis=0)).sum(axis=1) > 0).sum()) + 1
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": n_iter,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(w, n_kept_total / n_iter, sum(totals) / n_iter, mb, n_iter, args.lora, adamw=args.adamw),
            "online": {"ms_mean": statistics.mean(per_it), "ms_min": min(per_it), "ms_max": max(per_it),
                       "kept_chunks_min": min(kept_per_it), "kept_chunks_max": max(kept_per_it),
                       "chunks_min": min(totals), "chunks_max": max(totals),
                       "keep_prob_refreshes": refreshes, "t_rc": w.t_rc,
                       "keep_probs_first": (q_np[0] / float(1 << 24)).round(4).tolist(),
                       "keep_probs_last": (q_np[-1] / float(1 << 24)).round(4).tolist()},
            "roofline": roofline_of(prof, peaks, n_iter, flops_per_kept_chunk(w, args.lora) * n_kept_total / n_iter, ms_step, None),
            "kernel_classes": class_table(prof, n_iter),
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d / n_iter),
                    "d2h_bytes_per_step": int(d2h / n_iter), "ms_per_step": ms_e2e / n_iter},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "loss": loss_val, "device_status": status,
            "memory": {"workspace_bytes": int(hs.ws.numel()), "peak_allocated_bytes": int(peak_alloc)},
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_leg(args, w, batches[0], weights, base)
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 10; the ragged workload: 50 iterations)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C1")
    ap.add_argument("--mb", type=int, default=0, help="chunks per micro-batch (0: up to 384)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=2, help="kept chunks the CPU baseline leg runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-masked-full", action="store_true", help="skip the keep-every-chunk leg of the medium workload")
    ap.add_argument("--dp", action="store_true",
                    help="data parallel instead of replicas: the ranks share one batch and all-reduce the gradients")
    ap.add_argument("--lora", type=int, default=0, metavar="RANK",
                    help="fine-tune low-rank adapters of this rank (alpha = rank) with the base weights frozen")
    ap.add_argument("--adamw", action="store_true",
                    help="follow every actor update with the optimizer step (clip + AdamW), inside the timed region")
    args = ap.parse_args()
    from paper_2605_16154_b200 import launch
    if args.impl == "cuda" and launch.needs_relaunch(args.gpus, os.environ):
        cmd = launch.torchrun_command(args.gpus, os.path.abspath(__file__), sys.argv[1:])
        os.execv(cmd[0], cmd)
    if args.steps is None:
        args.steps = launch.default_steps(args.workload, args.impl)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
