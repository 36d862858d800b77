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

# DRAM traffic of the dominant kernel from one ncu capture (profiles/gemm_tc2_kernel_M19968_N3072_K1024_ncu.md):
# dram__bytes_read.sum + dram__bytes_write.sum = 119.6 MB for the QKV-shaped launch at M = 19968 rows against
# 169.9 MB of algorithmic bytes; traffic grows in proportion to the rows for a fixed weight matrix.
GEMM_TRAFFIC_CAPTURE = {"rows": 19968, "n": 3072, "k": 1024, "dram_bytes": 119.6e6, "algorithmic_bytes": 169.9e6}

METRIC = "kept_chunks_per_s_actor_fwd_bwd"
UNIT = "chunks/s"
ACT = 56


def flops_per_kept_chunk(w) -> float:
    """Linear layers fwd + dgrad + wgrad, causal attention fwd + bwd, head."""
    S, d, L = w.S, w.d, w.L
    return 6.0 * S * 16 * d * d * L + 7.0 * S * S * d * L + 6.0 * ACT * d * 256


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
def oracle_sample_step(w, rb, weights, seed, n_sample):
    """One oracle pass: PCM control plane on the whole batch, actor forward + backward on the first
    n_sample kept chunks.  Returns (seconds for the control plane, seconds for the actor sample, n_kept)."""
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
    ao.fwd_bwd(weights, X, tgt, lpo, adv_c, w.H, w.P, w.eps_low, w.eps_high, 1.0 / (ACT * len(kept)))
    t_actor = time.perf_counter() - t1
    return t_pcm, t_actor, len(kept)


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([int(p.get("num_threads", 1)) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    """The oracle as it stands, timed on the host cores, on the same workload and metric."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2605_16154_b200 import synth
    w = synth.WORKLOADS[args.workload]
    rb = synth.make_rollouts(w)
    weights = synth.make_weights(w)
    n_sample = 1
    est = []
    for it in range(args.warmup + args.steps):
        t_pcm, t_actor, n_kept = oracle_sample_step(w, rb, weights, w.seed, n_sample)
        if it >= args.warmup:
            est.append(t_pcm + t_actor * n_kept / n_sample)
    ms = 1e3 * sum(est) / len(est)
    value = n_kept / (ms / 1e3)
    sample = (f"per step: control plane on the full batch + actor fwd/bwd on {n_sample} of {n_kept} kept chunks, "
              f"scaled by {n_kept}/{n_sample} (chunks are independent sequences)")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": {"workload": w.name, "kept_chunks_per_step": n_kept},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
# CUDA path
# ------------------------------------------------------------------------------------------------
def run_cuda(args):
    import torch
    import torch.distributed as dist

    from paper_2605_16154_b200 import build as _build
    _build.build()
    from paper_2605_16154_b200 import binding as B, dist_util, pipeline as PL, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    w = synth.WORKLOADS[args.workload]
    td = PL.torch_dtype(w)
    seed = dist_util.replica_seed(w.seed, rank)    # every rank works on its own batch (replicas, no exchange)
    rb = synth.make_rollouts(w, seed)
    weights = synth.make_weights(w)
    lengths = np.diff(rb["traj_off"])
    total = int(rb["traj_off"][-1])
    n_kept = PL.n_kept_of(w.budget, rb["traj_off"])
    mb = args.mb if args.mb > 0 else min(n_kept, 384)

    # host inputs in pinned memory (what an end-to-end caller owns)
    gen = torch.Generator().manual_seed(seed)
    h_obs = torch.empty((total, w.P, w.d), dtype=td).pin_memory()
    for c0 in range(0, total, 256):                 # N(0,1) prefixes, rounded to the model dtype
        c1 = min(total, c0 + 256)
        h_obs[c0:c1] = torch.randn((c1 - c0, w.P, w.d), generator=gen, dtype=torch.float32).to(td)
    h = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in rb.items()}

    model = PL.upload_model(w, weights)
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=seed, max_traj=w.n_traj)
    d_in = {k: v.cuda() for k, v in h.items()}
    d_obs = h_obs.cuda()

    # behaviour-policy log-probs: a forward-only pass of the library over every chunk, plus noise
    ident = B.Context(w.n_phases, int(lengths.max()), w.G, max_traj=w.n_traj)
    d_lpo = torch.zeros((total, ACT), dtype=torch.float32, device="cuda")
    batch = B.make_batch(d_in["traj_off"], d_in["tok"], d_in["phase"], d_in["reward"], int(lengths.max()), d_obs, d_lpo)
    ws_fwd = None
    zero_adv = torch.zeros(w.n_traj, dtype=torch.float32, device="cuda")
    for c0 in range(0, total, 512):
        c1 = min(total, c0 + 512)
        idx = torch.arange(c0, c1, dtype=torch.int32, device="cuda")
        off = torch.clamp(d_in["traj_off"].to(torch.int32) - c0, 0, c1 - c0).to(torch.int32).contiguous()
        pk_all = B.grpo_pack_chunks(ident, batch, model, idx, off, zero_adv, B.Packed(model, c1 - c0))
        _, lp, _, _ = B.grpo_actor_fwd_bwd(model, pk_all, flags=B.GRPO_FWD_ONLY, mb_chunks=128, workspace=ws_fwd)
        d_lpo[c0:c1] = lp
        del pk_all
    ident.close()
    d_lpo += torch.from_numpy(synth.logp_noise(seed, total, 0.1)).cuda()
    h_lpo = d_lpo.cpu().pin_memory()
    torch.cuda.empty_cache()

    # preallocated outputs and workspace
    packed = B.Packed(model, n_kept)
    ws = torch.empty(B.grpo_workspace_bytes(model, mb, 0) + 256, dtype=torch.uint8, device="cuda")
    samp = {"kept_idx": torch.empty(w.n_traj * w.budget, dtype=torch.int32, device="cuda"),
            "kept_off": torch.empty(w.n_traj + 1, dtype=torch.int32, device="cuda"),
            "kept_per_phase": torch.empty(w.n_phases, dtype=torch.int32, device="cuda")}
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    logp = torch.empty((n_kept, ACT), dtype=torch.float32, device="cuda")
    model.alloc_grads()

    def step(it, bt):
        Cc, valid, _, adv = B.pcm_score_phases(ctx, bt)
        _, q = B.pcm_update_keep_probs(ctx, Cc, valid)
        kept_idx, kept_off, _ = B.pcm_sample_chunks(ctx, bt, q, it, out=samp)
        B.grpo_pack_chunks(ctx, bt, model, kept_idx, kept_off, adv, packed)
        B.grpo_actor_fwd_bwd(model, packed, w.eps_low, w.eps_high, 0.0, mb_chunks=mb, workspace=ws, want_stats=False,
                             logp=logp, loss=loss)

    kept_host = torch.empty(w.n_traj * w.budget, dtype=torch.int32).pin_memory()

    def step_e2e(it):
        """Host buffers in, loss out.  The mask is applied before the big transfer: the control plane runs on
        the small arrays first, the kept chunk ids come back (a few KB), and only the kept chunks'
        observation prefixes cross the bus."""
        for k in ("traj_off", "tok", "phase", "reward"):
            d_in[k].copy_(h[k], non_blocking=True)
        d_lpo.copy_(h_lpo, non_blocking=True)
        Cc, valid, _, adv = B.pcm_score_phases(ctx, batch)
        _, q = B.pcm_update_keep_probs(ctx, Cc, valid)
        kept_idx, kept_off, _ = B.pcm_sample_chunks(ctx, batch, q, it, out=samp)
        kept_host.copy_(kept_idx, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for c in kept_host[:n_kept].tolist():
            d_obs[c].copy_(h_obs[c], non_blocking=True)
        B.grpo_pack_chunks(ctx, batch, model, kept_idx, kept_off, adv, packed)
        B.grpo_actor_fwd_bwd(model, packed, w.eps_low, w.eps_high, 0.0, mb_chunks=mb, workspace=ws, want_stats=False,
                             logp=logp, loss=loss)
        return float(loss.item())                  # device -> host read of the step's result

    chunk_bytes = w.P * w.d * h_obs.element_size()
    h2d = sum(v.numel() * v.element_size() for v in h.values()) + h_lpo.numel() * h_lpo.element_size() + \
        n_kept * chunk_bytes
    d2h = 4 + 4 * w.n_traj * w.budget

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

    it = 0
    for _ in range(max(args.warmup, 3)):
        step(it, batch); it += 1
    torch.cuda.synchronize()
    assert B.pcm_poll_status(ctx) == 0

    # ---- device-resident timing (with per-kernel-class event pairs) ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    B.pcm_profile_read()
    B.pcm_profile_enable(True)
    launches0 = B.pcm_launch_count()
    ms_total = timed(lambda i: step(i, batch), args.steps, it)
    it += args.steps
    launches = B.pcm_launch_count() - launches0
    B.pcm_profile_enable(False)
    prof = B.pcm_profile_read()
    clocks = sampler.stop() if rank == 0 else None

    # ---- end to end: host buffers, copies inside the timed region ----
    step_e2e(it); it += 1
    ms_e2e = timed(step_e2e, args.steps, it)
    it += args.steps
    loss_val = float(loss.item())
    status = B.pcm_poll_status(ctx)
    peak_alloc = torch.cuda.max_memory_allocated()

    if rank == 0:
        peaks = measured_peaks()
        ms_step = ms_total / args.steps
        value = dist_util.aggregate_throughput(n_kept, args.steps, ms_total, world)
        e2e_value = dist_util.aggregate_throughput(n_kept, args.steps, ms_e2e, world)
        g = prof["gemm"]
        achieved = g["flops"] / (g["ms"] * 1e9) if g["ms"] > 0 else 0.0
        peak = peaks["bf16_tflops_sustained"]
        step_tflops = flops_per_kept_chunk(w) * n_kept / (ms_step * 1e9)
        classes = {}
        for name, p in prof.items():
            if p["launches"] == 0:
                continue
            c = {"ms_per_step": p["ms"] / args.steps, "launches_per_step": p["launches"] / args.steps}
            if p["flops"] > 0:
                c["tflops"] = p["flops"] / (p["ms"] * 1e9)
            if p["bytes"] > 0:
                c["gbs"] = p["bytes"] / (p["ms"] * 1e6)
            classes[name] = c
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": w.name, "kept_chunks_per_step": n_kept, "chunks_per_step": total,
                       "tokens_per_step": n_kept * w.S, "mb_chunks": mb, "l2": "inputs_larger_than_l2",
                       "multi_gpu": "independent replicas, no collective"},
            "roofline": {"bound": "tensor", "kernel": "gemm_tc2_kernel", "achieved": achieved, "peak": peak,
                         "unit": "TFLOP/s", "frac": achieved / peak if peak else None,
                         "traffic": GEMM_TRAFFIC_CAPTURE["dram_bytes"] * (n_kept * w.S) / GEMM_TRAFFIC_CAPTURE["rows"]
                         if (w.d == 1024 and mb >= n_kept) else None,
                         "traffic_of": "QKV-shaped launch [tokens x 3072 x 1024], ncu capture at 19968 rows scaled by rows",
                         "peak_source": peaks["source"] + " bf16_tflops_sustained",
                         "launches_per_step": g["launches"] / args.steps,
                         "flops_per_launch": g["flops"] / max(1, g["launches"]),
                         "step_tflops": step_tflops, "step_frac": step_tflops / peak},
            "kernel_classes": classes,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "loss": loss_val, "device_status": status,
            "memory": {"workspace_bytes": int(ws.numel()), "peak_allocated_bytes": int(peak_alloc)},
        }
        if world == 1 and not args.no_cpu_baseline:
            t_pcm, t_actor, nk = oracle_sample_step(w, rb, weights, seed, args.cpu_sample)
            est = t_pcm + t_actor * nk / args.cpu_sample
            line["cpu_baseline"] = {
                "value": nk / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                "sample": (f"control plane on the full batch ({t_pcm:.2f} s) + actor fwd/bwd on {args.cpu_sample} of "
                           f"{nk} kept chunks ({t_actor:.2f} s), scaled by {nk}/{args.cpu_sample}")}
        print(json.dumps(line))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="C1")
    ap.add_argument("--mb", type=int, default=0, help="chunks per micro-batch (0: up to 384)")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--cpu-sample", type=int, default=2, help="kept chunks the CPU baseline leg runs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
