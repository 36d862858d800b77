"""Per-kernel measurements through the C ABI (CUDA events, warm-up, inputs larger than L2 where the
kernel is bandwidth bound).  One JSON line per case.

    python -m paper_2605_16154_b200.microbench gemm [--m 19968 --n 3072 --k 1024 --layout nt|nn|tn --out bf16|f32|acc]
    python -m paper_2605_16154_b200.microbench attention [--seqs 64 --S 312 --heads 16 --dh 64]
    python -m paper_2605_16154_b200.microbench pcm [--tasks 8192 --G 8 --T 128 --phases 10 --budget 24]
    python -m paper_2605_16154_b200.microbench pack [--kept 384 --P 256 --d 1024]
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from . import binding as B


def _time(fn, iters, warmup=3):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def bench_gemm(a):
    M, N, K = a.m, a.n, a.k
    g = torch.Generator(device="cuda").manual_seed(0)
    layouts = {"nt": (True, True), "nn": (True, False), "tn": (False, False)}   # forward, input-gradient, weight-gradient
    a_k, b_k = layouts[a.layout]
    A = torch.randn((M, K) if a_k else (K, M), generator=g, device="cuda").to(torch.bfloat16)
    Bm = torch.randn((N, K) if b_k else (K, N), generator=g, device="cuda").to(torch.bfloat16)
    if a.out == "acc":
        C = torch.zeros((M, N), dtype=torch.float32, device="cuda")
        fn = lambda: B.grpo_gemm(A, a_k, Bm, b_k, M, N, K, R=C, backend=a.backend | 4, C_out=C)
    else:
        C = torch.empty((M, N), dtype=torch.bfloat16 if a.out == "bf16" else torch.float32, device="cuda")
        fn = lambda: B.grpo_gemm(A, a_k, Bm, b_k, M, N, K, backend=a.backend | 4, C_out=C)
    ms = _time(fn, a.iters)
    print(json.dumps({"kernel": "gemm", "M": M, "N": N, "K": K, "layout": a.layout, "out": a.out, "ms": ms,
                      "tflops": 2.0 * M * N * K / (ms * 1e9)}))


def bench_attention(a):
    d = a.heads * a.dh
    g = torch.Generator(device="cuda").manual_seed(0)
    qkv = torch.randn((a.seqs * a.S, 3 * d), generator=g, device="cuda").to(torch.bfloat16)
    do = torch.randn((a.seqs * a.S, d), generator=g, device="cuda").to(torch.bfloat16)
    ms_f = _time(lambda: B.grpo_attention(qkv, a.seqs, a.S, a.heads, a.dh), a.iters)
    ms_fb = _time(lambda: B.grpo_attention(qkv, a.seqs, a.S, a.heads, a.dh, dout=do), a.iters)
    f_fwd = 2.0 * a.S * a.S * d * a.seqs
    print(json.dumps({"kernel": "attention", "seqs": a.seqs, "S": a.S, "heads": a.heads, "dh": a.dh, "fwd_ms": ms_f,
                      "bwd_ms": ms_fb - ms_f, "fwd_tflops": f_fwd / (ms_f * 1e9),
                      "bwd_tflops": 2.5 * f_fwd / ((ms_fb - ms_f) * 1e9)}))


def bench_pcm(a):
    """Scoring and sampling on a batch scaled up until the token array is far larger than L2."""
    n_traj, total = a.tasks * a.G, a.tasks * a.G * a.T
    g = torch.Generator(device="cuda").manual_seed(0)
    tok = torch.randint(0, 256, (total, 56), generator=g, device="cuda", dtype=torch.uint8)
    phase = ((torch.arange(total, device="cuda") % a.T) * a.phases // a.T).to(torch.uint8)
    reward = (torch.rand(n_traj, generator=g, device="cuda") < 0.4).to(torch.uint8)
    traj_off = (torch.arange(n_traj + 1, device="cuda") * a.T).to(torch.int32)
    ctx = B.Context(a.phases, a.budget, a.G, max_traj=n_traj)
    batch = B.make_batch(traj_off, tok, phase, reward, a.T)
    Cc, valid, _, _ = B.pcm_score_phases(ctx, batch)
    _, q = B.pcm_update_keep_probs(ctx, Cc, valid)
    out = {"kept_idx": torch.empty(n_traj * a.budget, dtype=torch.int32, device="cuda"),
           "kept_off": torch.empty(n_traj + 1, dtype=torch.int32, device="cuda"),
           "kept_per_phase": torch.empty(a.phases, dtype=torch.int32, device="cuda")}
    B.pcm_profile_read()
    B.pcm_profile_enable(True)
    for it in range(a.iters + 3):
        B.pcm_score_phases(ctx, batch)
        B.pcm_sample_chunks(ctx, batch, q, it, out=out)
        if it == 2:
            B.pcm_profile_read()          # drop the warm-up iterations
    B.pcm_profile_enable(False)
    prof_all = B.pcm_profile_read()
    prof, prof_s = prof_all["pcm_score"], prof_all["pcm_sample"]
    ms_score = _time(lambda: B.pcm_score_phases(ctx, batch), a.iters)
    ms_sample = _time(lambda: B.pcm_sample_chunks(ctx, batch, q, 1, out=out), a.iters)
    print(json.dumps({"kernel": "pcm", "n_traj": n_traj, "chunks": total, "input_bytes": total * 57,
                      "score_ms": ms_score, "score_gbs": total * 57 / (ms_score * 1e6),
                      "sample_ms": ms_sample, "sample_gbs": (total + 4 * n_traj * a.budget) / (ms_sample * 1e6),
                      "score_groups_kernel_ms": prof["ms"] / max(1, prof["launches"]),
                      "score_groups_kernel_gbs": prof["bytes"] / (prof["ms"] * 1e6) if prof["ms"] > 0 else None,
                      "sample_kernel_ms": prof_s["ms"] / max(1, prof_s["launches"]),
                      "status": B.pcm_poll_status(ctx)}))
    ctx.close()


def bench_pack(a):
    n_chunks = max(a.kept * 5, a.kept + 1)
    g = torch.Generator(device="cuda").manual_seed(0)
    obs = torch.randn((n_chunks, a.P, a.d), generator=g, device="cuda").to(torch.bfloat16)
    tok = torch.randint(0, 256, (n_chunks, 56), generator=g, device="cuda", dtype=torch.uint8)
    lpo = torch.zeros((n_chunks, 56), device="cuda")
    e_act = torch.randn((256, a.d), generator=g, device="cuda").to(torch.bfloat16)
    traj_off = torch.tensor([0, n_chunks], dtype=torch.int32, device="cuda")
    phase = torch.zeros(n_chunks, dtype=torch.uint8, device="cuda")
    reward = torch.zeros(1, dtype=torch.uint8, device="cuda")
    ctx = B.Context(1, a.kept, 1, max_traj=1)
    batch = B.make_batch(traj_off, tok, phase, reward, n_chunks, obs, lpo)
    kept_idx = (torch.arange(a.kept, device="cuda") * 5).to(torch.int32)
    kept_off = torch.tensor([0, a.kept], dtype=torch.int32, device="cuda")
    adv = torch.zeros(1, device="cuda")

    class _M:
        cfg = B.grpo_model_cfg(a.d, 1, a.d // 64, a.P, B.GRPO_BF16, 0)
        weights = {"e_act": e_act}
        S = a.P + 56
    out = B.Packed(_M, a.kept)
    ms = _time(lambda: B.grpo_pack_chunks(ctx, batch, _M, kept_idx, kept_off, adv, out), a.iters)
    nbytes = a.kept * (2 * a.P + 2 * 56) * a.d * 2
    print(json.dumps({"kernel": "pack", "kept": a.kept, "P": a.P, "d": a.d, "ms": ms, "gbs": nbytes / (ms * 1e6),
                      "status": B.pcm_poll_status(ctx)}))
    ctx.close()


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="what", required=True)
    g = sub.add_parser("gemm")
    g.add_argument("--m", type=int, default=19968); g.add_argument("--n", type=int, default=3072)
    g.add_argument("--k", type=int, default=1024); g.add_argument("--layout", default="nt", choices=["nt", "nn", "tn"])
    g.add_argument("--out", default="bf16", choices=["bf16", "f32", "acc"]); g.add_argument("--backend", type=int, default=2)
    g.add_argument("--iters", type=int, default=20)
    t = sub.add_parser("attention")
    t.add_argument("--seqs", type=int, default=64); t.add_argument("--S", type=int, default=312)
    t.add_argument("--heads", type=int, default=16); t.add_argument("--dh", type=int, default=64)
    t.add_argument("--iters", type=int, default=10)
    c = sub.add_parser("pcm")
    c.add_argument("--tasks", type=int, default=8192); c.add_argument("--G", type=int, default=8)
    c.add_argument("--T", type=int, default=128); c.add_argument("--phases", type=int, default=10)
    c.add_argument("--budget", type=int, default=24); c.add_argument("--iters", type=int, default=10)
    k = sub.add_parser("pack")
    k.add_argument("--kept", type=int, default=384); k.add_argument("--P", type=int, default=256)
    k.add_argument("--d", type=int, default=1024); k.add_argument("--iters", type=int, default=10)
    a = ap.parse_args()
    {"gemm": bench_gemm, "attention": bench_attention, "pcm": bench_pcm, "pack": bench_pack}[a.what](a)


if __name__ == "__main__":
    main()
