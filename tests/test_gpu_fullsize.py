"""Parity at the full size of the medium workload (C1), in the launch configuration bench.py times
(whole batch of 384 kept chunks in one micro-batch): selection and packed rows bit-exact against the
oracle, sampled outputs the oracle can compute one by one, and properties that hold at any size."""
import numpy as np
import pytest
import torch

from oracle import actor_oracle as ao
from oracle import pcm_oracle as po
from paper_2605_16154_b200 import synth
from tests.gpu_helpers import grads_to_numpy, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def c1():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    w = synth.WORKLOADS["C1"]
    rb = synth.make_rollouts(w)
    weights = synth.make_weights(w)
    total = int(rb["traj_off"][-1])
    obs = synth.obs_all(w, w.seed, total)
    lpo_all = (-np.log(256.0) + synth.logp_noise(w.seed, total, 0.3)).astype(np.float32)
    model = PL.upload_model(w, weights)
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=5, max_traj=w.n_traj)
    batch = PL.upload_rollouts(w, rb, obs=PL.dev(obs, torch.bfloat16), logp_old=PL.dev(lpo_all))
    adv, Cc, valid, p, q, kept_idx, kept_off, per_phase = PL.select(ctx, batch, 0)
    n_kept = PL.n_kept_of(w.budget, rb["traj_off"])
    pk = B.grpo_pack_chunks(ctx, batch, model, kept_idx, kept_off, adv, B.Packed(model, n_kept))
    assert B.pcm_poll_status(ctx) == 0
    return dict(B=B, PL=PL, w=w, rb=rb, weights=weights, obs=obs, lpo_all=lpo_all, model=model, ctx=ctx, batch=batch,
                adv=adv, q=q, kept_idx=kept_idx, kept_off=kept_off, pk=pk, n_kept=n_kept)


def test_selection_and_pack_bit_exact_at_full_size(c1):
    w, rb = c1["w"], c1["rb"]
    C_o, valid_o, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    _, q_o, _ = po.update_keep_probs(po.KeepProbState(w.n_phases, w.p_min, w.t_rc), C_o, valid_o)
    kept_o, off_o, _ = po.sample_chunks(rb["traj_off"], rb["phase"], q_o, w.budget, 5, 0)
    assert c1["n_kept"] == 384 == len(kept_o)
    assert np.array_equal(c1["kept_idx"].cpu().numpy()[:384], kept_o)
    assert np.array_equal(c1["kept_off"].cpu().numpy(), off_o)
    pk = c1["pk"]
    X = pk.X.float().cpu().numpy()
    e_act = c1["weights"]["e_act"]
    for j in (0, 57, 200, 383):                                   # sampled packed rows against their sources
        c = int(kept_o[j])
        assert np.array_equal(X[j, :w.P], c1["obs"][c])
        assert np.array_equal(X[j, w.P:], e_act[rb["tok"][c].astype(int)])
        assert np.array_equal(pk.tgt[j].cpu().numpy(), rb["tok"][c])
        assert np.array_equal(pk.lpo[j].cpu().numpy(), c1["lpo_all"][c])
    adv_o = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
    owner = np.searchsorted(rb["traj_off"], kept_o, side="right") - 1
    assert np.array_equal(pk.adv_c.cpu().numpy(), adv_o[owner])


def test_sampled_log_probs_and_batch_properties_at_full_size(c1):
    B, w, model, pk = c1["B"], c1["w"], c1["model"], c1["pk"]
    loss, logp, grads, stats = B.grpo_actor_fwd_bwd(model, pk, mb_chunks=384)
    g_full = {k: v.clone() for k, v in grads.items()}
    loss_full = float(loss.item())
    assert np.isfinite(loss_full) and stats.n_launches > 0
    # sampled chunks: the oracle's forward pass on one chunk at a time
    X = pk.X.float().cpu().numpy()
    tgt = pk.tgt.cpu().numpy()
    for j in (3, 311):
        lp_o = ao.logp_only(c1["weights"], X[j:j + 1], tgt[j:j + 1], w.H, w.P)
        assert np.max(np.abs(logp[j].cpu().numpy() - lp_o[0])) < 0.04
    # micro-batching changes only the fp32 accumulation order
    loss_mb, logp_mb, grads_mb, _ = B.grpo_actor_fwd_bwd(model, pk, mb_chunks=100)
    assert torch.equal(logp_mb, logp)
    assert abs(float(loss_mb.item()) - loss_full) < 1e-6
    for k in g_full:
        assert rel_fro(grads_mb[k].cpu().numpy(), g_full[k].cpu().numpy()) < 2e-3, k
    # the masked objective is a sum over kept chunks: two halves with the same scale add up to the whole
    scale = 1.0 / (56 * 384)
    halves = {k: torch.zeros_like(v) for k, v in g_full.items()}
    loss_sum = 0.0
    for lo, hi in ((0, 192), (192, 384)):
        sub = B.Packed(model, hi - lo)
        sub.X.copy_(pk.X[lo:hi]); sub.tgt.copy_(pk.tgt[lo:hi]); sub.lpo.copy_(pk.lpo[lo:hi])
        sub.adv_c.copy_(pk.adv_c[lo:hi]); sub.src.copy_(pk.src[lo:hi])
        l, _, g, _ = B.grpo_actor_fwd_bwd(model, sub, loss_scale=scale, mb_chunks=192)
        loss_sum += float(l.item())
        for k in halves:
            halves[k] += g[k]
    assert abs(loss_sum - loss_full) < 1e-6
    for k in g_full:
        assert rel_fro(halves[k].cpu().numpy(), g_full[k].cpu().numpy()) < 2e-3, k


def test_eight_chunk_update_of_the_full_model_against_the_oracle(c1):
    """Every kernel at the medium model's real width, depth and sequence length (8 layers, d = 1024,
    S = 312), on a batch small enough for the fp64 oracle."""
    B, PL, w, model, pk = c1["B"], c1["PL"], c1["w"], c1["model"], c1["pk"]
    sel = [5, 60, 111, 170, 250, 300, 340, 380]
    X = pk.X[sel].float().cpu().numpy()
    tgt = pk.tgt[sel].cpu().numpy()
    adv_c = np.array([1.0, -1.0] * 4, dtype=np.float32)           # zero-mean like a rollout group's advantages
    lp_o = ao.logp_only(c1["weights"], X, tgt, w.H, w.P)
    noise = synth.logp_noise(11, len(sel), 0.1).astype(np.float64)
    hi, lo, m = np.log(1.2), np.log(0.8), 0.05
    log_r = -noise
    log_r = np.where(np.abs(log_r - hi) < m, hi + 2 * m * np.sign(log_r - hi + 1e-30), log_r)
    log_r = np.where(np.abs(log_r - lo) < m, lo + 2 * m * np.sign(log_r - lo + 1e-30), log_r)
    lpo = (lp_o - log_r).astype(np.float32)
    loss_o, _, grads_o, stats_o = ao.fwd_bwd(c1["weights"], X, tgt, lpo, adv_c, w.H, w.P, 0.2, 0.2)
    sub = B.Packed(model, len(sel))
    sub.X.copy_(pk.X[sel]); sub.tgt.copy_(pk.tgt[sel]); sub.lpo.copy_(PL.dev(lpo)); sub.adv_c.copy_(PL.dev(adv_c))
    loss, logp, grads, stats = B.grpo_actor_fwd_bwd(model, sub)
    errs = {k: rel_fro(v, grads_o[k]) for k, v in grads_to_numpy(grads).items()}
    assert max(errs.values()) < 2e-2, (errs, float(loss.item()), loss_o)
    assert abs(float(loss.item()) - loss_o) < 1e-3
    assert stats.clip_frac == pytest.approx(stats_o["clip_frac"], abs=1e-6)


def test_full_batch_backward_against_the_oracle_through_zero_advantage_chunks(c1):
    """The 384-chunk update in one micro-batch (every GEMM, attention and norm launch at the shape bench.py
    times) against the fp64 oracle.  Eight chunks spread over the batch, one of them in the last row tile,
    keep their own advantage; the other 376 get A = 0.  A zero advantage gives an exactly zero surrogate term and
    an exactly zero gradient (Eq. 1, Eq. 11), so the expected loss and gradients are the oracle's on the
    eight chunks alone under the full batch's scale 1 / (56 * 384)."""
    B, PL, w, model, pk = c1["B"], c1["PL"], c1["w"], c1["model"], c1["pk"]
    sel = [0, 47, 101, 190, 255, 256, 340, 383]
    X = pk.X[sel].float().cpu().numpy()
    tgt = pk.tgt[sel].cpu().numpy()
    adv8 = pk.adv_c[sel].cpu().numpy().astype(np.float32)          # Eq. 1 advantages of the chunks' own trajectories
    assert adv8.min() < 0.0 < adv8.max()                             # both outcomes among the eight
    lp_o = ao.logp_only(c1["weights"], X, tgt, w.H, w.P)
    noise = synth.logp_noise(13, len(sel), 0.1).astype(np.float64)
    hi, lo, m = np.log(1.2), np.log(0.8), 0.05
    log_r = -noise
    log_r = np.where(np.abs(log_r - hi) < m, hi + 2 * m * np.sign(log_r - hi + 1e-30), log_r)
    log_r = np.where(np.abs(log_r - lo) < m, lo + 2 * m * np.sign(log_r - lo + 1e-30), log_r)
    lpo8 = (lp_o - log_r).astype(np.float32)
    scale = 1.0 / (56 * 384)
    loss_o, _, grads_o, _ = ao.fwd_bwd(c1["weights"], X, tgt, lpo8, adv8, w.H, w.P, 0.2, 0.2, scale)
    full = B.Packed(model, 384)
    full.X.copy_(pk.X); full.tgt.copy_(pk.tgt); full.lpo.copy_(pk.lpo); full.src.copy_(pk.src)
    adv_c = np.zeros(384, dtype=np.float32)
    adv_c[sel] = adv8
    full.adv_c.copy_(PL.dev(adv_c))
    full.lpo[sel] = PL.dev(lpo8)
    loss, logp, grads, stats = B.grpo_actor_fwd_bwd(model, full, mb_chunks=384)
    assert abs(float(loss.item()) - loss_o) < 1e-3
    assert np.max(np.abs(logp[sel].cpu().numpy() - lp_o)) < 0.04
    errs = {k: rel_fro(v, grads_o[k]) for k, v in grads_to_numpy(grads).items()}
    assert max(errs.values()) < 2e-2, errs


def test_attention_at_the_full_batch_shape_on_sampled_sequences_and_heads():
    """grpo_attention on the shape one C1 layer runs (384 sequences of 312 tokens, 16 heads of 64: every CTA of the
    persistent kernels walks about 40 items); forward and backward checked against the oracle on sampled
    (sequence, head) pairs, which are independent problems."""
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    n_seq, S, H, dh = 384, 312, 16, 64
    d = H * dh
    g = torch.Generator(device="cuda").manual_seed(3)
    qkv = torch.randn((n_seq * S, 3 * d), generator=g, device="cuda").to(torch.bfloat16)
    do = torch.randn((n_seq * S, d), generator=g, device="cuda").to(torch.bfloat16)
    out, lse, dqkv = B.grpo_attention(qkv, n_seq, S, H, dh, dout=do)
    rng = np.random.default_rng(0)
    picks = [(0, 0), (n_seq - 1, H - 1), (147, 5), (148, 6)] + [(int(rng.integers(n_seq)), int(rng.integers(H))) for _ in range(8)]
    for s_i, h_i in picks:
        rows = slice(s_i * S, (s_i + 1) * S)
        cols = lambda part: slice(part * d + h_i * dh, part * d + (h_i + 1) * dh)
        blk = qkv[rows].float().cpu().numpy().astype(np.float64)
        q, k, v = (blk[:, cols(i)][None, None] for i in range(3))
        o, p = ao.causal_attention(q, k, v)
        go = do[rows, h_i * dh:(h_i + 1) * dh].float().cpu().numpy().astype(np.float64)[None, None]
        dq, dk, dv = ao.causal_attention_bwd(go, q, k, v, p)
        got = dqkv[rows].float().cpu().numpy()
        assert rel_fro(out[rows, h_i * dh:(h_i + 1) * dh].float().cpu().numpy(), o[0, 0]) < 1e-2, (s_i, h_i)
        assert rel_fro(got[:, cols(0)], dq[0, 0]) < 2e-2, (s_i, h_i)
        assert rel_fro(got[:, cols(1)], dk[0, 0]) < 2e-2, (s_i, h_i)
        assert rel_fro(got[:, cols(2)], dv[0, 0]) < 2e-2, (s_i, h_i)
        lse_o = np.log(np.exp(q[0, 0] @ k[0, 0].T / np.sqrt(dh) + np.triu(np.full((S, S), -np.inf), 1)).sum(-1))
        assert np.max(np.abs(lse[s_i, h_i].cpu().numpy() - lse_o)) < 2e-2, (s_i, h_i)


def test_attention_backward_repeats_bit_identically_over_many_items_per_cta():
    """The one-pass backward keeps a dozen roles in step through barriers whose phases come around every other item;
    a mis-counted phase shows up as a bounded wait that expires or as a tile taken too early.  Sizes from 2 to 40 items
    per CTA, each run several times: every run must end without a device timeout and give the same bits (no atomics:
    the order of every accumulation is fixed), and one run is checked against the oracle on sampled (sequence, head)s."""
    from paper_2605_16154_b200 import binding as B
    S, H, dh = 312, 16, 64
    d = H * dh
    for n_seq in (19, 74, 150):
        g = torch.Generator(device="cuda").manual_seed(n_seq)
        qkv = torch.randn((n_seq * S, 3 * d), generator=g, device="cuda").to(torch.bfloat16)
        do = torch.randn((n_seq * S, d), generator=g, device="cuda").to(torch.bfloat16)
        first = None
        for rep in range(8):
            _, _, dqkv = B.grpo_attention(qkv, n_seq, S, H, dh, dout=do)
            if first is None:
                first = dqkv.clone()
            else:
                assert torch.equal(dqkv, first), (n_seq, rep)
        assert B.grpo_attention_wait_status() == 0
        for s_i, h_i in ((0, 0), (n_seq - 1, H - 1), (n_seq // 2, 7)):
            rows = slice(s_i * S, (s_i + 1) * S)
            cols = lambda part: slice(part * d + h_i * dh, part * d + (h_i + 1) * dh)
            blk = qkv[rows].float().cpu().numpy().astype(np.float64)
            q, k, v = (blk[:, cols(i)][None, None] for i in range(3))
            _, p = ao.causal_attention(q, k, v)
            go = do[rows, h_i * dh:(h_i + 1) * dh].float().cpu().numpy().astype(np.float64)[None, None]
            dq, dk, dv = ao.causal_attention_bwd(go, q, k, v, p)
            got = first[rows].float().cpu().numpy()
            for part, ref in enumerate((dq, dk, dv)):
                assert rel_fro(got[:, cols(part)], ref[0, 0]) < 2e-2, (n_seq, s_i, h_i, part)


def test_two_launch_attention_backward_stays_correct_at_head_dim_64():
    """PCM_ATTN_BWD=2 (read once per process, hence a child process) keeps head dim 64 on the dQ / dK-dV launches, which
    are also the head-dim-128 path: the same attention case as the parity tests, against the oracle."""
    import os
    import subprocess
    import sys
    code = r'''
import numpy as np, torch
from oracle import actor_oracle as ao
from paper_2605_16154_b200 import binding as B
n_seq, S, H, dh = 5, 312, 3, 64
d = H * dh
rng = np.random.default_rng(5)
qkv = torch.from_numpy(rng.standard_normal((n_seq * S, 3 * d)).astype(np.float32)).cuda().to(torch.bfloat16)
do = torch.from_numpy(rng.standard_normal((n_seq * S, d)).astype(np.float32)).cuda().to(torch.bfloat16)
out, lse, dqkv = B.grpo_attention(qkv, n_seq, S, H, dh, dout=do)
heads = lambda x: x.float().cpu().numpy().astype(np.float64).reshape(n_seq, S, H, dh).transpose(0, 2, 1, 3)
q, k, v = heads(qkv[:, :d]), heads(qkv[:, d:2 * d]), heads(qkv[:, 2 * d:])
o, p = ao.causal_attention(q, k, v)
ref = ao.causal_attention_bwd(heads(do), q, k, v, p)
back = lambda x: x.transpose(0, 2, 1, 3).reshape(n_seq * S, d)
got = dqkv.float().cpu().numpy()
err = max(np.linalg.norm(got[:, i * d:(i + 1) * d] - back(ref[i])) / np.linalg.norm(back(ref[i])) for i in range(3))
assert err < 2e-2, err
print("two-launch ok", err)
'''
    env = dict(os.environ, PCM_ATTN_BWD="2")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    res = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stdout + res.stderr
    assert "two-launch ok" in res.stdout
