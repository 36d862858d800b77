"""Pins for the actor-update oracle: central finite differences, library routines for the pieces,
and the invariants the paper fixes (Eq. 11 -> Eq. 2, Eq. 3, zero-signal cases)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import actor_oracle as ao
from oracle import pcm_oracle as po


def tiny_model(rng, d=16, L=2, H=2, V=256, gamma_std=0.2, scale=0.25):
    shapes = {"w_qkv": (L, 3 * d, d), "w_o": (L, d, d), "w_gu": (L, 8 * d, d), "w_d": (L, d, 4 * d),
              "g1": (L, d), "g2": (L, d), "gf": (d,), "w_h": (V, d), "e_act": (V, d)}
    W = {}
    for k, s in shapes.items():
        if k in ("g1", "g2", "gf"):
            W[k] = 1.0 + gamma_std * rng.standard_normal(s)
        else:
            W[k] = scale * rng.standard_normal(s)
    return W


def tiny_batch(rng, W, n=3, P=4, d=16):
    tgt = rng.integers(0, 256, size=(n, 56)).astype(np.uint8)
    X = np.concatenate([rng.standard_normal((n, P, d)), W["e_act"][tgt.astype(int)]], axis=1)
    adv = np.array([1.2, -0.8, 0.4])[:n]
    return X, tgt, adv


def rebuild_X(W, X, tgt, P):
    X2 = X.copy()
    X2[:, P:] = W["e_act"][tgt.astype(int)]
    return X2


@pytest.mark.parametrize("clip_active", [False, True])
def test_gradient_matches_central_finite_differences(clip_active):
    rng = np.random.default_rng(10 + clip_active)
    d, H, P = 16, 2, 4
    W = tiny_model(rng, d=d, H=H)
    X, tgt, adv = tiny_batch(rng, W, P=P, d=d)
    logp = ao.logp_only(W, X, tgt, H, P)
    sigma = 0.3 if clip_active else 0.01
    lpo = logp + sigma * rng.standard_normal(logp.shape)
    el, eh = 0.2, 0.4
    loss, _, grads, stats = ao.fwd_bwd(W, X, tgt, lpo, adv, H, P, el, eh, loss_scale=1.0)
    if clip_active:
        assert 0.1 < stats["clip_frac"] < 0.9
    else:
        assert stats["clip_frac"] == 0.0

    def f(Wp):
        return ao.loss_only(Wp, rebuild_X(Wp, X, tgt, P), tgt, lpo, adv, H, P, el, eh, 1.0)

    assert f(W) == pytest.approx(loss, rel=1e-13)
    for name in W:
        # random directions: <grad, v> against (f(W + h v) - f(W - h v)) / 2h
        for _ in range(3):
            v = rng.standard_normal(W[name].shape)
            h = 1e-6 if clip_active else 1e-5     # the clipped surrogate has kinks: stay close
            Wp = dict(W); Wp[name] = W[name] + h * v
            Wm = dict(W); Wm[name] = W[name] - h * v
            fd = (f(Wp) - f(Wm)) / (2 * h)
            an = float(np.sum(grads[name] * v))
            assert an == pytest.approx(fd, rel=(2e-5 if clip_active else 2e-6), abs=1e-8), name
        # single entries
        flat = W[name].reshape(-1)
        for idx in rng.choice(flat.size, size=min(12, flat.size), replace=False):
            h = (1e-6 if clip_active else 1e-5) * max(1.0, abs(flat[idx]))
            Wp = dict(W); a = W[name].copy(); a.reshape(-1)[idx] += h; Wp[name] = a
            Wm = dict(W); b = W[name].copy(); b.reshape(-1)[idx] -= h; Wm[name] = b
            fd = (f(Wp) - f(Wm)) / (2 * h)
            assert grads[name].reshape(-1)[idx] == pytest.approx(fd, rel=1e-5, abs=1e-8), (name, idx)


def _torch_forward(W, X, H, P):
    """The same model assembled from torch library routines in fp64."""
    Wt = {k: torch.tensor(v, dtype=torch.float64) for k, v in W.items()}
    x = torch.tensor(X, dtype=torch.float64)
    n, S, d = x.shape
    dh = d // H
    L = Wt["w_qkv"].shape[0]
    pos = torch.arange(S, dtype=torch.float64)
    inv = 10000.0 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh)
    ang = torch.outer(pos, inv)
    rot = torch.polar(torch.ones_like(ang), ang)                 # e^{i pos theta}

    def rope(t):                                                  # [n,S,H,dh] via complex multiply
        z = torch.complex(t[..., :dh // 2], t[..., dh // 2:]) * rot[None, :, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for l in range(L):
        h = F.rms_norm(x, (d,), Wt["g1"][l], eps=1e-5)
        qkv = F.linear(h, Wt["w_qkv"][l])
        q, k, v = (t.reshape(n, S, H, dh) for t in qkv.split(d, dim=-1))
        q, k = rope(q), rope(k)
        o = F.scaled_dot_product_attention(q.transpose(1, 2), k.transpose(1, 2), v.transpose(1, 2), is_causal=True)
        x = x + F.linear(o.transpose(1, 2).reshape(n, S, d), Wt["w_o"][l])
        h = F.rms_norm(x, (d,), Wt["g2"][l], eps=1e-5)
        g, u = F.linear(h, Wt["w_gu"][l]).split(4 * d, dim=-1)
        x = x + F.linear(F.silu(g) * u, Wt["w_d"][l])
    hf = F.rms_norm(x[:, P - 1:P + 55], (d,), Wt["gf"], eps=1e-5)
    return F.linear(hf, Wt["w_h"])


def test_forward_matches_library_routines():
    rng = np.random.default_rng(20)
    d, H, P = 32, 4, 7
    W = tiny_model(rng, d=d, H=H, L=3)
    X, tgt, _ = tiny_batch(rng, W, P=P, d=d)
    z, _ = ao.forward(W, X, H, P)
    zt = _torch_forward(W, X, H, P)
    assert np.allclose(z, zt.numpy(), rtol=1e-11, atol=1e-12)
    logp, prob = ao.log_softmax_at(z, tgt)
    lt = torch.log_softmax(zt, dim=-1).gather(-1, torch.tensor(tgt.astype(np.int64))[..., None])[..., 0]
    assert np.allclose(logp, lt.numpy(), rtol=1e-12, atol=1e-13)
    assert np.allclose(prob.sum(-1), 1.0, rtol=1e-13)


def test_gradient_matches_autograd_of_library_model():
    rng = np.random.default_rng(21)
    d, H, P = 32, 4, 5
    W = tiny_model(rng, d=d, H=H, L=2)
    X, tgt, adv = tiny_batch(rng, W, P=P, d=d)
    lpo = ao.logp_only(W, X, tgt, H, P) + 0.15 * rng.standard_normal((3, 56))
    loss, _, grads, _ = ao.fwd_bwd(W, X, tgt, lpo, adv, H, P, 0.2, 0.2)
    Wt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in W.items()}
    Xt = torch.tensor(X, dtype=torch.float64)
    Xt = torch.cat([Xt[:, :P], Wt["e_act"][torch.tensor(tgt.astype(np.int64))]], dim=1)

    z = _torch_forward_tracked(Wt, Xt, H, P)
    lp = torch.log_softmax(z, -1).gather(-1, torch.tensor(tgt.astype(np.int64))[..., None])[..., 0]
    r = torch.exp(lp - torch.tensor(lpo))
    A = torch.tensor(adv)[:, None]
    lt = -(torch.minimum(r * A, torch.clamp(r, 0.8, 1.2) * A)).sum() / (56 * 3)
    lt.backward()
    assert float(lt.detach()) == pytest.approx(loss, rel=1e-12)
    for k in W:
        assert np.allclose(grads[k], Wt[k].grad.numpy(), rtol=1e-8, atol=1e-12), k


def _torch_forward_tracked(Wt, x, H, P):
    n, S, d = x.shape
    dh = d // H
    L = Wt["w_qkv"].shape[0]
    ang = torch.outer(torch.arange(S, dtype=torch.float64),
                      10000.0 ** (-torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    cos, sin = torch.cos(ang)[None, :, None, :], torch.sin(ang)[None, :, None, :]

    def rope(t):
        a, b = t[..., :dh // 2], t[..., dh // 2:]
        return torch.cat([a * cos - b * sin, b * cos + a * sin], dim=-1)

    for l in range(L):
        h = F.rms_norm(x, (d,), Wt["g1"][l], eps=1e-5)
        q, k, v = (t.reshape(n, S, H, dh) for t in F.linear(h, Wt["w_qkv"][l]).split(d, dim=-1))
        o = F.scaled_dot_product_attention(rope(q).transpose(1, 2), rope(k).transpose(1, 2), v.transpose(1, 2), is_causal=True)
        x = x + F.linear(o.transpose(1, 2).reshape(n, S, d), Wt["w_o"][l])
        h = F.rms_norm(x, (d,), Wt["g2"][l], eps=1e-5)
        g, u = F.linear(h, Wt["w_gu"][l]).split(4 * d, dim=-1)
        x = x + F.linear(F.silu(g) * u, Wt["w_d"][l])
    return F.linear(F.rms_norm(x[:, P - 1:P + 55], (d,), Wt["gf"], eps=1e-5), Wt["w_h"])


def test_rope_properties():
    rng = np.random.default_rng(22)
    S, dh = 9, 8
    cos, sin = ao.rope_tables(S, dh)
    q = rng.standard_normal((1, S, 1, dh)); k = rng.standard_normal((1, S, 1, dh))
    rq, rk = ao.rope(q, cos, sin), ao.rope(k, cos, sin)
    assert np.allclose(rq[0, 0], q[0, 0])                                   # position 0 is the identity
    assert np.allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1))
    # scores depend on the position difference only: same vectors at (2,5) and (4,7)
    q2 = np.tile(q[:, :1], (1, S, 1, 1)); k2 = np.tile(k[:, :1], (1, S, 1, 1))
    a, b = ao.rope(q2, cos, sin), ao.rope(k2, cos, sin)
    assert np.dot(a[0, 5, 0], b[0, 2, 0]) == pytest.approx(np.dot(a[0, 7, 0], b[0, 4, 0]), rel=1e-12)
    g = rng.standard_normal(rq.shape)
    assert np.sum(ao.rope(q, cos, sin) * g) == pytest.approx(np.sum(q * ao.rope_bwd(g, cos, sin)), rel=1e-12)


def _setup_masked(rng):
    d, H, P, n_traj, N, Kc = 16, 2, 3, 4, 6, 3
    W = tiny_model(rng, d=d, H=H)
    total = n_traj * N
    obs = rng.standard_normal((total, P, d))
    tok = rng.integers(0, 256, size=(total, 56)).astype(np.uint8)
    phase = np.tile(np.arange(N) * Kc // N, n_traj).astype(np.uint8)
    traj_off = (np.arange(n_traj + 1) * N).astype(np.int32)
    reward = np.array([1, 0, 0, 1], dtype=np.uint8)
    adv = po.advantages(reward, 4)
    lpo_all = -5.5 + 0.2 * rng.standard_normal((total, 56))
    return dict(W=W, H=H, P=P, obs=obs, tok=tok, phase=phase, traj_off=traj_off, adv=adv, lpo=lpo_all, total=total, Kc=Kc)


def _grad_for(s, kept, loss_scale):
    X, tgt, lpo, adv_c, _ = po.pack_chunks(lambda c: s["obs"][c], s["tok"], s["lpo"], s["adv"], s["traj_off"],
                                           np.asarray(kept, dtype=np.int32), s["W"]["e_act"])
    return ao.fwd_bwd(s["W"], X, tgt, lpo, adv_c, s["H"], s["P"], 0.2, 0.2, loss_scale)


def test_mask_all_equals_full_grpo_and_phase_decomposition():
    s = _setup_masked(np.random.default_rng(23))
    scale = 1.0 / 4
    all_idx = np.arange(s["total"])
    # sampler with budget >= N_i keeps every chunk: the masked update is the full update (Eq. 11 -> Eq. 2)
    kept, off, _ = po.sample_chunks(s["traj_off"], s["phase"], [1 << 24] * 3, 99, seed=1, it=0)
    assert np.array_equal(kept, all_idx)
    loss_full, _, g_full, _ = _grad_for(s, all_idx, scale)
    # Eq. 3: the gradient decomposes by phase
    acc = {k: np.zeros_like(v) for k, v in g_full.items()}
    loss_sum = 0.0
    for c in range(s["Kc"]):
        l_c, _, g_c, _ = _grad_for(s, all_idx[s["phase"] == c], scale)
        loss_sum += l_c
        for k in acc:
            acc[k] += g_c[k]
    assert loss_sum == pytest.approx(loss_full, rel=1e-12)
    for k in acc:
        assert np.allclose(acc[k], g_full[k], rtol=1e-9, atol=1e-14), k
    # chunks are independent sequences: permuting the packed order changes nothing
    perm = np.random.default_rng(1).permutation(s["total"])
    loss_p, _, g_p, _ = _grad_for(s, all_idx[perm], scale)
    assert loss_p == pytest.approx(loss_full, rel=1e-12)
    for k in acc:
        assert np.allclose(g_p[k], g_full[k], rtol=1e-9, atol=1e-14), k


def test_unclipped_on_policy_loss_is_eq11_and_zero_signal_cases():
    s = _setup_masked(np.random.default_rng(24))
    kept = np.array([0, 2, 7, 13, 20], dtype=np.int32)
    X, tgt, _, adv_c, _ = po.pack_chunks(lambda c: s["obs"][c], s["tok"], s["lpo"], s["adv"], s["traj_off"], kept, s["W"]["e_act"])
    logp = ao.logp_only(s["W"], X, tgt, s["H"], s["P"])
    # with logp_old = logp the ratio is 1 and the gradient equals that of -scale * sum A log pi (Eq. 11)
    loss, _, g, st = ao.fwd_bwd(s["W"], X, tgt, logp, adv_c, s["H"], s["P"], 0.2, 0.2, 1.0)
    assert st["clip_frac"] == 0.0 and loss == pytest.approx(-np.sum(adv_c) * 56, rel=1e-12)
    h = 1e-5
    v = np.random.default_rng(2).standard_normal(s["W"]["w_h"].shape)
    def eq11(Wp):
        return -np.sum(adv_c[:, None] * ao.logp_only(Wp, X, tgt, s["H"], s["P"]))
    Wp = dict(s["W"]); Wp["w_h"] = s["W"]["w_h"] + h * v
    Wm = dict(s["W"]); Wm["w_h"] = s["W"]["w_h"] - h * v
    assert np.sum(g["w_h"] * v) == pytest.approx((eq11(Wp) - eq11(Wm)) / (2 * h), rel=1e-6)
    # a group with uniform rewards has zero advantages, hence exactly zero gradient
    _, _, g0, _ = ao.fwd_bwd(s["W"], X, tgt, logp, np.zeros(len(kept)), s["H"], s["P"], 0.2, 0.2, 1.0)
    assert all(np.all(v == 0.0) for v in g0.values())


# ---- entropy bonus and chunk-level ratio (App. E; Eq. 2 / Eq. 11 written per chunk) -----------------
@pytest.mark.parametrize("ratio_level,sigma", [("token", 0.01), ("token", 0.3), ("chunk", 0.001), ("chunk", 0.04)])
def test_entropy_and_chunk_ratio_gradient_matches_finite_differences(ratio_level, sigma):
    rng = np.random.default_rng(40)
    d, H, P = 16, 2, 4
    W = tiny_model(rng, d=d, H=H)
    X, tgt, adv = tiny_batch(rng, W, P=P, d=d)
    lpo = ao.logp_only(W, X, tgt, H, P) + sigma * rng.standard_normal((3, 56))
    el, eh, coef = 0.2, 0.4, 0.05
    loss, _, grads, stats = ao.fwd_bwd(W, X, tgt, lpo, adv, H, P, el, eh, loss_scale=1.0, entropy_coef=coef,
                                        ratio_level=ratio_level)
    if sigma in (0.3, 0.04):
        assert 0.0 < stats["clip_frac"] < 1.0
    else:
        assert stats["clip_frac"] == 0.0

    def f(Wp):
        return ao.loss_only(Wp, rebuild_X(Wp, X, tgt, P), tgt, lpo, adv, H, P, el, eh, 1.0, coef, ratio_level)

    assert f(W) == pytest.approx(loss, rel=1e-13)
    for name in W:
        for _ in range(3):
            v = rng.standard_normal(W[name].shape)
            h = 1e-6
            Wp = dict(W); Wp[name] = W[name] + h * v
            Wm = dict(W); Wm[name] = W[name] - h * v
            fd = (f(Wp) - f(Wm)) / (2 * h)
            assert float(np.sum(grads[name] * v)) == pytest.approx(fd, rel=3e-5, abs=1e-7), name


def test_entropy_bonus_alone_matches_finite_differences_and_autograd():
    """A = 0 leaves only the entropy term: gradient against autograd of -coef * mean H from library ops."""
    rng = np.random.default_rng(41)
    d, H, P = 32, 4, 5
    W = tiny_model(rng, d=d, H=H, L=2)
    X, tgt, _ = tiny_batch(rng, W, P=P, d=d)
    lpo = ao.logp_only(W, X, tgt, H, P)
    coef = 0.7
    loss, _, grads, stats = ao.fwd_bwd(W, X, tgt, lpo, np.zeros(3), H, P, 0.2, 0.4, entropy_coef=coef)
    Wt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in W.items()}
    Xt = torch.tensor(X, dtype=torch.float64)
    Xt = torch.cat([Xt[:, :P], Wt["e_act"][torch.tensor(tgt.astype(np.int64))]], dim=1)
    z = _torch_forward_tracked(Wt, Xt, H, P)
    ent = torch.distributions.Categorical(logits=z).entropy()
    lt = -coef * ent.mean()
    lt.backward()
    assert float(lt.detach()) == pytest.approx(loss, rel=1e-12)
    assert stats["entropy"] == pytest.approx(float(ent.mean().detach()), rel=1e-12)
    for k in W:
        assert np.allclose(grads[k], Wt[k].grad.numpy(), rtol=1e-8, atol=1e-13), k


def test_full_paper_loss_matches_autograd_of_library_model():
    """Asymmetric clip (0.2, 0.4) + entropy coefficient 1e-3, token-level and chunk-level ratios."""
    rng = np.random.default_rng(42)
    d, H, P = 32, 4, 5
    W = tiny_model(rng, d=d, H=H, L=2)
    X, tgt, adv = tiny_batch(rng, W, P=P, d=d)
    base = ao.logp_only(W, X, tgt, H, P)
    for level, sigma in (("token", 0.25), ("chunk", 0.04)):
        lpo = base + sigma * rng.standard_normal((3, 56))
        loss, _, grads, stats = ao.fwd_bwd(W, X, tgt, lpo, adv, H, P, 0.2, 0.4, entropy_coef=1e-3, ratio_level=level)
        Wt = {k: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k, v in W.items()}
        Xt = torch.tensor(X, dtype=torch.float64)
        Xt = torch.cat([Xt[:, :P], Wt["e_act"][torch.tensor(tgt.astype(np.int64))]], dim=1)
        z = _torch_forward_tracked(Wt, Xt, H, P)
        lsm = torch.log_softmax(z, -1)
        lp = lsm.gather(-1, torch.tensor(tgt.astype(np.int64))[..., None])[..., 0]
        if level == "token":
            r = torch.exp(lp - torch.tensor(lpo)); A = torch.tensor(adv)[:, None]; denom = 56 * 3
        else:
            r = torch.exp(lp.sum(-1) - torch.tensor(lpo).sum(-1)); A = torch.tensor(adv); denom = 3
        pg = -(torch.minimum(r * A, torch.clamp(r, 0.8, 1.4) * A)).sum() / denom
        lt = pg - 1e-3 * (-(lsm.exp() * lsm).sum(-1)).mean()
        lt.backward()
        assert float(lt.detach()) == pytest.approx(loss, rel=1e-12)
        for k in W:
            assert np.allclose(grads[k], Wt[k].grad.numpy(), rtol=1e-8, atol=1e-12), (level, k)


def test_zero_head_gives_uniform_policy_entropy_log256_and_no_entropy_gradient():
    rng = np.random.default_rng(43)
    W = tiny_model(rng)
    W["w_h"] = np.zeros_like(W["w_h"])
    X, tgt, adv = tiny_batch(rng, W)
    lpo = np.full((3, 56), -np.log(256.0))
    loss, logp, grads, stats = ao.fwd_bwd(W, X, tgt, lpo, np.zeros(3), 2, 4, entropy_coef=0.5)
    assert stats["entropy"] == pytest.approx(np.log(256.0), rel=1e-14)
    assert loss == pytest.approx(-0.5 * np.log(256.0), rel=1e-14)
    assert np.allclose(logp, -np.log(256.0))
    assert all(np.abs(g).max() < 1e-15 for g in grads.values())          # the uniform policy maximises H


def test_chunk_level_ratio_on_policy_identity_and_joint_clipping():
    rng = np.random.default_rng(44)
    W = tiny_model(rng)
    X, tgt, adv = tiny_batch(rng, W)
    base = ao.logp_only(W, X, tgt, 2, 4)
    # on-policy: every ratio is 1, both forms give -scale * A * grad(sum of log-probs)
    _, _, g_tok, _ = ao.fwd_bwd(W, X, tgt, base, adv, 2, 4, loss_scale=0.01)
    _, _, g_chk, st = ao.fwd_bwd(W, X, tgt, base, adv, 2, 4, loss_scale=0.01, ratio_level="chunk")
    assert st["mean_ratio"] == pytest.approx(1.0, abs=1e-12)
    for k in W:
        assert np.allclose(g_tok[k], g_chk[k], rtol=1e-9, atol=1e-14), k
    # every token ratio e^0.01 is inside the clip range, the joint ratio e^0.56 is not
    lpo = base - 0.01
    _, _, _, st_tok = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, 0.2, 0.4)
    loss, _, g, st_chk = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, 0.2, 0.4, ratio_level="chunk")
    assert st_tok["clip_frac"] == 0.0
    assert st_chk["mean_ratio"] == pytest.approx(np.exp(0.56), rel=1e-12)
    assert st_chk["clip_frac"] == pytest.approx(2 / 3)                     # the two chunks with A > 0
    assert loss == pytest.approx(-(1.4 * 1.2 + np.exp(0.56) * -0.8 + 1.4 * 0.4) / 3, rel=1e-12)
    # only the A < 0 chunk (index 1) still carries gradient: compare with that chunk alone
    _, _, g1, _ = ao.fwd_bwd(W, X[1:2], tgt[1:2], lpo[1:2], adv[1:2], 2, 4, 0.2, 0.4, loss_scale=1 / 3, ratio_level="chunk")
    for k in W:
        assert np.allclose(g[k], g1[k], rtol=1e-9, atol=1e-14), k


# ------------------------------------------------------------------ LoRA (App. E: r = 32, alpha = 32)
def tiny_lora(rng, W, rank=4, alpha=6.0, b_scale=0.2):
    L, d = W["g1"].shape
    dims = {"qkv": (d, 3 * d), "o": (d, d), "gu": (d, 8 * d), "d": (4 * d, d)}
    lo = {"rank": rank, "alpha": alpha}
    for name, (fin, fout) in dims.items():
        lo["a_" + name] = 0.3 * rng.standard_normal((L, rank, fin))
        lo["b_" + name] = b_scale * rng.standard_normal((L, fout, rank))
    return lo


def merged_weights(W, lo):
    s = lo["alpha"] / lo["rank"]
    Wm = dict(W)
    for name in ao.LORA_PROJ:
        Wm["w_" + name] = W["w_" + name] + s * np.einsum("lor,lri->loi", lo["b_" + name], lo["a_" + name])
    return Wm


def test_lora_with_zero_b_is_the_dense_model():
    rng = np.random.default_rng(41)
    W = tiny_model(rng)
    X, tgt, adv = tiny_batch(rng, W)
    lo = tiny_lora(rng, W, b_scale=0.0)
    z0, _ = ao.forward(W, X, 2, 4)
    z1, _ = ao.forward(W, X, 2, 4, lora=lo)
    assert np.array_equal(z0, z1)
    # B = 0: no signal reaches A, and dB is what the dense weight gradient projects onto A
    lpo = ao.logp_only(W, X, tgt, 2, 4) + 0.01 * rng.standard_normal((3, 56))
    _, _, g_dense, _ = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, loss_scale=1.0)
    _, _, g, _ = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, loss_scale=1.0, lora=lo)
    s = lo["alpha"] / lo["rank"]
    for name in ao.LORA_PROJ:
        assert g["w_" + name] is None
        assert np.all(g["a_" + name] == 0.0)
        expect = s * np.einsum("loi,lri->lor", g_dense["w_" + name], lo["a_" + name])
        assert np.allclose(g["b_" + name], expect, rtol=1e-11, atol=1e-13)


def test_lora_equals_the_merged_dense_model_and_its_chain_rule():
    rng = np.random.default_rng(42)
    W = tiny_model(rng)
    X, tgt, adv = tiny_batch(rng, W)
    lo = tiny_lora(rng, W)
    Wm = merged_weights(W, lo)
    z_l, _ = ao.forward(W, X, 2, 4, lora=lo)
    z_m, _ = ao.forward(Wm, X, 2, 4)
    assert np.allclose(z_l, z_m, rtol=1e-11, atol=1e-12)
    assert not np.allclose(z_l, ao.forward(W, X, 2, 4)[0], atol=1e-3)          # the adapters do change the policy
    lpo = ao.logp_only(Wm, X, tgt, 2, 4) + 0.2 * rng.standard_normal((3, 56))
    loss_m, _, g_m, st_m = ao.fwd_bwd(Wm, X, tgt, lpo, adv, 2, 4, 0.2, 0.4, loss_scale=1.0, entropy_coef=1e-3)
    loss_l, _, g_l, st_l = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, 0.2, 0.4, loss_scale=1.0, entropy_coef=1e-3, lora=lo)
    assert loss_l == pytest.approx(loss_m, rel=1e-12)
    assert 0.0 < st_l["clip_frac"] == pytest.approx(st_m["clip_frac"])
    s = lo["alpha"] / lo["rank"]
    for name in ao.LORA_PROJ:
        dW = g_m["w_" + name]                                                   # W_eff = W + s B A
        assert np.allclose(g_l["a_" + name], s * np.einsum("lor,loi->lri", lo["b_" + name], dW), rtol=1e-10, atol=1e-12)
        assert np.allclose(g_l["b_" + name], s * np.einsum("loi,lri->lor", dW, lo["a_" + name]), rtol=1e-10, atol=1e-12)
    for name in ("g1", "g2", "gf", "w_h", "e_act"):                             # the rest sees the same function
        assert np.allclose(g_l[name], g_m[name], rtol=1e-10, atol=1e-12), name


def test_lora_gradient_matches_central_finite_differences():
    rng = np.random.default_rng(43)
    W = tiny_model(rng)
    X, tgt, adv = tiny_batch(rng, W)
    lo = tiny_lora(rng, W)
    lpo = ao.logp_only(W, X, tgt, 2, 4, lora=lo) + 0.01 * rng.standard_normal((3, 56))
    loss, _, g, _ = ao.fwd_bwd(W, X, tgt, lpo, adv, 2, 4, 0.2, 0.4, loss_scale=1.0, lora=lo)

    def f(lp):
        return ao.loss_only(W, X, tgt, lpo, adv, 2, 4, 0.2, 0.4, 1.0, lora=lp)

    assert f(lo) == pytest.approx(loss, rel=1e-13)
    for name in ao.LORA_PROJ:
        for key in ("a_" + name, "b_" + name):
            v = rng.standard_normal(lo[key].shape)
            h = 1e-5
            lp = dict(lo); lp[key] = lo[key] + h * v
            lm = dict(lo); lm[key] = lo[key] - h * v
            fd = (f(lp) - f(lm)) / (2 * h)
            assert float(np.sum(g[key] * v)) == pytest.approx(fd, rel=2e-6, abs=1e-9), key
            flat = lo[key].reshape(-1)
            for idx in rng.choice(flat.size, size=6, replace=False):
                lp = dict(lo); a = lo[key].copy(); a.reshape(-1)[idx] += h; lp[key] = a
                lm = dict(lo); b = lo[key].copy(); b.reshape(-1)[idx] -= h; lm[key] = b
                fd = (f(lp) - f(lm)) / (2 * h)
                assert g[key].reshape(-1)[idx] == pytest.approx(fd, rel=1e-5, abs=1e-9), (key, idx)
