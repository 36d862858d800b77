"""CPU oracle for the actor update: decoder-only policy forward, masked GRPO loss (Eq. 11 with the
PPO clip the paper's implementation uses, App. E) and its exact reverse-mode gradient, in fp64.

TEST INFRASTRUCTURE ONLY.  Plain numpy written from the definitions; it shares no code with the CUDA
path and must never be imported by it.  Only the tests, the smoke check and the benchmark's
CPU-baseline leg may call it.

Parity status: the gradient is pinned by central finite differences of `loss_only` on a 2-layer d=16
model; the pieces are pinned by textbook definitions (softmax attention as a double loop, RMSNorm,
single-row log-softmax); Eq. 11 -> Eq. 2 (mask keeps every chunk), the per-phase decomposition Eq. 3,
and the zero-gradient cases are checked as invariants.  The entropy bonus and the chunk-level ratio are
pinned by finite differences, by autograd of a library model, by H = log 256 for a zero head, and by the
on-policy identity (chunk-level and token-level gradients coincide at r = 1 for equal scales).

LoRA (App. E "Training": rank r = 32, alpha = 32): with `lora` given, every linear layer of the decoder computes
y = x W^T + (alpha / r) (x A^T) B^T with the base weight W frozen; the low-rank branch is evaluated as written
(never merged into W) and gradients go to A and B, the norm gains, the head and the action embedding.  Pinned by
finite differences over A and B, by B = 0 giving the dense model's logits, and by the merged-weight identity
(logits equal those of W + (alpha / r) B A; dA, dB equal the chain rule through the dense model's dW).

Model (every kept chunk is its own sequence of S = P + 56 tokens): pre-norm decoder, RMSNorm,
rotary position embedding on q and k (base 10000, pairs (i, i + dh/2)), causal softmax attention
scaled by 1/sqrt(dh), SwiGLU MLP with hidden width 4d, final RMSNorm, linear head over 256 bins.
Position P-1+j predicts action token j.  Every linear weight is stored [out, in]: y = x @ W.T.
"""
from __future__ import annotations

from typing import Dict, Tuple

import numpy as np

ACT_DIM = 56
RMS_EPS = 1e-5
ROPE_BASE = 10000.0


def _f64(a):
    return np.asarray(a, dtype=np.float64)


def rmsnorm(x, gamma):
    """y = x * rsqrt(mean(x^2) + eps) * gamma over the last axis."""
    rstd = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + RMS_EPS)
    return x * rstd * gamma, rstd


def rmsnorm_bwd(dy, x, rstd, gamma):
    n = x * rstd
    dn = dy * gamma
    dgamma = np.sum((dy * n).reshape(-1, x.shape[-1]), axis=0)
    dx = rstd * (dn - n * np.mean(dn * n, axis=-1, keepdims=True))
    return dx, dgamma


def rope_tables(S: int, dh: int) -> Tuple[np.ndarray, np.ndarray]:
    half = dh // 2
    inv_freq = ROPE_BASE ** (-(np.arange(half, dtype=np.float64) * 2.0) / dh)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def rope(x, cos, sin):
    """x [n, S, H, dh]; rotates pair (i, i + dh/2) by angle pos * base^(-2i/dh)."""
    half = x.shape[-1] // 2
    x1, x2 = x[..., :half], x[..., half:]
    c, s = cos[None, :, None, :], sin[None, :, None, :]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def rope_bwd(dy, cos, sin):
    """Transpose of the rotation = rotation by the negative angle."""
    half = dy.shape[-1] // 2
    d1, d2 = dy[..., :half], dy[..., half:]
    c, s = cos[None, :, None, :], sin[None, :, None, :]
    return np.concatenate([d1 * c + d2 * s, d2 * c - d1 * s], axis=-1)


def silu(x):
    return x / (1.0 + np.exp(-x))


def causal_attention(q, k, v):
    """softmax(q k^T / sqrt(dh) + causal mask) v for q, k, v of shape [n, H, S, dh]; returns (o, p)."""
    S, dh = q.shape[-2], q.shape[-1]
    causal = np.triu(np.ones((S, S), dtype=bool), k=1)       # True where key position > query position
    s = (q @ k.transpose(0, 1, 3, 2)) / np.sqrt(dh)          # [n, H, S(query), S(key)]
    s = np.where(causal[None, None], -np.inf, s)
    s = s - s.max(axis=-1, keepdims=True)
    p = np.exp(s)
    p = p / p.sum(axis=-1, keepdims=True)
    return p @ v, p


def causal_attention_bwd(do, q, k, v, p):
    """Gradients of causal_attention w.r.t. q, k, v given do = dL/do (all [n, H, S, dh])."""
    dh = q.shape[-1]
    dv = p.transpose(0, 1, 3, 2) @ do
    dp = do @ v.transpose(0, 1, 3, 2)
    ds = p * (dp - np.sum(dp * p, axis=-1, keepdims=True)) / np.sqrt(dh)
    return ds @ k, ds.transpose(0, 1, 3, 2) @ q, dv


LORA_PROJ = ("qkv", "o", "gu", "d")


def lora_linear(x, W, A=None, B=None, scale=1.0):
    """y = x W^T, plus the adapter's low-rank branch scale * (x A^T) B^T when A [r, in], B [out, r] are given."""
    y = x @ W.T
    if A is not None:
        y = y + scale * ((x @ A.T) @ B.T)
    return y


def lora_linear_bwd(dy, x, W, A=None, B=None, scale=1.0):
    """Input gradient of lora_linear and, with an adapter, (dA, dB); the base weight is frozen there.
    Without an adapter returns (dx, dW)."""
    in_f, out_f = W.shape[1], W.shape[0]
    dy2, x2 = dy.reshape(-1, out_f), x.reshape(-1, in_f)
    if A is None:
        return dy @ W, dy2.T @ x2
    u = dy @ B                                              # [.., r]
    dx = dy @ W + scale * (u @ A)
    dA = scale * (u.reshape(-1, A.shape[0]).T @ x2)
    dB = scale * (dy2.T @ (x2 @ A.T))
    return dx, (dA, dB)


def _adapter(lora, name, l):
    if lora is None:
        return None, None, 1.0
    return _f64(lora["a_" + name][l]), _f64(lora["b_" + name][l]), float(lora["alpha"]) / float(lora["rank"])


def forward(weights: Dict[str, np.ndarray], X, H: int, P: int, keep_cache: bool = True, lora=None):
    """X [n, S, d] -> (z [n, 56, V] logits at the scored positions, cache)."""
    Wt = {k: _f64(v) for k, v in weights.items()}
    x = _f64(X)
    n, S, d = x.shape
    L = Wt["w_qkv"].shape[0]
    dh = d // H
    cos, sin = rope_tables(S, dh)
    layers = []
    for l in range(L):
        x_in = x
        h1, rstd1 = rmsnorm(x_in, Wt["g1"][l])
        qkv = lora_linear(h1, Wt["w_qkv"][l], *_adapter(lora, "qkv", l))
        # heads as [n, H, S, dh]
        q = rope(qkv[..., :d].reshape(n, S, H, dh), cos, sin).transpose(0, 2, 1, 3)
        k = rope(qkv[..., d:2 * d].reshape(n, S, H, dh), cos, sin).transpose(0, 2, 1, 3)
        v = qkv[..., 2 * d:].reshape(n, S, H, dh).transpose(0, 2, 1, 3)
        o, p = causal_attention(q, k, v)
        o = o.transpose(0, 2, 1, 3).reshape(n, S, d)
        x_mid = x_in + lora_linear(o, Wt["w_o"][l], *_adapter(lora, "o", l))
        h2, rstd2 = rmsnorm(x_mid, Wt["g2"][l])
        gu = lora_linear(h2, Wt["w_gu"][l], *_adapter(lora, "gu", l))
        g, u = gu[..., :4 * d], gu[..., 4 * d:]
        act = silu(g) * u
        x = x_mid + lora_linear(act, Wt["w_d"][l], *_adapter(lora, "d", l))
        if keep_cache:
            layers.append(dict(x_in=x_in, rstd1=rstd1, h1=h1, q=q, k=k, v=v, p=p, o=o, x_mid=x_mid,
                               rstd2=rstd2, h2=h2, g=g, u=u, act=act))
    x_sc = x[:, P - 1:P - 1 + ACT_DIM, :]
    hf, rstdf = rmsnorm(x_sc, Wt["gf"])
    z = hf @ Wt["w_h"].T
    cache = dict(layers=layers, x_sc=x_sc, rstdf=rstdf, hf=hf, cos=cos, sin=sin, shape=(n, S, d), W=Wt)
    return z, cache


def log_softmax_at(z, tgt):
    """log-prob of token tgt under softmax(z) along the last axis; returns (logp, softmax)."""
    m = z.max(axis=-1, keepdims=True)
    lse = m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True))
    logp_all = z - lse
    logp = np.take_along_axis(logp_all, np.asarray(tgt, dtype=np.int64)[..., None], axis=-1)[..., 0]
    return logp, np.exp(logp_all)


def surrogate(logp, logp_old, adv_c, eps_low, eps_high, loss_scale):
    """Token-level clipped surrogate.  r = exp(logp - logp_old);
    loss = -loss_scale * sum min(r A, clip(r, 1-eps_low, 1+eps_high) A).
    Returns (loss, dloss/dlogp, ratio, active) where `active` marks terms whose gradient is r A:
    (A >= 0 and r <= 1+eps_high) or (A < 0 and r >= 1-eps_low)."""
    A = _f64(adv_c)[:, None]
    r = np.exp(logp - _f64(logp_old))
    s = np.minimum(r * A, np.clip(r, 1.0 - eps_low, 1.0 + eps_high) * A)
    loss = -loss_scale * float(np.sum(s))
    active = ((A >= 0) & (r <= 1.0 + eps_high)) | ((A < 0) & (r >= 1.0 - eps_low))
    dlogp = np.where(active, -loss_scale * A * r, 0.0)
    return loss, dlogp, r, active


def surrogate_chunk(logp, logp_old, adv_c, eps_low, eps_high, loss_scale):
    """Chunk-level clipped surrogate: the chunk's action is the joint of its 56 tokens, so
    log pi(a_ik | s_ik) = sum_j logp_j (the quantity Eq. 2 / Eq. 11 write) and one ratio per chunk,
    r = exp(sum_j logp_j - sum_j logp_old_j), goes through the same clip.
    loss = -loss_scale * sum_chunks min(r A, clip(r) A).  Returns (loss, dloss/dlogp [n,56], r [n], active [n])."""
    A = _f64(adv_c)
    r = np.exp(logp.sum(axis=-1) - _f64(logp_old).sum(axis=-1))
    s = np.minimum(r * A, np.clip(r, 1.0 - eps_low, 1.0 + eps_high) * A)
    loss = -loss_scale * float(np.sum(s))
    active = ((A >= 0) & (r <= 1.0 + eps_high)) | ((A < 0) & (r >= 1.0 - eps_low))
    dl = np.where(active, -loss_scale * A * r, 0.0)
    return loss, np.repeat(dl[:, None], logp.shape[-1], axis=-1), r, active


def entropy_rows(z):
    """Shannon entropy H = -sum_v p_v log p_v of softmax(z) along the last axis, and log p."""
    m = z.max(axis=-1, keepdims=True)
    logp_all = z - (m + np.log(np.exp(z - m).sum(axis=-1, keepdims=True)))
    return -(np.exp(logp_all) * logp_all).sum(axis=-1), logp_all


def objective(z, tgt, logp_old, adv_c, eps_low, eps_high, loss_scale, entropy_coef=0.0, ratio_level="token"):
    """Surrogate minus entropy bonus (App. E: entropy coefficient 1e-3, no KL term):
        loss = surrogate loss - entropy_coef * mean over the scored positions of H(pi(. | s)).
    Returns (loss, dloss/dz, logp, ratio, active, mean entropy)."""
    logp, prob = log_softmax_at(z, tgt)
    if ratio_level == "chunk":
        loss, dlogp, r, active = surrogate_chunk(logp, logp_old, adv_c, eps_low, eps_high, loss_scale)
    else:
        loss, dlogp, r, active = surrogate(logp, logp_old, adv_c, eps_low, eps_high, loss_scale)
    onehot = np.zeros_like(prob)
    np.put_along_axis(onehot, np.asarray(tgt, dtype=np.int64)[..., None], 1.0, axis=-1)
    dz = dlogp[..., None] * (onehot - prob)
    Hrow, logp_all = entropy_rows(z)
    if entropy_coef != 0.0:
        n_rows = Hrow.size
        loss = loss - entropy_coef * float(Hrow.sum()) / n_rows
        # dH/dz_v = -p_v (log p_v + H)
        dz = dz + (entropy_coef / n_rows) * prob * (logp_all + Hrow[..., None])
    return loss, dz, logp, r, active, float(Hrow.mean())


def logp_only(weights, X, tgt, H, P, lora=None):
    z, _ = forward(weights, X, H, P, keep_cache=False, lora=lora)
    return log_softmax_at(z, tgt)[0]


def loss_only(weights, X, tgt, logp_old, adv_c, H, P, eps_low, eps_high, loss_scale, entropy_coef=0.0,
              ratio_level="token", lora=None):
    z, _ = forward(weights, X, H, P, keep_cache=False, lora=lora)
    return objective(z, tgt, logp_old, adv_c, eps_low, eps_high, loss_scale, entropy_coef, ratio_level)[0]


def fwd_bwd(weights, X, tgt, logp_old, adv_c, H, P, eps_low=0.2, eps_high=0.2, loss_scale=None, entropy_coef=0.0,
            ratio_level="token", lora=None):
    """Masked GRPO actor update on the packed batch of kept chunks (Eq. 11).

    Returns (loss, logp [n,56], grads dict with the shapes of `weights`, stats).  `loss_scale`
    defaults to the mean over the surrogate's terms: 1/(56 n) with one ratio per token, 1/n with one
    ratio per chunk.  No gradient flows to the observation prefix; the embedding gradient collects
    the rows at the action-token positions.  With `lora` the four base matrices of every layer are frozen:
    their entries in `grads` are None and `grads` gains a_qkv, b_qkv, a_o, b_o, a_gu, b_gu, a_d, b_d."""
    n, S, d = np.asarray(X).shape
    if loss_scale is None:
        loss_scale = 1.0 / (ACT_DIM * n) if ratio_level == "token" else 1.0 / n
    z, cache = forward(weights, X, H, P, lora=lora)
    Wt = cache["W"]
    L = Wt["w_qkv"].shape[0]
    dh = d // H
    cos, sin = cache["cos"], cache["sin"]
    tgt = np.asarray(tgt, dtype=np.int64)
    loss, dz, logp, r, active, mean_H = objective(z, tgt, logp_old, adv_c, eps_low, eps_high, loss_scale,
                                                  entropy_coef, ratio_level)              # dz [n,56,V]
    grads = {k: np.zeros_like(v) for k, v in Wt.items()}
    if lora is not None:
        for name in LORA_PROJ:
            grads["w_" + name] = None
            grads["a_" + name] = np.zeros(np.asarray(lora["a_" + name]).shape)
            grads["b_" + name] = np.zeros(np.asarray(lora["b_" + name]).shape)

    def linear_bwd(name, l, dy, x_in_):
        """dx of projection `name` in layer l; stores dW, or (dA, dB) when the base weight is frozen."""
        A, B, sc = _adapter(lora, name, l)
        dx_, gw = lora_linear_bwd(dy, x_in_, Wt["w_" + name][l], A, B, sc)
        if lora is None:
            grads["w_" + name][l] = gw
        else:
            grads["a_" + name][l], grads["b_" + name][l] = gw
        return dx_

    V = dz.shape[-1]
    grads["w_h"] = dz.reshape(n * ACT_DIM, V).T @ cache["hf"].reshape(n * ACT_DIM, d)
    dhf = dz @ Wt["w_h"]
    dx_sc, grads["gf"] = rmsnorm_bwd(dhf, cache["x_sc"], cache["rstdf"], Wt["gf"])
    dx = np.zeros((n, S, d))
    dx[:, P - 1:P - 1 + ACT_DIM, :] = dx_sc

    for l in reversed(range(L)):
        c = cache["layers"][l]
        # x = x_mid + act @ W_d^T
        dact = linear_bwd("d", l, dx, c["act"])
        sg = 1.0 / (1.0 + np.exp(-c["g"]))
        dg = dact * c["u"] * (sg * (1.0 + c["g"] * (1.0 - sg)))
        du = dact * (c["g"] * sg)
        dgu = np.concatenate([dg, du], axis=-1)
        dh2 = linear_bwd("gu", l, dgu, c["h2"])
        dxm, grads["g2"][l] = rmsnorm_bwd(dh2, c["x_mid"], c["rstd2"], Wt["g2"][l])
        dx_mid = dx + dxm
        # x_mid = x_in + o @ W_o^T
        do = linear_bwd("o", l, dx_mid, c["o"]).reshape(n, S, H, dh).transpose(0, 2, 1, 3)   # [n, H, S, dh]
        dq, dk, dv = causal_attention_bwd(do, c["q"], c["k"], c["v"], c["p"])
        dq = rope_bwd(dq.transpose(0, 2, 1, 3), cos, sin)                           # [n, S, H, dh]
        dk = rope_bwd(dk.transpose(0, 2, 1, 3), cos, sin)
        dv = dv.transpose(0, 2, 1, 3)
        dqkv = np.concatenate([dq.reshape(n, S, d), dk.reshape(n, S, d), dv.reshape(n, S, d)], axis=-1)
        dh1 = linear_bwd("qkv", l, dqkv, c["h1"])
        dxi, grads["g1"][l] = rmsnorm_bwd(dh1, c["x_in"], c["rstd1"], Wt["g1"][l])
        dx = dx_mid + dxi

    # embedding gradient: rows at the action positions P .. P+55 hold E_act[token]
    dE = np.zeros_like(Wt["e_act"])
    for j in range(n):
        for t in range(ACT_DIM):
            dE[tgt[j, t]] += dx[j, P + t]
    grads["e_act"] = dE
    stats = dict(clip_frac=float(1.0 - active.mean()), mean_ratio=float(r.mean()), entropy=mean_H)
    return loss, logp, grads, stats
