"""Shared set-up for the GPU parity tests: builds one problem on the host from the seeded generators,
runs the oracle on it, and mirrors the same inputs onto the device."""
import numpy as np
import torch

from oracle import actor_oracle as ao
from oracle import pcm_oracle as po
from paper_2605_16154_b200 import synth


def rel_fro(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a - b))


def host_problem(w, seed=None, budget=None, sigma=0.1, lpo_mode="oracle", max_kept=None, clip_margin=0.0,
                 eps=(0.2, 0.2)):
    """Rollouts -> oracle selection -> oracle pack; logp_old = oracle log-probs + seeded noise.

    The clipped surrogate's gradient switches off discontinuously at ratio = 1 +- eps, so a token whose
    ratio sits on a boundary is decided by rounding.  With clip_margin > 0 the noise is moved so that
    no oracle ratio lies within that margin (in log space) of either boundary: the comparison then
    covers what is uniquely defined."""
    seed = w.seed if seed is None else seed
    budget = w.budget if budget is None else budget
    rb = synth.make_rollouts(w, seed)
    weights = synth.make_weights(w, seed)
    adv = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
    C, valid, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    _, q, _ = po.update_keep_probs(po.KeepProbState(w.n_phases, w.p_min, w.t_rc), C, valid)
    kept, off, _ = po.sample_chunks(rb["traj_off"], rb["phase"], q, budget, 7 + seed, 0)
    if max_kept is not None:
        kept = kept[:max_kept]
    obs = {int(c): synth.obs_chunk(w, seed, int(c)) for c in kept}
    total = int(rb["traj_off"][-1])
    lpo_all = np.zeros((total, 56), dtype=np.float32)
    X, tgt, _, adv_c, src = po.pack_chunks(lambda c: obs[c], rb["tok"], lpo_all, adv, rb["traj_off"], kept, weights["e_act"])
    if lpo_mode == "oracle":
        lp = ao.logp_only(weights, X, tgt, w.H, w.P)
        noise = synth.logp_noise(seed, len(kept), sigma).astype(np.float64)
        if clip_margin > 0.0:
            log_r = -noise                                   # log ratio seen by the oracle
            hi, lo = np.log(1.0 + eps[1]), np.log(1.0 - eps[0])
            log_r = np.where(np.abs(log_r - hi) < clip_margin, hi + 2 * clip_margin * np.sign(log_r - hi + 1e-30), log_r)
            log_r = np.where(np.abs(log_r - lo) < clip_margin, lo + 2 * clip_margin * np.sign(log_r - lo + 1e-30), log_r)
            noise = -log_r
        lpo = (lp + noise).astype(np.float32)
    else:   # constant near-uniform behaviour policy: heavy clipping
        lpo = (-np.log(256.0) + synth.logp_noise(seed, len(kept), sigma)).astype(np.float32)
    return dict(w=w, rb=rb, weights=weights, adv=adv, kept=kept, off=off, X=X, tgt=tgt, lpo=lpo, adv_c=adv_c, src=src,
                q=q, obs=obs)


def device_packed(B, PL, model, hp):
    w = hp["w"]
    pk = B.Packed(model, len(hp["kept"]))
    pk.X.copy_(PL.dev(hp["X"].astype(np.float32), PL.torch_dtype(w)))
    pk.tgt.copy_(PL.dev(hp["tgt"]))
    pk.lpo.copy_(PL.dev(hp["lpo"]))
    pk.adv_c.copy_(PL.dev(hp["adv_c"].astype(np.float32)))
    pk.src.copy_(PL.dev(hp["src"]))
    return pk


def oracle_update(hp, eps_low=0.2, eps_high=0.2, loss_scale=None, entropy_coef=0.0, ratio_level="token"):
    w = hp["w"]
    return ao.fwd_bwd(hp["weights"], hp["X"], hp["tgt"], hp["lpo"], hp["adv_c"], w.H, w.P, eps_low, eps_high, loss_scale,
                      entropy_coef, ratio_level)


def grads_to_numpy(grads):
    return {k: v.detach().cpu().numpy() for k, v in grads.items()}
