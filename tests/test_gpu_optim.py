"""Optimizer step on the device against the fp64 oracle, chained with the actor update."""
import numpy as np
import pytest
import torch

from oracle import actor_oracle as ao
from oracle import optim_oracle as oo
from paper_2605_16154_b200 import synth
from tests.gpu_helpers import device_packed, host_problem, rel_fro

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    return B, PL


def test_fp32_training_chain_matches_the_oracle():
    """Three iterations of (actor update -> clip -> AdamW) on the tiny fp32 workload."""
    B, PL = _mods()
    w = synth.WORKLOADS["C0"].with_(gamma_std=0.1)
    hp = host_problem(w)
    model = PL.upload_model(w, hp["weights"])
    pk = device_packed(B, PL, model, hp)
    opt = B.AdamW(model, lr=1e-3, max_grad_norm=0.01)               # a clip that bites and a visible step
    params = {k: v.astype(np.float64) for k, v in hp["weights"].items()}
    m = {k: np.zeros_like(v) for k, v in params.items()}
    v = {k: np.zeros_like(v) for k, v in params.items()}
    for step in range(1, 4):
        B.grpo_actor_fwd_bwd(model, pk)
        norm_gpu = float(opt.step().item())
        Xo = hp["X"].copy().astype(np.float64)
        Xo[:, w.P:] = params["e_act"][hp["tgt"].astype(int)]        # the packed action rows follow the updated embedding
        _, _, grads_o, _ = ao.fwd_bwd(params, Xo, hp["tgt"], hp["lpo"], hp["adv_c"], w.H, w.P, 0.2, 0.2)
        norm_o = oo.adamw_step(params, grads_o, m, v, step, lr=1e-3, max_norm=0.01)
        assert norm_o > 0.01                                        # clipping is active
        assert norm_gpu == pytest.approx(norm_o, rel=2e-5)
        pk.X[:, w.P:] = model.weights["e_act"][pk.tgt.long()]       # re-embed the action tokens with the new table
        for k in params:
            assert rel_fro(opt.master[k].cpu().numpy() - hp["weights"][k], params[k] - hp["weights"][k]) < 5e-4, (step, k)
            assert torch.equal(model.weights[k], opt.master[k])     # fp32 model: the weights are the masters


def test_bf16_weights_are_the_rounded_masters_and_moments_follow_the_gradients():
    B, PL = _mods()
    w = synth.WORKLOADS["C1"].with_(n_tasks=1, G=4, T=8, n_phases=4, budget=2, P=40, d=256, L=2, H=4, gamma_std=0.1,
                                    force_mixed=True, p_succ=0.5)
    hp = host_problem(w, seed=2, max_kept=5, clip_margin=0.05)
    model = PL.upload_model(w, hp["weights"])
    pk = device_packed(B, PL, model, hp)
    opt = B.AdamW(model, lr=1e-4, weight_decay=0.01, max_grad_norm=2.0)
    _, _, grads, _ = B.grpo_actor_fwd_bwd(model, pk)
    g = {k: t.clone() for k, t in grads.items()}
    before = {k: t.clone() for k, t in opt.master.items()}
    norm = float(opt.step().item())
    total = np.sqrt(sum(float((t.double() ** 2).sum()) for t in g.values()))
    assert norm == pytest.approx(total, rel=1e-5)
    params = {k: t.double().cpu().numpy() for k, t in before.items()}
    mo = {k: np.zeros_like(x) for k, x in params.items()}
    vo = {k: np.zeros_like(x) for k, x in params.items()}
    f32 = lambda x: float(np.float32(x))                            # the ABI carries the hyper-parameters as fp32
    oo.adamw_step(params, {k: t.cpu().numpy() for k, t in g.items()}, mo, vo, 1, lr=f32(1e-4), beta1=f32(0.9),
                  beta2=f32(0.999), eps=f32(1e-8), weight_decay=f32(0.01), max_norm=2.0)
    for k in params:
        # the fp32 master can only move in steps of its own ulp (6e-8 at 1.0): compare the weights, not the deltas
        assert np.allclose(opt.master[k].cpu().numpy(), params[k], rtol=2.5e-7, atol=1e-10), k
        assert rel_fro(opt.m[k].cpu().numpy(), mo[k]) < 2e-6 and rel_fro(opt.v[k].cpu().numpy(), vo[k]) < 2e-6, k
        assert torch.equal(model.weights[k], opt.master[k].to(torch.bfloat16)), k


def test_argument_errors():
    B, PL = _mods()
    w = synth.WORKLOADS["C0"]
    hp = host_problem(w)
    model = PL.upload_model(w, hp["weights"])
    model.alloc_grads()
    opt = B.AdamW(model, beta1=1.5)
    with pytest.raises(B.PcmError):
        opt.step()


@pytest.mark.parametrize("train_small", [True, False])
def test_lora_training_chain_matches_the_oracle(train_small):
    """Three iterations of (actor update with adapters -> clip -> AdamW on what is trained), fp32 mode."""
    B, PL = _mods()
    w = synth.WORKLOADS["C0"].with_(gamma_std=0.1)
    hp = host_problem(w)
    lo = synth.make_lora(w, 8, 12.0, b_std=0.05)
    model = PL.upload_model(w, hp["weights"])
    lora = PL.upload_lora(w, model, lo)
    pk = device_packed(B, PL, model, hp)
    opt = B.LoraAdamW(model, lora, train_small=train_small, lr=1e-3, max_grad_norm=0.01)
    small = ("g1", "g2", "gf", "w_h", "e_act") if train_small else ()
    weights = {k: v.astype(np.float64) for k, v in hp["weights"].items()}
    ad = {k: lo[k].astype(np.float64) for k in synth.LORA_NAMES}
    start = {**{k: weights[k].copy() for k in small}, **{k: ad[k].copy() for k in ad}}
    m = {k: np.zeros_like(v) for k, v in start.items()}
    v = {k: np.zeros_like(v) for k, v in start.items()}
    frozen_before = {k: model.weights[k].clone() for k in ("w_qkv", "w_o", "w_gu", "w_d")}
    for step in range(1, 4):
        B.grpo_actor_fwd_bwd(model, pk, lora=lora)
        norm_gpu = float(opt.step().item())
        Xo = hp["X"].copy().astype(np.float64)
        Xo[:, w.P:] = weights["e_act"][hp["tgt"].astype(int)]
        lo_now = dict(lo, **ad)
        _, _, grads_o, _ = ao.fwd_bwd(weights, Xo, hp["tgt"], hp["lpo"], hp["adv_c"], w.H, w.P, 0.2, 0.2, lora=lo_now)
        params = {**{k: weights[k] for k in small}, **ad}
        norm_o = oo.adamw_step(params, {k: grads_o[k] for k in params}, m, v, step, lr=1e-3, max_norm=0.01)
        for k in small:
            weights[k] = params[k]
        for k in ad:
            ad[k] = params[k]
        assert norm_o > 0.01
        assert norm_gpu == pytest.approx(norm_o, rel=2e-5)
        pk.X[:, w.P:] = model.weights["e_act"][pk.tgt.long()]
        for k in params:
            assert rel_fro(opt.master[k].cpu().numpy() - start[k], params[k] - start[k]) < 5e-4, (step, k)
            live = lora.tensors[k] if k in lora.tensors else model.weights[k]
            assert torch.equal(live, opt.master[k]), k
    for k, t in frozen_before.items():
        assert torch.equal(model.weights[k], t), k
    if not train_small:
        for k in ("g1", "g2", "gf", "w_h", "e_act"):
            assert np.array_equal(model.weights[k].cpu().numpy(), hp["weights"][k].astype(np.float32)), k


def test_lora_optimizer_wants_all_or_none_of_the_small_tensor_sets():
    B, PL = _mods()
    w = synth.WORKLOADS["C0"]
    hp = host_problem(w)
    model = PL.upload_model(w, hp["weights"])
    lora = PL.upload_lora(w, model, synth.make_lora(w, 8, 8.0))
    model.alloc_grads()
    lora.alloc_grads()
    opt = B.LoraAdamW(model, lora, train_small=True)
    opt.c_small[1] = None                    # moments missing while the rest is given
    with pytest.raises(B.PcmError):
        opt.step()
