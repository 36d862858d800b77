"""LoRA fine-tuning path (App. E: rank 32, alpha 32) against the fp64 oracle: adapter gradients, the gradients of
the tensors that stay trainable, loss and log-probs.  fp32 mode at 1e-5; bf16 on the tensor-core kernels (adapter
branch as a continuation of the contraction) at the bf16 tolerances."""
import numpy as np
import pytest
import torch

from oracle import actor_oracle as ao
from paper_2605_16154_b200 import synth
from tests.gpu_helpers import device_packed, grads_to_numpy, host_problem, rel_fro
from tests.test_gpu_actor import BF16_CASES, BF16_GRAD_TOL, BF16_LOSS_TOL, F32_TOL

pytestmark = pytest.mark.gpu
TRAINABLE = ("g1", "g2", "gf", "w_h", "e_act")


def _mods():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    return B, PL


def _lpo_from_lora_policy(hp, lo, w, margin):
    """Behaviour log-probs = the adapted policy's own (oracle) + seeded noise kept clear of the clip boundaries."""
    lp = ao.logp_only(hp["weights"], hp["X"], hp["tgt"], w.H, w.P, lora=lo)
    log_r = -synth.logp_noise(w.seed + 3, len(hp["kept"]), 0.1).astype(np.float64)
    for b in (np.log(1.2), np.log(0.8)):
        log_r = np.where(np.abs(log_r - b) < margin, b + 2 * margin * np.sign(log_r - b + 1e-30), log_r)
    return (lp - log_r).astype(np.float32)


def _run(B, PL, hp, lo, mb, entropy_coef=0.0):
    w = hp["w"]
    model = PL.upload_model(w, hp["weights"])
    lora = PL.upload_lora(w, model, lo)
    pk = device_packed(B, PL, model, hp)
    loss, logp, grads, stats = B.grpo_actor_fwd_bwd(model, pk, 0.2, 0.2, mb_chunks=mb, lora=lora, entropy_coef=entropy_coef)
    ref = ao.fwd_bwd(hp["weights"], hp["X"], hp["tgt"], hp["lpo"], hp["adv_c"], w.H, w.P, 0.2, 0.2,
                     entropy_coef=entropy_coef, lora=lo)
    got_g = grads_to_numpy(grads)
    got_g.update(grads_to_numpy(lora.grads))
    return model, lora, pk, (float(loss.item()), logp, got_g, stats), ref


@pytest.mark.parametrize("rank,alpha", [(8, 12.0), (32, 32.0)])
def test_lora_fp32_mode(rank, alpha):
    B, PL = _mods()
    w = synth.WORKLOADS["C0"].with_(gamma_std=0.1)
    hp = host_problem(w)
    lo = synth.make_lora(w, rank, alpha, b_std=0.05)
    hp["lpo"] = _lpo_from_lora_policy(hp, lo, w, 0.0)
    model, lora, pk, got, ref = _run(B, PL, hp, lo, mb=7, entropy_coef=1e-3)
    assert abs(got[0] - ref[0]) <= F32_TOL * abs(ref[0]) + 1e-9
    assert np.max(np.abs(got[1].cpu().numpy() - ref[1])) < 1e-5 * np.max(np.abs(ref[1]))
    for k in synth.LORA_NAMES + TRAINABLE:
        assert rel_fro(got[2][k], ref[2][k]) < F32_TOL, k
        assert np.max(np.abs(got[2][k] - ref[2][k])) <= F32_TOL * np.max(np.abs(ref[2][k])), k
    # the frozen matrices' gradient buffers were not touched
    assert all(float(model.grads[k].abs().max()) == 0.0 for k in ("w_qkv", "w_o", "w_gu", "w_d"))
    # accumulate doubles the adapter gradients
    B.grpo_actor_fwd_bwd(model, pk, 0.2, 0.2, mb_chunks=5, lora=lora, entropy_coef=1e-3, flags=B.GRPO_ACCUMULATE)
    for k in synth.LORA_NAMES:
        assert rel_fro(lora.grads[k].cpu().numpy(), 2 * ref[2][k]) < F32_TOL, k


@pytest.mark.parametrize("case,rank,alpha", [("small", 32, 32.0), ("c1_layer", 32, 32.0), ("small", 64, 32.0),
                                             ("small", 16, 8.0), ("c3_layer", 32, 32.0)])
def test_lora_bf16_on_the_tensor_core_kernels(case, rank, alpha):
    B, PL = _mods()
    kw = dict(BF16_CASES[case])
    max_kept = kw.pop("max_kept")
    w = synth.WORKLOADS["C1"].with_(gamma_std=0.1, force_mixed=True, p_succ=0.5, **kw)
    hp = host_problem(w, seed=2, max_kept=max_kept)
    lo = synth.make_lora(w, rank, alpha, seed=2, b_std=0.02)
    hp["lpo"] = _lpo_from_lora_policy(hp, lo, w, 0.05)
    model, lora, pk, got, ref = _run(B, PL, hp, lo, mb=2)
    assert abs(got[0] - ref[0]) < BF16_LOSS_TOL
    assert np.max(np.abs(got[1].cpu().numpy() - ref[1])) < 0.04
    errs = {k: rel_fro(got[2][k], ref[2][k]) for k in synth.LORA_NAMES + TRAINABLE}
    assert max(errs.values()) < BF16_GRAD_TOL, errs
    assert got[3].clip_frac == pytest.approx(ref[3]["clip_frac"], abs=1e-6)
    # the adapters do move the policy: the dense model's log-probs differ visibly
    lp_dense = ao.logp_only(hp["weights"], hp["X"], hp["tgt"], w.H, w.P)
    assert np.max(np.abs(lp_dense - ref[1])) > 0.01


def test_fresh_adapter_reproduces_the_dense_policy_bit_for_bit():
    """B = 0: the continuation adds exact zeros to the accumulator, so log-probs equal the dense call's."""
    B, PL = _mods()
    kw = dict(BF16_CASES["small"])
    max_kept = kw.pop("max_kept")
    w = synth.WORKLOADS["C1"].with_(gamma_std=0.1, force_mixed=True, p_succ=0.5, **kw)
    hp = host_problem(w, seed=2, max_kept=max_kept)
    lo = synth.make_lora(w, 32, 32.0, seed=2, b_std=0.0)
    model = PL.upload_model(w, hp["weights"])
    lora = PL.upload_lora(w, model, lo)
    pk = device_packed(B, PL, model, hp)
    _, logp_dense, _, _ = B.grpo_actor_fwd_bwd(model, pk, flags=B.GRPO_FWD_ONLY)
    _, logp_lora, _, _ = B.grpo_actor_fwd_bwd(model, pk, flags=B.GRPO_FWD_ONLY, lora=lora)
    assert torch.equal(logp_dense, logp_lora)
    _, _, _, _ = B.grpo_actor_fwd_bwd(model, pk, lora=lora)
    assert all(float(lora.grads[k].abs().max()) == 0.0 for k in ("a_qkv", "a_o", "a_gu", "a_d"))   # no signal reaches A
    assert all(float(lora.grads[k].abs().max()) > 0.0 for k in ("b_qkv", "b_o", "b_gu", "b_d"))


def test_lora_argument_errors():
    B, PL = _mods()
    w = synth.WORKLOADS["C0"]
    hp = host_problem(w)
    model = PL.upload_model(w, hp["weights"])
    pk = device_packed(B, PL, model, hp)
    lo = synth.make_lora(w, 8, 8.0)
    lora = PL.upload_lora(w, model, lo)
    lora.c.rank = 12                                        # not a multiple of 8
    with pytest.raises(B.PcmError):
        B.grpo_actor_fwd_bwd(model, pk, lora=lora)
    lora.c.rank = 8
    lora.c.alpha = 0.0
    with pytest.raises(B.PcmError):
        B.grpo_actor_fwd_bwd(model, pk, lora=lora)
