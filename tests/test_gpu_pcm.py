"""CUDA path vs oracle for the PCM control plane and the pack step: bit-exact."""
import numpy as np
import pytest
import torch

from oracle import pcm_oracle as po
from paper_2605_16154_b200 import synth

pytestmark = pytest.mark.gpu


def _mods():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    return B, PL


def _np(t):
    return t.detach().cpu().numpy()


@pytest.mark.parametrize("name", ["C0", "C1", "C3", "C4"])
def test_score_update_sample_bit_exact(name):
    B, PL = _mods()
    w = synth.WORKLOADS[name]
    rb = synth.make_rollouts(w)
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=1234 + w.seed, max_traj=w.n_traj)
    batch = PL.upload_rollouts(w, rb)
    adv, Cc, valid, p, q, kept_idx, kept_off, per_phase = PL.select(ctx, batch, it=7)
    assert B.pcm_poll_status(ctx) == 0
    C_o, valid_o, nvalid_o, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    assert np.array_equal(_np(Cc).view(np.uint64), C_o.view(np.uint64))            # bit-exact fp64
    assert np.array_equal(_np(valid), valid_o)
    adv_o = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
    assert np.array_equal(_np(adv).view(np.uint32), adv_o.view(np.uint32))
    st = po.KeepProbState(w.n_phases, w.p_min, w.t_rc)
    p_o, q_o, _ = po.update_keep_probs(st, C_o, valid_o)
    assert np.array_equal(_np(q).astype(np.int64), q_o)
    assert np.array_equal(_np(p), p_o.astype(np.float32))
    k_o, off_o, pp_o = po.sample_chunks(rb["traj_off"], rb["phase"], q_o, w.budget, 1234 + w.seed, 7)
    n_kept = int(off_o[-1])
    assert np.array_equal(_np(kept_off), off_o)
    assert np.array_equal(_np(kept_idx)[:n_kept], k_o)
    assert np.array_equal(_np(per_phase), pp_o)
    ctx.close()


def test_online_chain_50_iterations_ragged():
    """C4: rollouts resampled every iteration, keep-probability state carried across iterations."""
    B, PL = _mods()
    w = synth.WORKLOADS["C4"]
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=99, max_traj=w.n_traj)
    st = po.KeepProbState(w.n_phases, w.p_min, w.t_rc)
    refreshes = []
    for it in range(50):
        rb = synth.make_rollouts(w, seed=it)
        batch = PL.upload_rollouts(w, rb)
        adv, Cc, valid, p, q, kept_idx, kept_off, per_phase = PL.select(ctx, batch, it)
        C_o, valid_o, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
        p_o, q_o, refreshed = po.update_keep_probs(st, C_o, valid_o)
        if refreshed:
            refreshes.append(it)
        k_o, off_o, pp_o = po.sample_chunks(rb["traj_off"], rb["phase"], q_o, w.budget, 99, it)
        assert np.array_equal(_np(Cc).view(np.uint64), C_o.view(np.uint64)), it
        assert np.array_equal(_np(q).astype(np.int64), q_o), it
        assert np.array_equal(_np(kept_off), off_o), it
        assert np.array_equal(_np(kept_idx)[: int(off_o[-1])], k_o), it
        assert np.array_equal(_np(per_phase), pp_o), it
        if it == 22:      # stop and resume from an exported state blob
            blob = B.pcm_state_export(ctx)
            ctx.close()
            ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=99, max_traj=w.n_traj)
            B.pcm_state_import(ctx, blob)
    assert refreshes == list(range(0, 50, 5))
    assert B.pcm_poll_status(ctx) == 0
    ctx.close()


def test_sampler_edge_cases():
    """Budget above every length (keep all), lengths below the budget, single-chunk and empty
    trajectories, arbitrary (non-contiguous) phase labels, more than one tile of 32 chunks."""
    B, PL = _mods()
    rng = np.random.default_rng(0)
    lengths = np.array([1, 0, 5, 33, 64, 2, 100, 31, 32, 7, 257, 3], dtype=np.int64)
    traj_off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    total = int(traj_off[-1])
    Kc = 6
    rb = {"traj_off": traj_off, "tok": rng.integers(0, 256, (total, 56), dtype=np.uint8),
          "phase": rng.integers(0, Kc, total).astype(np.uint8), "reward": np.array([1, 0] * 6, dtype=np.uint8)}
    w = synth.WORKLOADS["C0"].with_(n_phases=Kc, G=4)
    for budget in (1, 6, 40, 500):
        ctx = B.Context(Kc, budget, 4, 5, 0.1, 1e-6, seed=(1 << 40) + 17, max_traj=12)
        batch = PL.upload_rollouts(w, rb)
        q_np = np.array([1 << 24, 1677722, 5000000, 1, 9999999, 1 << 23], dtype=np.int64)
        q = torch.from_numpy(q_np.astype(np.int32)).cuda()
        it = (3 << 32) + 5
        kept_idx, kept_off, per_phase = B.pcm_sample_chunks(ctx, batch, q, it)
        k_o, off_o, pp_o = po.sample_chunks(traj_off, rb["phase"], q_np, budget, (1 << 40) + 17, it)
        assert np.array_equal(_np(kept_off), off_o)
        assert np.array_equal(_np(kept_idx)[: int(off_o[-1])], k_o)
        assert np.array_equal(_np(per_phase), pp_o)
        assert B.pcm_poll_status(ctx) == 0
        ctx.close()


def test_score_edge_cases_and_status_word():
    B, PL = _mods()
    rng = np.random.default_rng(1)
    # long runs inside one phase (> 256 chunks between flushes), uniform groups, a missing phase
    lengths = np.array([700, 3, 1, 650, 10, 10, 10, 10], dtype=np.int64)
    traj_off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    total = int(traj_off[-1])
    phase = np.zeros(total, dtype=np.uint8)
    phase[traj_off[3]: traj_off[3] + 600] = 1
    phase[traj_off[4]:] = rng.integers(0, 3, total - traj_off[4]).astype(np.uint8)
    rb = {"traj_off": traj_off, "tok": np.full((total, 56), 255, dtype=np.uint8), "phase": phase,
          "reward": np.array([1, 0, 0, 0, 1, 1, 1, 1], dtype=np.uint8)}
    rb["tok"][traj_off[3]:] = rng.integers(0, 256, (total - traj_off[3], 56), dtype=np.uint8)
    w = synth.WORKLOADS["C0"].with_(n_phases=3, G=4)
    ctx = B.Context(3, 2, 4, 5, 0.1, 1e-6, seed=0, max_traj=8)
    batch = PL.upload_rollouts(w, rb)
    Cc, valid, n_valid, adv = B.pcm_score_phases(ctx, batch)
    C_o, valid_o, nv_o, _, _ = po.score_phases(traj_off, rb["tok"], phase, rb["reward"], 4, 3)
    assert np.array_equal(_np(Cc).view(np.uint64), C_o.view(np.uint64))
    assert np.array_equal(_np(valid), valid_o) and np.array_equal(_np(n_valid), nv_o)
    assert B.pcm_poll_status(ctx) == 0
    # a phase label beyond n_phases is reported through the status word, not by a fault
    bad = dict(rb)
    bad["phase"] = phase.copy()
    bad["phase"][5] = 9
    B.pcm_score_phases(ctx, PL.upload_rollouts(w, bad))
    assert B.pcm_poll_status(ctx) == -7
    assert B.pcm_poll_status(ctx) == 0
    ctx.close()


def test_host_argument_errors():
    B, PL = _mods()
    with pytest.raises(B.PcmError):
        B.Context(0, 3, 8)                      # no phases
    with pytest.raises(B.PcmError):
        B.Context(4, 3, 8, p_min=0.0)           # floor must be positive
    ctx = B.Context(4, 3, 8, max_traj=8)
    w = synth.WORKLOADS["C0"]
    rb = synth.make_rollouts(w)
    batch = PL.upload_rollouts(w, rb)
    batch.n_traj = 7                             # not a multiple of the group size
    with pytest.raises(B.PcmError):
        B.pcm_score_phases(ctx, batch)
    with pytest.raises(B.PcmError):
        B.pcm_state_import(ctx, b"\0" * 10)
    ctx.close()


@pytest.mark.parametrize("case", ["C0", "bf16_wide", "bf16_ragged"])
def test_pack_bit_exact(case):
    B, PL = _mods()
    if case == "C0":
        w = synth.WORKLOADS["C0"]
    elif case == "bf16_wide":
        w = synth.WORKLOADS["C1"].with_(n_tasks=1, G=4, T=9, budget=4)          # 512 KB prefixes, 2 KB rows
    else:
        w = synth.WORKLOADS["C4"].with_(n_tasks=1, G=4, d=2048, P=37, len_lo=3, len_hi_succ=9, len_hi_fail=12,
                                        n_phases=3, budget=5)
    rb = synth.make_rollouts(w, seed=3)
    total = int(rb["traj_off"][-1])
    e_act = synth.round_to_dtype(np.random.default_rng(2).standard_normal((256, w.d)).astype(np.float32), w.dtype)
    obs = synth.obs_all(w, 5, total)
    lpo = np.random.default_rng(3).standard_normal((total, 56)).astype(np.float32)
    adv = po.advantages(rb["reward"], w.G).astype(np.float32)
    q = [1 << 24] * w.n_phases
    kept, off, _ = po.sample_chunks(rb["traj_off"], rb["phase"], q, w.budget, 5, 0)
    X_o, tgt_o, lpo_o, advc_o, src_o = po.pack_chunks(lambda c: obs[c], rb["tok"], lpo, adv, rb["traj_off"], kept, e_act)

    td = PL.torch_dtype(w)
    ctx = B.Context(w.n_phases, w.budget, w.G, max_traj=w.n_traj)
    batch = PL.upload_rollouts(w, rb, obs=PL.dev(obs, td), logp_old=PL.dev(lpo))

    class _M:      # only what pack needs from a model
        cfg = B.grpo_model_cfg(w.d, w.L, w.H, w.P, PL.model_dtype(w), 0)
        weights = {"e_act": PL.dev(e_act, td)}
        S = w.S
    out = B.Packed(_M, len(kept))
    out.X.fill_(7.0)
    B.grpo_pack_chunks(ctx, batch, _M, PL.dev(kept), PL.dev(off), PL.dev(adv), out)
    assert B.pcm_poll_status(ctx) == 0
    assert np.array_equal(_np(out.X.float()), X_o.astype(np.float32))      # values exact in the dtype => bit-exact
    assert np.array_equal(_np(out.tgt), tgt_o)
    assert np.array_equal(_np(out.lpo), lpo_o)
    assert np.array_equal(_np(out.adv_c), advc_o)
    assert np.array_equal(_np(out.src), src_o)
    ctx.close()


@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("name", ["C0", "C4"])
def test_ablation_samplers_bit_exact(name, mode):
    """Random masking and full masking (RQ4): keep-probabilities, offsets and kept ids against the oracle
    over a chain of iterations; full masking keeps chunks of one phase only."""
    B, PL = _mods()
    w = synth.WORKLOADS[name]
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=5, max_traj=w.n_traj, mode=mode)
    st = po.KeepProbState(w.n_phases, w.p_min, w.t_rc, mode=mode)
    for it in range(7):
        rb = synth.make_rollouts(w, seed=100 + it)
        batch = PL.upload_rollouts(w, rb)
        adv, Cc, valid, p, q, kept_idx, kept_off, per_phase = PL.select(ctx, batch, it)
        C_o, valid_o, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
        p_o, q_o, _ = po.update_keep_probs(st, C_o, valid_o)
        k_o, off_o, pp_o = po.sample_chunks(rb["traj_off"], rb["phase"], q_o, w.budget, 5, it)
        assert np.array_equal(_np(q).astype(np.int64), q_o), it
        assert np.array_equal(_np(p), p_o.astype(np.float32)), it
        assert np.array_equal(_np(kept_off), off_o), it
        assert np.array_equal(_np(kept_idx)[: int(off_o[-1])], k_o), it
        assert np.array_equal(_np(per_phase), pp_o), it
        if mode == 2:
            assert np.count_nonzero(_np(per_phase)) == 1 and int(np.count_nonzero(q_o)) == 1
        else:
            lens = np.diff(rb["traj_off"])
            assert np.array_equal(np.diff(off_o), np.minimum(lens, w.budget))
    assert B.pcm_poll_status(ctx) == 0
    ctx.close()


def test_bad_mask_mode_is_rejected():
    B, _ = _mods()
    with pytest.raises(RuntimeError):
        B.Context(4, 4, 4, mode=3)


def _float_actions(rb, seed, scale_spread=True):
    """Continuous stand-in for the chunk actions: bin centres plus seeded jitter, magnitudes over several decades."""
    rng = np.random.default_rng(seed)
    base = -1.0 + (rb["tok"].astype(np.float64) + 0.5) / 128.0
    act = base + 0.01 * rng.standard_normal(base.shape)
    if scale_spread:
        act = act * np.exp(rng.uniform(-8, 3, size=(act.shape[0], 1)))
    return act.astype(np.float32)


@pytest.mark.parametrize("name", ["C0", "C4"])
def test_float_action_scoring_bit_exact(name):
    B, PL = _mods()
    w = synth.WORKLOADS[name]
    rb = synth.make_rollouts(w)
    ctx = B.Context(w.n_phases, w.budget, w.G, w.t_rc, w.p_min, 1e-6, seed=0, max_traj=w.n_traj)
    batch = PL.upload_rollouts(w, rb)
    for spread in (False, True):
        act = _float_actions(rb, 3, spread)
        Cc, valid, n_valid, adv = B.pcm_score_phases_f32(ctx, batch, PL.dev(act))
        C_o, valid_o, nv_o, _, _, bad = po.score_phases_float(rb["traj_off"], act, rb["phase"], rb["reward"], w.G, w.n_phases)
        assert bad == 0 and B.pcm_poll_status(ctx) == 0
        assert np.array_equal(_np(Cc).view(np.uint64), C_o.view(np.uint64))
        assert np.array_equal(_np(valid), valid_o) and np.array_equal(_np(n_valid), nv_o)
        adv_o = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
        assert np.array_equal(_np(adv).view(np.uint32), adv_o.view(np.uint32))
    # exact bin centres: the float entry point reproduces the token entry point to rounding
    centres = (-1.0 + (rb["tok"].astype(np.float64) + 0.5) / 128.0).astype(np.float32)
    C_f = _np(B.pcm_score_phases_f32(ctx, batch, PL.dev(centres))[0])
    C_t = _np(B.pcm_score_phases(ctx, batch)[0])
    assert np.allclose(C_f, C_t, rtol=1e-14, atol=0)
    ctx.close()


def test_float_action_scoring_edge_cases():
    B, PL = _mods()
    rng = np.random.default_rng(2)
    lengths = np.array([700, 3, 1, 0, 10, 10, 11, 10], dtype=np.int64)       # long, odd, single and empty trajectories
    traj_off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    total = int(traj_off[-1])
    phase = rng.integers(0, 3, total).astype(np.uint8)
    phase[:650] = 1                                                          # one long run in a single phase
    reward = np.array([1, 0, 0, 1, 1, 1, 1, 1], dtype=np.uint8)              # second group uniform
    act = (rng.standard_normal((total, 56)) * 10.0 ** rng.integers(-7, 4, size=(total, 1))).astype(np.float32)
    act = np.clip(act, -4096, 4096)
    act[5, 3] = 4096.0; act[6, 3] = -4096.0; act[7, 0] = 1e-30; act[8, 0] = -0.0
    w = synth.WORKLOADS["C0"].with_(n_phases=3, G=4)
    rb = {"traj_off": traj_off, "tok": np.zeros((total, 56), dtype=np.uint8), "phase": phase, "reward": reward}
    ctx = B.Context(3, 2, 4, 5, 0.1, 1e-6, seed=0, max_traj=8)
    batch = PL.upload_rollouts(w, rb)
    Cc, valid, n_valid, _ = B.pcm_score_phases_f32(ctx, batch, PL.dev(act))
    C_o, valid_o, nv_o, _, _, bad = po.score_phases_float(traj_off, act, phase, reward, 4, 3)
    assert bad == 0 and B.pcm_poll_status(ctx) == 0
    assert np.array_equal(_np(Cc).view(np.uint64), C_o.view(np.uint64))
    assert np.array_equal(_np(valid), valid_o) and np.array_equal(_np(n_valid), nv_o) and nv_o.max() == 1
    # values outside the range count as zero and are reported, on both sides
    act_bad = act.copy(); act_bad[2, 9] = np.nan; act_bad[701, 0] = np.inf; act_bad[10, 55] = -5000.0
    Cc, _, _, _ = B.pcm_score_phases_f32(ctx, batch, PL.dev(act_bad))
    C_b, _, _, _, _, bad = po.score_phases_float(traj_off, act_bad, phase, reward, 4, 3)
    assert bad == 3 and np.array_equal(_np(Cc).view(np.uint64), C_b.view(np.uint64))
    assert B.pcm_poll_status(ctx) == -7 and B.pcm_poll_status(ctx) == 0
    # host checks: misaligned action pointer, group too large for the 64-bit sums
    with pytest.raises(RuntimeError):
        B.pcm_score_phases_f32(ctx, batch, PL.dev(np.zeros(total * 56 + 1, dtype=np.float32))[1:].view(total, 56))
    big = B.make_batch(PL.dev(traj_off), None, PL.dev(phase), PL.dev(reward), 70000)
    with pytest.raises(RuntimeError):
        B.pcm_score_phases_f32(ctx, big, PL.dev(act))
    ctx.close()
