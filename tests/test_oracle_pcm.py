"""Pins for the PCM control-plane oracle: closed forms, brute force, enumeration of the sampling
law and published Philox known answers.  None of the expected values comes from the oracle itself."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import pcm_oracle as po
from paper_2605_16154_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ Eq. 1
@pytest.mark.parametrize("G,s", [(8, 1), (8, 4), (10, 3), (16, 15)])
def test_advantage_closed_form(G, s):
    # binary rewards with s successes: sigma = sqrt(s/G (1 - s/G))
    r = np.array([1] * s + [0] * (G - s), dtype=np.uint8)
    A = po.advantages(r, G, eps=1e-6)
    f = s / G
    sig = math.sqrt(f * (1 - f))
    assert np.allclose(A[:s], (1 - f) / (sig + 1e-6), rtol=1e-14)
    assert np.allclose(A[s:], -f / (sig + 1e-6), rtol=1e-14)
    assert abs(A.sum()) < 1e-12          # zero mean within the group (proof of Lemma 1)


def test_advantage_uniform_groups_are_zero():
    r = np.array([1] * 8 + [0] * 8 + [1, 0, 0, 0, 0, 0, 0, 0], dtype=np.uint8)
    A = po.advantages(r, 8)
    assert np.all(A[:16] == 0.0)
    assert A[16] > 0 and np.all(A[17:] < 0)


# ------------------------------------------------------------------ Eq. 5
def _batch(n_traj, N, Kc, rng, reward):
    traj_off = np.arange(n_traj + 1, dtype=np.int32) * N
    phase = np.tile((np.arange(N) * Kc // N).astype(np.uint8), n_traj)
    tok = rng.integers(0, 256, size=(n_traj * N, 56), dtype=np.uint8)
    return traj_off, tok, phase, np.asarray(reward, dtype=np.uint8)


def test_score_zero_when_outcomes_coincide():
    # Lemma 1 special case: success and failure action tokens identical -> no signal, exactly 0
    rng = np.random.default_rng(0)
    traj_off, tok, phase, reward = _batch(8, 16, 4, rng, [1, 0] * 4)
    tok = np.tile(tok[:16], (8, 1))      # every trajectory carries the same chunks
    C, valid, n_valid, _, _ = po.score_phases(traj_off, tok, phase, reward, 8, 4)
    assert np.all(valid == 1) and np.all(C == 0.0)


def test_score_closed_form_constant_tokens():
    # success tokens all t1, failure tokens all t2 in phase 1 -> C = (2/256) |t1 - t2| sqrt(56)
    rng = np.random.default_rng(1)
    traj_off, tok, phase, reward = _batch(8, 16, 4, rng, [1, 1, 1, 0, 0, 0, 0, 1])
    t1, t2 = 200, 77
    for i in range(8):
        sl = slice(i * 16, (i + 1) * 16)
        tok[sl][phase[sl] == 1] = t1 if reward[i] else t2
    C, valid, _, _, _ = po.score_phases(traj_off, tok, phase, reward, 8, 4)
    assert valid[1] == 1
    assert C[1] == pytest.approx((2.0 / 256.0) * abs(t1 - t2) * math.sqrt(56), rel=1e-14)


def test_score_matches_float_definition_brute_force():
    # Eq. 5 written directly on de-tokenised float actions with library mean / norm
    rng = np.random.default_rng(2)
    G, Kc, n_traj = 4, 3, 12
    lengths = rng.integers(3, 9, size=n_traj)
    traj_off = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    total = int(traj_off[-1])
    tok = rng.integers(0, 256, size=(total, 56), dtype=np.uint8)
    phase = rng.integers(0, Kc, size=total).astype(np.uint8)      # arbitrary, non-contiguous labels
    reward = np.array([1, 0, 0, 1, 1, 1, 1, 1, 0, 1, 0, 0], dtype=np.uint8)   # group 1 is uniform
    C, valid, n_valid, Cg, vg = po.score_phases(traj_off, tok, phase, reward, G, Kc)
    a = -1.0 + (tok.astype(np.float64) + 0.5) * (2.0 / 256.0)
    owner = np.repeat(np.arange(n_traj), lengths)
    for c in range(Kc):
        vals = []
        for g in range(n_traj // G):
            in_g = (owner // G) == g
            succ = in_g & (reward[owner] == 1) & (phase == c)
            fail = in_g & (reward[owner] == 0) & (phase == c)
            if succ.any() and fail.any():
                vals.append(np.linalg.norm(a[succ].mean(0) - a[fail].mean(0)))
                assert vg[g, c] == 1 and Cg[g, c] == pytest.approx(vals[-1], rel=1e-12, abs=1e-15)
            else:
                assert vg[g, c] == 0
        assert n_valid[c] == len(vals)
        if vals:
            assert C[c] == pytest.approx(np.mean(vals), rel=1e-12)
    assert np.all(vg[1] == 0)            # uniform-reward group contributes nothing


def test_score_skips_phase_missing_from_one_outcome():
    rng = np.random.default_rng(3)
    traj_off, tok, phase, reward = _batch(4, 8, 4, rng, [1, 0, 0, 0])
    # the only successful trajectory never visits phase 3
    phase[0:8] = np.array([0, 0, 1, 1, 2, 2, 2, 2], dtype=np.uint8)
    C, valid, _, _, _ = po.score_phases(traj_off, tok, phase, reward, 4, 4)
    assert list(valid) == [1, 1, 1, 0] and C[3] == 0.0


def test_score_statistical_shape_on_synthetic_rollouts():
    # E||.||^2 ~ 56 (delta^2 + sigma^2 (1/n+ + 1/n-)) in the divergent phase, noise floor elsewhere
    w = synth.WORKLOADS["C0"]
    b = synth.make_rollouts(w, seed=0)
    C, valid, _, _, _ = po.score_phases(b["traj_off"], b["tok"], b["phase"], b["reward"], w.G, w.n_phases)
    assert np.all(valid == 1)
    assert C[2] == pytest.approx(0.5 * math.sqrt(56), rel=0.05)
    assert np.all(np.delete(C, 2) < 0.5)


# ------------------------------------------------------------------ Eq. 7-9
def test_keep_probs_hand_example():
    st = po.KeepProbState(3, p_min=0.1, t_rc=5)
    p, q, refreshed = po.update_keep_probs(st, [4.0, 1.0, 0.2], [1, 1, 1])
    assert refreshed
    assert p[0] == 1.0 and p[1] == pytest.approx(0.25, rel=1e-15) and p[2] == 0.1
    assert q[0] == 1 << 24 and q[1] == pytest.approx(0.25 * 2 ** 24, abs=1) and q[2] == round(0.1 * 2 ** 24)


def test_keep_probs_schedule_bounds_and_freeze():
    rng = np.random.default_rng(4)
    K = 5
    st = po.KeepProbState(K, p_min=0.1, t_rc=5)
    refresh_steps, prev = [], None
    window = []
    for t in range(23):
        C = rng.random(K) * np.array([5, 1, 0.01, 0.3, 2.0])
        window.append(C)
        p, q, refreshed = po.update_keep_probs(st, C, [1] * K)
        assert np.all(p >= 0.1) and np.all(p <= 1.0) and p.max() == 1.0
        if refreshed:
            refresh_steps.append(t)
            S = np.sum(window, axis=0)                  # Eq. 8 by library sum
            expect = np.maximum(0.1, S / S.max())
            assert np.allclose(p, expect, rtol=1e-13)
            window = []
        else:
            assert np.array_equal(p, prev)              # held fixed between refreshes
        prev = p
    assert refresh_steps == [0, 5, 10, 15, 20]


def test_keep_probs_scale_invariance_and_zero_scores():
    Cs = np.random.default_rng(5).random((11, 4))
    out = []
    for lam in (1.0, 1024.0):       # power of two: exact in floating point
        st = po.KeepProbState(4)
        out.append([po.update_keep_probs(st, lam * C, [1, 1, 1, 1])[0] for C in Cs])
    assert np.array_equal(np.array(out[0]), np.array(out[1]))
    st = po.KeepProbState(4)
    p, q, refreshed = po.update_keep_probs(st, [0, 0, 0, 0], [0, 0, 0, 0])
    assert refreshed and np.all(p == 1.0) and np.all(q == 1 << 24)
    # a skipped phase counts as 0 in the sum
    st = po.KeepProbState(2)
    p, _, _ = po.update_keep_probs(st, [3.0, 9.0], [1, 0])
    assert p[0] == 1.0 and p[1] == 0.1


# ------------------------------------------------------------------ Philox + Eq. 10
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        assert list(po.philox4x32_10(v[0:4], v[4:6])) == v[6:10]


def _pl_inclusion_exact(weights, m):
    """Inclusion probabilities of successive sampling by enumerating every ordered draw."""
    n = len(weights)
    inc = np.zeros(n)
    for seq in itertools.permutations(range(n), m):
        pr, rem = 1.0, float(sum(weights))
        for k in seq:
            pr *= weights[k] / rem
            rem -= weights[k]
        for k in seq:
            inc[k] += pr
    return inc


def test_sampler_counts_sorted_unique_and_small_trajectories():
    w = synth.WORKLOADS["C4"]
    b = synth.make_rollouts(w, seed=3)
    q = [int(round(p * 2 ** 24)) for p in (1, .1, .1, .5, .1, .1, .1, .3, .1, .1)]
    kept, off, per_phase = po.sample_chunks(b["traj_off"], b["phase"], q, 50, seed=9, it=2)
    for i in range(w.n_traj):
        a, e = b["traj_off"][i], b["traj_off"][i + 1]
        ks = kept[off[i]:off[i + 1]]
        assert len(ks) == min(50, e - a)                 # |K_i| = min(B, N_i)
        assert np.all(np.diff(ks) > 0) and ks[0] >= a and ks[-1] < e
    assert per_phase.sum() == len(kept)
    assert np.array_equal(np.bincount(b["phase"][kept], minlength=10), per_phase)


def test_sampler_inclusion_frequencies_match_plackett_luce_over_1e5_seeds():
    phase = (np.arange(16) * 4 // 16).astype(np.uint8)
    p = [1.0, 0.25, 0.1, 0.6]
    q = [int(round(x * 2 ** 24)) for x in p]
    exact = _pl_inclusion_exact([p[c] for c in phase], 3)
    assert exact.sum() == pytest.approx(3.0, rel=1e-12)
    n_seeds = 100_000
    counts = np.zeros(16)
    traj_off = np.array([0, 16], dtype=np.int32)
    for seed in range(n_seeds):
        kept, _, _ = po.sample_chunks(traj_off, phase, q, 3, seed=seed, it=0)
        counts[kept] += 1
    freq = counts / n_seeds
    sigma = np.sqrt(exact * (1 - exact) / n_seeds)
    assert np.all(np.abs(freq - exact) < 4 * sigma)
    assert np.all(freq[phase == 2] > 0)                  # floor-weight phase is never excluded


def test_sampler_uniform_weights_give_B_over_N():
    traj_off = np.array([0, 10], dtype=np.int32)
    phase = np.zeros(10, dtype=np.uint8)
    counts = np.zeros(10)
    n = 20_000
    for it in range(n):
        kept, _, _ = po.sample_chunks(traj_off, phase, [1 << 24], 4, seed=123, it=it)
        counts[kept] += 1
    assert np.all(np.abs(counts / n - 0.4) < 4 * math.sqrt(0.4 * 0.6 / n))


def test_sampler_agrees_with_exponential_race():
    # successive sampling is equal in law to keeping the m smallest of E_k / w_k, E_k ~ Exp(1)
    rng = np.random.default_rng(7)
    wts = np.array([1.0, 1.0, 0.1, 0.1, 0.5, 0.5, 0.5, 0.2])
    q = [int(round(x * 2 ** 24)) for x in wts]
    phase = np.arange(8, dtype=np.uint8)
    n = 40_000
    race = np.zeros(8)
    for _ in range(n):
        race[np.argsort(rng.exponential(size=8) / wts)[:3]] += 1
    mine = np.zeros(8)
    for it in range(n):
        kept, _, _ = po.sample_chunks(np.array([0, 8], dtype=np.int32), phase, q, 3, seed=5, it=it)
        mine[kept] += 1
    f1, f2 = race / n, mine / n
    assert np.all(np.abs(f1 - f2) < 4 * np.sqrt((f1 * (1 - f1) + f2 * (1 - f2)) / n))


def test_sampler_draw_is_first_prefix_exceeding_x():
    # x = floor(bits * W / 2^64): bits = 0 picks the first chunk, bits = 2^64 - 1 the last
    assert po.sample_one_trajectory([5, 7, 9], 1, [0]) == [0]
    assert po.sample_one_trajectory([5, 7, 9], 1, [(1 << 64) - 1]) == [2]
    # x = 5 is the first value beyond chunk 0's mass
    bits = ((5 << 64) // 21) + 1
    assert po.sample_one_trajectory([5, 7, 9], 1, [bits]) == [1]
    assert po.sample_one_trajectory([5, 7, 9], 3, [0, 0, 0]) == [0, 1, 2]


# ------------------------------------------------------------------ pack
def test_pack_round_trip():
    rng = np.random.default_rng(8)
    P, d, total = 3, 4, 10
    obs = rng.standard_normal((total, P, d)).astype(np.float32)
    tok = rng.integers(0, 256, size=(total, 56), dtype=np.uint8)
    lpo = rng.standard_normal((total, 56)).astype(np.float32)
    e_act = rng.standard_normal((256, d)).astype(np.float32)
    traj_off = np.array([0, 4, 10], dtype=np.int32)
    adv = np.array([0.5, -2.0], dtype=np.float32)
    kept = np.array([1, 3, 4, 9], dtype=np.int32)
    X, tgt, l2, adv_c, src = po.pack_chunks(lambda c: obs[c], tok, lpo, adv, traj_off, kept, e_act)
    assert X.shape == (4, P + 56, d)
    for j, c in enumerate(kept):
        assert np.array_equal(X[j, :P], obs[c])
        for t in range(56):
            assert np.array_equal(X[j, P + t], e_act[tok[c, t]])
        assert np.array_equal(tgt[j], tok[c]) and np.array_equal(l2[j], lpo[c])
    assert list(adv_c) == [0.5, 0.5, -2.0, -2.0] and list(src) == list(kept)


# ---- ablation samplers of RQ4 (random masking, full masking) ------------------------------------
def test_random_masking_keeps_unit_weights_whatever_the_scores():
    st = po.KeepProbState(4, p_min=0.1, t_rc=2, mode=1)
    for C in ([5.0, 1.0, 0.0, 0.25], [0.0, 9.0, 1.0, 1.0], [1.0, 1.0, 1.0, 1.0]):
        p, q, _ = po.update_keep_probs(st, C, [1, 1, 1, 1])
        assert p.tolist() == [1.0] * 4 and q.tolist() == [1 << 24] * 4


def test_random_masking_is_uniform_over_chunks():
    """Inclusion frequency B/N for every chunk, independent of its phase (binomial 5-sigma band)."""
    N, Bk, n_seeds = 9, 3, 20000
    phase = np.array([0, 0, 0, 1, 1, 2, 2, 2, 2], dtype=np.uint8)
    traj_off = np.array([0, N], dtype=np.int32)
    q = np.full(3, 1 << 24, dtype=np.int64)
    cnt = np.zeros(N)
    for s in range(n_seeds):
        k, off, _ = po.sample_chunks(traj_off, phase, q, Bk, s, 0)
        assert off[-1] == Bk
        cnt[k] += 1
    f, sd = Bk / N, math.sqrt(Bk / N * (1 - Bk / N) / n_seeds)
    assert np.all(np.abs(cnt / n_seeds - f) < 5 * sd)


def test_full_masking_keeps_only_the_highest_scoring_phase():
    st = po.KeepProbState(4, p_min=0.1, t_rc=2, mode=2)
    p, q, _ = po.update_keep_probs(st, [0.5, 3.0, 3.0, 1.0], [1, 1, 1, 1])      # tie: the first arg-max wins
    assert p.tolist() == [0.0, 1.0, 0.0, 0.0] and q.tolist() == [0, 1 << 24, 0, 0]
    # trajectories with 5, 2 and 0 chunks in phase 1; budget 3
    phase = np.array([0, 1, 1, 2, 1, 1, 1, 3,   1, 0, 1,   0, 2, 3], dtype=np.uint8)
    traj_off = np.array([0, 8, 11, 14], dtype=np.int32)
    for it in range(50):
        k, off, per_phase = po.sample_chunks(traj_off, phase, q, 3, 77, it)
        assert off.tolist() == [0, 3, 5, 5]                                    # min(B, chunks of that phase)
        assert np.all(phase[k] == 1) and per_phase.tolist() == [0, 5, 0, 0]
        assert k[3:].tolist() == [8, 10]                                       # below the budget: all of them
        assert set(k[:3].tolist()) <= {1, 2, 4, 5, 6} and len(set(k[:3].tolist())) == 3
    # all five candidates of the first trajectory get drawn over the iterations
    seen = set()
    for it in range(200):
        seen |= set(po.sample_chunks(traj_off, phase, q, 3, 77, it)[0][:3].tolist())
    assert seen == {1, 2, 4, 5, 6}


def test_full_masking_follows_the_buffered_sum_not_the_last_step():
    st = po.KeepProbState(3, p_min=0.1, t_rc=2, mode=2)
    po.update_keep_probs(st, [1.0, 0.0, 0.0], [1, 1, 1])                        # step 0 refreshes: phase 0
    po.update_keep_probs(st, [0.0, 5.0, 0.0], [1, 1, 1])                        # buffered, p unchanged
    assert st.p == [1.0, 0.0, 0.0]
    p, _, refreshed = po.update_keep_probs(st, [0.0, 0.0, 4.0], [1, 1, 1])      # S = (0, 5, 4)
    assert refreshed and p.tolist() == [0.0, 1.0, 0.0]


def test_default_mode_unchanged_by_the_ablation_switch():
    a, b = po.KeepProbState(5, 0.1, 3), po.KeepProbState(5, 0.1, 3, mode=0)
    rng = np.random.default_rng(3)
    for _ in range(10):
        C = rng.random(5)
        pa, qa, _ = po.update_keep_probs(a, C, [1] * 5)
        pb, qb, _ = po.update_keep_probs(b, C, [1] * 5)
        assert np.array_equal(pa, pb) and np.array_equal(qa, qb) and np.all(qa >= round(0.1 * (1 << 24)))


# ---- Eq. 5 on continuous actions ------------------------------------------------------------------
def test_float_scoring_matches_the_plain_definition_in_extended_precision():
    """Brute force of Eq. 5 with exact rational arithmetic on the float32 inputs."""
    from fractions import Fraction
    rng = np.random.default_rng(11)
    G, Kc, n_traj = 4, 3, 8
    lens = rng.integers(3, 9, size=n_traj)
    traj_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    N = int(traj_off[-1])
    act = (rng.standard_normal((N, 56)) * np.exp(rng.uniform(-3, 2, size=(N, 1)))).astype(np.float32)
    phase = rng.integers(0, Kc, size=N).astype(np.uint8)
    reward = np.array([1, 0, 0, 1, 1, 1, 0, 1], dtype=np.uint8)
    C, valid, nv, Cg, vg, bad = po.score_phases_float(traj_off, act, phase, reward, G, Kc)
    assert bad == 0
    for g in range(2):
        for c in range(Kc):
            rows = {0: [], 1: []}
            for i in range(g * G, (g + 1) * G):
                for ch in range(traj_off[i], traj_off[i + 1]):
                    if phase[ch] == c:
                        rows[int(reward[i])].append(ch)
            if not rows[0] or not rows[1]:
                assert vg[g, c] == 0
                continue
            tot = Fraction(0)
            for dim in range(56):
                m1 = sum(Fraction(float(act[ch, dim])) for ch in rows[1]) / len(rows[1])
                m0 = sum(Fraction(float(act[ch, dim])) for ch in rows[0]) / len(rows[0])
                tot += (m1 - m0) ** 2
            assert Cg[g, c] == pytest.approx(math.sqrt(float(tot)), rel=1e-12, abs=1e-9)
    for c in range(Kc):
        if valid[c]:
            assert C[c] == pytest.approx(np.mean([Cg[g, c] for g in range(2) if vg[g, c]]), rel=1e-15)


def test_float_scoring_on_bin_centres_equals_token_scoring():
    """De-tokenised actions a = -1 + (tok + 1/2) / 128 are exact in float32: both entry points agree."""
    w = synth.WORKLOADS["C0"]
    rb = synth.make_rollouts(w)
    act = (-1.0 + (rb["tok"].astype(np.float64) + 0.5) / 128.0).astype(np.float32)
    C_t, v_t, n_t, Cg_t, vg_t = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    C_f, v_f, n_f, Cg_f, vg_f, bad = po.score_phases_float(rb["traj_off"], act, rb["phase"], rb["reward"], w.G, w.n_phases)
    assert bad == 0 and np.array_equal(v_t, v_f) and np.array_equal(n_t, n_f) and np.array_equal(vg_t, vg_f)
    assert np.allclose(Cg_f, Cg_t, rtol=1e-14, atol=0) and np.allclose(C_f, C_t, rtol=1e-14, atol=0)


def test_float_scoring_is_invariant_to_chunk_order_and_flags_bad_values():
    rng = np.random.default_rng(12)
    G, Kc = 4, 2
    traj_off = np.array([0, 5, 9, 15, 20], dtype=np.int32)
    act = (rng.standard_normal((20, 56)) * 10.0 ** rng.integers(-6, 3, size=(20, 1))).astype(np.float32)
    phase = rng.integers(0, Kc, size=20).astype(np.uint8)
    reward = np.array([1, 0, 1, 0], dtype=np.uint8)
    ref = po.score_phases_float(traj_off, act, phase, reward, G, Kc)
    # reverse the chunks inside every trajectory: the sets per (phase, outcome) are unchanged
    perm = np.concatenate([np.arange(traj_off[i], traj_off[i + 1])[::-1] for i in range(4)])
    got = po.score_phases_float(traj_off, act[perm], phase[perm], reward, G, Kc)
    assert np.array_equal(ref[0].view(np.uint64), got[0].view(np.uint64))          # bit-identical
    # translation by a constant vector cancels in the difference of means (values on the 2^-32 grid stay exact)
    shift = np.float32(0.5)
    sh = po.score_phases_float(traj_off, (act.astype(np.float64) + 0.5).astype(np.float32), phase, reward, G, Kc)
    assert np.allclose(sh[0], ref[0], rtol=1e-5)
    bad = act.copy(); bad[3, 7] = np.nan; bad[11, 0] = np.inf; bad[12, 55] = 5000.0
    out = po.score_phases_float(traj_off, bad, phase, reward, G, Kc)
    assert out[5] == 3
    zeroed = act.copy(); zeroed[3, 7] = 0; zeroed[11, 0] = 0; zeroed[12, 55] = 0
    assert np.array_equal(out[0], po.score_phases_float(traj_off, zeroed, phase, reward, G, Kc)[0])
