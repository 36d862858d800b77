"""CPU oracle for the PCM control plane (advantages, phase scores, keep-probabilities, sampling, pack).

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 / exact-integer numpy and Python loops written from the
paper's equations; it shares no code with the CUDA path and must never be imported by it.  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may call it.

Parity status: every function here is pinned by tests that do not use the function itself
(closed forms, brute force, enumeration of the sampling law, published Philox known answers).

Notation follows the paper: G rollouts per group, K phases (n_phases), budget B, floor p_min,
refresh window T_rc, chunk (i, k) with phase phi(i, k).
"""
from __future__ import annotations

import math
from typing import List, Sequence, Tuple

import numpy as np

ACT_DIM = 56
BIN_WIDTH = 2.0 / 256.0        # action range [-1, 1) split into 256 bins
Q_ONE = 1 << 24                # integer weight that represents keep-probability 1


# ----------------------------------------------------------------------------------------------
# Eq. 1 - group-relative advantage
# ----------------------------------------------------------------------------------------------
def advantages(reward: np.ndarray, G: int, eps: float = 1e-6) -> np.ndarray:
    """A_i = (r_i - mu_r) / (sigma_r + eps) with the population (1/G) standard deviation (Eq. 1).

    Sums run over the group's members in index order; a group whose rewards are all equal gets
    exactly zero advantages (numerator 0)."""
    r = np.asarray(reward, dtype=np.float64)
    out = np.zeros(r.size, dtype=np.float64)
    for g in range(r.size // G):
        s = 0.0
        for j in range(G):
            s = s + r[g * G + j]
        mu = s / G
        v = 0.0
        for j in range(G):
            dlt = r[g * G + j] - mu
            v = v + dlt * dlt
        sigma = math.sqrt(v / G)
        for j in range(G):
            out[g * G + j] = (r[g * G + j] - mu) / (sigma + eps)
    return out


# ----------------------------------------------------------------------------------------------
# Eq. 5 - success-failure action variance per phase
# ----------------------------------------------------------------------------------------------
def detokenize(tok: np.ndarray) -> np.ndarray:
    """Bin-centre action value of each token: a = -1 + (tok + 1/2) * 2/256."""
    return -1.0 + (np.asarray(tok, dtype=np.float64) + 0.5) * BIN_WIDTH


def score_phases(traj_off, tok, phase, reward, G: int, n_phases: int):
    """Batch-level phase scores C_c (Eq. 5).

    For every group with both outcomes present, and every phase that has chunks from both a
    successful and a failed rollout of that group, C_{c,g} is the Euclidean norm of the difference
    between the mean 56-dim chunk action over success chunks and over failure chunks.  Groups with
    uniform rewards are ignored and a phase missing from one outcome is skipped (Sec. 4.1, App. E.2).
    The batch score is the arithmetic mean of C_{c,g} over the groups where it is defined, summed
    in ascending group order.

    The affine de-tokenisation cancels in the difference of means, so the means are taken over the
    integer token ids (exact) and the bin width is applied once at the end.

    Returns (C float64[n_phases], valid uint8[n_phases], n_valid_groups int32[n_phases],
             C_group float64[n_groups, n_phases], valid_group uint8[n_groups, n_phases]).
    """
    traj_off = np.asarray(traj_off)
    n_traj = traj_off.size - 1
    n_groups = n_traj // G
    C_group = np.zeros((n_groups, n_phases), dtype=np.float64)
    valid_group = np.zeros((n_groups, n_phases), dtype=np.uint8)
    for g in range(n_groups):
        # integer sums and counts per (phase, outcome)
        S = np.zeros((n_phases, 2, ACT_DIM), dtype=np.int64)
        n = np.zeros((n_phases, 2), dtype=np.int64)
        for i in range(g * G, (g + 1) * G):
            o = int(reward[i])
            for ch in range(int(traj_off[i]), int(traj_off[i + 1])):
                c = int(phase[ch])
                S[c, o] += tok[ch].astype(np.int64)
                n[c, o] += 1
        for c in range(n_phases):
            if n[c, 1] == 0 or n[c, 0] == 0:
                continue
            acc = 0.0
            for dim in range(ACT_DIM):
                m_succ = float(S[c, 1, dim]) / float(n[c, 1])
                m_fail = float(S[c, 0, dim]) / float(n[c, 0])
                diff = m_succ - m_fail
                acc = acc + diff * diff
            C_group[g, c] = math.sqrt(acc) * BIN_WIDTH
            valid_group[g, c] = 1
    C = np.zeros(n_phases, dtype=np.float64)
    valid = np.zeros(n_phases, dtype=np.uint8)
    n_valid = np.zeros(n_phases, dtype=np.int32)
    for c in range(n_phases):
        s = 0.0
        cnt = 0
        for g in range(n_groups):
            if valid_group[g, c]:
                s = s + C_group[g, c]
                cnt += 1
        n_valid[c] = cnt
        if cnt > 0:
            C[c] = s / float(cnt)
            valid[c] = 1
    return C, valid, n_valid, C_group, valid_group


ACT_FIX_BITS = 32            # continuous actions are summed as integers in units of 2^-32
ACT_ABS_MAX = 4096.0         # |a| bound that keeps every sum below 2^63 for up to 2^18 chunks per group


def score_phases_float(traj_off, act, phase, reward, G: int, n_phases: int):
    """Eq. 5 on continuous chunk actions: act is float32 [n_chunks, 56] (the 7-DoF x 8-step action of each
    chunk as the policy emitted it, before or instead of tokenisation).

    Same groups, skip rules and reductions as score_phases.  So that the result does not depend on
    the order of a floating-point sum, every action value is first read as the integer
    round-half-even(a * 2^32) (exact for |a| >= 2^-9 in float32, off by at most 2^-33 below), the sums over
    chunks are exact integers, and the means, differences, squares, the ascending-dimension sum and the
    square root are individually rounded fp64 operations; the unit 2^-32 is applied once at the end.
    A value that is not finite or exceeds ACT_ABS_MAX in magnitude is counted as 0 and reported in `bad`.

    Returns (C, valid, n_valid_groups, C_group, valid_group, bad) with the shapes of score_phases.
    """
    traj_off = np.asarray(traj_off)
    act = np.asarray(act, dtype=np.float32)
    n_groups = (traj_off.size - 1) // G
    C_group = np.zeros((n_groups, n_phases), dtype=np.float64)
    valid_group = np.zeros((n_groups, n_phases), dtype=np.uint8)
    unit = 2.0 ** (-ACT_FIX_BITS)
    bad = 0
    for g in range(n_groups):
        S = [[[0] * ACT_DIM for _ in range(2)] for _ in range(n_phases)]      # Python ints: exact
        n = [[0, 0] for _ in range(n_phases)]
        for i in range(g * G, (g + 1) * G):
            o = 1 if reward[i] else 0
            for ch in range(int(traj_off[i]), int(traj_off[i + 1])):
                c = int(phase[ch])
                row = act[ch]
                for dim in range(ACT_DIM):
                    a = float(row[dim])
                    if not (abs(a) <= ACT_ABS_MAX):                           # also catches NaN
                        bad += 1
                        continue
                    S[c][o][dim] += int(round(a * 4294967296.0))              # a * 2^32 is exact in fp64
                n[c][o] += 1
        for c in range(n_phases):
            if n[c][1] == 0 or n[c][0] == 0:
                continue
            acc = 0.0
            for dim in range(ACT_DIM):
                diff = float(S[c][1][dim]) / float(n[c][1]) - float(S[c][0][dim]) / float(n[c][0])
                acc = acc + diff * diff
            C_group[g, c] = math.sqrt(acc) * unit
            valid_group[g, c] = 1
    C = np.zeros(n_phases, dtype=np.float64)
    valid = np.zeros(n_phases, dtype=np.uint8)
    n_valid = np.zeros(n_phases, dtype=np.int32)
    for c in range(n_phases):
        s = 0.0
        cnt = 0
        for g in range(n_groups):
            if valid_group[g, c]:
                s = s + C_group[g, c]
                cnt += 1
        n_valid[c] = cnt
        if cnt > 0:
            C[c] = s / float(cnt)
            valid[c] = 1
    return C, valid, n_valid, C_group, valid_group, bad


# ----------------------------------------------------------------------------------------------
# Eq. 7-9, Algorithm 1 - online keep-probability update
# ----------------------------------------------------------------------------------------------
class KeepProbState:
    """Phase-score buffers B_c, the step counter and the current keep-probabilities p_c."""

    def __init__(self, n_phases: int, p_min: float = 0.1, t_rc: int = 5, mode: int = 0):
        self.mode = int(mode)              # 0 PCM (Eq. 8-9); 1 random masking; 2 full masking (ablations of RQ4)
        self.n_phases = n_phases
        self.p_min = float(p_min)
        self.t_rc = int(t_rc)
        self.buf: List[List[float]] = [[] for _ in range(n_phases)]
        self.step = 0
        self.p = [1.0] * n_phases          # value before the first refresh (never used: step 0 refreshes)
        self.n_refresh = 0


def update_keep_probs(state: KeepProbState, C: Sequence[float], valid: Sequence[int]):
    """Append C^(t) to the buffers (Eq. 7); on the first batch or when the buffer holds T_rc
    entries, collapse to S_c, max-normalise the shares (Eq. 8), floor at p_min (Eq. 9) and clear
    the buffers (Algorithm 1); otherwise p_c is unchanged.

    Eq. 8 is followed literally: S_c, then the share rho_c = S_c / sum S (sum in ascending c), then
    rho~_c = rho_c / max rho.  A phase skipped in a step contributes 0 to its sum.  When every
    S_c is zero (0/0 in Eq. 8) the previous p_c is kept.  Returns (p float64[K], q int64[K],
    refreshed) where q_c = round-half-even(p_c * 2^24) is the integer weight the sampler uses.
    """
    K = state.n_phases
    for c in range(K):
        state.buf[c].append(float(C[c]) if valid[c] else 0.0)
    refreshed = False
    if state.step == 0 or len(state.buf[0]) == state.t_rc:
        S = [0.0] * K
        for c in range(K):
            s = 0.0
            for v in state.buf[c]:
                s = s + v
            S[c] = s
        s_tot = 0.0
        for c in range(K):
            s_tot = s_tot + S[c]
        if state.mode == 1:
            pass                                     # random masking: every phase keeps weight 1 (uniform sampling)
        elif s_tot > 0.0:
            rho = [S[c] / s_tot for c in range(K)]
            rho_max = 0.0
            c_max = 0
            for c in range(K):
                if rho[c] > rho_max:
                    rho_max = rho[c]
                    c_max = c
            for c in range(K):
                if state.mode == 2:                  # full masking: only the single highest-C_c phase survives
                    state.p[c] = 1.0 if c == c_max else 0.0
                else:
                    rho_t = rho[c] / rho_max
                    state.p[c] = rho_t if rho_t > state.p_min else state.p_min
        for c in range(K):
            state.buf[c] = []
        refreshed = True
        state.n_refresh += 1
    state.step += 1
    p = np.array(state.p, dtype=np.float64)
    q = np.array([int(round(pc * Q_ONE)) for pc in state.p], dtype=np.int64)  # round(): half to even
    return p, q, refreshed


# ----------------------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11)
# ----------------------------------------------------------------------------------------------
_PHILOX_M0 = 0xD2511F53
_PHILOX_M1 = 0xCD9E8D57
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_M32 = 0xFFFFFFFF


def philox4x32_10(ctr: Sequence[int], key: Sequence[int]) -> Tuple[int, int, int, int]:
    c0, c1, c2, c3 = (int(x) & _M32 for x in ctr)
    k0, k1 = (int(x) & _M32 for x in key)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> 32, p0 & _M32
        hi1, lo1 = p1 >> 32, p1 & _M32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0) & _M32, lo1, (hi0 ^ c3 ^ k1) & _M32, lo0
        k0 = (k0 + _PHILOX_W0) & _M32
        k1 = (k1 + _PHILOX_W1) & _M32
    return c0, c1, c2, c3


def draw_bits(seed: int, it: int, traj: int, draw: int) -> int:
    """64 random bits for draw number `draw` of trajectory `traj` at iteration `it`.
    key = (seed low, seed high); counter = (it low, traj, draw, it high)."""
    o = philox4x32_10((it & _M32, traj, draw, (it >> 32) & _M32), (seed & _M32, (seed >> 32) & _M32))
    return o[0] | (o[1] << 32)


# ----------------------------------------------------------------------------------------------
# Eq. 10 - fixed-budget weighted sampling without replacement
# ----------------------------------------------------------------------------------------------
def sample_one_trajectory(weights: Sequence[int], m: int, bits: Sequence[int]) -> List[int]:
    """Successive (Plackett-Luce) sampling: m times, pick a remaining chunk with probability
    proportional to its integer weight and remove it (chunks of weight 0 are never picked; the caller
    passes m <= number of positive weights).  Draw r maps its 64 random bits to
    x = floor(bits * W_remaining / 2^64) and selects the first remaining chunk, in index order,
    whose running weight sum exceeds x.  Returns the kept chunk positions in ascending order."""
    w = [int(v) for v in weights]
    kept = []
    W = sum(w)                      # total weight of the chunks still available
    for r in range(m):
        x = (int(bits[r]) * W) >> 64
        run = 0
        pick = -1
        for k, wk in enumerate(w):
            if wk == 0:
                continue
            run += wk
            if run > x:
                pick = k
                break
        kept.append(pick)
        W -= w[pick]
        w[pick] = 0
    return sorted(kept)


def sample_chunks(traj_off, phase, q, budget: int, seed: int, it: int):
    """Eq. 10 for every trajectory: |K_i| = min(B, N_i) chunks with weights w_ik = q[phi(i,k)].

    Returns kept_idx int32[n_kept] (global chunk ids, trajectory-major, ascending within a
    trajectory), kept_off int32[n_traj+1], kept_per_phase int32[K]."""
    traj_off = np.asarray(traj_off)
    n_traj = traj_off.size - 1
    kept_idx: List[int] = []
    kept_off = np.zeros(n_traj + 1, dtype=np.int32)
    kept_per_phase = np.zeros(len(q), dtype=np.int32)
    for i in range(n_traj):
        a, b = int(traj_off[i]), int(traj_off[i + 1])
        weights = [int(q[int(phase[ch])]) for ch in range(a, b)]
        m = min(budget, sum(1 for wk in weights if wk > 0))      # |K_i| = min(B, N_i) over the chunks that can be kept
        bits = [draw_bits(seed, it, i, r) for r in range(m)]
        for k in sample_one_trajectory(weights, m, bits):
            kept_idx.append(a + k)
            kept_per_phase[int(phase[a + k])] += 1
        kept_off[i + 1] = len(kept_idx)
    return np.array(kept_idx, dtype=np.int32), kept_off, kept_per_phase


# ----------------------------------------------------------------------------------------------
# physical shrinking (Sec. 4.5, Algorithm 1): dense batch of the kept chunks only
# ----------------------------------------------------------------------------------------------
def pack_chunks(obs_of_chunk, tok, logp_old, adv, traj_off, kept_idx, e_act):
    """X[j] = [obs prefix of chunk kept_idx[j] ; E_act[token] for its 56 action tokens]; targets,
    old log-probs and the owning trajectory's advantage are gathered alongside.

    obs_of_chunk(c) returns the [P, d] prefix of global chunk c.  Returns X [n, S, d] (dtype of
    e_act), tgt uint8[n,56], lpo [n,56], adv_c [n], src int32[n]."""
    traj_off = np.asarray(traj_off)
    n = len(kept_idx)
    rows = []
    tgt = np.zeros((n, ACT_DIM), dtype=np.uint8)
    lpo = np.zeros((n, ACT_DIM), dtype=np.asarray(logp_old).dtype)
    adv_c = np.zeros(n, dtype=np.asarray(adv).dtype)
    src = np.zeros(n, dtype=np.int32)
    for j, c in enumerate(kept_idx):
        c = int(c)
        i = int(np.searchsorted(traj_off, c, side="right")) - 1
        emb = np.stack([e_act[int(t)] for t in tok[c]])
        rows.append(np.concatenate([np.asarray(obs_of_chunk(c)), emb], axis=0))
        tgt[j] = tok[c]
        lpo[j] = logp_old[c]
        adv_c[j] = adv[i]
        src[j] = c
    X = np.stack(rows) if rows else np.zeros((0, 0, 0))
    return X, tgt, lpo, adv_c, src
