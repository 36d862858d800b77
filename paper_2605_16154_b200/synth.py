"""Seeded synthetic rollouts, observations and weights.

This module only *draws data*: rewards, trajectory lengths, phase labels, action tokens,
observation-prefix embeddings, model weights and log-prob noise.  It holds none of the method's
arithmetic (no advantages, scores, keep-probabilities, sampling, packing, forward or backward) so
that both the CPU oracle and the CUDA path can be fed from it without sharing any computation.

The shapes mirror the manipulation workloads the paper trains on: binary rewards, groups of G
rollouts per task, chunks of 8 actions x 7 degrees of freedom = 56 action tokens over 256 bins,
trajectories of tens to hundreds of chunks partitioned into a handful of phases, with success and
failure behaviour diverging in one or two phases only (Sec. 5.1, App. E, Fig. 1).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, Optional

import numpy as np

ACT_DIM = 56      # 8 actions x 7 DoF per chunk (Sec. 5.1)
N_BINS = 256      # action-token vocabulary


@dataclass(frozen=True)
class Workload:
    name: str
    n_tasks: int
    G: int                      # rollouts per group
    n_phases: int               # the paper's K
    budget: int                 # the paper's B (kept chunks per trajectory)
    P: int                      # observation-prefix tokens per chunk
    d: int
    L: int
    H: int
    dtype: str                  # "f32" | "bf16"
    p_succ: float
    T: int = 0                  # fixed chunks per trajectory (0 => ragged)
    len_lo: int = 0
    len_hi_succ: int = 0
    len_hi_fail: int = 0
    n_div_phases: int = 2       # phases in which failures diverge
    div_phase_fixed: int = -1   # >=0: that phase index diverges in every task
    shift_lo: float = 0.3
    shift_hi: float = 1.0
    phase_cuts: str = "equal"   # "equal" | "random"
    force_mixed: bool = False   # redraw rewards until every group has both outcomes
    seed: int = 1
    p_min: float = 0.1
    t_rc: int = 5
    eps_low: float = 0.2
    eps_high: float = 0.2
    gamma_std: float = 0.0      # RMSNorm gain jitter around 1 (tests use > 0)

    @property
    def n_traj(self) -> int:
        return self.n_tasks * self.G

    @property
    def S(self) -> int:
        return self.P + ACT_DIM

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # Tiny fp32 case: 1 task, G=8, 16 chunks in 4 equal phases, failures shifted by 0.5 in phase 2.
    "C0": Workload("C0", n_tasks=1, G=8, n_phases=4, budget=3, P=32, d=128, L=2, H=4, dtype="f32",
                   p_succ=0.5, T=16, n_div_phases=1, div_phase_fixed=2, shift_lo=0.5, shift_hi=0.5,
                   force_mixed=True, seed=0),
    # Medium bf16 case the headline metric is quoted on.
    "C1": Workload("C1", n_tasks=4, G=8, n_phases=8, budget=12, P=256, d=1024, L=8, H=16,
                   dtype="bf16", p_succ=0.4, T=64, seed=1),
    # Same model and data, mask keeps all 64 chunks (plain GRPO actor update).
    "C2": Workload("C2", n_tasks=4, G=8, n_phases=8, budget=64, P=256, d=1024, L=8, H=16,
                   dtype="bf16", p_succ=0.4, T=64, seed=1),
    # Large bf16 case.
    "C3": Workload("C3", n_tasks=16, G=8, n_phases=10, budget=24, P=256, d=2048, L=24, H=16,
                   dtype="bf16", p_succ=0.3, T=128, seed=1),
    # Ragged and skewed: lengths 40..200 (successes stop by 120), divergence in one phase.
    "C4": Workload("C4", n_tasks=8, G=16, n_phases=10, budget=16, P=256, d=1024, L=8, H=16,
                   dtype="bf16", p_succ=0.4, len_lo=40, len_hi_succ=120, len_hi_fail=200,
                   n_div_phases=1, phase_cuts="random", seed=0),
}


# ----------------------------------------------------------------------------------------------
# bf16 <-> fp32 bit conversions (round to nearest even); storage helpers, not method arithmetic
# ----------------------------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array whose values are exactly representable in `dtype`."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x))
    return x


# ----------------------------------------------------------------------------------------------
# rollouts
# ----------------------------------------------------------------------------------------------
def make_rollouts(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    """One batch of rollouts in CSR form.

    Returns traj_off int32[n_traj+1], tok uint8[sum_N, 56], phase uint8[sum_N], reward uint8[n_traj].
    Draw order: rewards, lengths, phase cuts, phase means, divergence pattern, actions.
    """
    seed = w.seed if seed is None else seed
    rng = np.random.Generator(np.random.PCG64(seed))
    n_traj, G, Kc = w.n_traj, w.G, w.n_phases

    # rewards
    reward = (rng.random(n_traj) < w.p_succ).astype(np.uint8)
    if w.force_mixed:
        for g in range(w.n_tasks):
            while True:
                s = int(reward[g * G:(g + 1) * G].sum())
                if 0 < s < G:
                    break
                reward[g * G:(g + 1) * G] = (rng.random(G) < w.p_succ).astype(np.uint8)

    # lengths
    if w.T > 0:
        lengths = np.full(n_traj, w.T, dtype=np.int64)
    else:
        u = rng.random(n_traj)
        span = np.where(reward == 1, w.len_hi_succ - w.len_lo + 1, w.len_hi_fail - w.len_lo + 1)
        lengths = w.len_lo + np.floor(u * span).astype(np.int64)
    traj_off = np.zeros(n_traj + 1, dtype=np.int32)
    traj_off[1:] = np.cumsum(lengths)
    total = int(traj_off[-1])

    # phase labels (contiguous in time)
    phase = np.empty(total, dtype=np.uint8)
    for i in range(n_traj):
        n = int(lengths[i])
        k = np.arange(n)
        if w.phase_cuts == "equal":
            lab = (k * Kc) // n
        else:
            cuts = np.sort(rng.choice(np.arange(1, n), size=Kc - 1, replace=False))
            lab = np.searchsorted(cuts, k, side="right")
        phase[traj_off[i]:traj_off[i + 1]] = lab.astype(np.uint8)

    # per-task phase means and divergence pattern
    mu = rng.uniform(-0.3, 0.3, size=(w.n_tasks, Kc, ACT_DIM))
    shift = np.zeros((w.n_tasks, Kc))
    if w.div_phase_fixed >= 0:
        shift[:, w.div_phase_fixed] = rng.uniform(w.shift_lo, w.shift_hi, size=w.n_tasks)
    elif w.phase_cuts == "random":
        # skewed: one divergent phase shared by all tasks of this batch
        c = int(rng.integers(0, Kc))
        shift[:, c] = rng.uniform(w.shift_lo, w.shift_hi, size=w.n_tasks)
    else:
        for t in range(w.n_tasks):
            cs = rng.choice(Kc, size=w.n_div_phases, replace=False)
            shift[t, cs] = rng.uniform(w.shift_lo, w.shift_hi, size=w.n_div_phases)
    direction = rng.choice(np.array([-1.0, 1.0]), size=(w.n_tasks, Kc, ACT_DIM))

    # actions -> tokens
    tok = np.empty((total, ACT_DIM), dtype=np.uint8)
    for i in range(n_traj):
        t = i // G
        lab = phase[traj_off[i]:traj_off[i + 1]].astype(np.int64)
        a = mu[t, lab] + 0.1 * rng.standard_normal((lab.size, ACT_DIM))
        if reward[i] == 0:
            a = a + shift[t, lab][:, None] * direction[t, lab]
        tok[traj_off[i]:traj_off[i + 1]] = np.clip(np.floor((a + 1.0) * 128.0), 0, 255).astype(np.uint8)

    return {"traj_off": traj_off, "tok": tok, "phase": phase, "reward": reward}


# ----------------------------------------------------------------------------------------------
# observation prefixes: every chunk has its own counter-based stream, so any subset of chunks can
# be regenerated without materialising the rest
# ----------------------------------------------------------------------------------------------
def obs_chunk(w: Workload, seed: int, chunk_id: int) -> np.ndarray:
    """fp32 [P, d] prefix embeddings of one chunk, iid N(0,1) rounded to the workload dtype."""
    rng = np.random.Generator(np.random.Philox(key=[np.uint64(seed) + np.uint64(0x0B5), np.uint64(chunk_id)]))
    x = rng.standard_normal((w.P, w.d), dtype=np.float32)
    return round_to_dtype(x, w.dtype)


def obs_all(w: Workload, seed: int, n_chunks: int) -> np.ndarray:
    out = np.empty((n_chunks, w.P, w.d), dtype=np.float32)
    for c in range(n_chunks):
        out[c] = obs_chunk(w, seed, c)
    return out


# ----------------------------------------------------------------------------------------------
# weights: every linear weight is stored [out_features, in_features]
# ----------------------------------------------------------------------------------------------
WEIGHT_NAMES = ("w_qkv", "w_o", "w_gu", "w_d", "g1", "g2", "gf", "w_h", "e_act")


def weight_shapes(w: Workload) -> Dict[str, tuple]:
    d, L = w.d, w.L
    return {
        "w_qkv": (L, 3 * d, d),     # rows 0..d-1 query, d..2d-1 key, 2d..3d-1 value
        "w_o": (L, d, d),
        "w_gu": (L, 8 * d, d),      # rows 0..4d-1 gate, 4d..8d-1 up
        "w_d": (L, d, 4 * d),
        "g1": (L, d),
        "g2": (L, d),
        "gf": (d,),
        "w_h": (N_BINS, d),         # action head
        "e_act": (N_BINS, d),       # action-token embedding
    }


def make_weights(w: Workload, seed: Optional[int] = None) -> Dict[str, np.ndarray]:
    seed = w.seed if seed is None else seed
    rng = np.random.Generator(np.random.PCG64(seed + 7919))
    out = {}
    for name, shape in weight_shapes(w).items():
        if name in ("g1", "g2", "gf"):
            x = 1.0 + w.gamma_std * rng.standard_normal(shape, dtype=np.float32)
        else:
            x = 0.02 * rng.standard_normal(shape, dtype=np.float32)
        out[name] = round_to_dtype(x.astype(np.float32), w.dtype)
    return out


LORA_NAMES = ("a_qkv", "b_qkv", "a_o", "b_o", "a_gu", "b_gu", "a_d", "b_d")


def lora_shapes(w: Workload, rank: int) -> Dict[str, tuple]:
    """A [L, rank, in_features], B [L, out_features, rank] for the four linear maps of a layer."""
    d, L = w.d, w.L
    return {"a_qkv": (L, rank, d), "b_qkv": (L, 3 * d, rank), "a_o": (L, rank, d), "b_o": (L, d, rank),
            "a_gu": (L, rank, d), "b_gu": (L, 8 * d, rank), "a_d": (L, rank, 4 * d), "b_d": (L, d, rank)}


def make_lora(w: Workload, rank: int = 32, alpha: float = 32.0, seed: Optional[int] = None, b_std: float = 0.02):
    """Adapter tensors (App. E: rank 32, alpha 32).  A ~ N(0, 1/in_features), B ~ N(0, b_std^2): a fresh adapter
    has B = 0 (b_std = 0); a non-zero B stands for an adapter part-way through training."""
    seed = w.seed if seed is None else seed
    rng = np.random.Generator(np.random.PCG64(seed + 15485863))
    out = {"rank": rank, "alpha": float(alpha)}
    for name, shape in lora_shapes(w, rank).items():
        std = 1.0 / np.sqrt(shape[2]) if name.startswith("a_") else b_std
        out[name] = round_to_dtype((std * rng.standard_normal(shape, dtype=np.float32)).astype(np.float32), w.dtype)
    return out


def logp_noise(seed: int, n_chunks: int, sigma: float = 0.1) -> np.ndarray:
    """fp32 [n_chunks, 56] noise added to a policy's log-probs to stand in for the behaviour policy."""
    rng = np.random.Generator(np.random.PCG64(seed + 104729))
    return (sigma * rng.standard_normal((n_chunks, ACT_DIM))).astype(np.float32)
