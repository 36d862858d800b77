"""CPU oracle for the gripper-based phase labelling rule (Sec. 5.1 "Phase Labeling", App. E.2).

TEST INFRASTRUCTURE ONLY; shares no code with the CUDA path.

Parity status: pinned by hand-labelled gripper traces in tests/test_oracle_label.py (expected labels
worked out from the rule's text, not from this function).

Phases: 0 approach, 1 pre-grasp, 2 active-grip, 3 release-ramp, 4 tail.  g_f[j] is the fraction of
the chunk's timesteps with the gripper-close command active; it is compared through integer counts
(count / n >= 3/4  <=>  4 count >= 3 n, etc.) so that both sides take the same decisions.

Readings where the rule leaves room:
  * a sustained-close interval is a maximal run of chunks with g_f >= 0.75;
  * "up to three chunks immediately before / after": the three chunk positions next to the interval; each
    of them that meets the phase's own condition (pre-grasp 0.1 <= g_f < 0.5, release-ramp g_f < 0.5) is
    claimed, so a gripper that opens through 0.5 -> 0.25 -> 0 still yields a release ramp;
  * overlapping windows: active-grip > pre-grasp > release-ramp > approach > tail;
  * a chunk no rule has claimed is approach when a sustained interval starts later, tail when it lies after
    the last sustained interval and g_f < 0.1, and approach otherwise (e.g. a rollout that never grasps).
"""
from __future__ import annotations

from typing import List, Sequence

import numpy as np

APPROACH, PRE_GRASP, ACTIVE_GRIP, RELEASE_RAMP, TAIL = 0, 1, 2, 3, 4
_PRIORITY = {ACTIVE_GRIP: 4, PRE_GRASP: 3, RELEASE_RAMP: 2, APPROACH: 1, TAIL: 0}


def chunk_counts(grip_close: Sequence[int], chunk_len: int):
    """(count of close commands, number of timesteps) per chunk of a trajectory."""
    T = len(grip_close)
    out = []
    for k in range((T + chunk_len - 1) // chunk_len):
        seg = grip_close[k * chunk_len:(k + 1) * chunk_len]
        out.append((int(np.sum(np.asarray(seg) != 0)), len(seg)))
    return out


def label_trajectory(counts) -> List[int]:
    N = len(counts)
    ge = lambda j, num, den: den * counts[j][0] >= num * counts[j][1]     # g_f[j] >= num / den
    label = [None] * N

    def claim(j, ph):
        if label[j] is None or _PRIORITY[ph] > _PRIORITY[label[j]]:
            label[j] = ph

    for j in range(N):
        if ge(j, 1, 2):
            claim(j, ACTIVE_GRIP)
    # sustained-close intervals
    intervals = []
    j = 0
    while j < N:
        if ge(j, 3, 4):
            s = j
            while j + 1 < N and ge(j + 1, 3, 4):
                j += 1
            intervals.append((s, j))
        j += 1
    for s, e in intervals:
        for k in range(max(0, s - 3), s):
            if ge(k, 1, 10) and not ge(k, 1, 2):
                claim(k, PRE_GRASP)
        for k in range(e + 1, min(N, e + 4)):
            if not ge(k, 1, 2):
                claim(k, RELEASE_RAMP)
    last_start = intervals[-1][0] if intervals else -1
    last_end = intervals[-1][1] if intervals else -1
    for j in range(N):
        if label[j] is None:
            if j < last_start:
                label[j] = APPROACH
            elif last_end >= 0 and j > last_end and not ge(j, 1, 10):
                label[j] = TAIL
            else:
                label[j] = APPROACH
    return label


def label_phases(step_off, grip_close, chunk_len: int = 8):
    """All trajectories: step_off [n_traj+1] CSR offsets in timesteps.  Returns (phase uint8[sum N_i],
    traj_off int32[n_traj+1]) with N_i = ceil(T_i / chunk_len)."""
    phases, traj_off = [], [0]
    for i in range(len(step_off) - 1):
        lab = label_trajectory(chunk_counts(grip_close[int(step_off[i]):int(step_off[i + 1])], chunk_len))
        phases.extend(lab)
        traj_off.append(len(phases))
    return np.array(phases, dtype=np.uint8), np.array(traj_off, dtype=np.int32)
