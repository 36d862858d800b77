"""Phase labelling on the device against the oracle: bit-exact labels on random gripper traces."""
import numpy as np
import pytest
import torch

from oracle import label_oracle as lo

pytestmark = pytest.mark.gpu


def _random_traces(rng, n_traj):
    """Piecewise-constant close commands with noise: approach, closing ramp, hold, release, sometimes twice."""
    steps, off = [], [0]
    for _ in range(n_traj):
        T = int(rng.integers(1, 700))
        g = np.zeros(T, dtype=np.uint8)
        for _ in range(int(rng.integers(0, 3))):
            s = int(rng.integers(0, T)); e = min(T, s + int(rng.integers(1, 200)))
            g[s:e] = 1
        flip = rng.random(T) < 0.08
        g = np.where(flip, 1 - g, g).astype(np.uint8)
        steps.append(g)
        off.append(off[-1] + T)
    return np.concatenate(steps), np.array(off, dtype=np.int32)


@pytest.mark.parametrize("chunk_len", [8, 5])
def test_labels_bit_exact(chunk_len):
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    rng = np.random.default_rng(chunk_len)
    grip, step_off = _random_traces(rng, 96)
    ph_o, traj_off = lo.label_phases(step_off, grip, chunk_len)
    assert set(np.unique(ph_o)) == {0, 1, 2, 3, 4}                 # every phase occurs in the sample
    ctx = B.Context(5, 12, 8, max_traj=96)
    ph = B.pcm_label_phases(ctx, PL.dev(traj_off), PL.dev(step_off), PL.dev(grip), chunk_len)
    assert B.pcm_poll_status(ctx) == 0
    assert np.array_equal(ph.cpu().numpy(), ph_o)
    # chunk offsets that do not match ceil(T / chunk_len) are reported, not read out of bounds
    bad = traj_off.copy()
    bad[1:] += 1
    B.pcm_label_phases(ctx, PL.dev(bad), PL.dev(step_off), PL.dev(grip), chunk_len,
                       phase=torch.zeros(int(bad[-1]), dtype=torch.uint8, device="cuda"))
    assert B.pcm_poll_status(ctx) == -7
    ctx.close()
