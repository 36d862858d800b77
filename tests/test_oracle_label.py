"""Pins for the phase-labelling oracle: gripper traces labelled by hand from the rule's text."""
import numpy as np

from oracle import label_oracle as lo

A, P, G, R, T = lo.APPROACH, lo.PRE_GRASP, lo.ACTIVE_GRIP, lo.RELEASE_RAMP, lo.TAIL


def _trace(fracs, L=8):
    """A per-timestep close-command trace whose chunk j has close fraction fracs[j] (multiples of 1/8)."""
    out = []
    for f in fracs:
        n = int(round(f * L))
        out += [1] * n + [0] * (L - n)
    return out


def _labels(fracs):
    return lo.label_trajectory(lo.chunk_counts(_trace(fracs), 8))


def test_single_grasp_cycle():
    #        open  open  .25   .375  1     1     .875  .5    .25   0     0     0     0
    fr = [0, 0, .25, .375, 1, 1, .875, .5, .25, 0, 0, 0, 0]
    # chunks 2,3: closing begun right before sustained closure -> pre-grasp; 4..6 sustained, 7 (>= 0.5) active;
    # the release window is chunks 7,8,9: 7 stays active-grip (priority), 8 and 9 (below 0.5) -> release-ramp;
    # 10.. open after the final release window -> tail
    assert _labels(fr) == [A, A, P, P, G, G, G, G, R, R, T, T, T]


def test_release_ramp_and_tail():
    fr = [0, .125, 1, 1, .25, 0, 0, 0, 0]
    # 1: 0.125 >= 0.1 directly before the interval -> pre-grasp; 4,5,6: three chunks after it below 0.5 -> release;
    # 7,8: open after the final release window -> tail
    assert _labels(fr) == [A, P, G, G, R, R, R, T, T]


def test_pre_grasp_window_is_at_most_three_and_needs_partial_closure():
    fr = [.25, .25, .25, .25, .25, 1, 0]
    # only the three chunks next to the interval; the earlier half-open chunks are approach
    assert _labels(fr) == [A, A, P, P, P, G, R]
    fr = [.25, 0, .25, 1]
    # the window is chunks 0..2; the fully open chunk 1 does not qualify (needs >= 0.1)
    assert _labels(fr) == [P, A, P, G]


def test_two_grasps_priorities_between_windows():
    fr = [0, 1, .25, .25, 1, 0, 0, 0, 0, .625, 0]
    # chunks 2,3 lie after grasp 1 (release window) and before grasp 2 (pre-grasp window): pre-grasp wins;
    # 5,6,7 release after the last sustained interval; 8 open -> tail; 9 (0.625) active-grip by the softer
    # threshold although not sustained; 10 open after the last sustained interval -> tail
    assert _labels(fr) == [A, G, P, P, G, R, R, R, T, G, T]


def test_no_grasp_at_all_and_partial_last_chunk():
    assert _labels([0, .25, 0, .375]) == [A, A, A, A]
    # 19 timesteps = 2 full chunks + 3 steps; the last chunk's fraction is 3/3
    trace = [0] * 8 + [1, 1, 0, 0, 0, 0, 0, 0] + [1, 1, 1]
    counts = lo.chunk_counts(trace, 8)
    assert counts == [(0, 8), (2, 8), (3, 3)]
    assert lo.label_trajectory(counts) == [A, P, G]


def test_csr_interface():
    t1, t2 = _trace([0, 1, 0]), _trace([.25, 1])
    ph, off = lo.label_phases(np.array([0, len(t1), len(t1) + len(t2)]), np.array(t1 + t2, dtype=np.uint8), 8)
    assert list(off) == [0, 3, 5] and list(ph) == [A, G, R, P, G]
