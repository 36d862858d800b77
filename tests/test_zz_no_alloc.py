"""The allocation-free scoring entry point against the ordinary one.

Some callers may not allocate device memory while they run: a training or serving loop whose memory
plan is frozen, a control thread beside the robot that must not block on the allocator, a plugin that
only receives pointers.  pcm_score_phases_static serves them from a fixed scratch array inside the
library.  Here it is called twice in a row through the C ABI, on two different batches (the second
smaller, so stale contents of the shared scratch would show), and must reproduce pcm_score_phases
and the CPU oracle bit for bit - the same bar the other scoring tests use.  Collected last on purpose: a run that stops
at the first failure has then already executed every other test."""
import numpy as np
import pytest
import torch

from oracle import pcm_oracle as po
from paper_2605_16154_b200 import synth

pytestmark = pytest.mark.gpu


def test_static_scoring_matches_context_scoring_twice_in_a_row():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    dev = torch.device("cuda")
    for name, seed in (("C3", 5), ("C4", 6)):            # 16 groups of 8, then 8 groups of 16 (ragged)
        w = synth.WORKLOADS[name]
        rb = synth.make_rollouts(w, seed)
        batch = PL.upload_rollouts(w, rb)
        ctx = B.Context(w.n_phases, w.budget, w.G, max_traj=w.n_traj)
        C_ref, valid_ref, nvalid_ref, adv_ref = B.pcm_score_phases(ctx, batch)
        out = {"C": torch.full((w.n_phases,), -1.0, dtype=torch.float64, device=dev),
               "valid": torch.full((w.n_phases,), 7, dtype=torch.uint8, device=dev),
               "n_valid": torch.full((w.n_phases,), -1, dtype=torch.int32, device=dev),
               "adv": torch.full((w.n_traj,), 9.0, dtype=torch.float32, device=dev),
               "status": torch.full((1,), 77, dtype=torch.int32, device=dev)}
        before = torch.cuda.memory_allocated()
        B.pcm_score_phases_static(w.n_phases, w.G, 1e-6, batch, out)
        torch.cuda.synchronize()
        assert torch.cuda.memory_allocated() == before                # the call created no tensor
        assert int(out["status"].item()) == 0
        assert np.array_equal(out["C"].cpu().numpy().view(np.uint64), C_ref.cpu().numpy().view(np.uint64))
        assert torch.equal(out["valid"], valid_ref) and torch.equal(out["n_valid"], nvalid_ref)
        assert np.array_equal(out["adv"].cpu().numpy().view(np.uint32), adv_ref.cpu().numpy().view(np.uint32))
        # and against the CPU oracle: the two entry points share a kernel, so a fault common to both would pass above
        C_o, valid_o, nvalid_o, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
        adv_o = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
        assert np.array_equal(out["C"].cpu().numpy().view(np.uint64), np.asarray(C_o, dtype=np.float64).view(np.uint64))
        assert np.array_equal(out["valid"].cpu().numpy(), np.asarray(valid_o, dtype=np.uint8))
        assert np.array_equal(out["n_valid"].cpu().numpy(), np.asarray(nvalid_o, dtype=np.int32))
        assert np.array_equal(out["adv"].cpu().numpy().view(np.uint32), adv_o.view(np.uint32))
        ctx.close()


def test_static_scoring_rejects_batches_beyond_its_scratch_and_reports_bad_labels():
    from paper_2605_16154_b200 import binding as B, pipeline as PL
    dev = torch.device("cuda")
    w = synth.WORKLOADS["C0"]
    rb = synth.make_rollouts(w)
    out = {"C": torch.zeros(w.n_phases, dtype=torch.float64, device=dev),
           "valid": torch.zeros(w.n_phases, dtype=torch.uint8, device=dev),
           "status": torch.zeros(1, dtype=torch.int32, device=dev)}
    batch = PL.upload_rollouts(w, rb)
    batch.n_traj = (B.STATIC_MAX_GROUPS + 1) * w.G                   # more groups than the scratch holds
    with pytest.raises(B.PcmError) as e:
        B.pcm_score_phases_static(w.n_phases, w.G, 1e-6, batch, out)
    assert e.value.code == -2
    bad = dict(rb)
    bad["phase"] = rb["phase"].copy()
    bad["phase"][3] = 31
    B.pcm_score_phases_static(w.n_phases, w.G, 1e-6, PL.upload_rollouts(w, bad), out)
    assert int(out["status"].item()) != 0
    B.pcm_score_phases_static(w.n_phases, w.G, 1e-6, PL.upload_rollouts(w, rb), out)
    assert int(out["status"].item()) == 0                            # cleared at the start of every call
