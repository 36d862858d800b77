"""Data-parallel actor update on CPU (gloo, world size 2): the kept chunks of ONE selection are dealt out by
trajectory, every rank differentiates its share under the global loss scale, and one all-reduce of the flat
gradient buffer must give the full-batch gradient (Eq. 11 is a sum over kept chunks).  The per-rank update is the
oracle's here: what is under test is the partition and the reduction, which is all the multi-GPU path adds."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_16154_b200 import dist_util, synth


def _problem():
    from oracle import pcm_oracle as po
    w = synth.WORKLOADS["C0"].with_(n_tasks=2, d=32, L=1, H=1, P=6, budget=3, gamma_std=0.1)
    rb = synth.make_rollouts(w, 3)
    weights = synth.make_weights(w, 3)
    adv = po.advantages(rb["reward"], w.G, 1e-6).astype(np.float32)
    C, valid, _, _, _ = po.score_phases(rb["traj_off"], rb["tok"], rb["phase"], rb["reward"], w.G, w.n_phases)
    _, q, _ = po.update_keep_probs(po.KeepProbState(w.n_phases, w.p_min, w.t_rc), C, valid)
    kept, off, _ = po.sample_chunks(rb["traj_off"], rb["phase"], q, w.budget, 9, 0)
    return w, rb, weights, adv, kept, off


def _grads_for(w, rb, weights, adv, kept, off, scale):
    from oracle import actor_oracle as ao
    from oracle import pcm_oracle as po
    obs = {int(c): synth.obs_chunk(w, 3, int(c)) for c in kept}
    total = int(rb["traj_off"][-1])
    lpo_all = (-np.log(256.0) + synth.logp_noise(3, total, 0.2)).astype(np.float32)
    X, tgt, lpo, adv_c, _ = po.pack_chunks(lambda c: obs[c], rb["tok"], lpo_all, adv, rb["traj_off"], kept, weights["e_act"])
    loss, _, grads, _ = ao.fwd_bwd(weights, X, tgt, lpo, adv_c, w.H, w.P, 0.2, 0.2, scale)
    return loss, grads


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w, rb, weights, adv, kept, off = _problem()                       # every rank sees the same batch and selection
    idx_l, off_l = dist_util.partition_kept(torch.from_numpy(kept.astype(np.int32)), torch.from_numpy(off.astype(np.int32)),
                                            rank, world)
    lengths = np.diff(rb["traj_off"])
    assert idx_l.numel() == dist_util.local_kept_count(lengths, w.budget, rank, world) == int(off_l[-1])
    scale = 1.0 / (56 * len(kept))                                    # the global scale, not the share's
    loss, grads = _grads_for(w, rb, weights, adv, idx_l.numpy(), off_l.numpy(), scale)
    names = sorted(grads)
    flat = torch.cat([torch.from_numpy(np.ascontiguousarray(grads[k])).reshape(-1) for k in names] + [torch.tensor([loss], dtype=torch.float64)])
    dist_util.allreduce_sum(flat)
    out[rank] = (idx_l.numpy().copy(), off_l.numpy().copy(), flat.numpy().copy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_partition_by_trajectory_and_one_allreduce_gives_the_full_gradient():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29700 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    w, rb, weights, adv, kept, off = _problem()
    # the shares are disjoint, cover the selection, keep the order, and follow trajectory parity
    i0, o0, f0 = out[0]
    i1, o1, f1 = out[1]
    assert sorted(np.concatenate([i0, i1]).tolist()) == sorted(kept.tolist())
    owner = np.searchsorted(rb["traj_off"], kept, side="right") - 1
    assert np.array_equal(i0, kept[owner % 2 == 0]) and np.array_equal(i1, kept[owner % 2 == 1])
    assert np.array_equal(np.diff(o0) + np.diff(o1), np.diff(off))
    assert np.all(np.diff(o0)[1::2] == 0) and np.all(np.diff(o1)[0::2] == 0)
    # both ranks hold the same reduced buffer, equal to the single-process full-batch update
    assert np.array_equal(f0, f1)
    loss, grads = _grads_for(w, rb, weights, adv, kept, off, 1.0 / (56 * len(kept)))
    expect = np.concatenate([np.ascontiguousarray(grads[k]).reshape(-1) for k in sorted(grads)] + [np.array([loss])])
    assert np.allclose(f0, expect, rtol=1e-10, atol=1e-14)


def test_partition_without_a_process_group_is_the_identity_for_one_rank():
    kept = torch.tensor([3, 5, 9, 12, 13, 20], dtype=torch.int32)
    off = torch.tensor([0, 2, 2, 5, 6], dtype=torch.int32)
    idx, off_l = dist_util.partition_kept(kept, off, 0, 1)
    assert torch.equal(idx, kept) and torch.equal(off_l, off)
    idx, off_l = dist_util.partition_kept(kept, off, 1, 3)             # trajectories 1 (empty) and none other < 4 -> 1 only
    assert idx.numel() == 0 and off_l.tolist() == [0, 0, 0, 0, 0]
    idx, off_l = dist_util.partition_kept(kept, off, 0, 3)             # trajectories 0 and 3
    assert idx.tolist() == [3, 5, 20] and off_l.tolist() == [0, 2, 2, 2, 3]
    t = torch.ones(4)
    assert dist_util.allreduce_sum(t) is t
