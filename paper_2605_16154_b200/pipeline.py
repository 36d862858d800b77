"""Host-side glue: uploads synthetic inputs and chains the C-ABI calls of one iteration.

Argument marshalling only; nothing here computes any step of the method.
"""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as B
from . import synth


def dev(a: np.ndarray, dtype=None) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def model_dtype(w: synth.Workload) -> int:
    return B.GRPO_BF16 if w.dtype == "bf16" else B.GRPO_F32


def torch_dtype(w: synth.Workload):
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def upload_model(w: synth.Workload, weights: Dict[str, np.ndarray]) -> B.Model:
    """Weights hold values exactly representable in the workload dtype, so the cast is exact."""
    td = torch_dtype(w)
    return B.Model(w.d, w.L, w.H, w.P, model_dtype(w), {k: dev(v, td) for k, v in weights.items()})


def upload_rollouts(w: synth.Workload, rb: Dict[str, np.ndarray], obs: Optional[torch.Tensor] = None,
                    logp_old: Optional[torch.Tensor] = None) -> B.pcm_batch:
    lengths = np.diff(rb["traj_off"])
    return B.make_batch(dev(rb["traj_off"]), dev(rb["tok"]), dev(rb["phase"]), dev(rb["reward"]),
                        max(1, int(lengths.max())) if lengths.size else 1, obs, logp_old)


def n_kept_of(budget: int, traj_off: np.ndarray) -> int:
    return int(np.minimum(np.diff(traj_off), budget).sum())


def select(ctx: B.Context, batch: B.pcm_batch, it: int):
    """Eq. 1, 5, 7-10: returns (adv, C, valid, p, q, kept_idx, kept_off, kept_per_phase)."""
    Cc, valid, _, adv = B.pcm_score_phases(ctx, batch)
    p, q = B.pcm_update_keep_probs(ctx, Cc, valid)
    kept_idx, kept_off, per_phase = B.pcm_sample_chunks(ctx, batch, q, it)
    return adv, Cc, valid, p, q, kept_idx, kept_off, per_phase


def upload_lora(w: synth.Workload, model: B.Model, lora: Dict) -> B.Lora:
    td = torch_dtype(w)
    return B.Lora(model, int(lora["rank"]), float(lora["alpha"]), {k: dev(lora[k], td) for k in synth.LORA_NAMES})
