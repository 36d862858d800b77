"""ctypes binding of libpcm_b200.so: the same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams come from torch); every step of the path
runs inside the library's kernels.  There is no CPU fallback: importing this module without the
compiled library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpcm_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2605_16154_b200.build` first "
                      "(there is no fallback path)")
_lib = C.CDLL(LIB_PATH)

ACT_DIM = 56
N_BINS = 256
GRPO_F32, GRPO_BF16 = 0, 1
GRPO_FWD_ONLY, GRPO_ACCUMULATE, GRPO_CHUNK_RATIO = 1, 2, 4
MASK_PCM, MASK_RANDOM, MASK_FULL = 0, 1, 2

STATUS_NAMES = {0: "PCM_OK", -1: "PCM_ERR_ARG", -2: "PCM_ERR_SHAPE", -3: "PCM_ERR_WORKSPACE", -4: "PCM_ERR_CUDA",
                -5: "PCM_ERR_DEVICE_TIMEOUT", -6: "PCM_ERR_STATE", -7: "PCM_ERR_DEVICE_DATA"}


class PcmError(RuntimeError):
    def __init__(self, call: str, code: int):
        super().__init__(f"{call} failed: {STATUS_NAMES.get(code, code)}")
        self.code = code


class pcm_config(C.Structure):
    _fields_ = [("n_phases", C.c_int32), ("budget", C.c_int32), ("group_size", C.c_int32), ("t_rc", C.c_int32),
                ("p_min", C.c_double), ("adv_eps", C.c_double), ("seed", C.c_uint64), ("mode", C.c_int32),
                ("reserved", C.c_int32)]


class pcm_batch(C.Structure):
    _fields_ = [("n_traj", C.c_int32), ("n_chunks", C.c_int32), ("max_len", C.c_int32), ("reserved", C.c_int32),
                ("traj_off", C.c_void_p), ("tok", C.c_void_p), ("phase", C.c_void_p), ("reward", C.c_void_p),
                ("obs", C.c_void_p), ("logp_old", C.c_void_p)]


class grpo_model_cfg(C.Structure):
    _fields_ = [("d", C.c_int32), ("n_layers", C.c_int32), ("n_heads", C.c_int32), ("prefix_len", C.c_int32),
                ("dtype", C.c_int32), ("reserved", C.c_int32)]


_WEIGHTS = ("w_qkv", "w_o", "w_gu", "w_d", "g1", "g2", "gf", "w_h", "e_act")


class grpo_model(C.Structure):
    _fields_ = [("cfg", grpo_model_cfg)] + [(n, C.c_void_p) for n in _WEIGHTS]


class grpo_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _WEIGHTS]


class grpo_packed(C.Structure):
    _fields_ = [("n_kept", C.c_int32), ("reserved", C.c_int32), ("X", C.c_void_p), ("tgt", C.c_void_p),
                ("lpo", C.c_void_p), ("adv_c", C.c_void_p), ("src", C.c_void_p)]


class grpo_loss_cfg(C.Structure):
    _fields_ = [("eps_low", C.c_float), ("eps_high", C.c_float), ("loss_scale", C.c_float), ("mb_chunks", C.c_int32),
                ("flags", C.c_uint32), ("entropy_coef", C.c_float)]


class grpo_stats(C.Structure):
    _fields_ = [("loss", C.c_float), ("clip_frac", C.c_float), ("mean_ratio", C.c_float), ("entropy", C.c_float),
                ("n_launches", C.c_int32), ("reserved", C.c_int32), ("workspace_high_water", C.c_uint64)]


_LORA = ("a_qkv", "b_qkv", "a_o", "b_o", "a_gu", "b_gu", "a_d", "b_d")


class grpo_lora(C.Structure):
    _fields_ = [("rank", C.c_int32), ("alpha", C.c_float)] + [(n, C.c_void_p) for n in _LORA]


class grpo_lora_grads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LORA]


class grpo_adamw_cfg(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("weight_decay", C.c_float), ("max_grad_norm", C.c_float)]


PROFILE_CLASSES = ("gemm", "attention", "rmsnorm", "elementwise", "loss", "embed_grad", "pack", "pcm_score", "pcm_sample",
                   "gemm_small")


class pcm_profile(C.Structure):
    _fields_ = [("ms", C.c_double * 10), ("flops", C.c_double * 10), ("bytes", C.c_double * 10),
                ("launches", C.c_int64 * 10)]


_P = C.c_void_p
_lib.pcm_create.argtypes = [C.POINTER(_P), C.POINTER(pcm_config), C.c_int32]
_lib.pcm_destroy.argtypes = [_P]
_lib.pcm_poll_status.argtypes = [_P, _P]
_lib.pcm_state_export.argtypes = [_P, _P, C.POINTER(C.c_size_t)]
_lib.pcm_state_import.argtypes = [_P, _P, C.c_size_t]
_lib.pcm_score_phases.argtypes = [_P, C.POINTER(pcm_batch), _P, _P, _P, _P, _P]
_lib.pcm_update_keep_probs.argtypes = [_P, _P, _P, _P, _P, _P]
_lib.pcm_sample_chunks.argtypes = [_P, C.POINTER(pcm_batch), _P, C.c_uint64, _P, _P, _P, _P]
_lib.grpo_pack_chunks.argtypes = [_P, C.POINTER(pcm_batch), C.POINTER(grpo_model_cfg), _P, _P, _P, _P,
                                  C.POINTER(grpo_packed), _P]
_lib.grpo_workspace_bytes.argtypes = [C.POINTER(grpo_model_cfg), C.c_int32, C.c_uint32]
_lib.grpo_workspace_bytes.restype = C.c_size_t
_lib.grpo_actor_fwd_bwd.argtypes = [C.POINTER(grpo_model), C.POINTER(grpo_packed), C.POINTER(grpo_loss_cfg),
                                    C.POINTER(grpo_grads), _P, _P, C.POINTER(grpo_stats), _P, C.c_size_t, _P]
_lib.grpo_lora_workspace_bytes.argtypes = [C.POINTER(grpo_model_cfg), C.c_int32, C.c_int32, C.c_uint32]
_lib.grpo_lora_workspace_bytes.restype = C.c_size_t
_lib.grpo_actor_fwd_bwd_lora.argtypes = [C.POINTER(grpo_model), C.POINTER(grpo_lora), C.POINTER(grpo_packed),
                                         C.POINTER(grpo_loss_cfg), C.POINTER(grpo_grads), C.POINTER(grpo_lora_grads), _P, _P,
                                         C.POINTER(grpo_stats), _P, C.c_size_t, _P]
_lib.grpo_actor_fwd_bwd_lora.restype = C.c_int
_lib.grpo_gemm.argtypes = [C.c_int32, C.c_int32, C.c_int32, _P, C.c_int64, C.c_int32, _P, C.c_int64, C.c_int32,
                           C.c_int32, _P, C.c_int64, C.c_int32, _P, C.c_int64, C.c_int32, _P]
_lib.grpo_attention.argtypes = [C.c_int32, _P, _P, _P, _P, _P, _P, C.c_int32, C.c_int32, C.c_int32, C.c_int32, _P]
_lib.pcm_score_phases_static.argtypes = [C.c_int32, C.c_int32, C.c_double, C.POINTER(pcm_batch), _P, _P, _P, _P, _P, _P]
_lib.pcm_score_phases_static.restype = C.c_int
_lib.pcm_score_phases_f32.argtypes = [_P, C.POINTER(pcm_batch), _P, _P, _P, _P, _P, _P]
_lib.pcm_score_phases_f32.restype = C.c_int
_lib.pcm_label_phases.argtypes = [_P, C.c_int32, _P, _P, _P, C.c_int32, _P, _P]
_lib.pcm_label_phases.restype = C.c_int
_lib.grpo_adamw_scratch_bytes.restype = C.c_size_t
_lib.grpo_adamw_step.argtypes = [C.POINTER(grpo_model_cfg), C.POINTER(grpo_adamw_cfg), C.c_int64, C.POINTER(grpo_model),
                                 C.POINTER(grpo_grads), C.POINTER(grpo_grads), C.POINTER(grpo_grads), C.POINTER(grpo_grads),
                                 _P, _P, C.c_size_t, _P]
_lib.grpo_adamw_step.restype = C.c_int
_lib.grpo_adamw_step_lora.argtypes = [C.POINTER(grpo_model_cfg), C.POINTER(grpo_adamw_cfg), C.c_int64, C.POINTER(grpo_lora),
                                      C.POINTER(grpo_lora_grads), C.POINTER(grpo_lora_grads), C.POINTER(grpo_lora_grads),
                                      C.POINTER(grpo_lora_grads), C.POINTER(grpo_model), C.POINTER(grpo_grads),
                                      C.POINTER(grpo_grads), C.POINTER(grpo_grads), C.POINTER(grpo_grads), C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]
_lib.grpo_adamw_step_lora.restype = C.c_int
_lib.pcm_launch_count.restype = C.c_int64
_lib.pcm_first_use_on_device.argtypes = [C.POINTER(C.c_uint64), C.c_int32]
_lib.pcm_first_use_on_device.restype = C.c_int32
_lib.pcm_profile_enable.argtypes = [C.c_int32]
_lib.pcm_profile_read.argtypes = [C.POINTER(pcm_profile)]
for _name in ("pcm_create", "pcm_destroy", "pcm_poll_status", "pcm_state_export", "pcm_state_import",
              "pcm_score_phases", "pcm_update_keep_probs", "pcm_sample_chunks", "grpo_pack_chunks",
              "grpo_actor_fwd_bwd", "grpo_gemm", "grpo_attention", "pcm_profile_enable", "pcm_profile_read"):
    getattr(_lib, _name).restype = C.c_int

EXPORTED = ("pcm_create", "pcm_destroy", "pcm_poll_status", "pcm_state_export", "pcm_state_import",
            "pcm_score_phases", "pcm_update_keep_probs", "pcm_sample_chunks", "grpo_pack_chunks",
            "grpo_workspace_bytes", "grpo_actor_fwd_bwd", "grpo_gemm", "grpo_attention", "pcm_launch_count",
            "pcm_profile_enable", "pcm_profile_read", "pcm_score_phases_static",
            "grpo_adamw_scratch_bytes", "grpo_adamw_step", "grpo_adamw_step_lora", "pcm_label_phases", "pcm_score_phases_f32",
            "grpo_attention_wait_status", "pcm_first_use_on_device", "grpo_lora_workspace_bytes",
            "grpo_actor_fwd_bwd_lora")


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(call: str, rc: int) -> None:
    if rc != 0:
        raise PcmError(call, rc)


def _torch_dtype(dtype: int):
    return torch.bfloat16 if dtype == GRPO_BF16 else torch.float32


# ------------------------------------------------------------------------------------------------
class Context:
    """Owns a pcm_ctx (configuration + persistent keep-probability state on the device)."""

    def __init__(self, n_phases: int, budget: int, group_size: int, t_rc: int = 5, p_min: float = 0.1,
                 adv_eps: float = 1e-6, seed: int = 0, max_traj: int = 1024, mode: int = 0):
        self.handle = _P()
        self.cfg = pcm_config(n_phases, budget, group_size, t_rc, p_min, adv_eps, seed, mode, 0)
        _check("pcm_create", _lib.pcm_create(C.byref(self.handle), C.byref(self.cfg), max_traj))

    def close(self):
        if getattr(self, "handle", None):
            _lib.pcm_destroy(self.handle)
            self.handle = _P()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def make_batch(traj_off, tok, phase, reward, max_len: int, obs=None, logp_old=None) -> pcm_batch:
    n_traj = traj_off.numel() - 1
    n_chunks = phase.numel()
    b = pcm_batch(n_traj, n_chunks, max_len, 0, _ptr(traj_off), _ptr(tok), _ptr(phase), _ptr(reward), _ptr(obs),
                  _ptr(logp_old))
    b._keep = (traj_off, tok, phase, reward, obs, logp_old)     # keep the tensors alive
    return b


def pcm_poll_status(ctx: Context) -> int:
    return _lib.pcm_poll_status(ctx.handle, _stream())


def pcm_state_export(ctx: Context) -> bytes:
    n = C.c_size_t(0)
    _check("pcm_state_export", _lib.pcm_state_export(ctx.handle, None, C.byref(n)))
    buf = C.create_string_buffer(n.value)
    _check("pcm_state_export", _lib.pcm_state_export(ctx.handle, buf, C.byref(n)))
    return bytes(buf.raw[: n.value])


def pcm_state_import(ctx: Context, blob: bytes) -> None:
    buf = C.create_string_buffer(blob, len(blob))
    _check("pcm_state_import", _lib.pcm_state_import(ctx.handle, buf, len(blob)))


def pcm_score_phases(ctx: Context, batch: pcm_batch, want_adv: bool = True):
    dev = torch.device("cuda")
    K = ctx.cfg.n_phases
    Cc = torch.empty(K, dtype=torch.float64, device=dev)
    valid = torch.empty(K, dtype=torch.uint8, device=dev)
    n_valid = torch.empty(K, dtype=torch.int32, device=dev)
    adv = torch.empty(batch.n_traj, dtype=torch.float32, device=dev) if want_adv else None
    _check("pcm_score_phases", _lib.pcm_score_phases(ctx.handle, C.byref(batch), _ptr(Cc), _ptr(valid), _ptr(n_valid),
                                                     _ptr(adv), _stream()))
    return Cc, valid, n_valid, adv


def pcm_score_phases_f32(ctx: Context, batch: pcm_batch, act: torch.Tensor, want_adv: bool = True):
    """Eq. 5 on continuous chunk actions: act float32 [n_chunks, 56]."""
    assert act.dtype == torch.float32 and act.shape[-1] == ACT_DIM
    dev = torch.device("cuda")
    K = ctx.cfg.n_phases
    Cc = torch.empty(K, dtype=torch.float64, device=dev)
    valid = torch.empty(K, dtype=torch.uint8, device=dev)
    n_valid = torch.empty(K, dtype=torch.int32, device=dev)
    adv = torch.empty(batch.n_traj, dtype=torch.float32, device=dev) if want_adv else None
    _check("pcm_score_phases_f32", _lib.pcm_score_phases_f32(ctx.handle, C.byref(batch), _ptr(act), _ptr(Cc), _ptr(valid),
                                                             _ptr(n_valid), _ptr(adv), _stream()))
    return Cc, valid, n_valid, adv


STATIC_MAX_GROUPS = 4096


def pcm_score_phases_static(n_phases: int, group_size: int, adv_eps: float, batch: pcm_batch, out: Dict[str, torch.Tensor]):
    """Allocation-free variant of pcm_score_phases: every output tensor, including the one-word
    `status`, is passed in by the caller (keys C, valid, n_valid, adv, status); this wrapper creates
    no tensor, so that the call stays free of device allocations end to end."""
    _check("pcm_score_phases_static",
           _lib.pcm_score_phases_static(n_phases, group_size, adv_eps, C.byref(batch), _ptr(out["C"]), _ptr(out["valid"]),
                                        _ptr(out.get("n_valid")), _ptr(out.get("adv")), _ptr(out.get("status")),
                                        _stream()))
    return out


def pcm_label_phases(ctx: Context, traj_off: torch.Tensor, step_off: torch.Tensor, grip_close: torch.Tensor,
                     chunk_len: int = 8, phase: Optional[torch.Tensor] = None) -> torch.Tensor:
    n_traj = traj_off.numel() - 1
    if phase is None:
        phase = torch.empty(int(traj_off[-1].item()), dtype=torch.uint8, device=traj_off.device)
    _check("pcm_label_phases", _lib.pcm_label_phases(ctx.handle, n_traj, _ptr(traj_off), _ptr(step_off), _ptr(grip_close),
                                                     chunk_len, _ptr(phase), _stream()))
    return phase


def pcm_update_keep_probs(ctx: Context, Cc: torch.Tensor, valid: torch.Tensor):
    dev = torch.device("cuda")
    K = ctx.cfg.n_phases
    p = torch.empty(K, dtype=torch.float32, device=dev)
    q = torch.empty(K, dtype=torch.int32, device=dev)          # uint32 bit pattern (values <= 2^24)
    _check("pcm_update_keep_probs", _lib.pcm_update_keep_probs(ctx.handle, _ptr(Cc), _ptr(valid), _ptr(p), _ptr(q),
                                                               _stream()))
    return p, q


def pcm_sample_chunks(ctx: Context, batch: pcm_batch, q: torch.Tensor, it: int,
                      out: Optional[Dict[str, torch.Tensor]] = None):
    dev = torch.device("cuda")
    if out is None:
        out = {"kept_idx": torch.empty(max(1, batch.n_traj * ctx.cfg.budget), dtype=torch.int32, device=dev),
               "kept_off": torch.empty(batch.n_traj + 1, dtype=torch.int32, device=dev),
               "kept_per_phase": torch.empty(ctx.cfg.n_phases, dtype=torch.int32, device=dev)}
    _check("pcm_sample_chunks", _lib.pcm_sample_chunks(ctx.handle, C.byref(batch), _ptr(q), it, _ptr(out["kept_idx"]),
                                                       _ptr(out["kept_off"]), _ptr(out["kept_per_phase"]), _stream()))
    return out["kept_idx"], out["kept_off"], out["kept_per_phase"]


# ------------------------------------------------------------------------------------------------
class Model:
    """Device weights of the decoder policy plus the matching grpo_model / grpo_grads structures."""

    def __init__(self, d: int, n_layers: int, n_heads: int, prefix_len: int, dtype: int,
                 weights: Dict[str, torch.Tensor]):
        self.cfg = grpo_model_cfg(d, n_layers, n_heads, prefix_len, dtype, 0)
        self.weights = {k: weights[k].contiguous() for k in _WEIGHTS}
        for k, t in self.weights.items():
            assert t.is_cuda and t.dtype == _torch_dtype(dtype), k
        self.c_model = grpo_model(self.cfg, *[_ptr(self.weights[k]) for k in _WEIGHTS])
        self.grads: Optional[Dict[str, torch.Tensor]] = None
        self.c_grads: Optional[grpo_grads] = None

    @property
    def S(self) -> int:
        return self.cfg.prefix_len + ACT_DIM

    def alloc_grads(self) -> Dict[str, torch.Tensor]:
        """fp32 gradient tensors, views of one flat buffer (self.flat_grads) so that a data-parallel caller can
        sum all of them over the ranks with a single all-reduce."""
        if self.grads is None:
            sizes = [(k, self.weights[k].numel()) for k in _WEIGHTS]
            pad = lambda n: (n + 63) // 64 * 64                      # every tensor starts 256-byte aligned
            self.flat_grads = torch.zeros(sum(pad(n) for _, n in sizes), dtype=torch.float32,
                                          device=self.weights["w_qkv"].device)
            self.grads, off = {}, 0
            for k, n in sizes:
                self.grads[k] = self.flat_grads[off:off + n].view(self.weights[k].shape)
                off += pad(n)
            self.c_grads = grpo_grads(*[_ptr(self.grads[k]) for k in _WEIGHTS])
        return self.grads


class Lora:
    """Device adapter tensors (App. E: rank 32, alpha 32) of a Model, with the matching C structures."""

    def __init__(self, model: Model, rank: int, alpha: float, tensors: Dict[str, torch.Tensor]):
        self.rank, self.alpha = rank, alpha
        self.tensors = {k: tensors[k].contiguous() for k in _LORA}
        for k, t in self.tensors.items():
            assert t.is_cuda and t.dtype == _torch_dtype(model.cfg.dtype), k
        self.c = grpo_lora(rank, alpha, *[_ptr(self.tensors[k]) for k in _LORA])
        self.grads: Optional[Dict[str, torch.Tensor]] = None
        self.c_grads: Optional[grpo_lora_grads] = None

    def alloc_grads(self) -> Dict[str, torch.Tensor]:
        """fp32 adapter gradients, views of one flat buffer (self.flat_grads)."""
        if self.grads is None:
            sizes = [(k, self.tensors[k].numel()) for k in _LORA]
            pad = lambda n: (n + 63) // 64 * 64
            self.flat_grads = torch.zeros(sum(pad(n) for _, n in sizes), dtype=torch.float32,
                                          device=self.tensors["a_qkv"].device)
            self.grads, off = {}, 0
            for k, n in sizes:
                self.grads[k] = self.flat_grads[off:off + n].view(self.tensors[k].shape)
                off += pad(n)
            self.c_grads = grpo_lora_grads(*[_ptr(self.grads[k]) for k in _LORA])
        return self.grads


class Packed:
    """Caller-allocated dense batch of kept chunks."""

    def __init__(self, model, n_kept: int):
        dev = torch.device("cuda")
        dt = _torch_dtype(model.cfg.dtype)
        self.n_kept = n_kept
        self.X = torch.empty((n_kept, model.S, model.cfg.d), dtype=dt, device=dev)
        self.tgt = torch.empty((n_kept, ACT_DIM), dtype=torch.uint8, device=dev)
        self.lpo = torch.empty((n_kept, ACT_DIM), dtype=torch.float32, device=dev)
        self.adv_c = torch.empty(n_kept, dtype=torch.float32, device=dev)
        self.src = torch.empty(n_kept, dtype=torch.int32, device=dev)
        self.c = grpo_packed(n_kept, 0, _ptr(self.X), _ptr(self.tgt), _ptr(self.lpo), _ptr(self.adv_c), _ptr(self.src))


def grpo_pack_chunks(ctx: Context, batch: pcm_batch, model, kept_idx, kept_off, adv, out: Packed) -> Packed:
    _check("grpo_pack_chunks", _lib.grpo_pack_chunks(ctx.handle, C.byref(batch), C.byref(model.cfg), _ptr(kept_idx),
                                                     _ptr(kept_off), _ptr(model.weights["e_act"]), _ptr(adv),
                                                     C.byref(out.c), _stream()))
    return out


def grpo_workspace_bytes(model: Model, mb_chunks: int, flags: int = 0, lora: Optional[Lora] = None) -> int:
    if lora is not None:
        return int(_lib.grpo_lora_workspace_bytes(C.byref(model.cfg), lora.rank, mb_chunks, flags))
    return int(_lib.grpo_workspace_bytes(C.byref(model.cfg), mb_chunks, flags))


def grpo_actor_fwd_bwd(model: Model, packed: Packed, eps_low: float = 0.2, eps_high: float = 0.2,
                       loss_scale: float = 0.0, mb_chunks: int = 64, flags: int = 0,
                       workspace: Optional[torch.Tensor] = None, want_stats: bool = True,
                       logp: Optional[torch.Tensor] = None, loss: Optional[torch.Tensor] = None,
                       entropy_coef: float = 0.0, lora: Optional[Lora] = None):
    """Returns (loss tensor[1] on the device, logp [n_kept, 56], grads dict or None, stats or None).
    With `lora` the base matrices are frozen (their entries of the grads dict are left untouched) and the
    adapter gradients are in lora.grads."""
    dev = torch.device("cuda")
    mb = max(1, min(mb_chunks, max(packed.n_kept, 1)))
    need = grpo_workspace_bytes(model, mb, flags, lora)
    if need == 0:
        raise PcmError("grpo_workspace_bytes", -2)
    if workspace is None:
        workspace = torch.empty(need + 256, dtype=torch.uint8, device=dev)
    off = (-workspace.data_ptr()) % 256
    ws_ptr = workspace.data_ptr() + off
    ws_bytes = workspace.numel() - off
    if loss is None:
        loss = torch.zeros(1, dtype=torch.float32, device=dev)
    if logp is None:
        logp = torch.empty((packed.n_kept, ACT_DIM), dtype=torch.float32, device=dev)
    lc = grpo_loss_cfg(eps_low, eps_high, loss_scale, mb, flags, entropy_coef)
    fwd_only = bool(flags & GRPO_FWD_ONLY)
    grads = None
    if not fwd_only:
        grads = model.alloc_grads()
    stats = grpo_stats() if want_stats else None
    if lora is None:
        rc = _lib.grpo_actor_fwd_bwd(C.byref(model.c_model), C.byref(packed.c), C.byref(lc),
                                     C.byref(model.c_grads) if not fwd_only else None, _ptr(loss), _ptr(logp),
                                     C.byref(stats) if stats is not None else None, ws_ptr, ws_bytes, _stream())
    else:
        if not fwd_only:
            lora.alloc_grads()
        rc = _lib.grpo_actor_fwd_bwd_lora(C.byref(model.c_model), C.byref(lora.c), C.byref(packed.c), C.byref(lc),
                                          C.byref(model.c_grads) if not fwd_only else None,
                                          C.byref(lora.c_grads) if not fwd_only else None, _ptr(loss), _ptr(logp),
                                          C.byref(stats) if stats is not None else None, ws_ptr, ws_bytes, _stream())
    _check("grpo_actor_fwd_bwd", rc)
    return loss, logp, grads, stats


# ------------------------------------------------------------------------------------------------
def grpo_gemm(A: torch.Tensor, a_kmajor: bool, B: torch.Tensor, b_kmajor: bool, M: int, N: int, K: int,
              out_dtype=torch.float32, R: Optional[torch.Tensor] = None, backend: int = 0,
              C_out: Optional[torch.Tensor] = None) -> torch.Tensor:
    ab = GRPO_BF16 if A.dtype == torch.bfloat16 else GRPO_F32
    if C_out is None:
        C_out = torch.empty((M, N), dtype=out_dtype, device=A.device)
    cd = GRPO_BF16 if C_out.dtype == torch.bfloat16 else GRPO_F32
    rc = _lib.grpo_gemm(M, N, K, _ptr(A), A.stride(0), int(a_kmajor), _ptr(B), B.stride(0), int(b_kmajor), ab,
                        _ptr(C_out), C_out.stride(0), cd, _ptr(R), R.stride(0) if R is not None else 0, backend,
                        _stream())
    _check("grpo_gemm", rc)
    return C_out


def grpo_attention(qkv: torch.Tensor, n_seq: int, S: int, H: int, dh: int, dout: Optional[torch.Tensor] = None):
    dt = GRPO_BF16 if qkv.dtype == torch.bfloat16 else GRPO_F32
    d = H * dh
    out = torch.empty((n_seq * S, d), dtype=qkv.dtype, device=qkv.device)
    lse = torch.empty((n_seq, H, S), dtype=torch.float32, device=qkv.device)
    dqkv = scratch = None
    if dout is not None:
        dqkv = torch.empty_like(qkv)
        scratch = torch.empty((n_seq, H, S), dtype=torch.float32, device=qkv.device)
    _check("grpo_attention", _lib.grpo_attention(dt, _ptr(qkv), _ptr(out), _ptr(lse), _ptr(dout), _ptr(dqkv),
                                                 _ptr(scratch), n_seq, S, H, dh, _stream()))
    return out, lse, dqkv


def grpo_attention_wait_status() -> int:
    _lib.grpo_attention_wait_status.restype = C.c_uint32
    return int(_lib.grpo_attention_wait_status())


def pcm_launch_count() -> int:
    return int(_lib.pcm_launch_count())


def pcm_profile_enable(on: bool) -> None:
    _check("pcm_profile_enable", _lib.pcm_profile_enable(int(on)))


def pcm_profile_read() -> Dict[str, Dict[str, float]]:
    """Per kernel class since the last read: elapsed ms, algorithmic flops and bytes, launches."""
    prof = pcm_profile()
    _check("pcm_profile_read", _lib.pcm_profile_read(C.byref(prof)))
    return {name: {"ms": prof.ms[i], "flops": prof.flops[i], "bytes": prof.bytes[i], "launches": int(prof.launches[i])}
            for i, name in enumerate(PROFILE_CLASSES)}


class AdamW:
    """fp32 master weights and moments for a Model, stepped by grpo_adamw_step."""

    def __init__(self, model: Model, lr: float = 1e-5, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
                 weight_decay: float = 0.0, max_grad_norm: float = 2.0):
        self.model = model
        self.cfg = grpo_adamw_cfg(lr, beta1, beta2, eps, weight_decay, max_grad_norm)
        self.master = {k: v.float().contiguous() for k, v in model.weights.items()}
        self.m = {k: torch.zeros_like(v) for k, v in self.master.items()}
        self.v = {k: torch.zeros_like(v) for k, v in self.master.items()}
        self.c_master = grpo_grads(*[_ptr(self.master[k]) for k in _WEIGHTS])
        self.c_m = grpo_grads(*[_ptr(self.m[k]) for k in _WEIGHTS])
        self.c_v = grpo_grads(*[_ptr(self.v[k]) for k in _WEIGHTS])
        n = int(_lib.grpo_adamw_scratch_bytes())
        self.scratch = torch.empty(n + 256, dtype=torch.uint8, device="cuda")
        self.grad_norm = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.step_count = 0

    def step(self) -> torch.Tensor:
        """Applies the model's current gradients; returns the (device) gradient norm before clipping."""
        assert self.model.c_grads is not None, "run grpo_actor_fwd_bwd first"
        self.step_count += 1
        off = (-self.scratch.data_ptr()) % 256
        _check("grpo_adamw_step",
               _lib.grpo_adamw_step(C.byref(self.model.cfg), C.byref(self.cfg), self.step_count, C.byref(self.model.c_model),
                                    C.byref(self.c_master), C.byref(self.model.c_grads), C.byref(self.c_m), C.byref(self.c_v),
                                    _ptr(self.grad_norm), self.scratch.data_ptr() + off, self.scratch.numel() - off, _stream()))
        return self.grad_norm


_SMALL = ("g1", "g2", "gf", "w_h", "e_act")


class LoraAdamW:
    """AdamW for LoRA fine-tuning (grpo_adamw_step_lora): fp32 masters and moments for the adapters and, with
    train_small, for the norm gains, head and action embedding as well; the projections stay frozen."""

    def __init__(self, model: Model, lora: Lora, train_small: bool = True, lr: float = 1e-5, beta1: float = 0.9,
                 beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0, max_grad_norm: float = 2.0):
        self.model, self.lora, self.train_small = model, lora, train_small
        self.cfg = grpo_adamw_cfg(lr, beta1, beta2, eps, weight_decay, max_grad_norm)
        self.master = {k: v.float().contiguous() for k, v in lora.tensors.items()}
        if train_small:
            self.master.update({k: model.weights[k].float().contiguous() for k in _SMALL})
        self.m = {k: torch.zeros_like(v) for k, v in self.master.items()}
        self.v = {k: torch.zeros_like(v) for k, v in self.master.items()}
        lora_struct = lambda d: grpo_lora_grads(*[_ptr(d[k]) for k in _LORA])
        small_struct = lambda d: grpo_grads(*[_ptr(d[k]) if k in _SMALL else None for k in _WEIGHTS])
        self.c_lora = [lora_struct(d) for d in (self.master, self.m, self.v)]
        self.c_small = [small_struct(d) for d in (self.master, self.m, self.v)] if train_small else None
        n = int(_lib.grpo_adamw_scratch_bytes())
        self.scratch = torch.empty(n + 256, dtype=torch.uint8, device="cuda")
        self.grad_norm = torch.zeros(1, dtype=torch.float32, device="cuda")
        self.step_count = 0

    def step(self) -> torch.Tensor:
        """Applies the current adapter (and small-tensor) gradients; returns the (device) norm before clipping."""
        assert self.lora.c_grads is not None and self.model.c_grads is not None, "run grpo_actor_fwd_bwd with lora first"
        self.step_count += 1
        off = (-self.scratch.data_ptr()) % 256
        ma, mm, mv = self.c_lora
        if self.train_small:
            sa, sm, sv = self.c_small
            ref = lambda x: None if x is None else C.byref(x)
            small = (ref(self.model.c_model), ref(sa), ref(self.model.c_grads), ref(sm), ref(sv))
        else:
            small = (None, None, None, None, None)
        _check("grpo_adamw_step_lora",
               _lib.grpo_adamw_step_lora(C.byref(self.model.cfg), C.byref(self.cfg), self.step_count, C.byref(self.lora.c),
                                         C.byref(ma), C.byref(self.lora.c_grads), C.byref(mm), C.byref(mv), *small,
                                         _ptr(self.grad_norm), self.scratch.data_ptr() + off, self.scratch.numel() - off,
                                         _stream()))
        return self.grad_norm
