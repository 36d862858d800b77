"""The shared library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "pcm_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b((?:pcm|grpo)_[a-z0-9_]+)\s*\(", text)))


def test_library_loads_and_exports_every_declared_symbol():
    from paper_2605_16154_b200 import build
    lib = ctypes.CDLL(build.build())
    names = _declared()
    assert {"pcm_score_phases", "pcm_update_keep_probs", "pcm_sample_chunks", "grpo_pack_chunks",
            "grpo_actor_fwd_bwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_struct_sizes_match_the_header_layout():
    from paper_2605_16154_b200 import binding as B
    assert ctypes.sizeof(B.pcm_config) == 48
    assert ctypes.sizeof(B.pcm_batch) == 16 + 6 * 8
    assert ctypes.sizeof(B.grpo_model_cfg) == 24
    assert ctypes.sizeof(B.grpo_model) == 24 + 9 * 8
    assert ctypes.sizeof(B.grpo_packed) == 8 + 5 * 8
    assert ctypes.sizeof(B.grpo_loss_cfg) == 24
    assert ctypes.sizeof(B.grpo_stats) == 32
    assert ctypes.sizeof(B.grpo_lora) == 8 + 8 * 8 and ctypes.sizeof(B.grpo_lora_grads) == 8 * 8
    assert set(B.EXPORTED) == set(_declared())


def test_host_side_argument_checks_need_no_gpu():
    from paper_2605_16154_b200 import binding as B
    cfg = B.grpo_model_cfg(100, 2, 3, 4, 1, 0)          # d not divisible by heads
    assert B._lib.grpo_workspace_bytes(ctypes.byref(cfg), 4, 0) == 0
    cfg = B.grpo_model_cfg(1024, 8, 16, 256, 1, 0)
    full = B._lib.grpo_workspace_bytes(ctypes.byref(cfg), 64, 0)
    fwd = B._lib.grpo_workspace_bytes(ctypes.byref(cfg), 64, B.GRPO_FWD_ONLY)
    assert 0 < fwd < full
    # activations kept per token per layer: 18 d bf16 + 2 d fp32 = 44 d bytes (+ small terms); in the last layer the
    # 30 d bytes after the attention exist for the 56 scored rows of a chunk's 312 only
    per_token = full / (64 * 312)
    expect = (7 * 44 + 14 + 30 * 56 / 312) * 1024
    assert expect < per_token < expect * 1.3
    lora = B._lib.grpo_lora_workspace_bytes(ctypes.byref(cfg), 32, 64, 0)
    assert full < lora < full * 1.02                     # adapters keep four [tokens][rank] products per layer
    assert B._lib.grpo_lora_workspace_bytes(ctypes.byref(cfg), 12, 64, 0) == 0
    assert B._lib.pcm_create(None, None, 0) == -1


def test_per_device_setup_mask_marks_each_device_once():
    """Kernel attributes are per device: the first launch on every device must set them, later ones must not."""
    from paper_2605_16154_b200 import binding as B
    mask = ctypes.c_uint64(0)
    f = B._lib.pcm_first_use_on_device
    assert f(ctypes.byref(mask), 0) == 1 and f(ctypes.byref(mask), 0) == 0
    assert f(ctypes.byref(mask), 1) == 1 and f(ctypes.byref(mask), 1) == 0 and f(ctypes.byref(mask), 0) == 0
    assert f(ctypes.byref(mask), 63) == 1 and f(ctypes.byref(mask), 63) == 0
    assert mask.value == (1 | 2 | (1 << 63))
    assert f(ctypes.byref(mask), 64) == 1 and f(ctypes.byref(mask), -1) == 1      # out of range: always set again
    assert mask.value == (1 | 2 | (1 << 63))
