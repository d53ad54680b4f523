"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, validates configurations and computes sizes (no compute call is made here)."""
import ctypes
import os
import re

import pytest

from paper_2604_16734_b200 import binding
from paper_2604_16734_b200.binding import KvcConfig, KVC_BF16, KVC_F32, KVC_EINVAL, KVC_ESTATE, KVC_OK

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_symbols():
    text = open(os.path.join(ROOT, "include", "kvc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvc_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = binding.lib()
    declared = _header_symbols()
    assert "kvc_create" in declared and "kvc_prefill_chunk" in declared and "kvc_cache_view" in declared \
        and "kvc_destroy" in declared
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in kvc.h but not exported"
    assert sorted(binding.EXPORTS) == declared


def _create(**kw):
    base = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=128, dtype=KVC_BF16, budget=256, max_chunk=64,
                obs_window=0, policy=0, softmax_scale=0.0, device=0, flags=0)
    base.update(kw)
    cfg = KvcConfig(**base)
    h = ctypes.c_void_p()
    rc = binding.lib().kvc_create(ctypes.byref(cfg), ctypes.byref(h))
    return rc, h


def test_create_validates_configuration():
    lib = binding.lib()
    rc, h = _create()
    assert rc == KVC_OK and h.value
    assert lib.kvc_destroy(h) == KVC_OK
    for bad in (dict(n_q_heads=7), dict(head_dim=96), dict(dtype=5), dict(budget=0), dict(max_chunk=0),
                dict(obs_window=257), dict(obs_window=-1), dict(policy=3), dict(n_layers=0),
                dict(n_q_heads=512, n_kv_heads=2), dict(budget=16, obs_window=0), dict(softmax_scale=-1.0)):
        rc, h = _create(**bad)
        assert rc == KVC_EINVAL and not h.value, bad
    assert lib.kvc_create(None, ctypes.byref(ctypes.c_void_p())) == KVC_EINVAL
    assert lib.kvc_destroy(None) == KVC_ESTATE
    # calls on a dead context are refused before anything touches a device
    assert lib.kvc_host_flush(None, None) == KVC_ESTATE
    assert lib.kvc_join(None, None) == KVC_ESTATE
    # a live context that never used the host entry point has nothing to flush (and needs no device to say so)
    rc, h = _create()
    assert rc == KVC_OK and lib.kvc_host_flush(h, None) == KVC_OK
    assert lib.kvc_destroy(h) == KVC_OK


def test_sizes_follow_the_memory_formula():
    lib = binding.lib()
    rc, h = _create(n_layers=32, n_q_heads=32, n_kv_heads=32, head_dim=128, budget=192, max_chunk=128)
    assert rc == KVC_OK
    a, b, c = ctypes.c_size_t(), ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.kvc_kv_bytes(h, 640, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)) == KVC_OK
    # Eq. 2: 2 x layers x heads x dim_head x precision x sequence length
    assert a.value == 2 * 32 * 32 * 128 * 2 * 192 == 96 * 2**20
    assert b.value == 2 * 32 * 32 * 128 * 2 * 384          # cap = roundup(192 + 128, 128)
    assert c.value == 2 * 32 * 32 * 128 * 2 * 640 == 320 * 2**20
    per_layer, ws = ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.kvc_cache_nbytes(h, ctypes.byref(per_layer), ctypes.byref(ws)) == KVC_OK
    assert per_layer.value >= b.value // 32 + 32 * 384 * 4 and per_layer.value % 256 == 0
    assert ws.value > 0
    # state errors without touching the device: layer never reset, bad arguments
    view = binding.KvcView()
    assert lib.kvc_cache_view(h, 0, 4096, ctypes.byref(view)) == KVC_ESTATE
    assert lib.kvc_cache_view(h, 99, 4096, ctypes.byref(view)) == KVC_EINVAL
    assert lib.kvc_launch_count(h) == 0
    assert lib.kvc_destroy(h) == KVC_OK


def test_fp32_config_and_error_text():
    lib = binding.lib()
    rc, h = _create(dtype=KVC_F32, head_dim=64, n_q_heads=4, n_kv_heads=1, budget=128, max_chunk=64)
    assert rc == KVC_OK
    assert isinstance(lib.kvc_last_error(h), bytes)
    assert lib.kvc_destroy(h) == KVC_OK


def test_binding_refuses_to_run_without_a_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        binding.Kvc(1, 4, 1, 64, torch.float32, 128, 64)
