"""CPU-side checks of the C ABI: the library loads, exports every declared symbol, validates arguments."""
import ctypes
import os
import re

import pytest

import paper_2602_16839_b200 as pt

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "ptenc.h")).read()
    return sorted(set(re.findall(r"PTENC_API\s+[\w\s\*]+?\b(ptenc_\w+)\s*\(", src)))


def test_every_declared_symbol_is_exported():
    names = _declared()
    assert len(names) >= 14
    raw = ctypes.CDLL(pt.LIB_PATH)
    for n in names:
        assert hasattr(raw, n), n
    assert sorted(pt.EXPORTS) == names


def test_strerror():
    assert pt.strerror(0) == "ok"
    for code in range(-7, 0):
        assert pt.strerror(code) not in ("ok", "unknown error")
    assert pt.strerror(-99) == "unknown error"


GOOD = dict(n_layers=2, batch=3, n_q_heads=8, n_kv_heads=2, head_dim=64, window=16)


def test_workspace_bytes_grows_with_window_not_with_length():
    a = pt.ptenc_workspace_bytes(pt.make_config(**GOOD))
    b = pt.ptenc_workspace_bytes(pt.make_config(**{**GOOD, "window": 32}))
    assert b > a > 2 * 2 * 3 * 2 * 16 * 64 * 2
    # the 7B-shaped configuration: two bf16 rings of 7 GiB each dominate
    big = pt.make_config(n_layers=28, batch=128, n_q_heads=28, n_kv_heads=4, head_dim=128, window=2048)
    n = pt.ptenc_workspace_bytes(big)
    assert 14 * 2**30 < n < 14.2 * 2**30


@pytest.mark.parametrize("patch,code", [
    (dict(n_layers=0), pt.binding.PTENC_EINVAL),
    (dict(window=0), pt.binding.PTENC_EINVAL),
    (dict(evict_chunk=0), pt.binding.PTENC_EINVAL),
    (dict(evict_chunk=17), pt.binding.PTENC_EINVAL),
    (dict(dtype=7), pt.binding.PTENC_EINVAL),
    (dict(normalize_mode=3), pt.binding.PTENC_EINVAL),
    (dict(n_q_heads=7), pt.binding.PTENC_ESHAPE),
    (dict(head_dim=12), pt.binding.PTENC_ESHAPE),
    (dict(head_dim=512), pt.binding.PTENC_ESHAPE),
    (dict(n_global=0), pt.binding.PTENC_ESHAPE),
    (dict(rank=129), pt.binding.PTENC_ESHAPE),
])
def test_bad_config_is_rejected_on_the_host(patch, code):
    cfg = pt.make_config(**{**GOOD, **patch})
    with pytest.raises(pt.PtencError) as e:
        pt.ptenc_workspace_bytes(cfg)
    assert e.value.code == code
    # create refuses the same configuration before touching the device
    h = ctypes.c_void_p()
    rc = pt.lib.ptenc_cache_create(ctypes.byref(cfg), 1024, 1 << 30, None, ctypes.byref(h))
    assert rc == code and not h.value


def test_create_rejects_null_misaligned_and_small_workspace():
    cfg = pt.make_config(**GOOD)
    h = ctypes.c_void_p()
    assert pt.lib.ptenc_cache_create(ctypes.byref(cfg), None, 1 << 30, None, ctypes.byref(h)) == pt.binding.PTENC_EINVAL
    assert pt.lib.ptenc_cache_create(ctypes.byref(cfg), 1024 + 16, 1 << 30, None, ctypes.byref(h)) == pt.binding.PTENC_EALIGN
    assert pt.lib.ptenc_cache_create(ctypes.byref(cfg), 4096, 1000, None, ctypes.byref(h)) == pt.binding.PTENC_EWORKSPACE
    for field, bad in (("attn_consumer_warps", 5), ("policy", 9), ("recent", -1)):
        cfg = pt.make_config(**GOOD)
        setattr(cfg, field, bad)
        assert pt.lib.ptenc_cache_create(ctypes.byref(cfg), 4096, 1 << 30, None, ctypes.byref(h)) == pt.binding.PTENC_EINVAL


def test_null_handle_is_an_error_not_a_crash():
    assert pt.lib.ptenc_cache_destroy(None) == pt.binding.PTENC_EINVAL
    assert pt.lib.ptenc_decode_step(None, 0, 16, 16, 16, None, 16, None) == pt.binding.PTENC_EINVAL
    assert pt.lib.ptenc_cache_status(None, None) == pt.binding.PTENC_EINVAL


def test_no_cpu_path():
    import torch
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    with pytest.raises(RuntimeError):
        pt.Cache(pt.make_config(**GOOD))
