"""The C-ABI library loads and exports what include/mtla.h declares; host-side validation.

No kernel is launched here: every call either needs no device or is rejected by argument
checks before anything is enqueued.
"""
import ctypes
import os
import re

import pytest

from paper_2505_13544_b200 import binding as M

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "mtla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mtla_[a-z_]+)\s*\(", text)))


def good_config(**kw):
    base = dict(d_model=512, n_heads=8, head_dim=64, latent_rank=256, rope_dim=32, stride=2,
                max_batch=4, max_tokens=64, max_prefill_tokens=32, dtype="bf16")
    base.update(kw)
    return M.make_config(**base)


def test_library_exports_every_declared_symbol():
    lib = M.load_library()
    names = declared_symbols()
    assert set(names) == set(M.EXPORTED_SYMBOLS)
    for name in names:
        assert getattr(lib, name) is not None


def test_arena_bytes_accounts_for_cache_and_rejects_bad_shapes():
    cfg = good_config()
    n = M.mtla_arena_bytes(cfg)
    cache = 4 * 32 * (256 + 32) * 2
    assert n > cache
    bigger = M.mtla_arena_bytes(good_config(max_tokens=128))
    assert bigger - n >= cache                      # 32 more slots for each of 4 sequences
    for bad in (dict(head_dim=48), dict(latent_rank=100), dict(rope_dim=16), dict(stride=0),
                dict(n_heads=64), dict(d_model=100), dict(hyper_dim=512), dict(max_batch=0)):
        assert M.mtla_arena_bytes(good_config(**bad)) == 0


def test_config_defaults_follow_the_paper():
    """Hyper-network width defaults to r/4 (Appendix: 256 -> 64)."""
    a = M.mtla_arena_bytes(good_config(hyper_dim=0))
    b = M.mtla_arena_bytes(good_config(hyper_dim=64))
    assert a == b


def test_create_rejects_bad_arguments_before_touching_the_device():
    lib = M.load_library()
    cfg = good_config()
    out = ctypes.c_void_p()
    w = M.mtla_weights()
    assert lib.mtla_create(None, ctypes.byref(w), 1024, 1 << 30, None, ctypes.byref(out)) == -1
    assert lib.mtla_create(ctypes.byref(cfg), ctypes.byref(w), 1024, 1 << 30, None,
                           ctypes.byref(out)) == -1          # null weight pointers
    bad = good_config(head_dim=48)
    assert lib.mtla_create(ctypes.byref(bad), ctypes.byref(w), 1024, 1 << 30, None,
                           ctypes.byref(out)) == -2
    assert out.value is None


def test_null_handle_calls_fail_cleanly():
    lib = M.load_library()
    assert lib.mtla_cache_bytes(None) == 0
    assert lib.mtla_destroy(None) == -1
    assert lib.mtla_reset(None) == -1
    assert lib.mtla_decode_step(None, None, 1, None, None) == -1
    assert lib.mtla_prefill(None, None, 1, 1, None, None) == -1
    assert lib.mtla_launch_count(None) == 0


def test_error_strings():
    assert M.error_string(0) == "ok"
    for code in range(-8, 0):
        assert M.error_string(code) != "unknown status"
    assert M.error_string(-99) == "unknown status"
    with pytest.raises(M.MTLAError) as e:
        M._check(-4, "probe")
    assert "capacity" in str(e.value)


def test_paged_arena_holds_the_pool_and_rejects_bad_paging():
    lib = M.load_library()
    cfg = good_config(max_tokens=1000)          # 500 slots -> 8 pages per sequence
    page = 64 * (256 + 32) * 2
    full = M.mtla_arena_bytes_paged(cfg)
    small = M.mtla_arena_bytes_paged(cfg, n_pages=5)
    assert full - small >= (4 * 8 - 5) * page - 4096
    assert M.mtla_arena_bytes_paged(cfg, n_pages=4 * 8 + 1) == 0      # more pages than could ever be used
    bad = M.mtla_paging(32, 0)                                        # pages are 64 slots
    assert lib.mtla_arena_bytes_paged(ctypes.byref(cfg), ctypes.byref(bad)) == 0
    assert lib.mtla_arena_bytes_paged(ctypes.byref(cfg), None) == 0


def test_baseline_arena_follows_the_cache_formula():
    """2 g d_h elements per token (Section 3), bf16."""
    lib = M.load_library()

    def arena(**kw):
        base = dict(d_model=512, n_heads=8, n_kv_heads=8, head_dim=64, max_batch=2, max_tokens=100,
                    rope_theta=0.0)
        base.update(kw)
        cfg = M.mtla_baseline_config(*[base[k] for k in ("d_model", "n_heads", "n_kv_heads", "head_dim",
                                                         "max_batch", "max_tokens", "rope_theta")])
        return lib.mtla_baseline_arena_bytes(ctypes.byref(cfg))

    per_token = 2 * 8 * 64 * 2
    assert arena(max_tokens=1100) - arena(max_tokens=100) >= 2 * 1000 * per_token
    assert arena(n_kv_heads=1) < arena(n_kv_heads=8)
    for bad in (dict(n_kv_heads=3), dict(head_dim=96), dict(n_heads=64, n_kv_heads=1), dict(max_batch=0)):
        assert arena(**bad) == 0
