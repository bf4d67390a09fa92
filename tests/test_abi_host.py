"""CPU-side checks of the C-ABI library: it loads, exports every declared symbol, and validates arguments
on the host before anything touches a device."""
import ctypes as C
import os
import re

import pytest

from paper_2601_22379_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "spla.h")).read()
    declared = set(re.findall(r"\b(spla_[a-z_]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_status_strings(lib):
    assert lib.spla_status_string(0) == b"ok"
    assert b"capacity" in lib.spla_status_string(binding.SPLA_ERR_CAPACITY)
    assert lib.spla_status_string(-99) == b"unknown status"
    assert lib.spla_last_cuda_error() == b""


def test_query_sizes_follow_the_documented_layouts(lib):
    cfg = binding.make_config(batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=32,
                              max_context=131072 + 64)
    sz = binding.query_sizes(cfg)
    max_blocks = 2049
    assert sz.k_cache == 4 * 8 * max_blocks * 64 * 128 * 2 == sz.v_cache
    assert sz.stats == 4 * 8 * max_blocks * 2 * 128 * 4
    assert sz.rla_state == 4 * 8 * 128 * 128 * 4
    assert sz.tok_lse == 4 * 8 * max_blocks * 64 * 4
    assert sz.seq_lens == 16
    assert 0 < sz.workspace < 64 << 20
    f32 = binding.make_config(batch=1, n_q_heads=1, n_kv_heads=1, head_dim=64, block_size=64, top_k=8,
                              max_context=4112, kv_dtype="f32")
    assert binding.query_sizes(f32).k_cache == 65 * 64 * 64 * 4
    # strided windows C = 32, s = 16 inside blocks of 64: three statistics records per block
    win = binding.make_config(batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=32,
                              max_context=131072 + 64, window_size=32, window_stride=16)
    assert win.n_windows == 3 and binding.query_sizes(win).stats == 3 * sz.stats
    assert binding.query_sizes(win).k_cache == sz.k_cache
    # 16-bit statistics: half the bytes, everything else unchanged
    half = binding.make_config(batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=32,
                               max_context=131072 + 64, flags=binding.SPLA_STATS_BF16)
    hs = binding.query_sizes(half)
    assert hs.stats * 2 == sz.stats and hs.k_cache == sz.k_cache and hs.workspace == sz.workspace


@pytest.mark.parametrize("kw,status", [
    (dict(n_q_heads=30), binding.SPLA_ERR_INVALID_ARG),          # G not an integer
    (dict(batch=0), binding.SPLA_ERR_INVALID_ARG),
    (dict(n_sink_blocks=20, n_local_blocks=20), binding.SPLA_ERR_INVALID_ARG),
    (dict(flags=64), binding.SPLA_ERR_INVALID_ARG),
    (dict(flags=128), binding.SPLA_ERR_INVALID_ARG),
    (dict(sm_scale=-1.0), binding.SPLA_ERR_INVALID_ARG),
    (dict(head_dim=96), binding.SPLA_ERR_UNSUPPORTED),
    (dict(block_size=48), binding.SPLA_ERR_UNSUPPORTED),
    (dict(top_k=65, n_sink_blocks=0, n_local_blocks=0), binding.SPLA_ERR_UNSUPPORTED),
    (dict(n_q_heads=8 * 17), binding.SPLA_ERR_UNSUPPORTED),
    (dict(max_context=64 * 32768 + 1), binding.SPLA_ERR_UNSUPPORTED),
    (dict(window_size=32), binding.SPLA_ERR_INVALID_ARG),                      # a window needs a stride
    (dict(window_stride=16), binding.SPLA_ERR_INVALID_ARG),
    (dict(window_size=128, window_stride=16), binding.SPLA_ERR_INVALID_ARG),   # wider than the block
    (dict(window_size=-1, window_stride=16), binding.SPLA_ERR_INVALID_ARG),
    (dict(window_size=8, window_stride=4), binding.SPLA_ERR_UNSUPPORTED),      # 15 windows per block: above 8
])
def test_bad_configurations_are_rejected_on_the_host(lib, kw, status):
    base = dict(batch=2, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=32, max_context=4096)
    base.update(kw)
    cfg = binding.make_config(**base)
    sz = binding.SplaSizes()
    assert lib.spla_query_sizes(C.byref(cfg), C.byref(sz)) == status
    handle = C.c_void_p()
    bufs = binding.SplaBuffers()
    assert lib.spla_init_cache(C.byref(cfg), C.byref(bufs), None, C.byref(handle)) == status
    assert not handle.value


def test_null_and_misaligned_buffers_are_rejected_before_any_launch(lib):
    cfg = binding.make_config(batch=1, n_q_heads=4, n_kv_heads=1, head_dim=128, block_size=64, top_k=8, max_context=1024)
    handle = C.c_void_p()
    assert lib.spla_query_sizes(None, None) == binding.SPLA_ERR_INVALID_ARG
    assert lib.spla_init_cache(C.byref(cfg), None, None, C.byref(handle)) == binding.SPLA_ERR_INVALID_ARG
    bufs = binding.SplaBuffers()                      # all NULL
    assert lib.spla_init_cache(C.byref(cfg), C.byref(bufs), None, C.byref(handle)) == binding.SPLA_ERR_INVALID_ARG
    fake = 0x7F0000000000
    sz = binding.query_sizes(cfg)
    bufs = binding.SplaBuffers(fake, fake, fake, fake, fake + 8, fake, fake, sz.workspace)   # tok_lse misaligned
    assert lib.spla_init_cache(C.byref(cfg), C.byref(bufs), None, C.byref(handle)) == binding.SPLA_ERR_INVALID_ARG
    bufs = binding.SplaBuffers(fake, fake, fake, fake, fake, fake, fake, sz.workspace - 1)   # workspace too small
    assert lib.spla_init_cache(C.byref(cfg), C.byref(bufs), None, C.byref(handle)) == binding.SPLA_ERR_INVALID_ARG
    assert lib.spla_append_tokens(None, None, None, None, 1, None) == binding.SPLA_ERR_INVALID_ARG
    assert lib.spla_decode(None, None, None, None, None, None, None, None) == binding.SPLA_ERR_INVALID_ARG
    assert lib.spla_sync_status(None, None) == binding.SPLA_ERR_INVALID_ARG
    assert lib.spla_destroy_cache(None) == binding.SPLA_OK


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.load(str(tmp_path / "libspla.so"))
