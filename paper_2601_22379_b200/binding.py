"""Thin ctypes binding of libspla.so: the same entry points as include/spla.h, argument marshalling only.

Every step of the decode path runs inside the CUDA library.  PyTorch is used here for device memory and
streams and nothing else; there is no CPU or eager fallback: if the shared library is missing or fails to load,
`load()` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

SPLA_OK, SPLA_ERR_INVALID_ARG, SPLA_ERR_CAPACITY, SPLA_ERR_CUDA, SPLA_ERR_UNSUPPORTED = 0, -1, -2, -3, -4
SPLA_ERR_TIMEOUT, SPLA_ERR_BOUNDS = -5, -6
SPLA_F32, SPLA_BF16 = 0, 1
SPLA_ADOPT_CONTENTS, SPLA_FIRST_ORDER, SPLA_NO_RLA, SPLA_GENERAL_KERNELS, SPLA_STATS_BF16, SPLA_DEBUG_BOUNDS = 1, 2, 4, 8, 16, 32

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libspla.so")

EXPORTS = ["spla_query_sizes", "spla_init_cache", "spla_append_tokens", "spla_decode", "spla_decode_selected",
           "spla_select_blocks_noalloc", "spla_select", "spla_append_decode", "spla_prefill",
           "spla_query_prefill_workspace",
           "spla_copy_scores", "spla_sync_status", "spla_set_length_bound", "spla_debug_wait_hook", "spla_destroy_cache",
           "spla_launch_count", "spla_status_string", "spla_last_cuda_error"]


class SplaConfig(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("block_size", C.c_int32), ("top_k", C.c_int32), ("max_context", C.c_int32),
                ("n_sink_blocks", C.c_int32), ("n_local_blocks", C.c_int32), ("kv_dtype", C.c_int32),
                ("q_dtype", C.c_int32), ("sm_scale", C.c_float), ("phi_scale", C.c_float), ("rms_eps", C.c_float),
                ("flags", C.c_uint32), ("window_size", C.c_int32), ("window_stride", C.c_int32)]

    @property
    def n_windows(self) -> int:
        """Selection windows per block (1 without strided windows)."""
        return (self.block_size - self.window_size) // self.window_stride + 1 if self.window_size > 0 else 1


class SplaBuffers(C.Structure):
    _fields_ = [("k_cache", C.c_void_p), ("v_cache", C.c_void_p), ("stats", C.c_void_p), ("rla_state", C.c_void_p),
                ("tok_lse", C.c_void_p), ("seq_lens", C.c_void_p), ("workspace", C.c_void_p),
                ("workspace_bytes", C.c_size_t)]


class SplaSizes(C.Structure):
    _fields_ = [(n, C.c_size_t) for n in ("k_cache", "v_cache", "stats", "rla_state", "tok_lse", "seq_lens",
                                          "workspace")]


_lib = None


def load(path: str | None = None) -> C.CDLL:
    """Loads the shared library (once).  Raises if it is absent: there is nothing to fall back to."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise RuntimeError(f"{p} not found: build it with `python -m paper_2601_22379_b200.build` "
                           "(the SPLA path has no fallback implementation)")
    lib = C.CDLL(p)
    vp, i32 = C.c_void_p, C.c_int32
    lib.spla_query_sizes.argtypes = [C.POINTER(SplaConfig), C.POINTER(SplaSizes)]
    lib.spla_init_cache.argtypes = [C.POINTER(SplaConfig), C.POINTER(SplaBuffers), vp, C.POINTER(vp)]
    lib.spla_append_tokens.argtypes = [vp, vp, vp, vp, i32, vp]
    lib.spla_decode.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.spla_decode_selected.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
    lib.spla_select.argtypes = [vp, vp, vp, vp]
    lib.spla_append_decode.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.spla_select_blocks_noalloc.argtypes = [C.POINTER(SplaConfig), vp, vp, vp, vp, vp, vp, vp]
    lib.spla_prefill.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, C.c_size_t, vp]
    lib.spla_query_prefill_workspace.argtypes = [C.POINTER(SplaConfig), i32, C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.spla_copy_scores.argtypes = [vp, vp, vp]
    lib.spla_debug_wait_hook.argtypes = [vp, i32, i32]
    lib.spla_sync_status.argtypes = [vp, vp]
    lib.spla_set_length_bound.argtypes = [vp, i32]
    lib.spla_destroy_cache.argtypes = [vp]
    for name in EXPORTS[:-3]:
        getattr(lib, name).restype = C.c_int
    lib.spla_launch_count.argtypes = []
    lib.spla_launch_count.restype = C.c_ulonglong
    lib.spla_status_string.argtypes = [C.c_int]
    lib.spla_status_string.restype = C.c_char_p
    lib.spla_last_cuda_error.argtypes = []
    lib.spla_last_cuda_error.restype = C.c_char_p
    if path is None:
        _lib = lib
    return lib


class SplaError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = load()
        msg = lib.spla_status_string(status).decode()
        extra = lib.spla_last_cuda_error().decode() if status == SPLA_ERR_CUDA else ""
        super().__init__(f"{where}: {msg} ({status}) {extra}".strip())
        self.status = status


def _check(status: int, where: str):
    if status != SPLA_OK:
        raise SplaError(status, where)


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def make_config(*, batch, n_q_heads, n_kv_heads, head_dim, block_size, top_k, max_context, n_sink_blocks=1,
                n_local_blocks=4, kv_dtype="bf16", q_dtype=None, sm_scale=0.0, phi_scale=0.0, rms_eps=0.0,
                flags=0, window_size=0, window_stride=0) -> SplaConfig:
    code = {"bf16": SPLA_BF16, "f32": SPLA_F32}
    return SplaConfig(batch, n_q_heads, n_kv_heads, head_dim, block_size, top_k, max_context, n_sink_blocks,
                      n_local_blocks, code[kv_dtype], code[q_dtype or kv_dtype], sm_scale, phi_scale, rms_eps, flags,
                      window_size, window_stride)


def query_sizes(cfg: SplaConfig) -> SplaSizes:
    sz = SplaSizes()
    _check(load().spla_query_sizes(C.byref(cfg), C.byref(sz)), "spla_query_sizes")
    return sz


@dataclass
class _Bufs:
    k_cache: torch.Tensor
    v_cache: torch.Tensor
    stats: torch.Tensor
    rla_state: torch.Tensor
    tok_lse: torch.Tensor
    seq_lens: torch.Tensor
    workspace: torch.Tensor


NOALLOC_SCRATCH_BYTES = 4 << 20


def select_blocks_noalloc(cfg: SplaConfig, stats: torch.Tensor, seq_lens: torch.Tensor, q: torch.Tensor,
                          sel_idx: torch.Tensor, scores_out: torch.Tensor | None = None,
                          status_out: torch.Tensor | None = None) -> int:
    """Score + select for callers that may not allocate on the device: every tensor is passed in, the kernel's
    scratch is a fixed array inside the library.  Returns the status code (0 = ok) instead of raising, so that a
    caller can fall back to `SplaCache.decode` when the configuration exceeds the fixed scratch.  Calls share
    that scratch: never let two of them overlap on the GPU."""
    assert stats.is_cuda and stats.dtype == torch.float32 and stats.is_contiguous()
    assert seq_lens.dtype == torch.int32 and sel_idx.dtype == torch.int32 and q.is_contiguous()
    with torch.cuda.device(stats.device):
        return load().spla_select_blocks_noalloc(C.byref(cfg), stats.data_ptr(), seq_lens.data_ptr(), q.data_ptr(),
                                                 sel_idx.data_ptr(), _ptr(scores_out), _ptr(status_out), _stream())


def launch_count() -> int:
    """Kernels the library has launched (or recorded into a graph capture) from this thread so far."""
    return int(load().spla_launch_count())


class SplaCache:
    """Owns the device buffers (as torch tensors) of one cache and forwards to the C ABI.

    Shapes follow include/spla.h: k_cache/v_cache [batch, H_kv, max_blocks, B, d], stats
    [batch, H_kv, max_blocks, 2, d] (with strided windows [batch, H_kv, max_blocks, NW, 2, d]; fp32, or bfloat16
    with SPLA_STATS_BF16), rla_state
    [batch, H_kv, d, d], tok_lse [batch, H_kv, max_blocks * B].
    """

    def __init__(self, cfg: SplaConfig, device="cuda:0"):
        self.lib = load()
        self.cfg = cfg
        self.device = torch.device(device)
        sz = query_sizes(cfg)
        self.sizes = sz
        B, d = cfg.block_size, cfg.head_dim
        self.max_blocks = (cfg.max_context + B - 1) // B
        kv_t = torch.bfloat16 if cfg.kv_dtype == SPLA_BF16 else torch.float32
        self.kv_torch_dtype = kv_t
        self.q_torch_dtype = torch.bfloat16 if cfg.q_dtype == SPLA_BF16 else torch.float32
        shp = (cfg.batch, cfg.n_kv_heads, self.max_blocks)
        dev = self.device
        self.bufs = _Bufs(
            k_cache=torch.empty(*shp, B, d, dtype=kv_t, device=dev),
            v_cache=torch.empty(*shp, B, d, dtype=kv_t, device=dev),
            stats=torch.empty(*shp, *((cfg.n_windows,) if cfg.window_size > 0 else ()), 2, d, device=dev,
                              dtype=torch.bfloat16 if cfg.flags & SPLA_STATS_BF16 else torch.float32),
            rla_state=torch.empty(cfg.batch, cfg.n_kv_heads, d, d, dtype=torch.float32, device=dev),
            tok_lse=torch.empty(cfg.batch, cfg.n_kv_heads, self.max_blocks * B, dtype=torch.float32, device=dev),
            seq_lens=torch.empty(cfg.batch, dtype=torch.int32, device=dev),
            workspace=torch.empty(sz.workspace, dtype=torch.uint8, device=dev),
        )
        b = self.bufs
        assert b.k_cache.numel() * b.k_cache.element_size() == sz.k_cache
        assert b.stats.numel() * b.stats.element_size() == sz.stats and b.tok_lse.numel() * 4 == sz.tok_lse
        cb = SplaBuffers(b.k_cache.data_ptr(), b.v_cache.data_ptr(), b.stats.data_ptr(), b.rla_state.data_ptr(),
                         b.tok_lse.data_ptr(), b.seq_lens.data_ptr(), b.workspace.data_ptr(), sz.workspace)
        self.handle = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.spla_init_cache(C.byref(cfg), C.byref(cb), _stream(), C.byref(self.handle)),
                   "spla_init_cache")

    # -- the three calls of the path -------------------------------------------------------------------
    def append_tokens(self, k_new: torch.Tensor, v_new: torch.Tensor, n_new: torch.Tensor | None = None):
        """k_new, v_new: [batch, H_kv, max_new, d] contiguous device tensors of the cache dtype."""
        cfg = self.cfg
        assert k_new.is_cuda and k_new.is_contiguous() and v_new.is_contiguous()
        assert k_new.dtype == self.kv_torch_dtype and v_new.dtype == self.kv_torch_dtype
        assert k_new.shape == v_new.shape and k_new.shape[0] == cfg.batch and k_new.shape[1] == cfg.n_kv_heads
        assert k_new.shape[3] == cfg.head_dim
        if n_new is not None:
            assert n_new.dtype == torch.int32 and n_new.is_cuda and n_new.numel() == cfg.batch
        with torch.cuda.device(self.device):
            _check(self.lib.spla_append_tokens(self.handle, k_new.data_ptr(), v_new.data_ptr(), _ptr(n_new),
                                               k_new.shape[2], _stream()), "spla_append_tokens")

    def decode(self, q: torch.Tensor, rms_weight: torch.Tensor | None, out: torch.Tensor | None = None,
               sel_idx: torch.Tensor | None = None, dbg_o_sparse=None, dbg_o_rla=None) -> torch.Tensor:
        """q: [batch, H_q, d] of the query dtype; returns out [batch, H_q, d] fp32."""
        cfg = self.cfg
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.q_torch_dtype
        assert tuple(q.shape) == (cfg.batch, cfg.n_q_heads, cfg.head_dim)
        if out is None:
            out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.spla_decode(self.handle, q.data_ptr(), _ptr(rms_weight), out.data_ptr(), _ptr(sel_idx),
                                        _ptr(dbg_o_sparse), _ptr(dbg_o_rla), _stream()), "spla_decode")
        return out

    def append_decode(self, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor, rms_weight, out=None,
                      n_new: torch.Tensor | None = None, sel_idx=None, dbg_o_sparse=None, dbg_o_rla=None) -> torch.Tensor:
        """One step: `append_tokens(k_new, v_new, n_new)` then `decode(q, ...)`, as one call."""
        cfg = self.cfg
        assert k_new.is_cuda and k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape
        assert k_new.dtype == self.kv_torch_dtype and v_new.dtype == self.kv_torch_dtype
        assert tuple(k_new.shape[:2]) == (cfg.batch, cfg.n_kv_heads) and k_new.shape[3] == cfg.head_dim
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.q_torch_dtype
        assert tuple(q.shape) == (cfg.batch, cfg.n_q_heads, cfg.head_dim)
        if n_new is not None:
            assert n_new.dtype == torch.int32 and n_new.is_cuda and n_new.numel() == cfg.batch
        if out is None:
            out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.spla_append_decode(self.handle, k_new.data_ptr(), v_new.data_ptr(), _ptr(n_new),
                                               k_new.shape[2], q.data_ptr(), _ptr(rms_weight), out.data_ptr(),
                                               _ptr(sel_idx), _ptr(dbg_o_sparse), _ptr(dbg_o_rla), _stream()),
                   "spla_append_decode")
        return out

    def prefill(self, k_new: torch.Tensor, v_new: torch.Tensor, q: torch.Tensor, rms_weight, out=None, sel_idx=None,
                workspace_bytes: int | None = None) -> torch.Tensor:
        """Prefill-shaped forward: appends T tokens per sequence and returns the output of every position.
        k_new, v_new [batch, H_kv, T, d]; q [batch, T, H_q, d]; out [batch, T, H_q, d] fp32;
        sel_idx (optional) [batch, T, H_kv, top_k] int32.  `workspace_bytes`: scratch to use (default: the size the
        library recommends; at least the minimum it reports)."""
        cfg = self.cfg
        T = k_new.shape[2]
        assert k_new.is_cuda and k_new.is_contiguous() and v_new.is_contiguous() and k_new.shape == v_new.shape
        assert k_new.dtype == self.kv_torch_dtype and tuple(k_new.shape[:2]) == (cfg.batch, cfg.n_kv_heads)
        assert q.is_contiguous() and q.dtype == self.q_torch_dtype and tuple(q.shape) == (cfg.batch, T, cfg.n_q_heads, cfg.head_dim)
        lo, good = C.c_size_t(), C.c_size_t()
        _check(self.lib.spla_query_prefill_workspace(C.byref(cfg), T, C.byref(lo), C.byref(good)), "spla_query_prefill_workspace")
        nbytes = good.value if workspace_bytes is None else max(int(workspace_bytes), lo.value)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        if out is None:
            out = torch.empty(cfg.batch, T, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.spla_prefill(self.handle, k_new.data_ptr(), v_new.data_ptr(), q.data_ptr(), T, _ptr(rms_weight),
                                         out.data_ptr(), _ptr(sel_idx), ws.data_ptr(), nbytes, _stream()), "spla_prefill")
        self._prefill_ws = ws                                  # keep the scratch alive until the stream has used it
        return out

    def select(self, q: torch.Tensor, sel_idx: torch.Tensor | None = None) -> torch.Tensor:
        """Block scores + top-k only; returns sel_idx [batch, H_kv, top_k] int32."""
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.q_torch_dtype
        if sel_idx is None:
            sel_idx = self.new_sel_buffer()
        with torch.cuda.device(self.device):
            _check(self.lib.spla_select(self.handle, q.data_ptr(), sel_idx.data_ptr(), _stream()), "spla_select")
        return sel_idx

    def decode_selected(self, q, rms_weight, sel_in: torch.Tensor, out=None, dbg_o_sparse=None, dbg_o_rla=None):
        cfg = self.cfg
        assert q.is_cuda and q.is_contiguous() and q.dtype == self.q_torch_dtype
        assert sel_in.dtype == torch.int32 and sel_in.is_contiguous()
        assert tuple(sel_in.shape) == (cfg.batch, cfg.n_kv_heads, cfg.top_k)
        if out is None:
            out = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.spla_decode_selected(self.handle, q.data_ptr(), _ptr(rms_weight), sel_in.data_ptr(),
                                                 out.data_ptr(), _ptr(dbg_o_sparse), _ptr(dbg_o_rla), _stream()),
                   "spla_decode_selected")
        return out

    # -- helpers ------------------------------------------------------------------------------------------
    def scores(self) -> torch.Tensor:
        out = torch.empty(self.cfg.batch, self.cfg.n_kv_heads, self.max_blocks, dtype=torch.float32,
                          device=self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.spla_copy_scores(self.handle, out.data_ptr(), _stream()), "spla_copy_scores")
        return out

    def sync_status(self) -> int:
        with torch.cuda.device(self.device):
            return self.lib.spla_sync_status(self.handle, _stream())

    def debug_wait_hook(self, max_wait_polls: int, extra_expected_bytes: int):
        """Test hook: wait limit of the decode kernels' copy barriers and bytes they expect in excess (see spla.h)."""
        _check(self.lib.spla_debug_wait_hook(self.handle, max_wait_polls, extra_expected_bytes), "spla_debug_wait_hook")

    def set_length_bound(self, n: int):
        _check(self.lib.spla_set_length_bound(self.handle, n), "spla_set_length_bound")

    def new_sel_buffer(self) -> torch.Tensor:
        return torch.empty(self.cfg.batch, self.cfg.n_kv_heads, self.cfg.top_k, dtype=torch.int32, device=self.device)

    def close(self):
        if getattr(self, "handle", None) is not None and self.handle.value:
            self.lib.spla_destroy_cache(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
