"""ctypes binding over libmtla.so: argument marshalling only.

Every function here has the name of the C call it wraps (see include/mtla.h) and passes
torch tensors by data_ptr(); torch is used for device memory and streams, nothing else.
There is no CPU fallback: if the library cannot be built or loaded the import of a symbol
raises, and every non-zero status raises MTLAError.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass

import numpy as np
import torch

from .build import LIB_PATH, build_library

MTLA_DTYPE_FP32, MTLA_DTYPE_BF16 = 0, 1
MTLA_PATH_AUTO, MTLA_PATH_CUDA_CORE = 0, 1
_DTYPES = {torch.float32: MTLA_DTYPE_FP32, torch.bfloat16: MTLA_DTYPE_BF16,
           "fp32": MTLA_DTYPE_FP32, "bf16": MTLA_DTYPE_BF16}
_TORCH_DTYPES = {MTLA_DTYPE_FP32: torch.float32, MTLA_DTYPE_BF16: torch.bfloat16}

WEIGHT_NAMES = ("w_q", "w_qr", "w_r", "w_kr", "ln_gamma", "ln_beta", "w_k", "w_v", "w_o",
                "hyp_c_w", "hyp_c_b", "hyp_pe_w", "hyp_pe_b")

EXPORTED_SYMBOLS = (
    "mtla_arena_bytes", "mtla_create", "mtla_prefill", "mtla_decode_step",
    "mtla_decode_step_host", "mtla_cache_bytes", "mtla_destroy", "mtla_reset", "mtla_position",
    "mtla_cache_export", "mtla_cache_import", "mtla_check", "mtla_launch_count",
    "mtla_attention_variant", "mtla_attention_gang", "mtla_error_string", "mtla_profile_begin", "mtla_profile_end",
    "mtla_profile_end_stages", "mtla_decode_step_static", "mtla_profile_begin_attention",
    "mtla_arena_bytes_paged", "mtla_create_paged", "mtla_prefill_seqs", "mtla_beam_reorder",
    "mtla_seq_positions", "mtla_pages_in_use", "mtla_cache_export_seq", "mtla_cache_import_seqs",
    "mtla_page_pool_create", "mtla_page_pool_destroy", "mtla_page_pool_prepare",
    "mtla_page_pool_reorder", "mtla_page_pool_row", "mtla_page_pool_in_use", "mtla_page_pool_ref",
    "mtla_baseline_arena_bytes", "mtla_baseline_create", "mtla_selftest_wait_timeout",
    "mtla_clear_error", "mtla_stack_arena_bytes", "mtla_stack_create", "mtla_stack_prefill",
    "mtla_stack_decode_step", "mtla_stack_cache_bytes", "mtla_stack_layer", "mtla_stack_reset",
    "mtla_stack_check", "mtla_stack_launch_count", "mtla_stack_destroy",
    "mtla_train_workspace_bytes", "mtla_train_backward")

PAGE_SLOTS = 64

DECODE_STAGES = ("input_proj", "norm_gate_update", "absorb", "attention", "combine", "value_proj",
                 "output_proj")


class MTLAError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {error_string(status)} ({status})")


class mtla_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "d_model", "n_heads", "head_dim", "latent_rank", "rope_dim", "stride", "hyper_dim",
        "max_batch", "max_tokens", "max_prefill_tokens", "dtype")] + [
        ("ln_eps", ctypes.c_float), ("rope_theta", ctypes.c_float),
        ("kernel_path", ctypes.c_int32)]


class mtla_paging(ctypes.Structure):
    _fields_ = [("page_slots", ctypes.c_int32), ("n_pages", ctypes.c_int32)]


class mtla_baseline_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in (
        "d_model", "n_heads", "n_kv_heads", "head_dim", "max_batch", "max_tokens")] + [
        ("rope_theta", ctypes.c_float)]


class mtla_baseline_weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("w_q", "w_k", "w_v", "w_o")]


class mtla_weights(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in WEIGHT_NAMES]


LAYER_EXTRA_NAMES = ("ln1_gamma", "ln1_beta", "ln2_gamma", "ln2_beta", "w1", "b1", "w2", "b2")


class mtla_layer_weights(ctypes.Structure):
    _fields_ = [("attn", mtla_weights)] + [(n, ctypes.c_void_p) for n in LAYER_EXTRA_NAMES]


class mtla_grads(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in WEIGHT_NAMES]


class mtla_stack_config(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("ln_eps", ctypes.c_float)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads (building first if needed) the CUDA library; raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    build_library()
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
    cfg_p, w_p = ctypes.POINTER(mtla_config), ctypes.POINTER(mtla_weights)
    pg_p, i32_p = ctypes.POINTER(mtla_paging), ctypes.POINTER(ctypes.c_int32)
    sigs = {
        "mtla_baseline_arena_bytes": (sz, [ctypes.POINTER(mtla_baseline_config)]),
        "mtla_baseline_create": (ctypes.c_int, [ctypes.POINTER(mtla_baseline_config),
                                                ctypes.POINTER(mtla_baseline_weights), vp, sz, vp,
                                                ctypes.POINTER(vp)]),
        "mtla_arena_bytes_paged": (sz, [cfg_p, pg_p]),
        "mtla_create_paged": (ctypes.c_int, [cfg_p, pg_p, w_p, vp, sz, vp, ctypes.POINTER(vp)]),
        "mtla_prefill_seqs": (ctypes.c_int, [vp, i32, vp, i32, i32, vp, vp]),
        "mtla_beam_reorder": (ctypes.c_int, [vp, i32_p, i32, vp]),
        "mtla_cache_import_seqs": (ctypes.c_int, [vp, i32, vp, i32, i32, vp]),
        "mtla_seq_positions": (ctypes.c_int, [vp, i32_p, i32]),
        "mtla_pages_in_use": (ctypes.c_int64, [vp]),
        "mtla_cache_export_seq": (ctypes.c_int, [vp, i32, vp, sz, vp]),
        "mtla_page_pool_create": (vp, [i32, i32, i32]),
        "mtla_page_pool_destroy": (None, [vp]),
        "mtla_page_pool_prepare": (ctypes.c_int, [vp, i32, i32, i32, i32_p, i32]),
        "mtla_page_pool_reorder": (ctypes.c_int, [vp, i32_p, i32, i32]),
        "mtla_page_pool_row": (ctypes.c_int, [vp, i32, i32_p, i32]),
        "mtla_page_pool_in_use": (ctypes.c_int, [vp]),
        "mtla_page_pool_ref": (ctypes.c_int, [vp, i32]),
        "mtla_arena_bytes": (sz, [cfg_p]),
        "mtla_create": (ctypes.c_int, [cfg_p, w_p, vp, sz, vp, ctypes.POINTER(vp)]),
        "mtla_prefill": (ctypes.c_int, [vp, vp, i32, i32, vp, vp]),
        "mtla_decode_step": (ctypes.c_int, [vp, vp, i32, vp, vp]),
        "mtla_decode_step_host": (ctypes.c_int, [vp, vp, i32, vp, vp]),
        "mtla_decode_step_static": (ctypes.c_int, [vp, vp, i32, vp, vp]),
        "mtla_cache_bytes": (sz, [vp]),
        "mtla_destroy": (ctypes.c_int, [vp]),
        "mtla_reset": (ctypes.c_int, [vp]),
        "mtla_position": (ctypes.c_int, [vp, ctypes.POINTER(i32), ctypes.POINTER(i32),
                                         ctypes.POINTER(i32)]),
        "mtla_cache_export": (ctypes.c_int, [vp, vp, sz, vp]),
        "mtla_cache_import": (ctypes.c_int, [vp, vp, i32, i32, vp]),
        "mtla_check": (ctypes.c_int, [vp, vp]),
        "mtla_launch_count": (ctypes.c_int64, [vp]),
        "mtla_attention_variant": (ctypes.c_char_p, [vp]),
        "mtla_attention_gang": (ctypes.c_int32, [vp]),
        "mtla_profile_begin": (ctypes.c_int, [vp, i32]),
        "mtla_profile_begin_attention": (ctypes.c_int, [vp, i32]),
        "mtla_profile_end": (ctypes.c_int, [vp, ctypes.POINTER(ctypes.c_double),
                                            ctypes.POINTER(i32)]),
        "mtla_profile_end_stages": (ctypes.c_int, [vp, ctypes.POINTER(ctypes.c_double),
                                                   ctypes.POINTER(i32)]),
        "mtla_error_string": (ctypes.c_char_p, [ctypes.c_int]),
        "mtla_stack_arena_bytes": (sz, [cfg_p, ctypes.POINTER(mtla_stack_config)]),
        "mtla_stack_create": (ctypes.c_int, [cfg_p, ctypes.POINTER(mtla_stack_config),
                                             ctypes.POINTER(mtla_layer_weights), vp, vp, vp, sz, vp,
                                             ctypes.POINTER(vp)]),
        "mtla_stack_prefill": (ctypes.c_int, [vp, vp, i32, i32, vp, vp]),
        "mtla_stack_decode_step": (ctypes.c_int, [vp, vp, i32, vp, vp]),
        "mtla_stack_cache_bytes": (sz, [vp]),
        "mtla_stack_layer": (vp, [vp, i32]),
        "mtla_stack_reset": (ctypes.c_int, [vp]),
        "mtla_stack_check": (ctypes.c_int, [vp, vp]),
        "mtla_stack_launch_count": (ctypes.c_int64, [vp]),
        "mtla_stack_destroy": (ctypes.c_int, [vp]),
        "mtla_train_workspace_bytes": (sz, [vp, i32, i32]),
        "mtla_train_backward": (ctypes.c_int, [vp, vp, vp, i32, i32, vp, ctypes.POINTER(mtla_grads), vp,
                                               sz, vp]),
        "mtla_selftest_wait_timeout": (ctypes.c_int, [vp, i32, vp]),
        "mtla_clear_error": (ctypes.c_int, [vp, vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def error_string(status: int) -> str:
    return load_library().mtla_error_string(status).decode()


def _check(status: int, where: str) -> None:
    if status != 0:
        raise MTLAError(status, where)


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


@dataclass
class Handle:
    """A live layer: the C handle plus the torch tensors that must outlive it."""
    ptr: int
    config: mtla_config
    arena: torch.Tensor
    dtype: torch.dtype
    device: torch.device
    kv_heads: int = 0      # comparison layers: key/value heads per sequence (0: an MTLA layer)


def make_config(*, d_model, n_heads, head_dim, latent_rank, rope_dim, stride, hyper_dim=0,
                max_batch, max_tokens, max_prefill_tokens=0, dtype="bf16", ln_eps=0.0,
                rope_theta=0.0, kernel_path=0) -> mtla_config:
    return mtla_config(d_model, n_heads, head_dim, latent_rank, rope_dim, stride, hyper_dim,
                       max_batch, max_tokens, max_prefill_tokens, _DTYPES[dtype], ln_eps,
                       rope_theta, kernel_path)


def mtla_arena_bytes(cfg: mtla_config) -> int:
    return load_library().mtla_arena_bytes(ctypes.byref(cfg))


def mtla_create(cfg: mtla_config, weights: dict, device="cuda:0", stream=None,
                paging: mtla_paging | None = None) -> Handle:
    """weights: name -> CUDA tensor, row-major [in][out], dtype matching cfg.dtype.
    With `paging` the call is mtla_create_paged."""
    lib = load_library()
    nbytes = (lib.mtla_arena_bytes(ctypes.byref(cfg)) if paging is None
              else lib.mtla_arena_bytes_paged(ctypes.byref(cfg), ctypes.byref(paging)))
    if nbytes == 0:
        raise MTLAError(-2, "mtla_arena_bytes")
    device = torch.device(device)
    dtype = _TORCH_DTYPES[cfg.dtype]
    with torch.cuda.device(device):
        arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        base = (arena.data_ptr() + 1023) // 1024 * 1024
        w = mtla_weights()
        keep = []
        for name in WEIGHT_NAMES:
            t = weights.get(name)
            if t is None:
                setattr(w, name, None)
                continue
            if t.dtype != dtype or not t.is_cuda:
                raise TypeError(f"weight {name}: expected a {dtype} CUDA tensor")
            t = t.contiguous()
            keep.append(t)
            setattr(w, name, t.data_ptr())
        out = ctypes.c_void_p()
        st = _stream_ptr(stream)
        if paging is None:
            _check(lib.mtla_create(ctypes.byref(cfg), ctypes.byref(w), base, nbytes, st,
                                   ctypes.byref(out)), "mtla_create")
        else:
            _check(lib.mtla_create_paged(ctypes.byref(cfg), ctypes.byref(paging), ctypes.byref(w),
                                         base, nbytes, st, ctypes.byref(out)), "mtla_create_paged")
        torch.cuda.current_stream().synchronize()   # packing done: weight tensors may be freed
    return Handle(out.value, cfg, arena, dtype, device)


def _expect(t: torch.Tensor, h: Handle, shape, name: str, cuda=True) -> None:
    if t.dtype != h.dtype or tuple(t.shape) != tuple(shape) or not t.is_contiguous():
        raise TypeError(f"{name}: expected contiguous {h.dtype} tensor of shape {tuple(shape)}")
    if cuda != t.is_cuda:
        raise TypeError(f"{name}: expected a {'CUDA' if cuda else 'host'} tensor")


def mtla_prefill(h: Handle, x: torch.Tensor, y: torch.Tensor | None = None, want_output=True,
                 stream=None):
    """x [B][T][d] on the device; returns y [B][T][d] (or None when want_output is False)."""
    b, t, d = x.shape
    _expect(x, h, (b, t, h.config.d_model), "x")
    if want_output and y is None:
        y = torch.empty_like(x)
    if y is not None:
        _expect(y, h, x.shape, "y")
    _check(load_library().mtla_prefill(h.ptr, x.data_ptr(), b, t,
                                       y.data_ptr() if y is not None else None,
                                       _stream_ptr(stream)), "mtla_prefill")
    return y


def mtla_baseline_create(*, d_model, n_heads, n_kv_heads, head_dim, max_batch, max_tokens,
                         weights: dict, rope_theta=0.0, device="cuda:0", stream=None) -> Handle:
    """A comparison layer (MHA: n_kv_heads = n_heads, MQA: 1, GQA in between), bf16.
    weights: w_q, w_k, w_v, w_o as CUDA bf16 tensors, row-major [in][out]."""
    lib = load_library()
    cfg = mtla_baseline_config(d_model, n_heads, n_kv_heads, head_dim, max_batch, max_tokens,
                               rope_theta)
    nbytes = lib.mtla_baseline_arena_bytes(ctypes.byref(cfg))
    if nbytes == 0:
        raise MTLAError(-2, "mtla_baseline_arena_bytes")
    device = torch.device(device)
    with torch.cuda.device(device):
        arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        base = (arena.data_ptr() + 1023) // 1024 * 1024
        w = mtla_baseline_weights()
        keep = []
        for name in ("w_q", "w_k", "w_v", "w_o"):
            t = weights[name]
            if t.dtype != torch.bfloat16 or not t.is_cuda:
                raise TypeError(f"weight {name}: expected a bfloat16 CUDA tensor")
            t = t.contiguous()
            keep.append(t)
            setattr(w, name, t.data_ptr())
        out = ctypes.c_void_p()
        _check(lib.mtla_baseline_create(ctypes.byref(cfg), ctypes.byref(w), base, nbytes,
                                        _stream_ptr(stream), ctypes.byref(out)), "mtla_baseline_create")
        torch.cuda.current_stream().synchronize()
    # The generic calls read d_model / widths from an mtla_config: give them one that describes
    # the cache rows of this layer (2 d_h elements per row, n_kv_heads planes per sequence).
    shim = make_config(d_model=d_model, n_heads=n_heads, head_dim=head_dim, latent_rank=2 * head_dim,
                       rope_dim=0, stride=1, max_batch=max_batch, max_tokens=max_tokens, dtype="bf16")
    h = Handle(out.value, shim, arena, torch.bfloat16, device)
    h.kv_heads = n_kv_heads
    return h


def mtla_create_paged(cfg: mtla_config, weights: dict, n_pages: int = 0, device="cuda:0",
                      stream=None) -> Handle:
    """A layer whose cache lives in 64-slot pages, with a token count per sequence."""
    return mtla_create(cfg, weights, device, stream, paging=mtla_paging(PAGE_SLOTS, n_pages))


def mtla_arena_bytes_paged(cfg: mtla_config, n_pages: int = 0) -> int:
    pg = mtla_paging(PAGE_SLOTS, n_pages)
    return load_library().mtla_arena_bytes_paged(ctypes.byref(cfg), ctypes.byref(pg))


def mtla_prefill_seqs(h: Handle, seq0: int, x: torch.Tensor, y: torch.Tensor | None = None,
                      want_output=True, stream=None):
    """Prefill of the empty sequences seq0 .. seq0 + B - 1 of a paged handle; x [B][T][d]."""
    b, t, d = x.shape
    _expect(x, h, (b, t, h.config.d_model), "x")
    if want_output and y is None:
        y = torch.empty_like(x)
    if y is not None:
        _expect(y, h, x.shape, "y")
    _check(load_library().mtla_prefill_seqs(h.ptr, seq0, x.data_ptr(), b, t,
                                            y.data_ptr() if y is not None else None,
                                            _stream_ptr(stream)), "mtla_prefill_seqs")
    return y


def mtla_cache_import_seqs(h: Handle, seq0: int, cache: torch.Tensor, tokens: int, stream=None) -> None:
    """cache [B][ceil(tokens/s)][r + d_R] on the device, for the empty sequences seq0 .. seq0 + B - 1."""
    b = cache.shape[0]
    slots = -(-tokens // h.config.stride)
    _expect(cache, h, (b, slots, h.config.latent_rank + h.config.rope_dim), "cache")
    _check(load_library().mtla_cache_import_seqs(h.ptr, seq0, cache.data_ptr(), b, tokens,
                                                 _stream_ptr(stream)), "mtla_cache_import_seqs")


def _i32_array(values):
    """int32 C array of a sequence; a contiguous numpy int32 array is passed as it is (no copy),
    which is what a decoding loop that calls once per step should hand over."""
    if isinstance(values, np.ndarray) and values.dtype == np.int32 and values.flags.c_contiguous:
        return values.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    return (ctypes.c_int32 * len(values))(*[int(v) for v in values])


def mtla_beam_reorder(h: Handle, parents, stream=None) -> None:
    """Sequence b of the new batch continues old sequence parents[b]."""
    _check(load_library().mtla_beam_reorder(h.ptr, _i32_array(parents), len(parents),
                                            _stream_ptr(stream)), "mtla_beam_reorder")


def mtla_seq_positions(h: Handle) -> list[int]:
    """Tokens consumed by each sequence of the batch."""
    batch = mtla_position(h)[2]
    out = (ctypes.c_int32 * max(batch, 1))()
    _check(load_library().mtla_seq_positions(h.ptr, out, batch), "mtla_seq_positions")
    return list(out)[:batch]


def mtla_pages_in_use(h: Handle) -> int:
    return load_library().mtla_pages_in_use(h.ptr)


def mtla_cache_export_seq(h: Handle, seq: int, stream=None) -> torch.Tensor:
    """The slots of one sequence as a tensor [slots][r + d_R]."""
    tokens = mtla_seq_positions(h)[seq]
    slots = -(-tokens // h.config.stride)
    width = h.config.latent_rank + h.config.rope_dim
    out = torch.empty(slots, width, dtype=h.dtype, device=h.device)
    if out.numel():
        _check(load_library().mtla_cache_export_seq(h.ptr, seq, out.data_ptr(),
                                                    out.numel() * out.element_size(),
                                                    _stream_ptr(stream)), "mtla_cache_export_seq")
    return out


class PagePool:
    """The library's host-only page bookkeeping (mtla_page_pool_*); needs no GPU."""

    def __init__(self, n_pages: int, max_seqs: int, max_pages_per_seq: int):
        self._lib = load_library()
        self.max_pages = max_pages_per_seq
        self.ptr = self._lib.mtla_page_pool_create(n_pages, max_seqs, max_pages_per_seq)
        if not self.ptr:
            raise MTLAError(-1, "mtla_page_pool_create")

    def close(self) -> None:
        if self.ptr:
            self._lib.mtla_page_pool_destroy(self.ptr)
            self.ptr = None

    def prepare(self, seq: int, n_slots: int, write_slot: int = -1) -> list[tuple[int, int, int]]:
        """Returns the page copies (source, destination, rows) the call implies."""
        buf = (ctypes.c_int32 * 6)()
        n = self._lib.mtla_page_pool_prepare(self.ptr, seq, n_slots, write_slot, buf, 2)
        _check(min(n, 0), "mtla_page_pool_prepare")
        return [(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(n)]

    def reorder(self, parents, n_old: int) -> None:
        _check(self._lib.mtla_page_pool_reorder(self.ptr, _i32_array(parents), len(parents), n_old),
               "mtla_page_pool_reorder")

    def row(self, seq: int) -> list[int]:
        buf = (ctypes.c_int32 * self.max_pages)()
        n = self._lib.mtla_page_pool_row(self.ptr, seq, buf, self.max_pages)
        _check(min(n, 0), "mtla_page_pool_row")
        return list(buf)[:n]

    def in_use(self) -> int:
        return self._lib.mtla_page_pool_in_use(self.ptr)

    def ref(self, page: int) -> int:
        return self._lib.mtla_page_pool_ref(self.ptr, page)


def mtla_decode_step(h: Handle, x: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """x [B][d] on the device; returns y [B][d]."""
    b = x.shape[0]
    _expect(x, h, (b, h.config.d_model), "x")
    if y is None:
        y = torch.empty_like(x)
    _expect(y, h, x.shape, "y")
    _check(load_library().mtla_decode_step(h.ptr, x.data_ptr(), b, y.data_ptr(),
                                           _stream_ptr(stream)), "mtla_decode_step")
    return y


def mtla_decode_step_static(h: Handle, x: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """mtla_decode_step with the attention split workspace taken from the library's built-in
    static array instead of allocated memory; x, y [B][d] on the device.  Raises MTLAError(-9)
    when the batch and layer shape need more than that array holds."""
    b = x.shape[0]
    _expect(x, h, (b, h.config.d_model), "x")
    if y is None:
        y = torch.empty_like(x)
    _expect(y, h, x.shape, "y")
    _check(load_library().mtla_decode_step_static(h.ptr, x.data_ptr(), b, y.data_ptr(),
                                                  _stream_ptr(stream)), "mtla_decode_step_static")
    return y


def mtla_decode_step_host(h: Handle, x_host: torch.Tensor, y_host: torch.Tensor, stream=None):
    """x_host, y_host [B][d] in (preferably pinned) host memory; copies are enqueued on the stream."""
    b = x_host.shape[0]
    _expect(x_host, h, (b, h.config.d_model), "x_host", cuda=False)
    _expect(y_host, h, x_host.shape, "y_host", cuda=False)
    _check(load_library().mtla_decode_step_host(h.ptr, x_host.data_ptr(), b, y_host.data_ptr(),
                                                _stream_ptr(stream)), "mtla_decode_step_host")
    return y_host


def mtla_cache_bytes(h: Handle) -> int:
    return load_library().mtla_cache_bytes(h.ptr)


def mtla_destroy(h: Handle) -> None:
    if h.ptr:
        _check(load_library().mtla_destroy(h.ptr), "mtla_destroy")
        h.ptr = 0


def mtla_reset(h: Handle) -> None:
    _check(load_library().mtla_reset(h.ptr), "mtla_reset")


def mtla_position(h: Handle) -> tuple[int, int, int]:
    """(tokens, slots, batch)."""
    t, s, b = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(load_library().mtla_position(h.ptr, ctypes.byref(t), ctypes.byref(s),
                                        ctypes.byref(b)), "mtla_position")
    return t.value, s.value, b.value


def mtla_cache_export(h: Handle, stream=None) -> torch.Tensor:
    """The cache in use as a tensor [B][slots][r + d_R]."""
    _, slots, batch = mtla_position(h)
    width = h.config.latent_rank + h.config.rope_dim
    shape = (batch, slots, width) if h.kv_heads == 0 else (batch, h.kv_heads, slots, width)
    out = torch.empty(*shape, dtype=h.dtype, device=h.device)
    if out.numel():
        _check(load_library().mtla_cache_export(h.ptr, out.data_ptr(),
                                                out.numel() * out.element_size(),
                                                _stream_ptr(stream)), "mtla_cache_export")
    return out


def mtla_cache_import(h: Handle, cache: torch.Tensor, tokens: int, stream=None) -> None:
    """cache [B][ceil(tokens/s)][r + d_R] on the device."""
    b = cache.shape[0]
    slots = -(-tokens // h.config.stride)
    width = h.config.latent_rank + h.config.rope_dim
    _expect(cache, h, (b, slots, width) if h.kv_heads == 0 else (b, h.kv_heads, slots, width), "cache")
    _check(load_library().mtla_cache_import(h.ptr, cache.data_ptr(), b, tokens,
                                            _stream_ptr(stream)), "mtla_cache_import")


def mtla_check(h: Handle, stream=None) -> None:
    _check(load_library().mtla_check(h.ptr, _stream_ptr(stream)), "mtla_check")


def mtla_selftest_wait_timeout(h: Handle, budget_us: int, stream=None) -> None:
    """Enqueues the one-CTA kernel whose bounded wait runs out after budget_us microseconds."""
    _check(load_library().mtla_selftest_wait_timeout(h.ptr, budget_us, _stream_ptr(stream)),
           "mtla_selftest_wait_timeout")


def mtla_clear_error(h: Handle, stream=None) -> None:
    _check(load_library().mtla_clear_error(h.ptr, _stream_ptr(stream)), "mtla_clear_error")


def mtla_launch_count(h: Handle) -> int:
    return load_library().mtla_launch_count(h.ptr)


def mtla_attention_gang(h: Handle) -> int:
    """Gang size of the latest decode step's attention launch (see include/mtla.h)."""
    return int(load_library().mtla_attention_gang(h.ptr))


def mtla_attention_variant(h: Handle) -> str:
    return load_library().mtla_attention_variant(h.ptr).decode()


def mtla_profile_begin(h: Handle, max_steps: int) -> None:
    _check(load_library().mtla_profile_begin(h.ptr, max_steps), "mtla_profile_begin")


def mtla_profile_begin_attention(h: Handle, max_steps: int) -> None:
    _check(load_library().mtla_profile_begin_attention(h.ptr, max_steps),
           "mtla_profile_begin_attention")


def mtla_profile_end(h: Handle) -> tuple[float, int]:
    """(summed decode-attention kernel time in ms, steps covered)."""
    ms, steps = ctypes.c_double(), ctypes.c_int32()
    _check(load_library().mtla_profile_end(h.ptr, ctypes.byref(ms), ctypes.byref(steps)),
           "mtla_profile_end")
    return ms.value, steps.value


def mtla_profile_end_stages(h: Handle) -> tuple[dict, int]:
    """({stage name: summed milliseconds}, steps covered) for the decode step's kernels."""
    ms, steps = (ctypes.c_double * len(DECODE_STAGES))(), ctypes.c_int32()
    _check(load_library().mtla_profile_end_stages(h.ptr, ms, ctypes.byref(steps)),
           "mtla_profile_end_stages")
    return dict(zip(DECODE_STAGES, list(ms))), steps.value


# --------------------------------------------------------------------------- decoder stacks

@dataclass
class Stack:
    """A live decoder stack: the C object plus the arena that must outlive it."""
    ptr: int
    config: mtla_config
    n_layers: int
    d_ff: int
    arena: torch.Tensor
    dtype: torch.dtype
    device: torch.device


def mtla_stack_arena_bytes(cfg: mtla_config, n_layers: int, d_ff: int) -> int:
    sc = mtla_stack_config(n_layers, d_ff, 0.0)
    return load_library().mtla_stack_arena_bytes(ctypes.byref(cfg), ctypes.byref(sc))


def mtla_stack_create(cfg: mtla_config, n_layers: int, d_ff: int, weights: dict, ln_eps: float = 0.0,
                      device="cuda:0", stream=None) -> Stack:
    """weights: {"layers": [per-layer dict of the attention weights plus ln1_gamma .. b2],
    "lnf_gamma", "lnf_beta"}, CUDA tensors of cfg.dtype, matrices row-major [in][out]."""
    lib = load_library()
    sc = mtla_stack_config(n_layers, d_ff, ln_eps)
    nbytes = lib.mtla_stack_arena_bytes(ctypes.byref(cfg), ctypes.byref(sc))
    if nbytes == 0:
        raise MTLAError(-2, "mtla_stack_arena_bytes")
    device = torch.device(device)
    dtype = _TORCH_DTYPES[cfg.dtype]
    keep = []

    def ptr(t, name):
        if t is None:
            return None
        if t.dtype != dtype or not t.is_cuda:
            raise TypeError(f"weight {name}: expected a {dtype} CUDA tensor")
        t = t.contiguous()
        keep.append(t)
        return t.data_ptr()

    with torch.cuda.device(device):
        arena = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
        base = (arena.data_ptr() + 1023) // 1024 * 1024
        arr = (mtla_layer_weights * n_layers)()
        for n, lw in enumerate(weights["layers"]):
            for name in WEIGHT_NAMES:
                setattr(arr[n].attn, name, ptr(lw.get(name), name))
            for name in LAYER_EXTRA_NAMES:
                setattr(arr[n], name, ptr(lw[name], name))
        out = ctypes.c_void_p()
        _check(lib.mtla_stack_create(ctypes.byref(cfg), ctypes.byref(sc), arr,
                                     ptr(weights["lnf_gamma"], "lnf_gamma"),
                                     ptr(weights["lnf_beta"], "lnf_beta"), base, nbytes,
                                     _stream_ptr(stream), ctypes.byref(out)), "mtla_stack_create")
        torch.cuda.current_stream().synchronize()   # packing done: weight tensors may be freed
    return Stack(out.value, cfg, n_layers, d_ff, arena, dtype, device)


def mtla_stack_prefill(s: Stack, x: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """x [B][T][d] on the device; returns the stack's output [B][T][d]."""
    b, t, d = x.shape
    _expect(x, s, (b, t, s.config.d_model), "x")
    if y is None:
        y = torch.empty_like(x)
    _expect(y, s, x.shape, "y")
    _check(load_library().mtla_stack_prefill(s.ptr, x.data_ptr(), b, t, y.data_ptr(),
                                             _stream_ptr(stream)), "mtla_stack_prefill")
    return y


def mtla_stack_decode_step(s: Stack, x: torch.Tensor, y: torch.Tensor | None = None, stream=None):
    """x [B][d] on the device; returns the stack's output [B][d]."""
    b = x.shape[0]
    _expect(x, s, (b, s.config.d_model), "x")
    if y is None:
        y = torch.empty_like(x)
    _expect(y, s, x.shape, "y")
    _check(load_library().mtla_stack_decode_step(s.ptr, x.data_ptr(), b, y.data_ptr(),
                                                 _stream_ptr(stream)), "mtla_stack_decode_step")
    return y


def mtla_stack_cache_bytes(s: Stack) -> int:
    return load_library().mtla_stack_cache_bytes(s.ptr)


def mtla_stack_layer(s: Stack, layer: int) -> Handle:
    """The attention handle of one layer, borrowed from the stack (never destroy it)."""
    p = load_library().mtla_stack_layer(s.ptr, layer)
    if not p:
        raise MTLAError(-1, "mtla_stack_layer")
    return Handle(p, s.config, s.arena, s.dtype, s.device)


def mtla_stack_reset(s: Stack) -> None:
    _check(load_library().mtla_stack_reset(s.ptr), "mtla_stack_reset")


def mtla_stack_check(s: Stack, stream=None) -> None:
    _check(load_library().mtla_stack_check(s.ptr, _stream_ptr(stream)), "mtla_stack_check")


def mtla_stack_launch_count(s: Stack) -> int:
    return load_library().mtla_stack_launch_count(s.ptr)


def mtla_stack_destroy(s: Stack) -> None:
    if s.ptr:
        _check(load_library().mtla_stack_destroy(s.ptr), "mtla_stack_destroy")
        s.ptr = 0


# --------------------------------------------------------------------------- training path

def weight_shapes(cfg: mtla_config) -> dict:
    """Shapes of the parameters (and of their gradients), row-major [in][out]."""
    d, nh, dh, r, dr = cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.latent_rank, cfg.rope_dim
    dw = cfg.hyper_dim or r // 4
    return {"w_q": (d, nh * dh), "w_qr": (d, nh * dr), "w_r": (d, r), "w_kr": (d, dr),
            "ln_gamma": (r,), "ln_beta": (r,), "w_k": (r, nh * dh), "w_v": (r, nh * dh),
            "w_o": (nh * dh, d), "hyp_c_w": (r, dw), "hyp_c_b": (dw,), "hyp_pe_w": (r, dw),
            "hyp_pe_b": (dw,)}


def mtla_train_backward(h: Handle, x: torch.Tensor, dy: torch.Tensor, stream=None):
    """The reverse of the mtla_prefill(h, x) that must directly precede this call.
    x, dy [B][T][d] fp32 on the device.  Returns (dx, {parameter name: gradient})."""
    b, t, d = x.shape
    _expect(x, h, (b, t, h.config.d_model), "x")
    _expect(dy, h, x.shape, "dy")
    lib = load_library()
    nbytes = lib.mtla_train_workspace_bytes(h.ptr, b, t)
    if nbytes == 0:
        raise MTLAError(-2, "mtla_train_workspace_bytes")
    with torch.cuda.device(h.device):
        ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=h.device)
        base = (ws.data_ptr() + 255) // 256 * 256
        dx = torch.empty_like(x)
        grads = {n: torch.empty(*shape, dtype=torch.float32, device=h.device)
                 for n, shape in weight_shapes(h.config).items()}
        g = mtla_grads(*[grads[n].data_ptr() for n in WEIGHT_NAMES])
        _check(lib.mtla_train_backward(h.ptr, x.data_ptr(), dy.data_ptr(), b, t, dx.data_ptr(),
                                       ctypes.byref(g), base, nbytes, _stream_ptr(stream)),
               "mtla_train_backward")
        torch.cuda.current_stream().synchronize()     # the workspace is released on return
    return dx, grads
