"""ctypes binding of libswaa.so: argument marshalling only.

Every function has the name of the C entry point it forwards to (include/swaa.h).  Tensors are
torch tensors used purely as device-memory handles: the binding checks dtype, device and contiguity,
reads sizes from the shapes, passes raw pointers, and raises ``SwaaError`` on a non-zero status.
There is no fallback path: if the shared library is missing or cannot be loaded, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

from .build import LIB_PATH

SWAA_OK = 0
SWAA_PHASE_PREFILL = 0
SWAA_PHASE_DECODE = 1

_lib = None


class SwaaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_str(status)} ({status})")


class _Policy(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("n_layers", "window", "n_sink", "fa_start", "fa_step", "fa_decode")] + \
               [("fa_mask", ctypes.POINTER(ctypes.c_uint8))]


@dataclass
class SwaaPolicy:
    """Mirror of the C struct swaa_policy (one SWAA configuration: window, FA layers, keep first, FA decode)."""
    n_layers: int
    window: int
    n_sink: int = 0
    fa_start: int = 0
    fa_step: int = 0
    fa_decode: bool = False
    fa_mask: list | None = None  # explicit FA set: one 0/1 entry per layer (replaces fa_start / fa_step)

    def _c(self) -> _Policy:
        mask = None
        if self.fa_mask is not None:
            if len(self.fa_mask) != self.n_layers:
                raise ValueError("SwaaPolicy.fa_mask must have n_layers entries")
            mask = (ctypes.c_uint8 * max(self.n_layers, 1))(*[int(bool(x)) for x in self.fa_mask])
        c = _Policy(self.n_layers, self.window, self.n_sink, self.fa_start, self.fa_step, int(bool(self.fa_decode)),
                    ctypes.cast(mask, ctypes.POINTER(ctypes.c_uint8)) if mask is not None else None)
        c._keepalive = mask  # the C struct only borrows the array
        return c


def lib_path() -> str:
    return LIB_PATH


def load_library():
    """Loads libswaa.so (built in-tree by ``build.build_library``); raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_10411_b200.build` "
                           "(there is no fallback implementation)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.swaa_prefill.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp]
    lib.swaa_prefill.restype = ci
    lib.swaa_prefill_chunked.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp]
    lib.swaa_prefill_chunked.restype = ci
    lib.swaa_prefill_chunked_mixed.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp]
    lib.swaa_prefill_chunked_mixed.restype = ci
    lib.swaa_prefill_paged_mixed.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf,
                                             vp, vp]
    lib.swaa_prefill_paged_mixed.restype = ci
    lib.swaa_prefill_context_parallel.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci,
                                                  ci, ci, cf, vp, vp]
    lib.swaa_prefill_context_parallel.restype = ci
    lib.swaa_prefill_backward_workspace_size.argtypes = [ci, ci, ci, ci, ci, ci]
    lib.swaa_prefill_backward_workspace_size.restype = ctypes.c_size_t
    lib.swaa_prefill_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp, ctypes.c_size_t, vp]
    lib.swaa_prefill_backward.restype = ci
    lib.swaa_prefill_paged.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp]
    lib.swaa_prefill_paged.restype = ci
    lib.swaa_lazy_ratio.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, vp, vp, vp]
    lib.swaa_lazy_ratio.restype = ci
    lib.swaa_decode_workspace_size.argtypes = [ci] * 8
    lib.swaa_decode_workspace_size.restype = ctypes.c_size_t
    lib.swaa_decode_num_blocks.argtypes = [ci] * 8
    lib.swaa_decode_num_blocks.restype = ci
    lib.swaa_decode.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, ctypes.c_size_t, vp]
    lib.swaa_decode.restype = ci
    lib.swaa_decode_paged_workspace_size.argtypes = [ci] * 9
    lib.swaa_decode_paged_workspace_size.restype = ctypes.c_size_t
    lib.swaa_decode_paged.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, ctypes.c_size_t, vp]
    lib.swaa_decode_paged.restype = ci
    lib.swaa_decode_partial_workspace_size.argtypes = [ci] * 8
    lib.swaa_decode_partial_workspace_size.restype = ctypes.c_size_t
    lib.swaa_decode_partial.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp, ctypes.c_size_t, vp]
    lib.swaa_decode_partial.restype = ci
    lib.swaa_decode_combine.argtypes = [vp, ci, ci, ci, ci, vp, vp]
    lib.swaa_decode_combine.restype = ci
    lib.swaa_decode_static.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, ci, ci, ci, cf, vp]
    lib.swaa_decode_static.restype = ci
    lib.swaa_schedule_is_full.argtypes = [ctypes.POINTER(_Policy), ci, ci]
    lib.swaa_schedule_is_full.restype = ci
    lib.swaa_schedule_fill.argtypes = [ctypes.POINTER(_Policy), ci, ctypes.POINTER(ctypes.c_uint8)]
    lib.swaa_schedule_fill.restype = ci
    lib.swaa_schedule_select_fa_layers.argtypes = [ctypes.POINTER(ctypes.c_float), ci, ci, ci, ci,
                                                   ctypes.POINTER(ctypes.c_uint8)]
    lib.swaa_schedule_select_fa_layers.restype = ci
    lib.swaa_prefill_tile_range.argtypes = [ci] * 7 + [ctypes.POINTER(ci)] * 3
    lib.swaa_prefill_tile_range.restype = ci
    lib.swaa_prefill_tile_needs_mask.argtypes = [ci] * 8
    lib.swaa_prefill_tile_needs_mask.restype = ci
    lib.swaa_prefill_block_m.restype = ci
    lib.swaa_prefill_block_n.restype = ci
    lib.swaa_trimmed_cache_slot.argtypes = [ctypes.c_longlong, ci, ci]
    lib.swaa_trimmed_cache_slot.restype = ctypes.c_longlong
    lib.swaa_trimmed_cache_len.argtypes = [ctypes.c_longlong, ci, ci]
    lib.swaa_trimmed_cache_len.restype = ctypes.c_longlong
    lib.swaa_status_str.argtypes = [ci]
    lib.swaa_status_str.restype = ctypes.c_char_p
    lib.swaa_last_device_status.argtypes = [vp]
    lib.swaa_last_device_status.restype = ci
    lib.swaa_kernel_launch_count.restype = ctypes.c_uint64
    _lib = lib
    return lib


def status_str(status: int) -> str:
    return load_library().swaa_status_str(int(status)).decode()


def _dev_ptr(t: torch.Tensor | None, dtype, name: str):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def swaa_prefill(q, k, v, out, cu_seqlens, max_seqlen: int, window: int, n_sink: int, is_full: bool,
                 scale: float = 0.0, lse=None, stream=None) -> None:
    """Forwards to C swaa_prefill.  q, out [T,Hq,D]; k, v [T,Hkv,D] bf16; cu_seqlens int32 [B+1]; lse f32 [Hq,T]."""
    lib = load_library()
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    if tuple(k.shape) != (T, Hkv, D) or tuple(v.shape) != (T, Hkv, D) or tuple(out.shape) != (T, Hq, D):
        raise ValueError("swaa_prefill: inconsistent tensor shapes")
    B = cu_seqlens.numel() - 1
    if lse is not None and tuple(lse.shape) != (Hq, T):
        raise ValueError("swaa_prefill: lse must be [Hq, T]")
    bf = torch.bfloat16
    rc = lib.swaa_prefill(_dev_ptr(q, bf, "q"), _dev_ptr(k, bf, "k"), _dev_ptr(v, bf, "v"), _dev_ptr(out, bf, "out"),
                          _dev_ptr(cu_seqlens, torch.int32, "cu_seqlens"), B, T, int(max_seqlen), Hq, Hkv, D,
                          int(window), int(n_sink), int(bool(is_full)), float(scale),
                          _dev_ptr(lse, torch.float32, "lse"), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill")


def swaa_prefill_chunked(q, k, v, out, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int, window: int,
                         n_sink: int, is_full: bool, scale: float = 0.0, lse=None, stream=None, is_full_seq=None) -> None:
    """Forwards to C swaa_prefill_chunked, or, when is_full_seq (uint8 [B], a mask policy per sequence) is given, to
    C swaa_prefill_chunked_mixed.  q, out [Tq,Hq,D]; k, v [Tk,Hkv,D] bf16; cu_seqlens_* int32 [B+1];
    lse f32 [Hq,Tq].  The queries of each sequence are the last len_q tokens of its len_k-token context."""
    lib = load_library()
    Tq, Hq, D = q.shape
    Tk, Hkv = k.shape[0], k.shape[1]
    if tuple(k.shape) != (Tk, Hkv, D) or tuple(v.shape) != (Tk, Hkv, D) or tuple(out.shape) != (Tq, Hq, D):
        raise ValueError("swaa_prefill_chunked: inconsistent tensor shapes")
    B = cu_seqlens_q.numel() - 1
    if cu_seqlens_k.numel() != B + 1:
        raise ValueError("swaa_prefill_chunked: cu_seqlens_q and cu_seqlens_k must have the same length")
    if lse is not None and tuple(lse.shape) != (Hq, Tq):
        raise ValueError("swaa_prefill_chunked: lse must be [Hq, Tq]")
    bf = torch.bfloat16
    if is_full_seq is not None:
        if is_full_seq.numel() != B:
            raise ValueError("swaa_prefill_chunked: is_full_seq must have one entry per sequence")
        rc = lib.swaa_prefill_chunked_mixed(_dev_ptr(q, bf, "q"), _dev_ptr(k, bf, "k"), _dev_ptr(v, bf, "v"),
                                            _dev_ptr(out, bf, "out"), _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                                            _dev_ptr(cu_seqlens_k, torch.int32, "cu_seqlens_k"),
                                            _dev_ptr(is_full_seq, torch.uint8, "is_full_seq"), B, Tq, Tk,
                                            int(max_seqlen_q), int(max_seqlen_k), Hq, Hkv, D, int(window), int(n_sink),
                                            float(scale), _dev_ptr(lse, torch.float32, "lse"), _stream_ptr(stream))
        if rc != SWAA_OK:
            raise SwaaError(rc, "swaa_prefill_chunked_mixed")
        return
    rc = lib.swaa_prefill_chunked(_dev_ptr(q, bf, "q"), _dev_ptr(k, bf, "k"), _dev_ptr(v, bf, "v"),
                                  _dev_ptr(out, bf, "out"), _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                                  _dev_ptr(cu_seqlens_k, torch.int32, "cu_seqlens_k"), B, Tq, Tk, int(max_seqlen_q),
                                  int(max_seqlen_k), Hq, Hkv, D, int(window), int(n_sink), int(bool(is_full)),
                                  float(scale), _dev_ptr(lse, torch.float32, "lse"), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill_chunked")


def prefill_backward_workspace_size(B, T, Hq, Hkv, D, n_sink) -> int:
    """Forwards to C swaa_prefill_backward_workspace_size (bytes)."""
    return int(load_library().swaa_prefill_backward_workspace_size(int(B), int(T), int(Hq), int(Hkv), int(D), int(n_sink)))


def swaa_prefill_backward(q, k, v, out, dout, lse, cu_seqlens, max_seqlen: int, window: int, n_sink: int, is_full: bool,
                          dq, dk, dv, workspace, scale: float = 0.0, stream=None) -> None:
    """Forwards to C swaa_prefill_backward.  q, out, dout, dq [T,Hq,D]; k, v, dk, dv [T,Hkv,D] bf16; lse f32 [Hq,T];
    workspace uint8 of prefill_backward_workspace_size(B, T, Hq, Hkv, D, n_sink) bytes."""
    lib = load_library()
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    for name, t, shp in (("k", k, (T, Hkv, D)), ("v", v, (T, Hkv, D)), ("out", out, (T, Hq, D)), ("dout", dout, (T, Hq, D)),
                         ("dq", dq, (T, Hq, D)), ("dk", dk, (T, Hkv, D)), ("dv", dv, (T, Hkv, D)), ("lse", lse, (Hq, T))):
        if tuple(t.shape) != shp:
            raise ValueError(f"swaa_prefill_backward: {name} must be {shp}")
    B = cu_seqlens.numel() - 1
    bf = torch.bfloat16
    rc = lib.swaa_prefill_backward(_dev_ptr(q, bf, "q"), _dev_ptr(k, bf, "k"), _dev_ptr(v, bf, "v"), _dev_ptr(out, bf, "out"),
                                   _dev_ptr(dout, bf, "dout"), _dev_ptr(lse, torch.float32, "lse"),
                                   _dev_ptr(cu_seqlens, torch.int32, "cu_seqlens"), B, T, int(max_seqlen), Hq, Hkv, D,
                                   int(window), int(n_sink), int(bool(is_full)), float(scale), _dev_ptr(dq, bf, "dq"),
                                   _dev_ptr(dk, bf, "dk"), _dev_ptr(dv, bf, "dv"),
                                   _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill_backward")


def swaa_prefill_paged(q, kpages, vpages, out, cu_seqlens_q, seqlens_k, block_table, max_seqlen_q: int, window: int,
                       n_sink: int, is_full: bool, scale: float = 0.0, lse=None, stream=None, is_full_seq=None) -> None:
    """Forwards to C swaa_prefill_paged (to C swaa_prefill_paged_mixed when is_full_seq, uint8 [B], is given).  q, out [Tq,Hq,D]; kpages, vpages [num_pages,page_size,Hkv,D] bf16;
    cu_seqlens_q int32 [B+1]; seqlens_k int32 [B]; block_table int32 [B,max_blocks]; lse f32 [Hq,Tq]."""
    lib = load_library()
    Tq, Hq, D = q.shape
    num_pages, page_size, Hkv, _ = kpages.shape
    if tuple(vpages.shape) != tuple(kpages.shape) or kpages.shape[3] != D or tuple(out.shape) != (Tq, Hq, D):
        raise ValueError("swaa_prefill_paged: inconsistent tensor shapes")
    B = cu_seqlens_q.numel() - 1
    if block_table.dim() != 2 or block_table.shape[0] != B or seqlens_k.numel() != B:
        raise ValueError("swaa_prefill_paged: block_table must be [B, max_blocks] and seqlens_k [B]")
    if lse is not None and tuple(lse.shape) != (Hq, Tq):
        raise ValueError("swaa_prefill_paged: lse must be [Hq, Tq]")
    bf = torch.bfloat16
    if is_full_seq is not None:
        if is_full_seq.numel() != B:
            raise ValueError("swaa_prefill_paged: is_full_seq must have one entry per sequence")
        rc = lib.swaa_prefill_paged_mixed(_dev_ptr(q, bf, "q"), _dev_ptr(kpages, bf, "kpages"),
                                          _dev_ptr(vpages, bf, "vpages"), _dev_ptr(out, bf, "out"),
                                          _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                                          _dev_ptr(seqlens_k, torch.int32, "seqlens_k"),
                                          _dev_ptr(block_table, torch.int32, "block_table"),
                                          _dev_ptr(is_full_seq, torch.uint8, "is_full_seq"), B, Tq, int(max_seqlen_q),
                                          block_table.shape[1], num_pages, page_size, Hq, Hkv, D, int(window),
                                          int(n_sink), float(scale), _dev_ptr(lse, torch.float32, "lse"),
                                          _stream_ptr(stream))
        if rc != SWAA_OK:
            raise SwaaError(rc, "swaa_prefill_paged_mixed")
        return
    rc = lib.swaa_prefill_paged(_dev_ptr(q, bf, "q"), _dev_ptr(kpages, bf, "kpages"), _dev_ptr(vpages, bf, "vpages"),
                                _dev_ptr(out, bf, "out"), _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                                _dev_ptr(seqlens_k, torch.int32, "seqlens_k"),
                                _dev_ptr(block_table, torch.int32, "block_table"), B, Tq, int(max_seqlen_q),
                                block_table.shape[1], num_pages, page_size, Hq, Hkv, D, int(window), int(n_sink),
                                int(bool(is_full)), float(scale), _dev_ptr(lse, torch.float32, "lse"),
                                _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill_paged")


def swaa_prefill_context_parallel(q, k_local, v_local, sink_k, sink_v, out, cu_seqlens_q, cu_seqlens_k, key_pos0,
                                  max_seqlen_q: int, max_seqlen_k: int, window: int, n_sink: int, scale: float = 0.0,
                                  lse=None, stream=None) -> None:
    """Forwards to C swaa_prefill_context_parallel.  q, out [Tq,Hq,D]; k_local, v_local [Tk,Hkv,D] bf16 (halo + own
    stretch, starting at position key_pos0[b]); sink_k, sink_v [B,sink_rows,Hkv,D] bf16 or None; key_pos0 int32 [B]."""
    lib = load_library()
    Tq, Hq, D = q.shape
    Tk, Hkv = k_local.shape[0], k_local.shape[1]
    if tuple(k_local.shape) != (Tk, Hkv, D) or tuple(v_local.shape) != (Tk, Hkv, D) or tuple(out.shape) != (Tq, Hq, D):
        raise ValueError("swaa_prefill_context_parallel: inconsistent tensor shapes")
    B = cu_seqlens_q.numel() - 1
    if cu_seqlens_k.numel() != B + 1 or key_pos0.numel() != B:
        raise ValueError("swaa_prefill_context_parallel: cu_seqlens_k must be [B+1] and key_pos0 [B]")
    sink_rows = 0
    if sink_k is not None:
        sink_rows = sink_k.shape[1]
        if tuple(sink_k.shape) != (B, sink_rows, Hkv, D) or tuple(sink_v.shape) != tuple(sink_k.shape):
            raise ValueError("swaa_prefill_context_parallel: sink_k, sink_v must be [B, sink_rows, Hkv, D]")
    if lse is not None and tuple(lse.shape) != (Hq, Tq):
        raise ValueError("swaa_prefill_context_parallel: lse must be [Hq, Tq]")
    bf = torch.bfloat16
    rc = lib.swaa_prefill_context_parallel(_dev_ptr(q, bf, "q"), _dev_ptr(k_local, bf, "k_local"),
                                           _dev_ptr(v_local, bf, "v_local"), _dev_ptr(sink_k, bf, "sink_k"),
                                           _dev_ptr(sink_v, bf, "sink_v"), _dev_ptr(out, bf, "out"),
                                           _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                                           _dev_ptr(cu_seqlens_k, torch.int32, "cu_seqlens_k"),
                                           _dev_ptr(key_pos0, torch.int32, "key_pos0"), B, Tq, Tk, int(max_seqlen_q),
                                           int(max_seqlen_k), sink_rows, Hq, Hkv, D, int(window), int(n_sink),
                                           float(scale), _dev_ptr(lse, torch.float32, "lse"), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill_context_parallel")


def swaa_lazy_ratio(q, k, v, cu_seqlens_q, cu_seqlens_k, max_seqlen_q: int, max_seqlen_k: int, recent: int, n_sink: int,
                    ratio, scratch_out, scratch_lse, scale: float = 0.0, stream=None) -> None:
    """Forwards to C swaa_lazy_ratio.  q [Tq,Hq,D]; k [Tk,Hkv,D] bf16; ratio f32 [Hq]; scratch_lse f32 [2,Hq,Tq].
    v and scratch_out are not used by the probe and may be None."""
    lib = load_library()
    Tq, Hq, D = q.shape
    Tk, Hkv = k.shape[0], k.shape[1]
    if tuple(scratch_lse.shape) != (2, Hq, Tq) or tuple(ratio.shape) != (Hq,):
        raise ValueError("swaa_lazy_ratio: inconsistent output / scratch shapes")
    B = cu_seqlens_q.numel() - 1
    bf = torch.bfloat16
    rc = lib.swaa_lazy_ratio(_dev_ptr(q, bf, "q"), _dev_ptr(k, bf, "k"), _dev_ptr(v, bf, "v"),
                             _dev_ptr(cu_seqlens_q, torch.int32, "cu_seqlens_q"),
                             _dev_ptr(cu_seqlens_k, torch.int32, "cu_seqlens_k"), B, Tq, Tk, int(max_seqlen_q),
                             int(max_seqlen_k), Hq, Hkv, D, int(recent), int(n_sink), float(scale),
                             _dev_ptr(ratio, torch.float32, "ratio"), _dev_ptr(scratch_out, bf, "scratch_out"),
                             _dev_ptr(scratch_lse, torch.float32, "scratch_lse"), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_lazy_ratio")


def decode_workspace_size(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) -> int:
    """Forwards to C swaa_decode_workspace_size (bytes)."""
    return int(load_library().swaa_decode_workspace_size(B, Hq, Hkv, D, Lmax, int(window), int(n_sink),
                                                         int(bool(is_full))))


def decode_num_blocks(B, Hq, Hkv, D, Lmax, window, n_sink, is_full) -> int:
    return int(load_library().swaa_decode_num_blocks(B, Hq, Hkv, D, Lmax, int(window), int(n_sink),
                                                     int(bool(is_full))))


def swaa_decode(q, kcache, vcache, out, seqlens, window: int, n_sink: int, is_full: bool, workspace,
                scale: float = 0.0, stream=None) -> None:
    """Forwards to C swaa_decode.  q, out [B,Hq,D]; caches [B,Lmax,Hkv,D] bf16; seqlens int32 [B];
    workspace: uint8 CUDA tensor of at least decode_workspace_size(...) bytes."""
    lib = load_library()
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = kcache.shape
    if tuple(kcache.shape) != (B, Lmax, Hkv, D) or tuple(vcache.shape) != (B, Lmax, Hkv, D) \
            or tuple(out.shape) != (B, Hq, D) or seqlens.numel() != B:
        raise ValueError("swaa_decode: inconsistent tensor shapes")
    bf = torch.bfloat16
    rc = lib.swaa_decode(_dev_ptr(q, bf, "q"), _dev_ptr(kcache, bf, "kcache"), _dev_ptr(vcache, bf, "vcache"),
                         _dev_ptr(out, bf, "out"), _dev_ptr(seqlens, torch.int32, "seqlens"), B, Lmax, Hq, Hkv, D,
                         int(window), int(n_sink), int(bool(is_full)), float(scale),
                         _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_decode")


def decode_paged_workspace_size(B, Hq, Hkv, D, max_blocks, page_size, window, n_sink, is_full) -> int:
    """Forwards to C swaa_decode_paged_workspace_size (bytes)."""
    return int(load_library().swaa_decode_paged_workspace_size(B, Hq, Hkv, D, int(max_blocks), int(page_size),
                                                               int(window), int(n_sink), int(bool(is_full))))


def swaa_decode_paged(q, kpages, vpages, out, block_table, seqlens, window: int, n_sink: int, is_full: bool, workspace,
                      scale: float = 0.0, stream=None) -> None:
    """Forwards to C swaa_decode_paged.  q, out [B,Hq,D]; kpages, vpages [num_pages,page_size,Hkv,D] bf16;
    block_table int32 [B,max_blocks]; seqlens int32 [B]; workspace uint8 of decode_paged_workspace_size(...) bytes."""
    lib = load_library()
    B, Hq, D = q.shape
    num_pages, page_size, Hkv, _ = kpages.shape
    if tuple(vpages.shape) != tuple(kpages.shape) or kpages.shape[3] != D or tuple(out.shape) != (B, Hq, D):
        raise ValueError("swaa_decode_paged: inconsistent tensor shapes")
    if block_table.dim() != 2 or block_table.shape[0] != B or seqlens.numel() != B:
        raise ValueError("swaa_decode_paged: block_table must be [B, max_blocks] and seqlens [B]")
    bf = torch.bfloat16
    rc = lib.swaa_decode_paged(_dev_ptr(q, bf, "q"), _dev_ptr(kpages, bf, "kpages"), _dev_ptr(vpages, bf, "vpages"),
                               _dev_ptr(out, bf, "out"), _dev_ptr(block_table, torch.int32, "block_table"),
                               _dev_ptr(seqlens, torch.int32, "seqlens"), B, block_table.shape[1], num_pages, page_size,
                               Hq, Hkv, D, int(window), int(n_sink), int(bool(is_full)), float(scale),
                               _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_decode_paged")


def decode_partial_workspace_size(B, Hq, Hkv, D, Lshard, window, n_sink, is_full) -> int:
    """Forwards to C swaa_decode_partial_workspace_size (bytes)."""
    return int(load_library().swaa_decode_partial_workspace_size(B, Hq, Hkv, D, int(Lshard), int(window), int(n_sink),
                                                                 int(bool(is_full))))


def swaa_decode_partial(q, kshard, vshard, partial_out, seqlens, key_pos0: int, window: int, n_sink: int, is_full: bool,
                        workspace, scale: float = 0.0, stream=None) -> None:
    """Forwards to C swaa_decode_partial.  q [B,Hq,D]; kshard, vshard [B,Lshard,Hkv,D] bf16 holding positions key_pos0..;
    partial_out f32 [B,Hq,D+2]; seqlens int32 [B] (total lengths)."""
    lib = load_library()
    B, Hq, D = q.shape
    _, Lshard, Hkv, _ = kshard.shape
    if tuple(kshard.shape) != (B, Lshard, Hkv, D) or tuple(vshard.shape) != (B, Lshard, Hkv, D) \
            or tuple(partial_out.shape) != (B, Hq, D + 2) or seqlens.numel() != B:
        raise ValueError("swaa_decode_partial: inconsistent tensor shapes")
    bf = torch.bfloat16
    rc = lib.swaa_decode_partial(_dev_ptr(q, bf, "q"), _dev_ptr(kshard, bf, "kshard"), _dev_ptr(vshard, bf, "vshard"),
                                 _dev_ptr(partial_out, torch.float32, "partial_out"),
                                 _dev_ptr(seqlens, torch.int32, "seqlens"), B, Lshard, int(key_pos0), Hq, Hkv, D,
                                 int(window), int(n_sink), int(bool(is_full)), float(scale),
                                 _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_decode_partial")


def swaa_decode_combine(partials, out, stream=None) -> None:
    """Forwards to C swaa_decode_combine.  partials f32 [P,B,Hq,D+2]; out bf16 [B,Hq,D]."""
    lib = load_library()
    P, B, Hq, D2 = partials.shape
    if tuple(out.shape) != (B, Hq, D2 - 2):
        raise ValueError("swaa_decode_combine: out must be [B, Hq, D]")
    rc = lib.swaa_decode_combine(_dev_ptr(partials, torch.float32, "partials"), P, B, Hq, D2 - 2,
                                 _dev_ptr(out, torch.bfloat16, "out"), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_decode_combine")


def trimmed_cache_slot(pos: int, window: int, n_sink: int) -> int:
    """Forwards to C swaa_trimmed_cache_slot."""
    return int(load_library().swaa_trimmed_cache_slot(int(pos), int(window), int(n_sink)))


def trimmed_cache_len(length: int, window: int, n_sink: int) -> int:
    """Forwards to C swaa_trimmed_cache_len."""
    return int(load_library().swaa_trimmed_cache_len(int(length), int(window), int(n_sink)))


DECODE_STATIC_SCRATCH_BYTES = 2 << 20


def swaa_decode_static(q, kcache, vcache, out, seqlens, window: int, n_sink: int, is_full: bool, scale: float = 0.0,
                       stream=None) -> None:
    """Forwards to C swaa_decode_static: decode with the library's built-in scratch array, for callers
    that cannot allocate a workspace.  Shapes whose scratch need exceeds DECODE_STATIC_SCRATCH_BYTES raise
    SwaaError(SWAA_ERR_WORKSPACE).  Calls on one GPU share the array: do not let two overlap."""
    lib = load_library()
    B, Hq, D = q.shape
    _, Lmax, Hkv, _ = kcache.shape
    if tuple(kcache.shape) != (B, Lmax, Hkv, D) or tuple(vcache.shape) != (B, Lmax, Hkv, D) \
            or tuple(out.shape) != (B, Hq, D) or seqlens.numel() != B:
        raise ValueError("swaa_decode_static: inconsistent tensor shapes")
    bf = torch.bfloat16
    rc = lib.swaa_decode_static(_dev_ptr(q, bf, "q"), _dev_ptr(kcache, bf, "kcache"), _dev_ptr(vcache, bf, "vcache"),
                                _dev_ptr(out, bf, "out"), _dev_ptr(seqlens, torch.int32, "seqlens"), B, Lmax, Hq, Hkv,
                                D, int(window), int(n_sink), int(bool(is_full)), float(scale), _stream_ptr(stream))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_decode_static")


def schedule_is_full(policy: SwaaPolicy, layer: int, phase: int) -> bool:
    c = policy._c()
    rc = load_library().swaa_schedule_is_full(ctypes.byref(c), int(layer), int(phase))
    if rc < 0:
        raise SwaaError(rc, "swaa_schedule_is_full")
    return bool(rc)


def schedule_fill(policy: SwaaPolicy, phase: int) -> list:
    c = policy._c()
    buf = (ctypes.c_uint8 * max(policy.n_layers, 1))()
    rc = load_library().swaa_schedule_fill(ctypes.byref(c), int(phase), buf)
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_schedule_fill")
    return [bool(buf[i]) for i in range(policy.n_layers)]


def schedule_select_fa_layers(ratio, n_lazy: int, fa_on_lazy: bool) -> list:
    """Forwards to C swaa_schedule_select_fa_layers.  ratio: [n_layers][n_heads] numbers on the host (per layer the
    output of swaa_lazy_ratio).  Returns the FA mask as a list of 0/1, usable as SwaaPolicy.fa_mask."""
    rows = [list(map(float, r)) for r in ratio]
    n_layers = len(rows)
    n_heads = len(rows[0]) if n_layers else 1
    if any(len(r) != n_heads for r in rows):
        raise ValueError("schedule_select_fa_layers: ragged ratio table")
    flat = (ctypes.c_float * max(n_layers * n_heads, 1))(*[x for r in rows for x in r])
    out = (ctypes.c_uint8 * max(n_layers, 1))()
    rc = load_library().swaa_schedule_select_fa_layers(flat, n_layers, n_heads, int(n_lazy), int(bool(fa_on_lazy)), out)
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_schedule_select_fa_layers")
    return [int(out[i]) for i in range(n_layers)]


def prefill_tile_range(L, m, BM, BN, window, n_sink, is_full):
    a, b, c = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    rc = load_library().swaa_prefill_tile_range(L, m, BM, BN, int(window), int(n_sink), int(bool(is_full)),
                                                ctypes.byref(a), ctypes.byref(b), ctypes.byref(c))
    if rc != SWAA_OK:
        raise SwaaError(rc, "swaa_prefill_tile_range")
    return a.value, b.value, c.value


def prefill_tile_needs_mask(L, m, n, BM, BN, window, n_sink, is_full) -> bool:
    rc = load_library().swaa_prefill_tile_needs_mask(L, m, n, BM, BN, int(window), int(n_sink), int(bool(is_full)))
    if rc < 0:
        raise SwaaError(rc, "swaa_prefill_tile_needs_mask")
    return bool(rc)


def prefill_block_shape():
    lib = load_library()
    return lib.swaa_prefill_block_m(), lib.swaa_prefill_block_n()


def last_device_status(stream=None) -> int:
    return int(load_library().swaa_last_device_status(_stream_ptr(stream)))


def kernel_launch_count() -> int:
    return int(load_library().swaa_kernel_launch_count())
