"""Python binding of the sparkattn C-ABI library (``libsparkattn.so``).

Argument marshalling only: every step of the path (block selection, FP8
quantisation, block-sparse attention) runs in the CUDA kernels behind the
``extern "C"`` entry points declared in ``include/sparkattn.h``.  PyTorch is
used for device memory and streams.  There is no CPU fallback: if the shared
library is missing or cannot be loaded, every call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparkattn.so")
VERSION = 1

OK = 0
E_INVALID_ARG = -1
E_UNSUPPORTED_SHAPE = -2
E_MISALIGNED = -3
E_WORKSPACE_TOO_SMALL = -4
E_CUDA = -5
E_DEVICE_TIMEOUT = -6
E_BAD_INDEX = -7
E_NO_DEVICE = -8

BF16 = 0
FP8_E4M3 = 1

EXPORTS = (
    "sparkattn_version", "sparkattn_status_string", "sparkattn_workspace_bytes", "sparkattn_select",
    "sparkattn_quant_fp8", "sparkattn_quant_fp8_per_token", "sparkattn_fwd", "sparkattn_read_status", "sparkattn_arena_bytes",
    "sparkattn_attention_host", "sparkattn_select_noalloc", "sparkattn_select_noalloc_max_bytes",
    "sparkattn_select_noalloc_status", "sparkattn_comp_workspace_bytes", "sparkattn_comp_state",
    "sparkattn_comp_apply", "sparkattn_select_window", "sparkattn_fwd_window", "sparkattn_brick_count",
    "sparkattn_brick_layout", "sparkattn_gather_tokens", "sparkattn_select_padded", "sparkattn_fwd_padded",
    "sparkattn_quant_fp8_pooled", "sparkattn_select_pooled", "sparkattn_fwd_gated_workspace_bytes", "sparkattn_fwd_gated",
)


class Shape(ctypes.Structure):
    """Mirror of ``sparkattn_shape_t``."""
    _fields_ = [
        ("struct_size", ctypes.c_uint32), ("version", ctypes.c_uint32),
        ("B", ctypes.c_int32), ("H", ctypes.c_int32), ("N", ctypes.c_int32), ("d", ctypes.c_int32),
        ("block", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64),
        ("softmax_scale", ctypes.c_float), ("pad", ctypes.c_uint32),
    ]


class SparkAttnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2609_23153_b200.build` "
                "(there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_size_t
        sp = ctypes.POINTER(Shape)
        L.sparkattn_version.restype = ctypes.c_int
        L.sparkattn_status_string.restype = ctypes.c_char_p
        L.sparkattn_status_string.argtypes = [ctypes.c_int]
        L.sparkattn_workspace_bytes.restype = sz
        L.sparkattn_workspace_bytes.argtypes = [sp, i32, i32]
        L.sparkattn_select.restype = ctypes.c_int
        L.sparkattn_select.argtypes = [sp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.sparkattn_quant_fp8.restype = ctypes.c_int
        L.sparkattn_quant_fp8.argtypes = [sp, vp, vp, vp, ctypes.c_uint32, vp]
        L.sparkattn_quant_fp8_pooled.restype = ctypes.c_int
        L.sparkattn_quant_fp8_pooled.argtypes = [sp, vp, vp, vp, i32, vp, sz, vp]
        L.sparkattn_select_pooled.restype = ctypes.c_int
        L.sparkattn_select_pooled.argtypes = [sp, i32, vp, vp, vp, sz, vp]
        L.sparkattn_quant_fp8_per_token.restype = ctypes.c_int
        L.sparkattn_quant_fp8_per_token.argtypes = [sp, vp, vp, vp, vp]
        L.sparkattn_fwd.restype = ctypes.c_int
        L.sparkattn_fwd.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.sparkattn_read_status.restype = ctypes.c_int
        L.sparkattn_read_status.argtypes = [vp, vp]
        L.sparkattn_brick_count.restype = ctypes.c_int64
        L.sparkattn_brick_count.argtypes = [vp, vp]
        L.sparkattn_brick_layout.restype = ctypes.c_int
        L.sparkattn_brick_layout.argtypes = [vp, vp, i32, vp, vp, vp, vp]
        L.sparkattn_gather_tokens.restype = ctypes.c_int
        L.sparkattn_gather_tokens.argtypes = [sp, vp, sp, vp, vp, vp, sz, vp]
        L.sparkattn_select_padded.restype = ctypes.c_int
        L.sparkattn_select_padded.argtypes = [sp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.sparkattn_fwd_padded.restype = ctypes.c_int
        L.sparkattn_fwd_padded.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
        L.sparkattn_arena_bytes.restype = sz
        L.sparkattn_arena_bytes.argtypes = [sp, i32, i32]
        L.sparkattn_attention_host.restype = ctypes.c_int
        L.sparkattn_attention_host.argtypes = [sp, i32, vp, vp, vp, i32, vp, vp, vp, sz, vp]
        L.sparkattn_select_noalloc.restype = ctypes.c_int
        L.sparkattn_select_noalloc.argtypes = [sp, vp, vp, i32, vp, vp, vp]
        L.sparkattn_select_noalloc_max_bytes.restype = sz
        L.sparkattn_select_noalloc_status.restype = ctypes.c_int
        L.sparkattn_select_noalloc_status.argtypes = [vp]
        L.sparkattn_select_window.restype = ctypes.c_int
        L.sparkattn_select_window.argtypes = [sp, vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
        L.sparkattn_fwd_window.restype = ctypes.c_int
        L.sparkattn_fwd_window.argtypes = [sp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, vp, vp, vp, sz, vp]
        L.sparkattn_comp_workspace_bytes.restype = sz
        L.sparkattn_comp_workspace_bytes.argtypes = [sp, vp]
        L.sparkattn_comp_state.restype = ctypes.c_int
        L.sparkattn_comp_state.argtypes = [sp, vp, vp, vp, i32, vp, vp, vp, vp, vp, sz, vp]
        L.sparkattn_comp_apply.restype = ctypes.c_int
        L.sparkattn_comp_apply.argtypes = [sp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, ctypes.c_float, vp, sz, vp]
        L.sparkattn_fwd_gated_workspace_bytes.restype = sz
        L.sparkattn_fwd_gated_workspace_bytes.argtypes = [sp, i32, vp]
        L.sparkattn_fwd_gated.restype = ctypes.c_int
        L.sparkattn_fwd_gated.argtypes = [sp, vp, vp, vp, vp, vp, i32, vp, i32, vp, vp, vp, vp, vp, ctypes.c_float, vp,
                                          vp, vp, sz, vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().sparkattn_status_string(int(status)).decode()


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise SparkAttnError(rc, where)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> ctypes.c_void_p:
    return ctypes.c_void_p(0 if t is None else t.data_ptr())


def make_shape(x: torch.Tensor, block: int, softmax_scale: float = 0.0) -> Shape:
    """Shape descriptor for a [B, H, N, d] tensor (d contiguous, arbitrary outer strides)."""
    if x.dim() != 4 or x.stride(3) != 1:
        raise ValueError("expected a [B, H, N, d] tensor with a contiguous last dimension")
    B, H, N, d = x.shape
    return Shape(ctypes.sizeof(Shape), VERSION, B, H, N, d, block, 0,
                 x.stride(0), x.stride(1), x.stride(2), float(softmax_scale), 0)


def _same_layout(ref: torch.Tensor, *others: torch.Tensor) -> None:
    for o in others:
        if o.shape != ref.shape or o.stride() != ref.stride():
            raise ValueError("tensors of one call must share shape and strides")


def workspace_bytes(shape: Shape, which: int, topk_or_kmax: int) -> int:
    return int(lib().sparkattn_workspace_bytes(ctypes.byref(shape), which, topk_or_kmax))


def alloc_workspace(shape: Shape, which: int, topk_or_kmax: int, device) -> torch.Tensor:
    n = workspace_bytes(shape, which, topk_or_kmax)
    if n == 0:
        raise SparkAttnError(E_UNSUPPORTED_SHAPE, "sparkattn_workspace_bytes")
    return torch.empty(n, dtype=torch.uint8, device=device)


def read_status(workspace: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
    return int(lib().sparkattn_read_status(_ptr(workspace), _stream_ptr(stream)))


def select(q: torch.Tensor, k: torch.Tensor, block: int, topk: int, *,
           kept_idx: Optional[torch.Tensor] = None, kept_cnt: Optional[torch.Tensor] = None,
           workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
           frame_tokens: int = 0, window: int = 0, block_valid: Optional[torch.Tensor] = None,
           ) -> Tuple[torch.Tensor, torch.Tensor]:
    """``sparkattn_select`` (``sparkattn_select_window`` when ``frame_tokens`` > 0, ``sparkattn_select_padded``
    with ``block_valid``, device int32 [nb]): q, k bf16 [B,H,N,d] on the device -> (kept_idx int32
    [B,H,nb,topk] ascending, kept_cnt int32 [B,H,nb])."""
    _same_layout(q, k)
    shape = make_shape(q, block)
    B, H, N, _ = q.shape
    nb = (N + block - 1) // block
    if kept_idx is None:
        kept_idx = torch.empty((B, H, nb, max(topk, 1)), dtype=torch.int32, device=q.device)
    if kept_cnt is None:
        kept_cnt = torch.empty((B, H, nb), dtype=torch.int32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(shape, 0, topk, q.device)
    if block_valid is not None:
        if frame_tokens > 0:
            raise ValueError("block_valid and a causal window cannot be combined")
        rc = lib().sparkattn_select_padded(ctypes.byref(shape), _ptr(q), _ptr(k), topk, _ptr(block_valid), _ptr(kept_idx),
                                           _ptr(kept_cnt), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
        _check(rc, "sparkattn_select_padded")
        return kept_idx, kept_cnt
    if frame_tokens > 0:
        rc = lib().sparkattn_select_window(ctypes.byref(shape), _ptr(q), _ptr(k), topk, frame_tokens, window,
                                           _ptr(kept_idx), _ptr(kept_cnt), _ptr(workspace), workspace.numel(),
                                           _stream_ptr(stream))
        _check(rc, "sparkattn_select_window")
        return kept_idx, kept_cnt
    rc = lib().sparkattn_select(ctypes.byref(shape), _ptr(q), _ptr(k), topk, _ptr(kept_idx), _ptr(kept_cnt),
                                _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_select")
    return kept_idx, kept_cnt


def select_noalloc(q: torch.Tensor, k: torch.Tensor, block: int, topk: int, kept_idx: torch.Tensor,
                   kept_cnt: Optional[torch.Tensor], stream: Optional[torch.cuda.Stream] = None) -> None:
    """``sparkattn_select_noalloc``: same selection as :func:`select`, for callers that
    must not allocate device memory at call time.  The caller passes the output
    buffers; the scratch is a fixed 32 MiB array inside the library, shared by all
    calls on the device (do not overlap calls; make the first call on a device
    before any stream capture)."""
    _same_layout(q, k)
    shape = make_shape(q, block)
    rc = lib().sparkattn_select_noalloc(ctypes.byref(shape), _ptr(q), _ptr(k), topk, _ptr(kept_idx), _ptr(kept_cnt),
                                        _stream_ptr(stream))
    _check(rc, "sparkattn_select_noalloc")


def quant_fp8(x: torch.Tensor, block: int, *, codes: Optional[torch.Tensor] = None,
              scales: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
              ) -> Tuple[torch.Tensor, torch.Tensor]:
    """``sparkattn_quant_fp8``: x bf16 [B,H,N,d] -> (codes uint8, same strides; scales fp32 [B,H,nb])."""
    shape = make_shape(x, block)
    B, H, N, _ = x.shape
    nb = (N + block - 1) // block
    if codes is None:
        codes = torch.empty_strided(x.shape, x.stride(), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty((B, H, nb), dtype=torch.float32, device=x.device)
    rc = lib().sparkattn_quant_fp8(ctypes.byref(shape), _ptr(x), _ptr(codes), _ptr(scales), 0, _stream_ptr(stream))
    _check(rc, "sparkattn_quant_fp8")
    return codes, scales


def quant_fp8_pooled(x: torch.Tensor, block: int, key_side: bool, select_workspace: torch.Tensor, *,
                     codes: Optional[torch.Tensor] = None, scales: Optional[torch.Tensor] = None,
                     stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """``sparkattn_quant_fp8_pooled``: :func:`quant_fp8` that also leaves the pooled block means of ``x`` (the query
    tensor, or the key tensor with ``key_side``) in ``select_workspace`` for :func:`select_pooled`."""
    shape = make_shape(x, block)
    B, H, N, _ = x.shape
    nb = (N + block - 1) // block
    if codes is None:
        codes = torch.empty_strided(x.shape, x.stride(), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty((B, H, nb), dtype=torch.float32, device=x.device)
    rc = lib().sparkattn_quant_fp8_pooled(ctypes.byref(shape), _ptr(x), _ptr(codes), _ptr(scales), 1 if key_side else 0,
                                          _ptr(select_workspace), select_workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_quant_fp8_pooled")
    return codes, scales


def select_pooled(ref: torch.Tensor, block: int, topk: int, workspace: torch.Tensor, *,
                  kept_idx: Optional[torch.Tensor] = None, kept_cnt: Optional[torch.Tensor] = None,
                  stream: Optional[torch.cuda.Stream] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """``sparkattn_select_pooled``: scores + top-k on the pooled means two :func:`quant_fp8_pooled` calls left in
    ``workspace``; ``ref`` is any [B,H,N,d] tensor of the problem (for the shape)."""
    shape = make_shape(ref, block)
    B, H, N, _ = ref.shape
    nb = (N + block - 1) // block
    if kept_idx is None:
        kept_idx = torch.empty((B, H, nb, max(topk, 1)), dtype=torch.int32, device=ref.device)
    if kept_cnt is None:
        kept_cnt = torch.empty((B, H, nb), dtype=torch.int32, device=ref.device)
    rc = lib().sparkattn_select_pooled(ctypes.byref(shape), topk, _ptr(kept_idx), _ptr(kept_cnt), _ptr(workspace),
                                       workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_select_pooled")
    return kept_idx, kept_cnt


def quant_fp8_per_token(x: torch.Tensor, *, codes: Optional[torch.Tensor] = None,
                        scales: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
                        ) -> Tuple[torch.Tensor, torch.Tensor]:
    """``sparkattn_quant_fp8_per_token``: x bf16 [B,H,N,d] -> (codes uint8, same strides; scales fp32 [B,H,N])."""
    shape = make_shape(x, 64 if x.shape[-1] == 64 else 128)
    B, H, N, _ = x.shape
    if codes is None:
        codes = torch.empty_strided(x.shape, x.stride(), dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty((B, H, N), dtype=torch.float32, device=x.device)
    rc = lib().sparkattn_quant_fp8_per_token(ctypes.byref(shape), _ptr(x), _ptr(codes), _ptr(scales), _stream_ptr(stream))
    _check(rc, "sparkattn_quant_fp8_per_token")
    return codes, scales


def fwd(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, kept_idx: torch.Tensor,
        kept_cnt: Optional[torch.Tensor], block: int, *,
        scales: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None,
        softmax_scale: float = 0.0, out: Optional[torch.Tensor] = None, return_lse: bool = False,
        workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
        check_status: bool = False, frame_tokens: int = 0, window: int = 0,
        block_valid: Optional[torch.Tensor] = None):
    """``sparkattn_fwd`` (``sparkattn_fwd_window`` when ``frame_tokens`` > 0, ``sparkattn_fwd_padded`` with
    ``block_valid``, device int32 [nb]).  bf16 q,k,v, or uint8
    E4M3 codes with ``scales=(q_scale, k_scale, v_scale)``.  Returns out bf16 [B,H,N,d] (and lse
    fp32 [B,H,N])."""
    _same_layout(q, k, v)
    shape = make_shape(q, block, softmax_scale)
    B, H, N, _ = q.shape
    dtype = BF16 if scales is None else FP8_E4M3
    kmax = kept_idx.shape[-1]
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if return_lse else None
    if workspace is None:
        workspace = alloc_workspace(shape, 1, kmax, q.device)
    sq, sk, sv = scales if scales is not None else (None, None, None)
    if block_valid is not None:
        if frame_tokens > 0:
            raise ValueError("block_valid and a causal window cannot be combined")
        rc = lib().sparkattn_fwd_padded(ctypes.byref(shape), dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(sq), _ptr(sk), _ptr(sv),
                                        _ptr(kept_idx), _ptr(kept_cnt), kmax, _ptr(block_valid), _ptr(out), _ptr(lse),
                                        _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    elif frame_tokens > 0:
        rc = lib().sparkattn_fwd_window(ctypes.byref(shape), dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(sq), _ptr(sk),
                                        _ptr(sv), _ptr(kept_idx), _ptr(kept_cnt), kmax, frame_tokens, window,
                                        _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    else:
        rc = lib().sparkattn_fwd(ctypes.byref(shape), dtype, _ptr(q), _ptr(k), _ptr(v), _ptr(sq), _ptr(sk), _ptr(sv),
                                 _ptr(kept_idx), _ptr(kept_cnt), kmax, _ptr(out), _ptr(lse), _ptr(workspace),
                                 workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_fwd")
    if check_status:
        _check(read_status(workspace, stream), "sparkattn_fwd (device status)")
    return (out, lse) if return_lse else out


def brick_layout(grid, brick, block: int, device="cuda:0", stream: Optional[torch.cuda.Stream] = None):
    """``sparkattn_brick_layout``: (gather int32 [bricks * block] with -1 for padding, block_valid int32 [bricks],
    scatter int32 [N]) for a (T, Hg, Wg) grid cut into (bt, bh, bw) bricks, one block per brick."""
    g = (ctypes.c_int32 * 3)(*[int(v) for v in grid])
    b = (ctypes.c_int32 * 3)(*[int(v) for v in brick])
    bricks = int(lib().sparkattn_brick_count(ctypes.cast(g, ctypes.c_void_p), ctypes.cast(b, ctypes.c_void_p)))
    if bricks == 0:
        raise SparkAttnError(E_INVALID_ARG, "sparkattn_brick_count")
    n = int(grid[0]) * int(grid[1]) * int(grid[2])
    gather = torch.empty(bricks * block, dtype=torch.int32, device=device)
    valid = torch.empty(bricks, dtype=torch.int32, device=device)
    scatter = torch.empty(n, dtype=torch.int32, device=device)
    rc = lib().sparkattn_brick_layout(ctypes.cast(g, ctypes.c_void_p), ctypes.cast(b, ctypes.c_void_p), block, _ptr(gather),
                                      _ptr(valid), _ptr(scatter), _stream_ptr(stream))
    _check(rc, "sparkattn_brick_layout")
    return gather, valid, scatter


def gather_tokens(x: torch.Tensor, index: torch.Tensor, *, out: Optional[torch.Tensor] = None,
                  workspace: Optional[torch.Tensor] = None, stream: Optional[torch.cuda.Stream] = None,
                  check_status: bool = False) -> torch.Tensor:
    """``sparkattn_gather_tokens``: out[b,h,i,:] = x[b,h,index[i],:] (zero row for index -1); x bf16 [B,H,N,d],
    index int32 [N_out] on the device, out bf16 [B,H,N_out,d]."""
    blk = 64 if x.shape[-1] == 64 else 128
    B, H, _, d = x.shape
    if index.dtype != torch.int32 or index.dim() != 1 or not index.is_contiguous():
        raise ValueError("index must be a contiguous 1-D int32 tensor")
    if out is None:
        out = torch.empty((B, H, index.numel(), d), dtype=x.dtype, device=x.device)
    src, dst = make_shape(x, blk), make_shape(out, blk)
    if workspace is None:
        workspace = torch.empty(256, dtype=torch.uint8, device=x.device)
    rc = lib().sparkattn_gather_tokens(ctypes.byref(src), _ptr(x), ctypes.byref(dst), _ptr(index), _ptr(out), _ptr(workspace),
                                       workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_gather_tokens")
    if check_status:
        _check(read_status(workspace, stream), "sparkattn_gather_tokens (device status)")
    return out


def arena_bytes(shape: Shape, dtype: int, topk: int) -> int:
    return int(lib().sparkattn_arena_bytes(ctypes.byref(shape), dtype, topk))


def attention_host(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, block: int, topk: int, *,
                   dtype: int = BF16, out: Optional[torch.Tensor] = None,
                   kept_idx: Optional[torch.Tensor] = None, arena: Optional[torch.Tensor] = None,
                   device="cuda:0", stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """``sparkattn_attention_host``: q, k, v contiguous bf16 HOST tensors (pinned for
    speed); runs copy-in, select, (quant,) fwd, copy-out and returns the host output."""
    for t in (q, k, v):
        if t.device.type != "cpu" or not t.is_contiguous() or t.dtype != torch.bfloat16:
            raise ValueError("attention_host expects contiguous bf16 CPU tensors")
    shape = make_shape(q, block)
    if out is None:
        out = torch.empty_like(q).pin_memory()
    if arena is None:
        arena = torch.empty(arena_bytes(shape, dtype, topk), dtype=torch.uint8, device=device)
    rc = lib().sparkattn_attention_host(ctypes.byref(shape), dtype, _ptr(q), _ptr(k), _ptr(v), topk, _ptr(out),
                                        _ptr(kept_idx), _ptr(arena), arena.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_attention_host")
    return out


def _rope_host(grid, axis: torch.Tensor, freq: torch.Tensor):
    g = (ctypes.c_int32 * 3)(*[int(x) for x in grid])
    a = axis.detach().to("cpu", torch.int32).contiguous()
    f = freq.detach().to("cpu", torch.float32).contiguous()
    if a.numel() != f.numel():
        raise ValueError("rope axis and frequency tables must have rank/2 entries each")
    return g, a, f


def comp_workspace_bytes(shape: Shape, grid) -> int:
    g = (ctypes.c_int32 * 3)(*[int(x) for x in grid])
    return int(lib().sparkattn_comp_workspace_bytes(ctypes.byref(shape), g))


def comp_state(k: torch.Tensor, v: torch.Tensor, pk: torch.Tensor, grid, axis: torch.Tensor, freq: torch.Tensor, *,
               state: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
               stream: Optional[torch.cuda.Stream] = None, check_status: bool = False) -> torch.Tensor:
    """``sparkattn_comp_state``: k, v bf16 [B,H,N,d]; pk bf16 [H,r,d]; grid (T,Hg,Wg); axis/freq the
    rotary tables (rank/2 entries, any device).  Returns the state fp32 [B,H,r,d]."""
    _same_layout(k, v)
    shape = make_shape(k, 128)
    B, H, _, d = k.shape
    rank = pk.shape[1]
    g, a, f = _rope_host(grid, axis, freq)
    if not pk.is_contiguous() or pk.shape != (H, rank, d):
        raise ValueError("pk must be contiguous [H, rank, d]")
    if state is None:
        state = torch.empty((B, H, rank, d), dtype=torch.float32, device=k.device)
    if workspace is None:
        workspace = torch.empty(max(comp_workspace_bytes(shape, grid), 256), dtype=torch.uint8, device=k.device)
    rc = lib().sparkattn_comp_state(ctypes.byref(shape), _ptr(k), _ptr(v), _ptr(pk), rank, g, _ptr(a), _ptr(f),
                                    _ptr(state), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_comp_state")
    if check_status:
        _check(read_status(workspace, stream), "sparkattn_comp_state (device status)")
    return state


def comp_apply(q: torch.Tensor, pq: torch.Tensor, state: torch.Tensor, gate: torch.Tensor, o_sparse: torch.Tensor,
               grid, axis: torch.Tensor, freq: torch.Tensor, *, eps: float = 1e-6,
               out: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None,
               stream: Optional[torch.cuda.Stream] = None, check_status: bool = False) -> torch.Tensor:
    """``sparkattn_comp_apply``: q, o_sparse bf16 [B,H,N,d]; pq bf16 [H,r,d]; state fp32 [B,H,r,d];
    gate fp32 [B,H,N].  Returns the fused output bf16 [B,H,N,d]."""
    _same_layout(q, o_sparse)
    shape = make_shape(q, 128)
    B, H, N, d = q.shape
    rank = pq.shape[1]
    g, a, f = _rope_host(grid, axis, freq)
    if not pq.is_contiguous() or pq.shape != (H, rank, d):
        raise ValueError("pq must be contiguous [H, rank, d]")
    if not state.is_contiguous() or state.shape != (B, H, rank, d) or state.dtype != torch.float32:
        raise ValueError("state must be contiguous fp32 [B, H, rank, d]")
    if not gate.is_contiguous() or gate.shape != (B, H, N) or gate.dtype != torch.float32:
        raise ValueError("gate must be contiguous fp32 [B, H, N]")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=torch.bfloat16, device=q.device)
    if workspace is None:
        workspace = torch.empty(max(comp_workspace_bytes(shape, grid), 256), dtype=torch.uint8, device=q.device)
    rc = lib().sparkattn_comp_apply(ctypes.byref(shape), _ptr(q), _ptr(pq), rank, g, _ptr(a), _ptr(f), _ptr(state),
                                    _ptr(gate), _ptr(o_sparse), _ptr(out), ctypes.c_float(eps), _ptr(workspace),
                                    workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_comp_apply")
    if check_status:
        _check(read_status(workspace, stream), "sparkattn_comp_apply (device status)")
    return out


def fwd_gated_workspace_bytes(shape: Shape, kmax: int, grid) -> int:
    g = (ctypes.c_int32 * 3)(*[int(x) for x in grid])
    return int(lib().sparkattn_fwd_gated_workspace_bytes(ctypes.byref(shape), kmax, g))


def fwd_gated(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, kept_idx: torch.Tensor,
              kept_cnt: Optional[torch.Tensor], pq: torch.Tensor, state: torch.Tensor, gate: torch.Tensor,
              grid, axis: torch.Tensor, freq: torch.Tensor, *, eps: float = 1e-6, softmax_scale: float = 0.0,
              out: Optional[torch.Tensor] = None, return_lse: bool = False, workspace: Optional[torch.Tensor] = None,
              stream: Optional[torch.cuda.Stream] = None, check_status: bool = False):
    """``sparkattn_fwd_gated``: the bf16 forward over 128-token blocks whose epilogue adds the gated
    compensation term.  Arguments as in ``fwd`` and ``comp_apply``; returns the module output bf16
    [B,H,N,d] (and the lse of the sparse branch, fp32 [B,H,N])."""
    _same_layout(q, k, v)
    shape = make_shape(q, 128, softmax_scale)
    B, H, N, d = q.shape
    rank = pq.shape[1]
    kmax = kept_idx.shape[-1]
    g, a, f = _rope_host(grid, axis, freq)
    if not pq.is_contiguous() or pq.shape != (H, rank, d):
        raise ValueError("pq must be contiguous [H, rank, d]")
    if not state.is_contiguous() or state.shape != (B, H, rank, d) or state.dtype != torch.float32:
        raise ValueError("state must be contiguous fp32 [B, H, rank, d]")
    if not gate.is_contiguous() or gate.shape != (B, H, N) or gate.dtype != torch.float32:
        raise ValueError("gate must be contiguous fp32 [B, H, N]")
    if out is None:
        out = torch.empty_strided(q.shape, q.stride(), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if return_lse else None
    if workspace is None:
        workspace = torch.empty(max(fwd_gated_workspace_bytes(shape, kmax, grid), 256), dtype=torch.uint8,
                                device=q.device)
    rc = lib().sparkattn_fwd_gated(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(kept_idx), _ptr(kept_cnt), kmax,
                                   _ptr(pq), rank, g, _ptr(a), _ptr(f), _ptr(state), _ptr(gate), ctypes.c_float(eps),
                                   _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel(), _stream_ptr(stream))
    _check(rc, "sparkattn_fwd_gated")
    if check_status:
        _check(read_status(workspace, stream), "sparkattn_fwd_gated (device status)")
    return (out, lse) if return_lse else out
