"""ctypes front-end of the CPU oracle (``sparkattn_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by
the benchmark's CPU-baseline leg.  The CUDA package never imports this module
and this module never imports the CUDA package.

All tensors are CPU torch tensors; bf16 data is passed as its raw 16-bit
pattern, FP8 data as raw E4M3 codes plus fp32 block scales.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sparkattn_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-shared", "-fPIC", "-Wall",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        L.oracle_e4m3_decode.restype = ctypes.c_double
        L.oracle_e4m3_decode.argtypes = [ctypes.c_uint8]
        L.oracle_e4m3_encode.restype = ctypes.c_uint8
        L.oracle_e4m3_encode.argtypes = [ctypes.c_float]
        L.oracle_attention.restype = ctypes.c_int
        L.oracle_select.restype = ctypes.c_int
        L.oracle_select_f64_diff.restype = ctypes.c_int64
        L.oracle_quant_fp8.restype = None
        L.oracle_quant_fp8_per_token.restype = None
        L.oracle_comp_state.restype = None
        L.oracle_comp_apply.restype = None
        L.oracle_pool.restype = None
        L.oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return ctypes.c_void_p(0)
    assert t.device.type == "cpu" and t.is_contiguous()
    return ctypes.c_void_p(t.data_ptr())


def _raw16(x: torch.Tensor) -> torch.Tensor:
    assert x.dtype == torch.bfloat16
    return x.contiguous().view(torch.int16)


def e4m3_decode(code: int) -> float:
    return float(_load().oracle_e4m3_decode(ctypes.c_uint8(code)))


def e4m3_encode(y: float) -> int:
    return int(_load().oracle_e4m3_encode(ctypes.c_float(y)))


def e4m3_encode_array(y: np.ndarray) -> np.ndarray:
    L = _load()
    y = np.ascontiguousarray(y, dtype=np.float32)
    out = np.empty(y.shape, dtype=np.uint8)
    yf, of = y.reshape(-1), out.reshape(-1)
    for i in range(yf.size):
        of[i] = L.oracle_e4m3_encode(ctypes.c_float(float(yf[i])))
    return out


def attention(
    q: torch.Tensor,
    k: torch.Tensor,
    v: torch.Tensor,
    kept_idx: torch.Tensor,
    kept_cnt: torch.Tensor,
    block: int,
    items: Optional[Sequence[Tuple[int, int]]] = None,
    scales: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None,
    softmax_scale: float = 0.0,
    frame_tokens: int = 0,
    window: int = 0,
    block_valid: Optional[torch.Tensor] = None,
):
    """ATT-0.  q, k, v: [H, N, d] bf16, or uint8 E4M3 codes with
    ``scales = (q_scale, k_scale, v_scale)`` each fp32 [H, nb].
    kept_idx int32 [H, nb, kmax], kept_cnt int32 [H, nb].
    Returns (out fp64 [n_items, block, d], lse fp64 [n_items, block]) for the
    (head, query-block) pairs in ``items`` (default: all, head-major).
    WIN-0: with ``frame_tokens`` = F > 0, key j counts for query i only if its frame j // F lies in
    (i // F - window, i // F]; a row with no such kept key gives out = 0, lse = -inf.
    ORD-0: with ``block_valid`` (int32 [nb]) block b holds block_valid[b] tokens followed by padding rows,
    which are neither keys nor evaluated as queries (their output rows stay 0)."""
    L = _load()
    H, N, d = q.shape
    nb = (N + block - 1) // block
    kmax = kept_idx.shape[-1]
    assert kept_idx.shape == (H, nb, kmax) and kept_cnt.shape == (H, nb)
    if items is None:
        items = [(h, i) for h in range(H) for i in range(nb)]
    it = torch.tensor(list(items), dtype=torch.int32).reshape(-1, 2).contiguous()
    n_items = it.shape[0]
    out = torch.zeros((n_items, block, d), dtype=torch.float64)
    lse = torch.zeros((n_items, block), dtype=torch.float64)
    if scales is None:
        dtype = 0
        qq, kk, vv = _raw16(q), _raw16(k), _raw16(v)
        sq = sk = sv = None
    else:
        dtype = 1
        assert q.dtype == torch.uint8
        qq, kk, vv = q.contiguous(), k.contiguous(), v.contiguous()
        sq, sk, sv = (s.contiguous().float() for s in scales)
    ki = kept_idx.contiguous().to(torch.int32)
    kc = kept_cnt.contiguous().to(torch.int32)
    rc = L.oracle_attention(
        ctypes.c_int(dtype), _ptr(qq), _ptr(kk), _ptr(vv), _ptr(sq), _ptr(sk), _ptr(sv),
        ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(d), ctypes.c_int(block),
        _ptr(ki), _ptr(kc), ctypes.c_int(kmax), ctypes.c_double(softmax_scale),
        _ptr(it), ctypes.c_int(n_items), ctypes.c_int(frame_tokens), ctypes.c_int(window),
        _ptr(None if block_valid is None else block_valid.contiguous().to(torch.int32)), _ptr(out), _ptr(lse))
    if rc != 0:
        raise ValueError("kept_idx holds a block index outside [0, nb)")
    return out, lse


def pool(x: torch.Tensor, block: int, block_valid: Optional[torch.Tensor] = None) -> torch.Tensor:
    """SEL-1 steps 1-2: pooled fp32 block means [H, nb, d] of a bf16 [H, N, d] tensor (ORD-0: over the first
    block_valid[b] tokens of block b)."""
    L = _load()
    H, N, d = x.shape
    nb = (N + block - 1) // block
    out = torch.empty((H, nb, d), dtype=torch.float32)
    L.oracle_pool(_ptr(_raw16(x)), ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(d),
                  ctypes.c_int(block), _ptr(None if block_valid is None else block_valid.contiguous().to(torch.int32)),
                  _ptr(out))
    return out


def select(q: torch.Tensor, k: torch.Tensor, block: int, topk: int, return_scores: bool = False,
           frame_tokens: int = 0, window: int = 0, block_valid: Optional[torch.Tensor] = None):
    """SEL-1.  q, k: [H, N, d] bf16.  Returns kept_idx int32 [H, nb, topk]
    (ascending), kept_cnt int32 [H, nb] (and the fp32 scores [H, nb, nb]).
    WIN-0: with ``frame_tokens`` > 0 only key blocks inside the causal frame window of the query
    block are candidates; kept_cnt = min(topk, candidates), unused list entries are -1."""
    L = _load()
    H, N, d = q.shape
    nb = (N + block - 1) // block
    idx = torch.empty((H, nb, topk), dtype=torch.int32)
    cnt = torch.empty((H, nb), dtype=torch.int32)
    scores = torch.empty((H, nb, nb), dtype=torch.float32) if return_scores else None
    rc = L.oracle_select(_ptr(_raw16(q)), _ptr(_raw16(k)), ctypes.c_int(H), ctypes.c_int(N),
                         ctypes.c_int(d), ctypes.c_int(block), ctypes.c_int(topk),
                         ctypes.c_int(frame_tokens), ctypes.c_int(window),
                         _ptr(None if block_valid is None else block_valid.contiguous().to(torch.int32)),
                         _ptr(idx), _ptr(cnt), _ptr(scores))
    if rc != 0:
        raise ValueError("topk must be in [1, nb]")
    return (idx, cnt, scores) if return_scores else (idx, cnt)


def select_f64_diff(q: torch.Tensor, k: torch.Tensor, block: int, topk: int, kept_idx: torch.Tensor):
    """Diagnostic: rows whose fp64 top-k set differs from ``kept_idx`` and the
    smallest relative gap between the k-th and (k+1)-th fp64 score."""
    L = _load()
    H, N, d = q.shape
    gap = ctypes.c_double(0.0)
    n = L.oracle_select_f64_diff(_ptr(_raw16(q)), _ptr(_raw16(k)), ctypes.c_int(H), ctypes.c_int(N),
                                 ctypes.c_int(d), ctypes.c_int(block), ctypes.c_int(topk),
                                 _ptr(kept_idx.contiguous().to(torch.int32)), ctypes.byref(gap))
    return int(n), float(gap.value)


def quant_fp8(x: torch.Tensor, block: int):
    """QNT-1.  x: [H, N, d] bf16.  Returns (codes uint8 [H, N, d], scales fp32 [H, nb])."""
    L = _load()
    H, N, d = x.shape
    nb = (N + block - 1) // block
    codes = torch.zeros((H, N, d), dtype=torch.uint8)
    scales = torch.zeros((H, nb), dtype=torch.float32)
    L.oracle_quant_fp8(_ptr(_raw16(x)), ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(d),
                       ctypes.c_int(block), _ptr(codes), _ptr(scales))
    return codes, scales


def quant_fp8_per_token(x: torch.Tensor):
    """QNT-1 with one scale per token.  x: [H, N, d] bf16.  Returns (codes uint8 [H, N, d], scales fp32 [H, N])."""
    L = _load()
    H, N, d = x.shape
    codes = torch.zeros((H, N, d), dtype=torch.uint8)
    scales = torch.zeros((H, N), dtype=torch.float32)
    L.oracle_quant_fp8_per_token(_ptr(_raw16(x)), ctypes.c_int(H), ctypes.c_int(N), ctypes.c_int(d),
                                 _ptr(codes), _ptr(scales))
    return codes, scales


def comp_state(k: torch.Tensor, v: torch.Tensor, pk: torch.Tensor, grid, axis: torch.Tensor, freq: torch.Tensor):
    """CMP-0, state: C[h] = sum_j k~_j v_j^T.  k, v bf16 [H, N, d]; pk bf16 [H, r, d]; grid (T, Hg, Wg);
    axis int32 [r/2] (0 = t, 1 = y, 2 = x); freq fp32 [r/2].  Returns fp64 [H, r, d]."""
    L = _load()
    H, N, d = k.shape
    r = pk.shape[1]
    assert grid[0] * grid[1] * grid[2] == N and pk.shape == (H, r, d)
    state = torch.zeros((H, r, d), dtype=torch.float64)
    g = torch.tensor(list(grid), dtype=torch.int32)
    L.oracle_comp_state(_ptr(_raw16(k)), _ptr(_raw16(v)), _ptr(_raw16(pk)), ctypes.c_int(H), ctypes.c_int(N),
                        ctypes.c_int(d), ctypes.c_int(r), _ptr(g), _ptr(axis.contiguous().to(torch.int32)),
                        _ptr(freq.contiguous().float()), _ptr(state))
    return state


def comp_apply(q: torch.Tensor, pq: torch.Tensor, state: torch.Tensor, gate: torch.Tensor, o_sparse: torch.Tensor,
               grid, axis: torch.Tensor, freq: torch.Tensor, rows, eps: float = 1e-6):
    """CMP-0, apply: O_i = O_s,i + g_i r_i RMSNorm(q~_i^T C) for the (head, token) pairs in ``rows``.
    Returns fp64 [len(rows), d]."""
    L = _load()
    H, N, d = q.shape
    r = pq.shape[1]
    rr = torch.tensor(list(rows), dtype=torch.int32).reshape(-1, 2).contiguous()
    out = torch.zeros((rr.shape[0], d), dtype=torch.float64)
    g = torch.tensor(list(grid), dtype=torch.int32)
    L.oracle_comp_apply(_ptr(_raw16(q)), _ptr(_raw16(pq)), _ptr(state.contiguous().double()),
                        _ptr(gate.contiguous().float()), _ptr(_raw16(o_sparse)), ctypes.c_int(H), ctypes.c_int(N),
                        ctypes.c_int(d), ctypes.c_int(r), _ptr(g), _ptr(axis.contiguous().to(torch.int32)),
                        _ptr(freq.contiguous().float()), ctypes.c_double(eps), _ptr(rr), ctypes.c_int(rr.shape[0]),
                        _ptr(out))
    return out


def brick_layout(grid, brick, block: int):
    """ORD-0, token order of 3-D bricks padded to whole blocks (the paper fixes contiguous blocks, Sec. 2, not
    the order of the tokens): the (T, Hg, Wg) grid is cut into bricks of (bt, bh, bw) cells with
    bt * bh * bw <= block, cut short at the far faces; bricks are visited in raster order of the brick grid,
    the cells of a brick in raster order inside it; every brick takes one block, its cells first, padding
    after them.  Written as that enumeration.  Returns (gather int32 [nbricks * block]: the raster index
    n = (t * Hg + y) * Wg + x of the token at each padded position, -1 for padding; block_valid int32
    [nbricks]; scatter int32 [N]: the padded position of raster token n)."""
    T, Hg, Wg = (int(v) for v in grid)
    bt, bh, bw = (int(v) for v in brick)
    assert bt * bh * bw <= block
    gather, valid = [], []
    for t0 in range(0, T, bt):
        for y0 in range(0, Hg, bh):
            for x0 in range(0, Wg, bw):
                cells = [(t * Hg + y) * Wg + x for t in range(t0, min(T, t0 + bt)) for y in range(y0, min(Hg, y0 + bh))
                         for x in range(x0, min(Wg, x0 + bw))]
                valid.append(len(cells))
                gather.extend(cells + [-1] * (block - len(cells)))
    gather = torch.tensor(gather, dtype=torch.int32)
    scatter = torch.empty(T * Hg * Wg, dtype=torch.int32)
    pos = torch.nonzero(gather >= 0).flatten()
    scatter[gather[pos].long()] = pos.to(torch.int32)
    return gather, torch.tensor(valid, dtype=torch.int32), scatter
