"""Host-side checks that need no GPU: the C-ABI library loads, exports every
symbol the public header declares, and rejects bad arguments before touching
the device."""
import ctypes
import os
import re

import pytest
import torch

import paper_2609_23153_b200 as sa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_23153_b200 import build
    build.build()
    return sa.lib()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "sparkattn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sparkattn_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared_symbols()
    assert set(sa.EXPORTS) <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in sparkattn.h but not exported"


def test_version_and_status_strings(lib):
    assert lib.sparkattn_version() == sa.VERSION
    seen = set()
    for code in range(0, -9, -1):
        s = sa.status_string(code)
        assert s and s != "unknown status" and s not in seen
        seen.add(s)
    assert sa.status_string(-99) == "unknown status"


def _shape(B=1, H=2, N=2048, d=64, block=64):
    return sa.Shape(ctypes.sizeof(sa.Shape), sa.VERSION, B, H, N, d, block, 0, H * N * d, N * d, d, 0.0, 0)


def test_shape_struct_matches_header_size():
    # 2*u32 + 6*i32 + 3*i64 + f32 + u32 = 64 bytes, no implicit padding
    assert ctypes.sizeof(sa.Shape) == 64


def test_workspace_sizes(lib):
    s = _shape()
    nb = 32
    assert sa.workspace_bytes(s, 1, 16) == 256
    assert sa.workspace_bytes(s, 0, 16) == 256 + 2 * nb * 64 * 4 + 2 * 64 * 32 * 4
    assert sa.workspace_bytes(s, 2, 0) == 256          # the gather call: status header only
    assert sa.workspace_bytes(s, 3, 16) == 0
    bad = _shape(d=96)
    assert sa.workspace_bytes(bad, 0, 16) == 0
    assert sa.arena_bytes(s, sa.BF16, 16) > 4 * 2 * 2048 * 64 * 2
    assert sa.arena_bytes(s, sa.BF16, 0) == 0


def test_argument_errors_are_caught_on_the_host(lib):
    s = _shape()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: validation fails first
    null = ctypes.c_void_p(0)
    st = ctypes.c_void_p(0)
    r = lib.sparkattn_select(ctypes.byref(s), null, fake, 4, fake, null, fake, 1 << 20, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select(ctypes.byref(s), fake, fake, 0, fake, null, fake, 1 << 20, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select(ctypes.byref(s), fake, fake, 33, fake, null, fake, 1 << 20, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select(ctypes.byref(s), fake, fake, 4, fake, null, fake, 16, st)
    assert r == sa.E_WORKSPACE_TOO_SMALL
    r = lib.sparkattn_select(ctypes.byref(s), ctypes.c_void_p(0x1008), fake, 4, fake, null, fake, 1 << 20, st)
    assert r == sa.E_MISALIGNED
    bad = _shape(d=96)
    assert lib.sparkattn_quant_fp8(ctypes.byref(bad), fake, fake, fake, 0, st) == sa.E_UNSUPPORTED_SHAPE
    assert lib.sparkattn_quant_fp8(ctypes.byref(s), fake, fake, fake, 1, st) == sa.E_INVALID_ARG
    odd = _shape()
    odd.stride_n = 72
    assert lib.sparkattn_quant_fp8(ctypes.byref(odd), fake, fake, fake, 0, st) == sa.E_MISALIGNED
    wrong = _shape()
    wrong.version = 7
    assert lib.sparkattn_quant_fp8(ctypes.byref(wrong), fake, fake, fake, 0, st) == sa.E_INVALID_ARG
    # fwd: FP8 needs scales and the 128/128 shape; kmax in range
    r = lib.sparkattn_fwd(ctypes.byref(s), sa.FP8_E4M3, fake, fake, fake, null, null, null, fake, null, 4, fake,
                          null, fake, 256, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_fwd(ctypes.byref(s), sa.FP8_E4M3, fake, fake, fake, fake, fake, fake, fake, null, 4, fake,
                          null, fake, 256, st)
    assert r == sa.E_UNSUPPORTED_SHAPE            # FP8 needs d = 128
    assert sa.workspace_bytes(_shape(d=64, block=64), 1, 4) == 256
    # d = 128 keeps checked copies of the kept lists behind the status words: per item, or per pair of 64-token blocks
    assert sa.workspace_bytes(_shape(d=128, block=128), 1, 4) == 256 + 256 + 2 * 16 * 4 * 4 + 2 * 4
    assert sa.workspace_bytes(_shape(d=128, block=64), 1, 4) == 256 + 256 + 2 * 16 * 8 * 4 + 2 * 4
    assert sa.workspace_bytes(_shape(d=128, block=64), 1, 0) == 0
    assert sa.workspace_bytes(_shape(d=64, block=128), 1, 4) == 0
    r = lib.sparkattn_fwd(ctypes.byref(s), sa.BF16, fake, fake, fake, null, null, null, fake, null, 40, fake,
                          null, fake, 256, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_fwd(ctypes.byref(s), 5, fake, fake, fake, null, null, null, fake, null, 4, fake,
                          null, fake, 256, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_fwd(ctypes.byref(s), sa.BF16, fake, fake, fake, null, null, null, fake, null, 4, fake,
                          null, fake, 8, st)
    assert r == sa.E_WORKSPACE_TOO_SMALL
    # causal window: frame size and window length must be positive; selection with a window needs kept_cnt
    r = lib.sparkattn_fwd_window(ctypes.byref(s), sa.BF16, fake, fake, fake, null, null, null, fake, null, 4, 0, 1, fake,
                                 null, fake, 256, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_fwd_window(ctypes.byref(s), sa.BF16, fake, fake, fake, null, null, null, fake, null, 4, 64, 0, fake,
                                 null, fake, 256, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select_window(ctypes.byref(s), fake, fake, 4, 64, 1, fake, null, fake, 1 << 20, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select_window(ctypes.byref(s), fake, fake, 4, 64, 1, fake, fake, fake, 16, st)
    assert r == sa.E_WORKSPACE_TOO_SMALL
    # compensation branch: d = 128 and rank 64 only; the grid must cover N; rotary tables checked
    s128 = _shape(d=128, block=128)
    grid = (ctypes.c_int32 * 3)(2, 32, 32)
    axis = (ctypes.c_int32 * 32)(*([0] * 32))
    freq = (ctypes.c_float * 32)(*([1.0] * 32))
    r = lib.sparkattn_comp_state(ctypes.byref(s), fake, fake, fake, 64, grid, axis, freq, fake, fake, 1 << 30, st)
    assert r == sa.E_UNSUPPORTED_SHAPE            # d = 64
    r = lib.sparkattn_comp_state(ctypes.byref(s128), fake, fake, fake, 32, grid, axis, freq, fake, fake, 1 << 30, st)
    assert r == sa.E_UNSUPPORTED_SHAPE            # rank 32
    bad_grid = (ctypes.c_int32 * 3)(2, 32, 31)
    r = lib.sparkattn_comp_state(ctypes.byref(s128), fake, fake, fake, 64, bad_grid, axis, freq, fake, fake, 1 << 30, st)
    assert r == sa.E_INVALID_ARG
    axis[5] = 3
    r = lib.sparkattn_comp_state(ctypes.byref(s128), fake, fake, fake, 64, grid, axis, freq, fake, fake, 1 << 30, st)
    assert r == sa.E_INVALID_ARG
    axis[5] = 0
    r = lib.sparkattn_comp_state(ctypes.byref(s128), fake, fake, fake, 64, grid, axis, freq, fake, fake, 256, st)
    assert r == sa.E_WORKSPACE_TOO_SMALL
    r = lib.sparkattn_comp_apply(ctypes.byref(s128), fake, fake, 64, grid, axis, freq, fake, fake, fake, fake,
                                 ctypes.c_float(0.0), fake, 1 << 20, st)
    assert r == sa.E_INVALID_ARG                  # eps must be positive
    assert lib.sparkattn_comp_workspace_bytes(ctypes.byref(s128), bad_grid) == 0
    assert lib.sparkattn_comp_workspace_bytes(ctypes.byref(s128), grid) > 256


def test_fused_quant_pool_entry_points_validate_on_the_host(lib):
    s = _shape()
    fake = ctypes.c_void_p(0x1000)
    null = ctypes.c_void_p(0)
    st = ctypes.c_void_p(0)
    need = sa.workspace_bytes(s, 0, 4)
    assert lib.sparkattn_quant_fp8_pooled(ctypes.byref(s), fake, fake, fake, 2, fake, need, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_quant_fp8_pooled(ctypes.byref(s), fake, fake, fake, 0, null, need, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_quant_fp8_pooled(ctypes.byref(s), fake, fake, fake, 1, fake, need - 1, st) == sa.E_WORKSPACE_TOO_SMALL
    assert lib.sparkattn_quant_fp8_pooled(ctypes.byref(s), fake, fake, fake, 1, ctypes.c_void_p(0x1010), need, st) == sa.E_MISALIGNED
    assert lib.sparkattn_select_pooled(ctypes.byref(s), 0, fake, null, fake, need, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_select_pooled(ctypes.byref(s), 33, fake, null, fake, need, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_select_pooled(ctypes.byref(s), 4, fake, null, fake, 16, st) == sa.E_WORKSPACE_TOO_SMALL
    assert lib.sparkattn_select_pooled(ctypes.byref(_shape(d=96)), 4, fake, null, fake, need, st) == sa.E_UNSUPPORTED_SHAPE


def test_binding_checks_layout():
    q = torch.zeros((1, 2, 128, 64), dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        sa.make_shape(q.transpose(2, 3), 64)
    s = sa.make_shape(q, 64)
    assert (s.B, s.H, s.N, s.d, s.block) == (1, 2, 128, 64, 64)
    assert (s.stride_b, s.stride_h, s.stride_n) == (2 * 128 * 64, 128 * 64, 64)
    # a [B, N, H, d] buffer viewed as [B, H, N, d]
    x = torch.zeros((1, 128, 2, 64), dtype=torch.bfloat16).permute(0, 2, 1, 3)
    s = sa.make_shape(x, 64)
    assert (s.stride_h, s.stride_n) == (64, 128)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(sa, "_lib", None)
    monkeypatch.setattr(sa, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        sa.lib()


def test_padded_brick_entry_points_validate_on_the_host(lib):
    s128 = _shape(d=128, block=128, N=4096)
    s64 = _shape()
    fake = ctypes.c_void_p(0x1000)
    null = ctypes.c_void_p(0)
    st = ctypes.c_void_p(0)
    grid = (ctypes.c_int32 * 3)(21, 45, 80)
    brick = (ctypes.c_int32 * 3)(3, 5, 8)
    gp, bp = ctypes.cast(grid, ctypes.c_void_p), ctypes.cast(brick, ctypes.c_void_p)
    lib.sparkattn_brick_count.restype = ctypes.c_int64
    assert lib.sparkattn_brick_count(gp, bp) == 7 * 9 * 10
    assert lib.sparkattn_brick_count(null, bp) == 0
    zero = (ctypes.c_int32 * 3)(3, 0, 8)
    assert lib.sparkattn_brick_count(gp, ctypes.cast(zero, ctypes.c_void_p)) == 0
    big = (ctypes.c_int32 * 3)(3, 9, 8)                                   # 216 cells > 128
    assert lib.sparkattn_brick_layout(gp, ctypes.cast(big, ctypes.c_void_p), 128, fake, fake, fake, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_brick_layout(gp, bp, 100, fake, fake, fake, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_brick_layout(gp, bp, 128, null, null, null, st) == sa.E_INVALID_ARG
    # select / fwd on padded bricks: block_valid required, N a multiple of the block, d = 128
    r = lib.sparkattn_select_padded(ctypes.byref(s128), fake, fake, 4, null, fake, null, fake, 1 << 24, st)
    assert r == sa.E_INVALID_ARG
    ragged = _shape(d=128, block=128, N=4000)
    r = lib.sparkattn_select_padded(ctypes.byref(ragged), fake, fake, 4, fake, fake, null, fake, 1 << 24, st)
    assert r == sa.E_INVALID_ARG
    r = lib.sparkattn_select_padded(ctypes.byref(s64), fake, fake, 4, fake, fake, null, fake, 1 << 24, st)
    assert r == sa.E_UNSUPPORTED_SHAPE
    r = lib.sparkattn_fwd_padded(ctypes.byref(s64), sa.BF16, fake, fake, fake, null, null, null, fake, fake, 4, fake, fake,
                                 null, fake, 1 << 24, st)
    assert r == sa.E_UNSUPPORTED_SHAPE
    r = lib.sparkattn_fwd_padded(ctypes.byref(s128), sa.BF16, fake, fake, fake, null, null, null, fake, fake, 4, null, fake,
                                 null, fake, 1 << 24, st)
    assert r == sa.E_INVALID_ARG
    # gather: shapes must agree in B, H, d; buffers must differ; workspace holds the status header
    other = _shape(d=128, block=128, N=4096)
    other.H = s128.H + 1
    assert lib.sparkattn_gather_tokens(ctypes.byref(s128), fake, ctypes.byref(other), fake, ctypes.c_void_p(0x2000), fake, 256, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_gather_tokens(ctypes.byref(s128), fake, ctypes.byref(s128), fake, fake, fake, 256, st) == sa.E_INVALID_ARG
    assert lib.sparkattn_gather_tokens(ctypes.byref(s128), fake, ctypes.byref(s128), fake, ctypes.c_void_p(0x2000), fake, 16, st) == sa.E_WORKSPACE_TOO_SMALL


def test_host_buffer_call_rejects_more_batches_than_head_groups(lib):
    """The host-buffer path runs at most 16 head groups and a group never spans two batch entries: B = 17
    must come back as an error at once (it used to loop for ever while sizing the groups)."""
    fake = ctypes.c_void_p(0x1000)
    st = ctypes.c_void_p(0)
    s = _shape(B=17, H=2, N=256, d=64, block=64)
    r = lib.sparkattn_attention_host(ctypes.byref(s), sa.BF16, fake, fake, fake, 2, fake, ctypes.c_void_p(0), fake, 1 << 40, st)
    assert r == sa.E_UNSUPPORTED_SHAPE
    # 16 batch entries of many heads still form 16 groups (one per batch entry): passes the group sizing
    # and stops at the arena-size check
    s = _shape(B=16, H=40, N=256, d=64, block=64)
    r = lib.sparkattn_attention_host(ctypes.byref(s), sa.BF16, fake, fake, fake, 2, fake, ctypes.c_void_p(0), fake, 256, st)
    assert r == sa.E_WORKSPACE_TOO_SMALL


def test_gated_forward_validates_on_the_host(lib):
    """sparkattn_fwd_gated: every argument check happens before the device is touched."""
    s = _shape(N=2048, d=128, block=128)
    fake = ctypes.c_void_p(0x1000)
    null = ctypes.c_void_p(0)
    st = ctypes.c_void_p(0)
    grid = (ctypes.c_int32 * 3)(2, 32, 32)
    axis = (ctypes.c_int32 * 32)(*([0] * 10 + [1] * 11 + [2] * 11))
    freq = (ctypes.c_float * 32)(*[0.01 * (m + 1) for m in range(32)])
    eps = ctypes.c_float(1e-6)
    need = lib.sparkattn_fwd_gated_workspace_bytes(ctypes.byref(s), 4, grid)
    assert need > sa.workspace_bytes(s, 1, 4)          # the plain forward's workspace plus the rotary table

    def call(shape=s, q=fake, kmax=4, rank=64, g=grid, ax=axis, e=eps, ws=fake, nbytes=need, state=fake):
        return lib.sparkattn_fwd_gated(ctypes.byref(shape), q, fake, fake, fake, null, kmax, fake, rank, g, ax, freq, state,
                                       fake, e, fake, null, ws, nbytes, st)

    assert call(q=null) == sa.E_INVALID_ARG
    assert call(state=null) == sa.E_INVALID_ARG
    assert call(kmax=0) == sa.E_INVALID_ARG
    assert call(kmax=17) == sa.E_INVALID_ARG                          # more than the 16 key blocks
    assert call(e=ctypes.c_float(0.0)) == sa.E_INVALID_ARG
    assert call(g=(ctypes.c_int32 * 3)(2, 32, 31)) == sa.E_INVALID_ARG     # grid does not multiply to N
    assert call(ax=(ctypes.c_int32 * 32)(*([3] * 32))) == sa.E_INVALID_ARG
    assert call(rank=32) == sa.E_UNSUPPORTED_SHAPE
    assert call(shape=_shape(N=2048, d=128, block=64)) == sa.E_UNSUPPORTED_SHAPE
    assert call(shape=_shape(N=2048, d=64, block=128)) == sa.E_UNSUPPORTED_SHAPE
    assert call(q=ctypes.c_void_p(0x1008)) == sa.E_MISALIGNED
    assert call(ws=ctypes.c_void_p(0x1010)) == sa.E_MISALIGNED
    assert call(nbytes=need - 1) == sa.E_WORKSPACE_TOO_SMALL
    assert lib.sparkattn_fwd_gated_workspace_bytes(ctypes.byref(_shape(N=2048, d=128, block=64)), 4, grid) == 0
    assert lib.sparkattn_fwd_gated_workspace_bytes(ctypes.byref(s), 4, (ctypes.c_int32 * 3)(2, 32, 31)) == 0
