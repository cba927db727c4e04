"""The allocation-free selection entry point against the regular one.

Some callers cannot allocate device memory at the moment they call the library
(a serving loop with a fixed memory plan, a host application whose allocator is
frozen after start-up, a plugin that only gets its input and output buffers).
``sparkattn_select_noalloc`` keeps its scratch in a fixed array inside the
library, so it must give exactly the lists ``sparkattn_select`` gives, call
after call, although every call re-uses the same scratch memory.

This file is collected last on purpose: it exercises library-global state."""
import ctypes

import pytest
import torch

import paper_2609_23153_b200 as sa
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(cfg_id, H, grid, sparsity):
    w = workloads.small_structured(H=H, d=128, grid=grid, block=128, sparsity=sparsity, cfg_id=cfg_id)
    q, k, _ = workloads.structured_qkv(w)
    return w, q.to(DEV), k.to(DEV)


def test_noalloc_select_matches_regular_select_on_two_calls_in_a_row():
    # two different problems back to back: the second call starts with the first call's
    # pooled means still in the shared scratch (and a larger one precedes a smaller one)
    cases = [_case(71, 4, (5, 14, 20), 0.8), _case(72, 2, (3, 10, 17), 0.5)]
    # the first call on a device is also the one-time set-up (the library image with the
    # scratch array gets loaded onto the device): make it before watching the free memory
    w0, q0, k0 = cases[1]
    sa.select_noalloc(q0, k0, w0.block, 1, torch.empty((1, w0.H, w0.nb, 1), dtype=torch.int32, device=DEV), None)
    torch.cuda.synchronize()
    for w, q, k in cases:
        ref_idx, ref_cnt = sa.select(q, k, w.block, w.topk)
        idx = torch.full_like(ref_idx, -1)
        cnt = torch.full_like(ref_cnt, -1)
        free_before = torch.cuda.mem_get_info()[0]
        sa.select_noalloc(q, k, w.block, w.topk, idx, cnt)
        assert sa.lib().sparkattn_select_noalloc_status(ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)) == sa.OK
        assert torch.cuda.mem_get_info()[0] == free_before          # nothing was allocated by the call
        assert torch.equal(idx, ref_idx) and torch.equal(cnt, ref_cnt)
    # and the same problem twice gives the same lists again
    w, q, k = cases[0]
    ref_idx, _ = sa.select(q, k, w.block, w.topk)
    for _ in range(2):
        idx = torch.full_like(ref_idx, -1)
        sa.select_noalloc(q, k, w.block, w.topk, idx, None)
        assert torch.equal(idx, ref_idx)


def test_noalloc_select_rejects_shapes_beyond_its_scratch():
    limit = sa.lib().sparkattn_select_noalloc_max_bytes()
    assert limit == 32 << 20
    # 64 heads x 75,600 tokens needs ~39 MB of pooled means: beyond the built-in array
    big = sa.Shape(ctypes.sizeof(sa.Shape), sa.VERSION, 1, 64, 75600, 128, 128, 0,
                   64 * 75600 * 128, 75600 * 128, 128, 0.0, 0)
    assert sa.workspace_bytes(big, 0, 18) > limit
    fake = ctypes.c_void_p(0x1000)  # never dereferenced: the size check comes first
    rc = sa.lib().sparkattn_select_noalloc(ctypes.byref(big), fake, fake, 18, fake, None, None)
    assert rc == sa.E_WORKSPACE_TOO_SMALL
    assert "workspace" in sa.status_string(rc)
    # the benchmark's largest shape fits
    w = workloads.WAN_14B_720P
    fits = sa.Shape(ctypes.sizeof(sa.Shape), sa.VERSION, 1, w.H, w.N, 128, 128, 0, w.H * w.N * 128, w.N * 128, 128, 0.0, 0)
    assert 0 < sa.workspace_bytes(fits, 0, w.topk) <= limit
