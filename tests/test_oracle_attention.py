"""Pins for the attention oracle (ATT-0): a dense library formula, an explicit
token-level mask, closed forms and invariants.  None of these re-use the
oracle's own loop."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads


def _dense_numpy(q, k, v, mask=None, scale=None):
    """softmax(Q K^T / sqrt(d) + mask) V in fp64 with library matmuls.
    q,k,v: [N, d] float64 arrays; mask: [N, N] of {0, -inf} or None."""
    d = q.shape[1]
    s = (q @ k.T) * (1.0 / math.sqrt(d) if scale is None else scale)
    if mask is not None:
        s = s + mask
    m = s.max(axis=1, keepdims=True)
    p = np.exp(s - m)
    l = p.sum(axis=1, keepdims=True)
    return (p @ v) / l, (m + np.log(l))[:, 0]


def _rand(H, N, d, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda: torch.randn((H, N, d), generator=g).to(torch.bfloat16)
    return mk(), mk(), mk()


def _flatten(out, lse, H, nb, block, N):
    """[H*nb, block, d] -> [H, N, d] dropping tail padding rows."""
    d = out.shape[-1]
    o = out.reshape(H, nb * block, d)[:, :N]
    l = lse.reshape(H, nb * block)[:, :N]
    return o.numpy(), l.numpy()


@pytest.mark.parametrize("N", [1, 63, 64, 65, 200])
def test_all_blocks_kept_equals_dense(N):
    H, d, block = 2, 32, 64
    q, k, v = _rand(H, N, d, 10 + N)
    nb = (N + block - 1) // block
    idx = torch.arange(nb, dtype=torch.int32).expand(H, nb, nb).contiguous()
    cnt = torch.full((H, nb), nb, dtype=torch.int32)
    out, lse = oracle.attention(q, k, v, idx, cnt, block)
    o, l = _flatten(out, lse, H, nb, block, N)
    for h in range(H):
        ro, rl = _dense_numpy(q[h].double().numpy(), k[h].double().numpy(), v[h].double().numpy())
        np.testing.assert_allclose(o[h], ro, rtol=0, atol=1e-12)
        np.testing.assert_allclose(l[h], rl, rtol=0, atol=1e-12)


def test_tiny_workload_dense_when_nothing_is_skipped():
    w = workloads.TINY
    q, k, v = workloads.tiny_inputs(w)
    q, k, v = q[0], k[0], v[0]
    nb = w.nb
    idx = torch.arange(nb, dtype=torch.int32).expand(w.H, nb, nb).contiguous()
    cnt = torch.full((w.H, nb), nb, dtype=torch.int32)
    items = [(h, i) for h in range(w.H) for i in (0, 7, nb - 1)]
    out, lse = oracle.attention(q, k, v, idx, cnt, w.block, items=items)
    for n, (h, i) in enumerate(items):
        ro, rl = _dense_numpy(q[h].double().numpy(), k[h].double().numpy(), v[h].double().numpy())
        rows = slice(i * w.block, (i + 1) * w.block)
        np.testing.assert_allclose(out[n].numpy(), ro[rows], atol=1e-12)
        np.testing.assert_allclose(lse[n].numpy(), rl[rows], atol=1e-12)


@pytest.mark.parametrize("N,block", [(256, 64), (200, 64), (130, 32)])
def test_block_mask_equals_dense_with_token_mask(N, block):
    H, d = 2, 16
    q, k, v = _rand(H, N, d, 77 + N)
    nb = (N + block - 1) // block
    keep = max(1, nb // 2)
    idx, cnt = workloads.random_block_mask(1, H, nb, keep, seed_base=5)
    idx, cnt = idx[0], cnt[0]
    out, lse = oracle.attention(q, k, v, idx, cnt, block, softmax_scale=0.37)
    o, l = _flatten(out, lse, H, nb, block, N)
    for h in range(H):
        mask = np.full((N, N), -np.inf)
        for qb in range(nb):
            for kb in idx[h, qb].tolist():
                mask[qb * block:(qb + 1) * block, kb * block:(kb + 1) * block] = 0.0
        ro, rl = _dense_numpy(q[h].double().numpy(), k[h].double().numpy(), v[h].double().numpy(), mask, 0.37)
        np.testing.assert_allclose(o[h], ro, atol=1e-12)
        np.testing.assert_allclose(l[h], rl, atol=1e-12)


def test_variable_counts_and_empty_list():
    H, N, d, block = 1, 192, 8, 64
    q, k, v = _rand(H, N, d, 3)
    idx = torch.tensor([[[2, 0, 0], [1, 2, 0], [0, 0, 0]]], dtype=torch.int32)
    cnt = torch.tensor([[1, 2, 0]], dtype=torch.int32)
    out, lse = oracle.attention(q, k, v, idx, cnt, block)
    o, l = _flatten(out, lse, H, 3, block, N)
    mask = np.full((N, N), -np.inf)
    mask[0:64, 128:192] = 0
    mask[64:128, 64:192] = 0
    ro, rl = _dense_numpy(q[0, :128].double().numpy(), k[0].double().numpy(), v[0].double().numpy(), mask[:128])
    np.testing.assert_allclose(o[0, :128], ro, atol=1e-12)
    np.testing.assert_allclose(l[0, :128], rl, atol=1e-12)
    assert np.all(o[0, 128:] == 0) and np.all(np.isneginf(l[0, 128:]))


def test_closed_forms():
    H, N, d, block = 1, 200, 8, 64  # tail block has 8 valid tokens
    q, k, v = _rand(H, N, d, 4)
    nb = 4
    idx = torch.tensor([[[1, 3], [0, 3], [2, 3], [3, 0]]], dtype=torch.int32)
    cnt = torch.full((1, nb), 2, dtype=torch.int32)
    vd = v[0].double().numpy()
    # Q = 0: uniform weights over the kept valid keys; lse = ln(#keys)
    out, lse = oracle.attention(torch.zeros_like(q), k, v, idx, cnt, block)
    o, l = _flatten(out, lse, H, nb, block, N)
    keys0 = np.r_[64:128, 192:200]
    np.testing.assert_allclose(o[0, :64], np.tile(vd[keys0].mean(0), (64, 1)), atol=1e-13)
    np.testing.assert_allclose(l[0, :64], math.log(72), atol=1e-13)
    # identical K rows give the same
    kc = k.clone(); kc[:] = k[0, 5]
    out, lse = oracle.attention(q, kc, v, idx, cnt, block)
    o2, _ = _flatten(out, lse, H, nb, block, N)
    np.testing.assert_allclose(o2[0, :64], np.tile(vd[keys0].mean(0), (64, 1)), atol=1e-12)
    # constant V
    vc = torch.full_like(v, 0.75)
    out, _ = oracle.attention(q, k, vc, idx, cnt, block)
    assert np.allclose(out.numpy()[0, :64], 0.75, atol=1e-14)
    # one dominant key: logit 60 above the others -> output is that V row
    qd = torch.zeros_like(q); kd = torch.zeros_like(k)
    qd[0, :, 0] = 8.0
    kd[0, 70, 0] = 60.0 * math.sqrt(d) / 8.0
    out, _ = oracle.attention(qd, kd, v, idx, cnt, block)
    np.testing.assert_allclose(out.numpy()[0, 3], vd[70], atol=1e-20, rtol=1e-12)
    # single kept block with a single valid key
    N1 = 129
    q1, k1, v1 = _rand(1, N1, d, 6)
    idx1 = torch.tensor([[[2], [2], [2]]], dtype=torch.int32)
    cnt1 = torch.ones((1, 3), dtype=torch.int32)
    out, lse = oracle.attention(q1, k1, v1, idx1, cnt1, 64)
    o1, _ = _flatten(out, lse, 1, 3, 64, N1)
    np.testing.assert_array_equal(o1[0], np.tile(v1[0, 128].double().numpy(), (N1, 1)))


def test_invariants():
    H, N, d, block = 2, 320, 16, 64
    q, k, v = _rand(H, N, d, 8)
    nb = 5
    idx, cnt = workloads.random_block_mask(1, H, nb, 3, seed_base=9)
    idx, cnt = idx[0], cnt[0]
    out, lse = oracle.attention(q, k, v, idx, cnt, block)
    # permuting a kept list changes nothing beyond summation order
    perm = idx.flip(-1).contiguous()
    out_p, lse_p = oracle.attention(q, k, v, perm, cnt, block)
    np.testing.assert_allclose(out_p.numpy(), out.numpy(), atol=1e-13)
    np.testing.assert_allclose(lse_p.numpy(), lse.numpy(), atol=1e-13)
    # output lies in the per-channel hull of the kept V rows
    o, _ = _flatten(out, lse, H, nb, block, N)
    for h in range(H):
        for qb in range(nb):
            rows = np.concatenate([np.arange(b * block, min(N, (b + 1) * block)) for b in idx[h, qb].tolist()])
            vv = v[h].double().numpy()[rows]
            blk = o[h, qb * block:(qb + 1) * block]
            assert np.all(blk <= vv.max(0) + 1e-12) and np.all(blk >= vv.min(0) - 1e-12)
    # shifting every logit of a row by a constant leaves O unchanged and moves lse by it:
    # append a channel: q' = [q, 1], k' = [k, alpha]  ->  s' = s + alpha * scale
    alpha = 3.0
    ones = torch.ones((H, N, 1), dtype=torch.bfloat16)
    qa = torch.cat([q, ones], -1); ka = torch.cat([k, alpha * ones], -1)
    sc = 1.0 / math.sqrt(d)
    out_a, lse_a = oracle.attention(qa, ka, torch.cat([v, ones], -1), idx, cnt, block, softmax_scale=sc)
    np.testing.assert_allclose(out_a.numpy()[..., :d], out.numpy(), atol=1e-12)
    np.testing.assert_allclose(lse_a.numpy(), lse.numpy() + alpha * sc, atol=1e-12)
    # the softmax weights sum to one: V = 1 gives exactly-normalised rows
    np.testing.assert_allclose(out_a.numpy()[..., d], 1.0, atol=1e-14)


def test_rejects_bad_index():
    q, k, v = _rand(1, 64, 8, 1)
    with pytest.raises(ValueError):
        oracle.attention(q, k, v, torch.tensor([[[5]]], dtype=torch.int32),
                         torch.ones((1, 1), dtype=torch.int32), 64)


def test_fp8_inputs_are_dequantised_exactly():
    """FP8 mode = bf16-free path: decode(code) * scale fed to the same definition."""
    H, N, d, block = 1, 160, 16, 64
    g = torch.Generator().manual_seed(12)
    codes = [torch.randint(0, 0x7F, (H, N, d), generator=g, dtype=torch.uint8) for _ in range(3)]
    for c in codes:  # random signs, avoid NaN codes
        c |= (torch.randint(0, 2, c.shape, generator=g, dtype=torch.uint8) << 7)
        c[(c & 0x7F) == 0x7F] = 0x7E
    nb = 3
    scales = [torch.rand((H, nb), generator=g) * 0.01 + 0.001 for _ in range(3)]
    idx = torch.tensor([[[0, 2], [1, 2], [0, 1]]], dtype=torch.int32)
    cnt = torch.full((1, 3), 2, dtype=torch.int32)
    out, lse = oracle.attention(codes[0], codes[1], codes[2], idx, cnt, block, scales=tuple(scales))
    table = torch.tensor([oracle.e4m3_decode(c) for c in range(256)], dtype=torch.float64)
    deq = []
    for c, s in zip(codes, scales):
        x = table[c.long()]
        x = x * s.double().repeat_interleave(block, dim=1)[:, :N, None]
        deq.append(x[0].numpy())
    mask = np.full((N, N), -np.inf)
    for qb in range(3):
        for kb in idx[0, qb].tolist():
            mask[qb * block:(qb + 1) * block, kb * block:(kb + 1) * block] = 0
    ro, rl = _dense_numpy(deq[0], deq[1], deq[2], mask)
    o, l = _flatten(out, lse, H, nb, block, N)
    np.testing.assert_allclose(o[0], ro, atol=1e-12, rtol=1e-12)
    np.testing.assert_allclose(l[0], rl, atol=1e-12)
