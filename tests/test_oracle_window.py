"""Pins for the causal frame window of the oracle (WIN-0: Sec. 1 mentions, without a formula, that the
method extends to auto-regressive generation by limiting attention to a causal window; read as: key j
counts for query i iff its frame j // F lies in (i // F - W, i // F]).  Independent formulations: library softmax over explicitly
masked logits, per-frame dense attention, brute-force candidate enumeration."""
import math

import numpy as np
import torch

import oracle


def _qkv(H, N, d, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda: torch.randn((H, N, d), generator=g).to(torch.bfloat16)
    return mk(), mk(), mk()


def _token_mask(N, F, W):
    f = torch.arange(N) // F
    return (f[None, :] <= f[:, None]) & (f[None, :] > f[:, None] - W)       # [query, key]


def _masked_reference(q, k, v, allowed):
    """fp64 softmax over the allowed keys with library ops; rows without any allowed key -> 0 / -inf."""
    s = (q.double() @ k.double().T) / math.sqrt(q.shape[-1])
    s = s.masked_fill(~allowed, float("-inf"))
    lse = torch.logsumexp(s, dim=-1)
    p = torch.exp(s - torch.where(torch.isinf(lse), torch.zeros_like(lse), lse)[:, None])
    p = torch.where(allowed, p, torch.zeros_like(p))
    return p @ v.double(), lse


def _all_blocks(H, nb):
    idx = torch.arange(nb, dtype=torch.int32).repeat(H, nb, 1)
    return idx, torch.full((H, nb), nb, dtype=torch.int32)


def test_full_lists_match_masked_library_softmax():
    H, N, d, blk, F = 2, 200, 16, 32, 50              # frames of 50 tokens straddle the 32-token blocks
    q, k, v = _qkv(H, N, d, 0)
    nb = (N + blk - 1) // blk
    idx, cnt = _all_blocks(H, nb)
    for W in (1, 2, 4, 7):
        out, lse = oracle.attention(q, k, v, idx, cnt, blk, frame_tokens=F, window=W)
        out = out.reshape(H, nb * blk, d)[:, :N]
        lse = lse.reshape(H, nb * blk)[:, :N]
        allowed = _token_mask(N, F, W)
        for h in range(H):
            ref, ref_lse = _masked_reference(q[h], k[h], v[h], allowed)
            assert torch.allclose(out[h], ref, atol=1e-12)
            assert torch.allclose(lse[h], ref_lse, atol=1e-12)


def test_window_of_one_frame_is_per_frame_attention():
    H, N, d, blk, F = 1, 192, 8, 64, 48
    q, k, v = _qkv(H, N, d, 1)
    nb = N // blk
    idx, cnt = _all_blocks(H, nb)
    out, _ = oracle.attention(q, k, v, idx, cnt, blk, frame_tokens=F, window=1)
    out = out.reshape(N, d)
    for f in range(N // F):
        sl = slice(f * F, (f + 1) * F)
        s = (q[0, sl].double() @ k[0, sl].double().T) / math.sqrt(d)
        ref = torch.softmax(s, dim=-1) @ v[0, sl].double()
        assert torch.allclose(out[sl], ref, atol=1e-12)


def test_sparse_lists_and_rows_without_admissible_keys():
    H, N, d, blk, F, W = 2, 230, 16, 32, 40, 2          # ragged last block (230 = 7 * 32 + 6)
    q, k, v = _qkv(H, N, d, 2)
    nb = (N + blk - 1) // blk
    g = torch.Generator().manual_seed(5)
    kmax = 3
    idx = torch.stack([torch.stack([torch.randperm(nb, generator=g)[:kmax] for _ in range(nb)]) for _ in range(H)]).to(torch.int32)
    cnt = torch.randint(0, kmax + 1, (H, nb), generator=g, dtype=torch.int32)
    out, lse = oracle.attention(q, k, v, idx, cnt, blk, frame_tokens=F, window=W)
    out = out.reshape(H, nb * blk, d)[:, :N]
    lse = lse.reshape(H, nb * blk)[:, :N]
    win = _token_mask(N, F, W)
    seen_empty = False
    for h in range(H):
        allowed = torch.zeros((N, N), dtype=torch.bool)
        for qb in range(nb):
            for t in range(int(cnt[h, qb])):
                kb = int(idx[h, qb, t])
                allowed[qb * blk:(qb + 1) * blk, kb * blk:(kb + 1) * blk] = True
        allowed &= win
        ref, ref_lse = _masked_reference(q[h], k[h], v[h], allowed)
        assert torch.allclose(out[h], ref, atol=1e-12)
        empty = ~allowed.any(dim=1)
        seen_empty |= bool(empty.any())
        assert torch.all(out[h][empty] == 0) and torch.all(torch.isneginf(lse[h][empty]))
        assert torch.allclose(lse[h][~empty], ref_lse[~empty], atol=1e-12)
    assert seen_empty


def test_select_candidates_by_brute_force():
    H, N, d, blk, F = 2, 230, 16, 32, 40
    q, k, _ = _qkv(H, N, d, 3)
    nb = (N + blk - 1) // blk
    for W, topk in ((1, 2), (2, 3), (3, nb)):
        idx, cnt, scores = oracle.select(q, k, blk, topk, return_scores=True, frame_tokens=F, window=W)
        win = _token_mask(N, F, W).numpy()
        for h in range(H):
            for qb in range(nb):
                rows = slice(qb * blk, min(N, (qb + 1) * blk))
                cand = [j for j in range(nb) if win[rows, j * blk:min(N, (j + 1) * blk)].any()]
                assert cand == list(range(cand[0], cand[-1] + 1))          # a contiguous run
                c = int(cnt[h, qb])
                assert c == min(topk, len(cand))
                kept = idx[h, qb, :c].tolist()
                assert kept == sorted(kept) and set(kept) <= set(cand)
                assert idx[h, qb, c:].tolist() == [-1] * (topk - c)
                sc = scores[h, qb].numpy()
                order = sorted(cand, key=lambda j: (-sc[j], j))[:c]
                assert sorted(order) == kept


def test_no_window_is_unchanged():
    H, N, d, blk = 1, 128, 8, 32
    q, k, v = _qkv(H, N, d, 4)
    a = oracle.select(q, k, blk, 2)
    b = oracle.select(q, k, blk, 2, frame_tokens=0, window=0)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    idx, cnt = a
    o1, l1 = oracle.attention(q, k, v, idx, cnt, blk)
    o2, l2 = oracle.attention(q, k, v, idx, cnt, blk, frame_tokens=N, window=1)   # one frame = everything
    assert torch.equal(o1, o2) and torch.equal(l1, l2)
