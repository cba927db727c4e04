"""Pins for ORD-0 of the oracle: tokens stored brick by brick, every brick padded to a whole block
(``oracle.brick_layout``), and the ``block_valid`` argument of ``oracle.attention`` / ``oracle.pool`` /
``oracle.select`` (padding rows are not keys, do not enter the pooled means, are not evaluated as queries).
Independent formulations: a library sort by (brick, cell) coordinates, library softmax over explicitly masked
logits, exact integer pooling, and the invariance of dense attention under the reordering."""
import math

import numpy as np
import pytest
import torch

import oracle

LAYOUTS = [((4, 6, 8), (2, 3, 4), 32), ((5, 7, 9), (2, 3, 4), 32), ((3, 5, 7), (2, 2, 4), 16), ((21, 45, 80), (3, 5, 8), 128),
           ((21, 30, 52), (3, 5, 4), 64), ((2, 3, 13), (1, 1, 5), 8), ((2, 3, 4), (1, 1, 1), 4)]


def _coords(grid):
    T, Hg, Wg = grid
    n = np.arange(T * Hg * Wg)
    return n // (Hg * Wg), (n // Wg) % Hg, n % Wg


@pytest.mark.parametrize("grid,brick,block", LAYOUTS)
def test_layout_is_the_sort_by_brick_then_cell(grid, brick, block):
    gather, valid, scatter = (t.numpy() for t in oracle.brick_layout(grid, brick, block))
    t, y, x = _coords(grid)
    bt, bh, bw = brick
    order = np.lexsort((x, y, t, x // bw, y // bh, t // bt))         # last key is the primary one
    assert np.array_equal(gather[gather >= 0], order.astype(np.int32))
    nbricks = -(-grid[0] // bt) * -(-grid[1] // bh) * -(-grid[2] // bw)
    assert len(valid) == nbricks and len(gather) == nbricks * block
    for b in range(nbricks):                                          # cells first, padding after them
        blk = gather[b * block:(b + 1) * block]
        assert np.all(blk[:valid[b]] >= 0) and np.all(blk[valid[b]:] == -1)
        tok = blk[:valid[b]]
        assert len({(a // bt, c // bh, e // bw) for a, c, e in zip(t[tok], y[tok], x[tok])}) == 1   # one brick
        assert valid[b] == (np.ptp(t[tok]) + 1) * (np.ptp(y[tok]) + 1) * (np.ptp(x[tok]) + 1)         # a full box
    assert np.array_equal(gather[scatter], np.arange(len(scatter)))
    assert valid.sum() == grid[0] * grid[1] * grid[2]


def test_layout_without_padding_when_bricks_tile_the_grid():
    gather, valid, scatter = oracle.brick_layout((4, 16, 32), (2, 8, 8), 128)
    assert torch.all(valid == 128) and torch.all(gather >= 0) and len(gather) == 4 * 16 * 32
    gather, valid, _ = oracle.brick_layout((3, 4, 16), (1, 1, 16), 16)      # bricks = raster strips: identity
    assert gather.tolist() == list(range(3 * 4 * 16))


def _qkv(H, N, d, seed):
    g = torch.Generator().manual_seed(seed)
    mk = lambda: torch.randn((H, N, d), generator=g).to(torch.bfloat16)
    return mk(), mk(), mk()


def test_attention_with_block_valid_matches_masked_library_softmax():
    H, blk, nb, d = 2, 16, 7, 8
    N = nb * blk
    q, k, v = _qkv(H, N, d, 0)
    g = torch.Generator().manual_seed(1)
    valid = torch.randint(1, blk + 1, (nb,), generator=g, dtype=torch.int32)
    valid[2] = blk
    kmax = 4
    idx = torch.stack([torch.stack([torch.randperm(nb, generator=g)[:kmax] for _ in range(nb)]) for _ in range(H)]).to(torch.int32)
    cnt = torch.randint(1, kmax + 1, (H, nb), generator=g, dtype=torch.int32)
    out, lse = oracle.attention(q, k, v, idx, cnt, blk, block_valid=valid)
    out = out.reshape(H, N, d)
    lse = lse.reshape(H, N)
    is_real = (torch.arange(N) % blk) < valid[torch.arange(N) // blk]
    for h in range(H):
        allowed = torch.zeros((N, N), dtype=torch.bool)
        for qb in range(nb):
            for t in range(int(cnt[h, qb])):
                kb = int(idx[h, qb, t])
                allowed[qb * blk:(qb + 1) * blk, kb * blk:(kb + 1) * blk] = True
        allowed &= is_real[None, :]
        s = (q[h].double() @ k[h].double().T) / math.sqrt(d)
        s = s.masked_fill(~allowed, float("-inf"))
        ref = torch.softmax(s, dim=-1) @ v[h].double()
        ref_lse = torch.logsumexp(s, dim=-1)
        assert torch.allclose(out[h][is_real], ref[is_real], atol=1e-12)
        assert torch.allclose(lse[h][is_real], ref_lse[is_real], atol=1e-12)
        assert torch.all(out[h][~is_real] == 0)                     # padding rows are not evaluated


def test_pool_and_select_with_block_valid():
    H, blk, nb, d = 2, 8, 9, 4
    N = nb * blk
    g = torch.Generator().manual_seed(2)
    # small integers: the fp32 sums are exact, so the mean is one correctly rounded division
    q = torch.randint(-8, 9, (H, N, d), generator=g).to(torch.bfloat16)
    k = torch.randint(-8, 9, (H, N, d), generator=g).to(torch.bfloat16)
    valid = torch.randint(1, blk + 1, (nb,), generator=g, dtype=torch.int32)
    pq = oracle.pool(q, blk, block_valid=valid).numpy()
    pk = oracle.pool(k, blk, block_valid=valid).numpy()
    for x, p in ((q, pq), (k, pk)):
        for b in range(nb):
            ssum = x[:, b * blk: b * blk + int(valid[b])].double().sum(dim=1).numpy()
            assert np.array_equal(p[:, b], (ssum.astype(np.float32) / np.float32(int(valid[b]))))
    topk = 3
    idx, cnt, scores = oracle.select(q, k, blk, topk, return_scores=True, block_valid=valid)
    for h in range(H):
        for i in range(nb):
            sc64 = [float(np.dot(pq[h, i].astype(np.float64), pk[h, j].astype(np.float64))) for j in range(nb)]
            assert np.allclose(scores[h, i].numpy(), sc64, rtol=1e-5, atol=1e-5)     # scores come from the masked means
            sc = scores[h, i].tolist()
            order = sorted(range(nb), key=lambda j: (-sc[j], j))[:topk]
            assert idx[h, i].tolist() == sorted(order) and int(cnt[h, i]) == topk


def test_dense_attention_is_invariant_under_the_padded_brick_order():
    grid, brick, blk = (3, 5, 7), (2, 2, 4), 16
    H, d = 2, 8
    N = grid[0] * grid[1] * grid[2]
    q, k, v = _qkv(H, N, d, 3)
    gather, valid, scatter = oracle.brick_layout(grid, brick, blk)
    nbr = len(valid)

    def to_bricks(x):
        y = torch.zeros((H, nbr * blk, d), dtype=x.dtype)
        pos = torch.nonzero(gather >= 0).flatten()
        y[:, pos] = x[:, gather[pos].long()]
        return y

    nb_r = (N + blk - 1) // blk
    dense_r = torch.arange(nb_r, dtype=torch.int32).repeat(H, nb_r, 1)
    ref, _ = oracle.attention(q, k, v, dense_r, torch.full((H, nb_r), nb_r, dtype=torch.int32), blk)
    ref = ref.reshape(H, nb_r * blk, d)[:, :N]
    dense_b = torch.arange(nbr, dtype=torch.int32).repeat(H, nbr, 1)
    out, _ = oracle.attention(to_bricks(q), to_bricks(k), to_bricks(v), dense_b, torch.full((H, nbr), nbr, dtype=torch.int32),
                              blk, block_valid=valid)
    out = out.reshape(H, nbr * blk, d)[:, scatter.long()]
    assert torch.allclose(out, ref, atol=1e-12)
