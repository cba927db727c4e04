"""Pins for the selection oracle (SEL-1): exact rational arithmetic rounded to
fp32 by hand, a brute-force sort, constructed inputs with known answers."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import workloads


def _round_f32(x: Fraction) -> Fraction:
    """Round an exact rational to the nearest fp32 (ties to even), by integers only."""
    if x == 0:
        return Fraction(0)
    s = -1 if x < 0 else 1
    a = abs(x)
    e = 0
    while a >= 2 ** 24:
        a /= 2; e += 1
    while a < 2 ** 23 and e > -149 - 23 + 23:  # stay above the subnormal grid 2^-149
        a *= 2; e -= 1
    if e < -149:  # clamp to the subnormal spacing
        a = a / (2 ** (-149 - e)); e = -149
    n = a.numerator // a.denominator
    r = a - n
    if r > Fraction(1, 2) or (r == Fraction(1, 2) and n % 2 == 1):
        n += 1
    return s * Fraction(n) * (Fraction(2) ** e)


def _bf16_exact(x: torch.Tensor):
    return [[Fraction(float(v)) for v in row] for row in x.float().tolist()]


def _pool_exact(x: torch.Tensor, block: int):
    """x [N, d] bf16 -> list over blocks of lists of Fractions, following the
    stated order: sequential fp32 adds then one fp32 divide."""
    N, d = x.shape
    rows = _bf16_exact(x)
    out = []
    for b in range((N + block - 1) // block):
        t0, t1 = b * block, min(N, (b + 1) * block)
        acc = [Fraction(0)] * d
        for t in range(t0, t1):
            acc = [_round_f32(acc[c] + rows[t][c]) for c in range(d)]
        out.append([_round_f32(a / (t1 - t0)) for a in acc])
    return out


def _score_exact(pq, pk):
    a = Fraction(0)
    for x, y in zip(pq, pk):
        a = _round_f32(x * y + a)
    return a


def test_round_f32_helper_matches_numpy():
    rng = np.random.default_rng(0)
    for v in rng.standard_normal(200) * 10.0 ** rng.integers(-3, 4, 200):
        assert float(_round_f32(Fraction(float(v)))) == float(np.float32(v))
    # an exact tie: 1 + 2^-24 rounds to even (1.0); 1 + 3*2^-24 rounds up to 1 + 2^-22
    assert _round_f32(Fraction(1) + Fraction(1, 2 ** 24)) == 1
    assert _round_f32(Fraction(1) + Fraction(3, 2 ** 24)) == Fraction(1) + Fraction(1, 2 ** 22)


@pytest.mark.parametrize("N,block,d", [(100, 16, 8), (64, 16, 4)])
def test_pool_and_scores_match_exact_arithmetic(N, block, d):
    g = torch.Generator().manual_seed(N)
    q = torch.randn((1, N, d), generator=g).to(torch.bfloat16)
    k = torch.randn((1, N, d), generator=g).to(torch.bfloat16)
    pq = oracle.pool(q, block)[0]
    pq_x = _pool_exact(q[0], block)
    pk_x = _pool_exact(k[0], block)
    nb = len(pq_x)
    for b in range(nb):
        for c in range(d):
            assert Fraction(float(pq[b, c])) == pq_x[b][c]
    topk = 3
    idx, cnt, scores = oracle.select(q, k, block, topk, return_scores=True)
    for i in range(nb):
        exact = [_score_exact(pq_x[i], pk_x[j]) for j in range(nb)]
        for j in range(nb):
            assert Fraction(float(scores[0, i, j])) == exact[j]
        order = sorted(range(nb), key=lambda j: (-exact[j], j))[:topk]
        assert idx[0, i].tolist() == sorted(order)
    assert torch.all(cnt == topk)


def test_topk_matches_bruteforce_sort_on_oracle_scores():
    w = workloads.small_structured(H=2, d=32, grid=(4, 12, 20), block=32, sparsity=0.8)
    q, k, _ = workloads.structured_qkv(w)
    idx, cnt, scores = oracle.select(q[0], k[0], w.block, w.topk, return_scores=True)
    for h in range(w.H):
        for i in range(w.nb):
            s = scores[h, i].tolist()
            order = sorted(range(w.nb), key=lambda j: (-s[j], j))[: w.topk]
            assert idx[h, i].tolist() == sorted(order)


def _onehot_rows(nb, block, d, which, scale=1.0):
    """[nb*block, d] bf16 whose block b has every token equal to scale[b] * e_{which[b]}."""
    x = torch.zeros((nb * block, d), dtype=torch.bfloat16)
    for b in range(nb):
        sc = scale[b] if isinstance(scale, (list, tuple)) else scale
        x[b * block:(b + 1) * block, which[b]] = sc
    return x


def test_constructed_ranking_and_tie_break():
    nb, block, d = 6, 8, 8
    # query block i looks along channel i; key block j has weight w[j] on every channel
    q = _onehot_rows(nb, block, d, list(range(nb)))[None]
    k = torch.zeros((1, nb * block, d), dtype=torch.bfloat16)
    wts = [1.0, 4.0, 2.0, 4.0, 0.5, 4.0]
    for j in range(nb):
        k[0, j * block:(j + 1) * block, :] = wts[j]
    idx, _ = oracle.select(q, k, block, 2)
    # three key blocks tie at 4.0: the two lowest indices win
    assert all(row == [1, 3] for row in idx[0].tolist())
    idx, _ = oracle.select(q, k, block, 4)
    assert all(row == [1, 2, 3, 5] for row in idx[0].tolist())
    idx, _ = oracle.select(q, k, block, nb)
    assert all(row == list(range(nb)) for row in idx[0].tolist())
    idx, _ = oracle.select(q, k, block, 1)
    assert all(row == [1] for row in idx[0].tolist())
    # negative scores rank below zero scores
    idx, _ = oracle.select(q, -k, block, 1)
    assert all(row == [4] for row in idx[0].tolist())


def test_tail_block_uses_mean_not_sum():
    # N = 2 blocks + 2 tokens. The tail key block has large entries but only 2
    # tokens: a sum-based score would rank it last, the mean ranks it first.
    block, d = 8, 4
    N = 2 * block + 2
    q = torch.ones((1, N, d), dtype=torch.bfloat16)
    k = torch.ones((1, N, d), dtype=torch.bfloat16)
    k[0, :block] = 1.0
    k[0, block:2 * block] = 2.0
    k[0, 2 * block:] = 3.0
    idx, _ = oracle.select(q, k, block, 1)
    assert all(row == [2] for row in idx[0].tolist())
    p = oracle.pool(k, block)
    assert p[0, 2].tolist() == [3.0] * d


def test_permutation_structure():
    # pooled q of block i = e_i, pooled k of block j = e_{perm[j]}: score(i,j) = [perm[j] == i]
    nb, block, d = 8, 4, 8
    perm = [3, 0, 6, 1, 7, 2, 5, 4]
    q = _onehot_rows(nb, block, d, list(range(nb)))[None]
    k = _onehot_rows(nb, block, d, perm)[None]
    idx, _ = oracle.select(q, k, block, 1)
    for i in range(nb):
        assert idx[0, i, 0].item() == perm.index(i)


def test_f64_diagnostic_agrees_on_structured_inputs():
    w = workloads.small_structured(H=2, d=64, grid=(6, 16, 24), block=64, sparsity=0.9)
    q, k, _ = workloads.structured_qkv(w)
    idx, _ = oracle.select(q[0], k[0], w.block, w.topk)
    ndiff, gap = oracle.select_f64_diff(q[0], k[0], w.block, w.topk, idx)
    assert ndiff == 0 and gap > 1e-6
    # and it does flag a wrong list
    bad = idx.clone()
    bad[0, 0, 0] = (bad[0, 0, 0] + 1) % w.nb if (bad[0, 0, 0] + 1) % w.nb not in bad[0, 0].tolist() else bad[0, 0, 0]
    bad[1, 2] = torch.sort(torch.randperm(w.nb)[: w.topk]).values.to(torch.int32)
    ndiff2, _ = oracle.select_f64_diff(q[0], k[0], w.block, w.topk, bad)
    assert ndiff2 >= 1


def test_budget_for_sparsity_matches_paper_block_work_ratio():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "block_work_ratio.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    nb = workloads.WAN_14B_720P.nb
    assert nb == 591 and workloads.WAN_1P3B_480P.nb == 256 and workloads.TINY.nb == 32
    for sa, sb, ratio, tol in rows:
        ka = workloads.kept_blocks_for_sparsity(float(sa), nb)
        kb = workloads.kept_blocks_for_sparsity(float(sb), nb)
        assert abs(ka / kb - float(ratio)) <= float(tol)
    assert workloads.WAN_14B_720P.topk == 18 and workloads.WAN_1P3B_480P.topk == 26
    assert workloads.kept_blocks_for_sparsity(0.0, nb) == nb
    assert workloads.kept_blocks_for_sparsity(0.9999, nb) == 1
