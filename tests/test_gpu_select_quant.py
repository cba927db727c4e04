"""GPU parity: sparkattn_select and sparkattn_quant_fp8 against the CPU oracle, bit for bit."""
import pytest
import torch

import oracle
import paper_2609_23153_b200 as sa
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _small_cases():
    return [
        workloads.small_structured(H=3, d=128, grid=(5, 12, 20), block=128, sparsity=0.8, cfg_id=11),   # N=1200: 9 full + tail 48
        workloads.small_structured(H=2, d=128, grid=(3, 16, 16), block=128, sparsity=0.5, cfg_id=12),   # N=768: no tail
        workloads.small_structured(H=2, d=64, grid=(3, 10, 21), block=64, sparsity=0.9, cfg_id=13),     # N=630: tail 54
        workloads.small_structured(H=1, d=64, grid=(1, 1, 37), block=64, sparsity=0.0, cfg_id=14),      # one ragged block
        workloads.small_structured(H=2, d=128, grid=(1, 1, 1), block=128, sparsity=0.0, cfg_id=15),     # N=1
        workloads.small_structured(H=2, d=128, grid=(4, 9, 25), block=64, sparsity=0.9, cfg_id=17),     # d=128, 64-token blocks, tail 4
    ]


@pytest.mark.parametrize("w", _small_cases(), ids=lambda w: f"{w.name}-N{w.N}-d{w.d}")
def test_select_matches_oracle(w):
    q, k, _ = workloads.structured_qkv(w)
    for topk in sorted({1, w.topk, w.nb}):
        ref_idx, ref_cnt = oracle.select(q[0], k[0], w.block, topk)
        idx, cnt = sa.select(q.to(DEV), k.to(DEV), w.block, topk)
        torch.cuda.synchronize()
        assert torch.equal(idx[0].cpu(), ref_idx)
        assert torch.equal(cnt[0].cpu(), ref_cnt)


def test_select_tiny_workload_and_ties():
    w = workloads.TINY
    q, k, _ = workloads.tiny_inputs(w)
    ref_idx, _ = oracle.select(q[0], k[0], w.block, 16)
    idx, _ = sa.select(q.to(DEV), k.to(DEV), w.block, 16)
    assert torch.equal(idx[0].cpu(), ref_idx)
    # exact ties: every key block identical -> lowest indices win
    kc = k.clone(); kc[:] = k[0, 0, 5]
    ref_idx, _ = oracle.select(q[0], kc[0], w.block, 7)
    idx, _ = sa.select(q.to(DEV), kc.to(DEV), w.block, 7)
    assert torch.equal(idx[0].cpu(), ref_idx)
    assert ref_idx[0, 0].tolist() == list(range(7))
    # zero queries: all scores +0/-0 -> still the lowest indices
    ref_idx, _ = oracle.select(torch.zeros_like(q[0]), -k[0], w.block, 5)
    idx, _ = sa.select(torch.zeros_like(q).to(DEV), (-k).to(DEV), w.block, 5)
    assert torch.equal(idx[0].cpu(), ref_idx)


def _crafted_qk(nb, block, d, pattern, tail=0):
    """Q/K whose pooled block scores are known exactly: channel 0 of key block j holds v_j on all its tokens,
    channel 0 of query block i holds a_i, every other channel is 0, so score(i, j) = a_i * v_j without rounding."""
    N = nb * block - tail
    j = torch.arange(nb)
    if pattern == "one_lane":          # the largest keys all sit in one lane (j % 32 == 5) of the selecting warp
        v = torch.where(j % 32 == 5, 64.0 + (j // 32).float(), ((j * 37) % 97).float() / 128.0)
    elif pattern == "ties":            # two values only: most of the kept keys are ties at the threshold
        v = (j % 3 == 0).float()
    elif pattern == "few_then_ties":   # three clear winners, then a long run of equal keys
        v = torch.where(j % 101 == 7, 5.0 + (j // 101).float(), torch.where((j % 4) != 1, 2.0, 0.25))
    else:
        raise ValueError(pattern)
    a = torch.tensor([1.0, -1.0, 0.5, -0.75, 2.0])[torch.arange(nb) % 5]      # sign flips reverse the order
    q = torch.zeros((1, 2, N, d), dtype=torch.bfloat16)
    k = torch.zeros((1, 2, N, d), dtype=torch.bfloat16)
    tok_blk = torch.arange(N) // block
    q[0, :, :, 0] = a[tok_blk].to(torch.bfloat16)
    k[0, 0, :, 0] = v[tok_blk].to(torch.bfloat16)
    k[0, 1, :, 0] = v.flip(0)[tok_blk].to(torch.bfloat16)
    return q, k


@pytest.mark.parametrize("nb,topk", [(100, 7), (300, 8), (300, 40), (1000, 30), (1000, 140), (1400, 12)])
@pytest.mark.parametrize("pattern", ["one_lane", "ties", "few_then_ties"])
def test_select_crafted_scores(nb, topk, pattern):
    """Score layouts aimed at the branches of the selection: many of the largest keys in one lane of the warp
    (the search over per-lane maxima must give way to the full search), long runs of ties at the threshold,
    every register-resident key count (nb <= 256, 640, 1280) and the shared-memory path above."""
    block, d = 64, 128
    q, k = _crafted_qk(nb, block, d, pattern, tail=13)
    ref_idx, ref_cnt = oracle.select(q[0], k[0], block, topk)
    idx, cnt = sa.select(q.to(DEV), k.to(DEV), block, topk)
    assert torch.equal(idx[0].cpu(), ref_idx)
    assert torch.equal(cnt[0].cpu(), ref_cnt)


@pytest.mark.parametrize("pattern", ["one_lane", "ties"])
def test_select_crafted_scores_with_window(pattern):
    nb, block, d, topk = 300, 64, 128, 9
    q, k = _crafted_qk(nb, block, d, pattern, tail=13)
    F, window = 1000, 6                       # frames of 1000 tokens straddle the 64-token blocks
    ref_idx, ref_cnt = oracle.select(q[0], k[0], block, topk, frame_tokens=F, window=window)
    idx, cnt = sa.select(q.to(DEV), k.to(DEV), block, topk, frame_tokens=F, window=window)
    assert torch.equal(idx[0].cpu(), ref_idx)
    assert torch.equal(cnt[0].cpu(), ref_cnt)


def test_select_strided_layout_and_batch():
    # [B, N, H, d] storage viewed as [B, H, N, d]; two batches
    w = workloads.small_structured(H=2, d=128, grid=(2, 10, 26), block=128, sparsity=0.75, cfg_id=16)
    qs, ks = [], []
    for b in range(2):
        q, k, _ = workloads.structured_qkv(workloads.small_structured(2, 128, (2, 10, 26), 128, 0.75, cfg_id=16 + b))
        qs.append(q[0]); ks.append(k[0])
    q = torch.stack(qs); k = torch.stack(ks)
    qd = q.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    kd = k.permute(0, 2, 1, 3).contiguous().to(DEV).permute(0, 2, 1, 3)
    idx, cnt = sa.select(qd, kd, w.block, w.topk)
    for b in range(2):
        ref_idx, _ = oracle.select(q[b], k[b], w.block, w.topk)
        assert torch.equal(idx[b].cpu(), ref_idx)


@pytest.mark.parametrize("w", _small_cases(), ids=lambda w: f"{w.name}-N{w.N}-d{w.d}")
def test_quant_matches_oracle(w):
    q, _, v = workloads.structured_qkv(w)
    for x in (q, v):
        ref_codes, ref_scales = oracle.quant_fp8(x[0], w.block)
        codes, scales = sa.quant_fp8(x.to(DEV), w.block)
        torch.cuda.synchronize()
        assert torch.equal(scales[0].cpu().view(torch.int32), ref_scales.view(torch.int32))
        assert torch.equal(codes[0].cpu(), ref_codes)


def test_quant_edge_values():
    H, N, d, block = 2, 300, 128, 128
    g = torch.Generator().manual_seed(21)
    x = (torch.randn((1, H, N, d), generator=g) * 4).to(torch.bfloat16)
    x[0, 0, :128] = 0                       # all-zero block
    x[0, 1, 130, 7] = -1000.0               # one huge negative element: the rest underflows towards zero
    x[0, 1, 131, 9] = 3.0e-3
    x[0, 0, 256:] *= 1e-20                  # tiny magnitudes in the tail block
    ref_codes, ref_scales = oracle.quant_fp8(x[0], block)
    # canary: rows past N of a padded buffer must stay untouched
    buf = torch.full((1, H, N + 20, d), 0xAB, dtype=torch.uint8, device=DEV)
    xd = torch.zeros((1, H, N + 20, d), dtype=torch.bfloat16, device=DEV)
    xd[:, :, :N] = x.to(DEV)
    codes, scales = sa.quant_fp8(xd[:, :, :N], block, codes=buf[:, :, :N])
    torch.cuda.synchronize()
    assert torch.equal(codes[0].cpu(), ref_codes)
    assert torch.equal(scales[0].cpu().view(torch.int32), ref_scales.view(torch.int32))
    assert torch.all(buf[:, :, N:] == 0xAB)


def test_select_and_quant_are_deterministic():
    w = workloads.small_structured(H=4, d=128, grid=(4, 12, 20), block=128, sparsity=0.8, cfg_id=19)
    q, k, v = (t.to(DEV) for t in workloads.structured_qkv(w))
    a = sa.select(q, k, w.block, w.topk)[0].clone()
    b = sa.select(q, k, w.block, w.topk)[0].clone()
    assert torch.equal(a, b)
    c1 = sa.quant_fp8(v, w.block)[0].clone()
    c2 = sa.quant_fp8(v, w.block)[0].clone()
    assert torch.equal(c1, c2)


@pytest.mark.parametrize("w", _small_cases(), ids=lambda w: f"{w.name}-N{w.N}-d{w.d}")
def test_per_token_quant_matches_oracle(w):
    q, _, v = workloads.structured_qkv(w)
    v = v * torch.logspace(-2, 1, w.N)[None, None, :, None].to(torch.bfloat16)   # widely varying row magnitudes
    v[0, 0, w.N // 2] = 0
    for x in (q, v):
        ref_codes, ref_scales = oracle.quant_fp8_per_token(x[0])
        codes, scales = sa.quant_fp8_per_token(x.to(DEV))
        torch.cuda.synchronize()
        assert torch.equal(scales[0].cpu().view(torch.int32), ref_scales.view(torch.int32))
        assert torch.equal(codes[0].cpu(), ref_codes)


def test_per_token_quant_strided_and_fullsize_sample():
    w = workloads.WAN_1P3B_480P
    q, _, _ = workloads.structured_qkv(w, device=DEV)
    qs = q.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)          # [B,N,H,d] storage
    codes, scales = sa.quant_fp8_per_token(qs)
    assert codes.stride() == qs.stride()
    for h in (0, 11):
        rc, rs = oracle.quant_fp8_per_token(q[0, h:h + 1].cpu())
        assert torch.equal(codes[0, h:h + 1].cpu(), rc) and torch.equal(scales[0, h:h + 1].cpu().view(torch.int32), rs.view(torch.int32))


def _pooled_from_workspace(ws, H, nb, d):
    """Pooled Q [H, nb, d] and pooled K [H, nb, d] out of a selection workspace (B = 1): pooled Q sits right
    behind the 256-byte header, pooled K transposed [H, d, nbp] (nbp = nb rounded up to 32) behind it."""
    nbp = (nb + 31) // 32 * 32
    f = ws[256:].view(torch.float32).cpu()
    pq = f[: H * nb * d].reshape(H, nb, d)
    pk = f[H * nb * d: H * nb * d + H * d * nbp].reshape(H, d, nbp)[:, :, :nb].transpose(1, 2).contiguous()
    return pq, pk


@pytest.mark.parametrize("w", _small_cases(), ids=lambda w: f"{w.name}-N{w.N}-d{w.d}")
def test_quant_with_pooling_and_select_from_pooled_match_oracle(w):
    """One pass over Q and one over K give codes, scales AND the selection's pooled means (same order of
    additions as the selection's own pooling: bit-exact against oracle.pool); scores + top-k on those means
    give the oracle's lists."""
    q, k, _ = workloads.structured_qkv(w)
    qd, kd = q.to(DEV), k.to(DEV)
    ws = sa.alloc_workspace(sa.make_shape(qd, w.block), 0, w.topk, DEV)
    ws.fill_(0x5A)                                           # stale contents must not matter
    cq, sq = sa.quant_fp8_pooled(qd, w.block, False, ws)
    ck, sk = sa.quant_fp8_pooled(kd, w.block, True, ws)
    for (codes, scales), x in (((cq, sq), q), ((ck, sk), k)):
        rc, rs = oracle.quant_fp8(x[0], w.block)
        assert torch.equal(codes[0].cpu(), rc)
        assert torch.equal(scales[0].cpu().view(torch.int32), rs.view(torch.int32))
    torch.cuda.synchronize()
    pq, pk = _pooled_from_workspace(ws, w.H, w.nb, w.d)
    assert torch.equal(pq.view(torch.int32), oracle.pool(q[0], w.block).view(torch.int32))
    assert torch.equal(pk.view(torch.int32), oracle.pool(k[0], w.block).view(torch.int32))
    for topk in sorted({1, w.topk, w.nb}):
        idx, cnt = sa.select_pooled(qd, w.block, topk, ws)
        ref_idx, ref_cnt = oracle.select(q[0], k[0], w.block, topk)
        assert sa.read_status(ws) == sa.OK
        assert torch.equal(idx[0].cpu(), ref_idx) and torch.equal(cnt[0].cpu(), ref_cnt)


def test_quant_with_pooling_strided_batch_equals_separate_calls():
    """[B, N, H, d] buffers viewed as [B, H, N, d], two batch entries: the fused pass must reproduce the separate
    sparkattn_quant_fp8 / sparkattn_select calls bit for bit."""
    H, d, block, topk = 3, 128, 128, 2
    g = torch.Generator().manual_seed(21)
    q = torch.randn((2, 700, H, d), generator=g).to(torch.bfloat16).to(DEV).permute(0, 2, 1, 3)
    k = torch.randn((2, 700, H, d), generator=g).to(torch.bfloat16).to(DEV).permute(0, 2, 1, 3)
    ws = sa.alloc_workspace(sa.make_shape(q, block), 0, topk, DEV)
    cq, sq = sa.quant_fp8_pooled(q, block, False, ws)
    ck, sk = sa.quant_fp8_pooled(k, block, True, ws)
    idx, cnt = sa.select_pooled(q, block, topk, ws)
    rq, rsq = sa.quant_fp8(q, block)
    rk, rsk = sa.quant_fp8(k, block)
    ridx, rcnt = sa.select(q, k, block, topk)
    assert cq.stride() == q.stride()
    assert torch.equal(cq, rq) and torch.equal(ck, rk)
    assert torch.equal(sq.view(torch.int32), rsq.view(torch.int32)) and torch.equal(sk.view(torch.int32), rsk.view(torch.int32))
    assert torch.equal(idx, ridx) and torch.equal(cnt, rcnt)
