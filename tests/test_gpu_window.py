"""GPU parity of the causal frame window (Sec. 1, auto-regressive extension) against the oracle:
window-restricted selection bit-exact, window-masked block-sparse attention within the bf16 / FP8
tolerances, rows without any admissible kept key (zero output, lse = -inf), and the benchmark shape on
sampled work items.  Both forward kernels are covered: d = 128 with 128-token blocks runs the
persistent pipelined kernel (64-token blocks in pairs), d = 64 the one-item-per-CTA kernel."""
import math

import pytest
import torch

import oracle
import paper_2609_23153_b200 as sa
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _relrms(got, ref):
    got, ref = got.double(), ref.double()
    return math.sqrt(float(((got - ref) ** 2).sum()) / max(float((ref ** 2).sum()), 1e-300)), float((got - ref).abs().max())


@pytest.mark.parametrize("H,d,grid,block,topk,window", [
    (2, 128, (6, 10, 23), 128, 4, 2),      # frames of 230 tokens straddle the 128-token blocks; ragged tail
    (3, 128, (12, 12, 15), 128, 6, 3),     # 180-token frames, 17 blocks per head
    (2, 128, (5, 9, 11), 64, 5, 1),        # 64-token blocks: pairs of query blocks on the persistent kernel
    (2, 64, (4, 8, 20), 64, 4, 2),         # d = 64
])
def test_select_and_fwd_with_window(H, d, grid, block, topk, window):
    w = workloads.small_structured(H, d, grid, block, 0.0, cfg_id=51 + H + block)
    F = grid[1] * grid[2]
    q, k, v = workloads.structured_qkv(w)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    idx, cnt = sa.select(qd, kd, block, topk, frame_tokens=F, window=window)
    ridx, rcnt = oracle.select(q[0], k[0], block, topk, frame_tokens=F, window=window)
    assert torch.equal(idx[0].cpu(), ridx) and torch.equal(cnt[0].cpu(), rcnt)
    assert int(rcnt.min()) < topk or window * F >= w.N          # the window does cut some lists short
    out, lse = sa.fwd(qd, kd, vd, idx, cnt, block, return_lse=True, check_status=True, frame_tokens=F, window=window)
    ref, ref_lse = oracle.attention(q[0], k[0], v[0], ridx, rcnt, block, frame_tokens=F, window=window)
    ref = ref.reshape(H, w.nb * block, d)[:, : w.N]
    ref_lse = ref_lse.reshape(H, w.nb * block)[:, : w.N]
    rel, mx = _relrms(out[0].cpu(), ref)
    assert rel <= 1e-2 and mx <= 3e-2
    fin = torch.isfinite(ref_lse)
    assert torch.equal(torch.isneginf(lse[0].cpu()), ~fin)
    assert float((lse[0].cpu().double()[fin] - ref_lse[fin]).abs().max()) <= 1e-2


def test_rows_without_admissible_keys_and_random_lists():
    """Random kept lists (not produced by the selector): many rows have no admissible kept key."""
    H, d, block, grid, window = 2, 128, 128, (8, 10, 16), 2
    w = workloads.small_structured(H, d, grid, block, 0.0, cfg_id=61)
    F = grid[1] * grid[2]
    q, k, v = workloads.structured_qkv(w)
    g = torch.Generator().manual_seed(7)
    kmax = 3
    idx = torch.stack([torch.stack([torch.randperm(w.nb, generator=g)[:kmax] for _ in range(w.nb)]) for _ in range(H)]).to(torch.int32)
    cnt = torch.randint(1, kmax + 1, (H, w.nb), generator=g, dtype=torch.int32)
    out, lse = sa.fwd(q.to(DEV), k.to(DEV), v.to(DEV), idx[None].to(DEV), cnt[None].to(DEV), block, return_lse=True,
                      check_status=True, frame_tokens=F, window=window)
    ref, ref_lse = oracle.attention(q[0], k[0], v[0], idx, cnt, block, frame_tokens=F, window=window)
    ref = ref.reshape(H, w.nb * block, d)[:, : w.N]
    ref_lse = ref_lse.reshape(H, w.nb * block)[:, : w.N]
    empty = torch.isneginf(ref_lse)
    assert bool(empty.any()) and bool((~empty).any())
    got = out[0].cpu()
    assert torch.all(got[empty] == 0) and torch.equal(torch.isneginf(lse[0].cpu()), empty)
    rel, mx = _relrms(got, ref)
    assert rel <= 1e-2 and mx <= 3e-2
    assert torch.isfinite(got.float()).all()


def test_fp8_with_window():
    H, d, block, grid, topk, window = 2, 128, 128, (6, 10, 23), 4, 2
    w = workloads.small_structured(H, d, grid, block, 0.0, cfg_id=63)
    F = grid[1] * grid[2]
    q, k, v = workloads.structured_qkv(w)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    idx, cnt = sa.select(qd, kd, block, topk, frame_tokens=F, window=window)
    cs = [sa.quant_fp8(t, block) for t in (qd, kd, vd)]
    out = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, block, scales=tuple(s for _, s in cs), check_status=True,
                 frame_tokens=F, window=window)
    ref, _ = oracle.attention(cs[0][0][0].cpu(), cs[1][0][0].cpu(), cs[2][0][0].cpu(), idx[0].cpu(), cnt[0].cpu(), block,
                              scales=tuple(s[0].cpu() for _, s in cs), frame_tokens=F, window=window)
    ref = ref.reshape(H, w.nb * block, d)[:, : w.N]
    rel, _ = _relrms(out[0].cpu(), ref)
    assert rel <= 5e-2 and torch.isfinite(out.float()).all()


def test_benchmark_shape_sampled():
    """Wan2.1-14B-720P shape (frames of 45 x 80 = 3600 tokens), window of 3 frames, 97 % budget."""
    w = workloads.WAN_14B_720P.with_heads(4)
    F, window = w.grid[1] * w.grid[2], 3
    q, k, v = workloads.structured_qkv(w, device=DEV)
    idx, cnt = sa.select(q, k, w.block, w.topk, frame_tokens=F, window=window)
    ridx, rcnt = oracle.select(q[0].cpu(), k[0].cpu(), w.block, w.topk, frame_tokens=F, window=window)
    assert torch.equal(idx[0].cpu(), ridx) and torch.equal(cnt[0].cpu(), rcnt)
    out = sa.fwd(q, k, v, idx, cnt, w.block, check_status=True, frame_tokens=F, window=window)
    g = torch.Generator().manual_seed(3)
    items = [(h, qb) for h in range(w.H) for qb in sorted({0, 27, 28, w.nb - 1} | {int(x) for x in torch.randint(0, w.nb, (3,), generator=g)})]
    ref, _ = oracle.attention(q[0].cpu(), k[0].cpu(), v[0].cpu(), ridx, rcnt, w.block, items=items, frame_tokens=F, window=window)
    got = torch.cat([out[0, h, qb * w.block: min(w.N, (qb + 1) * w.block)].cpu() for h, qb in items])
    want = torch.cat([ref[n, : min(w.N, (qb + 1) * w.block) - qb * w.block] for n, (h, qb) in enumerate(items)])
    rel, mx = _relrms(got, want)
    assert rel <= 1e-2 and mx <= 3e-2


def test_argument_errors():
    w = workloads.small_structured(1, 128, (2, 8, 16), 128, 0.0, cfg_id=65)
    q, k, v = (t.to(DEV) for t in workloads.structured_qkv(w))
    with pytest.raises(sa.SparkAttnError) as e:
        sa.select(q, k, 128, 1, frame_tokens=128, window=0)
    assert e.value.status == sa.E_INVALID_ARG
    idx, cnt = sa.select(q, k, 128, 1)
    with pytest.raises(sa.SparkAttnError) as e:
        sa.fwd(q, k, v, idx, cnt, 128, frame_tokens=128, window=-1)
    assert e.value.status == sa.E_INVALID_ARG
