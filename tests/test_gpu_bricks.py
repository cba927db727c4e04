"""GPU parity of the brick token order (bricks padded to whole blocks): layout and gather kernels bit-exact
against the oracle's enumeration, selection with per-block token counts bit-exact, forward with padding keys
masked within the bf16 / FP8 tolerances, and the whole chain raster -> bricks -> attention -> raster against
attention computed in raster order."""
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


@pytest.mark.parametrize("grid,brick,block", [((4, 6, 8), (2, 3, 4), 64), ((5, 7, 9), (2, 3, 4), 64), ((21, 45, 80), (3, 5, 8), 128),
                                              ((21, 30, 52), (3, 5, 4), 64), ((4, 16, 32), (2, 8, 8), 128), ((2, 3, 13), (1, 1, 5), 64)])
def test_layout_matches_oracle(grid, brick, block):
    gather, valid, scatter = sa.brick_layout(grid, brick, block)
    rg, rv, rs = oracle.brick_layout(grid, brick, block)
    assert torch.equal(gather.cpu(), rg) and torch.equal(valid.cpu(), rv) and torch.equal(scatter.cpu(), rs)


@pytest.mark.parametrize("d", [128, 64])
def test_gather_moves_rows_exactly(d):
    g = torch.Generator().manual_seed(d)
    B, H, N = 2, 3, 1000
    x = torch.randn((B, H, N, d), generator=g).to(torch.bfloat16).to(DEV)
    index = torch.randint(-1, N, (1500,), generator=g, dtype=torch.int32)
    index[7] = -1
    out = sa.gather_tokens(x, index.to(DEV), check_status=True)
    ref = torch.zeros((B, H, 1500, d), dtype=torch.bfloat16, device=DEV)
    real = index >= 0
    ref[:, :, real.to(DEV)] = x[:, :, index[real].long().to(DEV)]
    assert torch.equal(out, ref)
    # [B, N, H, d] storage viewed as [B, H, N, d]
    xs = x.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
    assert torch.equal(sa.gather_tokens(xs, index.to(DEV)), ref)
    # an index outside [0, N) other than -1: zero row and a status
    bad = index.clone(); bad[3] = N + 5
    ws = torch.empty(256, dtype=torch.uint8, device=DEV)
    out = sa.gather_tokens(x, bad.to(DEV), workspace=ws)
    assert sa.read_status(ws) == sa.E_BAD_INDEX
    assert torch.all(out[:, :, 3] == 0)


def _to_bricks(x, gather):
    return sa.gather_tokens(x, gather)


@pytest.mark.parametrize("grid,brick,block", [((6, 10, 23), (2, 4, 16), 128),     # bricks of 128, 92 (x tail), 64 (y tail) ... cells
                                              ((6, 10, 23), (2, 4, 8), 64),        # 64-token blocks: pairs of query blocks over merged lists
                                              ((5, 9, 21), (1, 3, 20), 64)])       # an odd number of bricks, 60 or 3 real rows
def test_select_and_fwd_with_block_valid_match_oracle(grid, brick, block):
    H, d, topk = 3, 128, 5
    w = workloads.small_structured(H, d, grid, block, 0.0, cfg_id=71)
    q, k, v = (t.to(DEV) for t in workloads.structured_qkv(w))
    gather, valid, scatter = sa.brick_layout(grid, brick, block)
    assert int(valid.min()) < block
    qb, kb, vb = (_to_bricks(t, gather) for t in (q, k, v))
    nbr = valid.numel()
    idx, cnt = sa.select(qb, kb, block, topk, block_valid=valid)
    ridx, rcnt = oracle.select(qb[0].cpu(), kb[0].cpu(), block, topk, block_valid=valid.cpu())
    assert torch.equal(idx[0].cpu(), ridx) and torch.equal(cnt[0].cpu(), rcnt)
    plain_idx, _ = sa.select(qb, kb, block, topk)
    assert not torch.equal(plain_idx, idx)                      # the token counts do change the ranking
    out, lse = sa.fwd(qb, kb, vb, idx, cnt, block, return_lse=True, check_status=True, block_valid=valid)
    ref, ref_lse = oracle.attention(qb[0].cpu(), kb[0].cpu(), vb[0].cpu(), ridx, rcnt, block, block_valid=valid.cpu())
    ref = ref.reshape(H, nbr * block, d)
    ref_lse = ref_lse.reshape(H, nbr * block)
    real = (gather >= 0).cpu()
    rel, mx = _relrms(out[0].cpu()[:, real], ref[:, real])
    assert rel <= 1e-2 and mx <= 3e-2
    assert float((lse[0].cpu().double()[:, real] - ref_lse[:, real]).abs().max()) <= 1e-2
    assert torch.isfinite(out.float()).all()
    # FP8 on the same lists
    cs = [sa.quant_fp8(t, block) for t in (qb, kb, vb)]
    out8 = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, block, scales=tuple(s for _, s in cs), check_status=True,
                  block_valid=valid)
    ref8, _ = oracle.attention(cs[0][0][0].cpu(), cs[1][0][0].cpu(), cs[2][0][0].cpu(), ridx, rcnt, block,
                               scales=tuple(s[0].cpu() for _, s in cs), block_valid=valid.cpu())
    rel8, _ = _relrms(out8[0].cpu()[:, real], ref8.reshape(H, nbr * block, d)[:, real])
    assert rel8 <= 5e-2


def test_dense_attention_through_the_brick_order_equals_raster_attention():
    grid, brick, block = (4, 9, 20), (2, 4, 10), 128            # bricks of 80, 20 (y tail) cells: every block padded
    H, d = 2, 128
    w = workloads.small_structured(H, d, grid, block, 0.0, cfg_id=73)
    q, k, v = (t.to(DEV) for t in workloads.structured_qkv(w))
    nb_r = w.nb
    dense_r = torch.arange(nb_r, dtype=torch.int32, device=DEV).repeat(1, H, nb_r, 1)
    ref = sa.fwd(q, k, v, dense_r, None, block, check_status=True)
    gather, valid, scatter = sa.brick_layout(grid, brick, block)
    nbr = valid.numel()
    qb, kb, vb = (_to_bricks(t, gather) for t in (q, k, v))
    dense_b = torch.arange(nbr, dtype=torch.int32, device=DEV).repeat(1, H, nbr, 1)
    outb = sa.fwd(qb, kb, vb, dense_b, None, block, check_status=True, block_valid=valid)
    back = sa.gather_tokens(outb, scatter, check_status=True)
    assert back.shape == ref.shape
    rel, mx = _relrms(back.cpu(), ref.cpu())
    assert rel <= 6e-3 and mx <= 3e-2                           # two bf16 results of the same exact attention


def test_benchmark_grid_sampled():
    """Wan2.1-14B-720P grid in 3 x 5 x 8 bricks (120 of 128 rows real in every block, 630 blocks), 97 % budget."""
    w = workloads.WAN_14B_720P.with_heads(2)
    brick, block = (3, 5, 8), 128
    q, k, v = workloads.structured_qkv(w, device=DEV)
    gather, valid, scatter = sa.brick_layout(w.grid, brick, block)
    assert valid.numel() == 630 and torch.all(valid == 120)
    qb, kb, vb = (_to_bricks(t, gather) for t in (q, k, v))
    topk = 19
    idx, cnt = sa.select(qb, kb, block, topk, block_valid=valid)
    ridx, rcnt = oracle.select(qb[0].cpu(), kb[0].cpu(), block, topk, block_valid=valid.cpu())
    assert torch.equal(idx[0].cpu(), ridx) and torch.equal(cnt[0].cpu(), rcnt)
    out = sa.fwd(qb, kb, vb, idx, cnt, block, check_status=True, block_valid=valid)
    items = [(h, i) for h in range(2) for i in (0, 1, 314, 629)]
    ref, _ = oracle.attention(qb[0].cpu(), kb[0].cpu(), vb[0].cpu(), ridx, rcnt, block, items=items, block_valid=valid.cpu())
    got = torch.stack([out[0, h, i * block: i * block + 120].cpu() for h, i in items])
    rel, mx = _relrms(got, ref[:, :120])
    assert rel <= 1e-2 and mx <= 3e-2
