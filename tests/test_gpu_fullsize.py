"""GPU parity at the benchmark's full sizes and launch configuration
(Wan2.1-1.3B-480P at 90 % and Wan2.1-14B-720P at 97 % sparsity).

The whole tensors go through the same calls bench.py times; the fp64 oracle
then recomputes a sample of (head, query block) work items one by one: for
every sampled head the first block, the ragged last block and a few seeded
random blocks.  Selection is compared in full for the sampled heads."""
import math

import pytest
import torch

import oracle
import paper_2609_23153_b200 as sa
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _sample_items(w, heads, n_random, seed):
    g = torch.Generator().manual_seed(seed)
    items = []
    for h in heads:
        qbs = {0, w.nb - 1} | {int(x) for x in torch.randint(1, w.nb - 1, (n_random,), generator=g)}
        items += [(h, i) for i in sorted(qbs)]
    return items


def _gather(out_dev, items, w):
    rows = []
    for h, qb in items:
        rows.append(out_dev[h, qb * w.block: min(w.N, (qb + 1) * w.block)].cpu())
    return torch.cat(rows)


def _ref_rows(ref, items, w):
    return torch.cat([ref[n, : min(w.N, (qb + 1) * w.block) - qb * w.block] for n, (h, qb) in enumerate(items)])


def _relrms(got, ref):
    got, ref = got.double(), ref.double()
    return math.sqrt(float(((got - ref) ** 2).sum()) / float((ref ** 2).sum())), float((got - ref).abs().max())


@pytest.mark.parametrize("name,heads,n_random", [("wan1p3b", list(range(12)), 6), ("wan14b", list(range(0, 40, 3)), 4)])
def test_fullsize_bf16_select_and_fwd(name, heads, n_random):
    w = workloads.WORKLOADS[name]
    q, k, v = workloads.structured_qkv(w, device=DEV)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    out, lse = sa.fwd(q, k, v, idx, cnt, w.block, return_lse=True, check_status=True)
    torch.cuda.synchronize()
    qh, kh, vh = (t[0, heads].cpu() for t in (q, k, v))
    ref_idx, ref_cnt = oracle.select(qh, kh, w.block, w.topk)
    assert torch.equal(idx[0, heads].cpu(), ref_idx), "kept-block lists differ from the oracle"
    assert torch.equal(cnt[0, heads].cpu(), ref_cnt)
    ndiff, gap = oracle.select_f64_diff(qh[:2], kh[:2], w.block, w.topk, ref_idx[:2])
    print(f"{name}: fp64 top-k differs on {ndiff} rows of 2 heads, min relative gap {gap:.3e}")
    local = _sample_items(w, range(len(heads)), n_random, seed=7)
    ref_out, ref_lse = oracle.attention(qh, kh, vh, ref_idx, ref_cnt, w.block, items=local)
    items = [(heads[h], i) for h, i in local]
    rel, mx = _relrms(_gather(out[0], items, w), _ref_rows(ref_out, local, w))
    dl = (_gather(lse[0][..., None], items, w)[:, 0].double() - _ref_rows(ref_lse[..., None], local, w)[:, 0]).abs().max().item()
    print(f"{name}: {len(items)} work items, relRMS {rel:.3e}, max abs {mx:.3e}, lse abs {dl:.3e}")
    assert rel <= 1e-2 and mx <= 3e-2 and dl <= 1e-2
    # properties that hold at any size: finite output everywhere, untouched nothing past N
    assert torch.isfinite(out.float()).all() and torch.isfinite(lse).all()


def test_fullsize_fp8_quant_and_fwd():
    w = workloads.WAN_14B_720P
    heads = [0, 13, 39]
    q, k, v = workloads.structured_qkv(w, device=DEV)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    cs = [sa.quant_fp8(t, w.block) for t in (q, k, v)]
    out = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, w.block, scales=tuple(s for _, s in cs), check_status=True)
    torch.cuda.synchronize()
    # codes and scales bit-exact on the sampled heads
    for (codes, scales), x in zip(cs, (q, k, v)):
        rc, rs = oracle.quant_fp8(x[0, heads].cpu(), w.block)
        assert torch.equal(codes[0, heads].cpu(), rc)
        assert torch.equal(scales[0, heads].cpu().view(torch.int32), rs.view(torch.int32))
    local = _sample_items(w, range(len(heads)), 2, seed=11)
    ref_out, _ = oracle.attention(*(c[0, heads].cpu() for c, _ in cs), idx[0, heads].cpu(), cnt[0, heads].cpu(), w.block,
                                  items=local, scales=tuple(s[0, heads].cpu() for _, s in cs))
    items = [(heads[h], i) for h, i in local]
    rel, mx = _relrms(_gather(out[0], items, w), _ref_rows(ref_out, local, w))
    got, ref = _gather(out[0], items, w).double(), _ref_rows(ref_out, local, w).double()
    worst_row = float((((got - ref) ** 2).sum(-1) / (ref ** 2).sum(-1).clamp_min(1e-300)).sqrt().max())
    print(f"wan14b fp8: {len(items)} work items, relRMS {rel:.3e}, max abs {mx:.3e}, worst row relRMS {worst_row:.3e}")
    assert rel <= 5e-2 and worst_row <= 1.5e-1
    assert torch.isfinite(out.float()).all()


def test_fullsize_fused_quant_pool_select_matches_separate_calls(wan14b_inputs):
    """The 40-head 75,600-token shape through the fused chain the benchmark's FP8 leg times (quantise + pool Q,
    quantise + pool K, scores + top-k on the pooled means): codes, scales and kept lists identical to the
    separate calls, which the other tests compare with the oracle."""
    w, (q, k, v), cs, host = wan14b_inputs
    ws = sa.alloc_workspace(sa.make_shape(q, w.block), 0, w.topk, DEV)
    cq, sq = sa.quant_fp8_pooled(q, w.block, False, ws)
    ck, sk = sa.quant_fp8_pooled(k, w.block, True, ws)
    idx, cnt = sa.select_pooled(q, w.block, w.topk, ws)
    assert sa.read_status(ws) == sa.OK
    ridx, rcnt = sa.select(q, k, w.block, w.topk)
    assert torch.equal(idx, ridx) and torch.equal(cnt, rcnt)
    assert torch.equal(cq, cs[0][0]) and torch.equal(ck, cs[1][0])
    assert torch.equal(sq.view(torch.int32), cs[0][1].view(torch.int32)) and torch.equal(sk.view(torch.int32), cs[1][1].view(torch.int32))
    heads = SWEEP_HEADS
    ref_idx, _ = oracle.select(*host["bf16"][:2], w.block, w.topk)
    assert torch.equal(idx[0, heads].cpu(), ref_idx)


def test_host_buffer_call_matches_device_call():
    w = workloads.WAN_1P3B_480P.with_heads(2)
    q, k, v = workloads.structured_qkv(w)
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    idx, cnt = sa.select(qd, kd, w.block, w.topk)
    for dtype in (sa.BF16, sa.FP8_E4M3):
        if dtype == sa.BF16:
            ref = sa.fwd(qd, kd, vd, idx, cnt, w.block)
        else:
            cs = [sa.quant_fp8(t, w.block) for t in (qd, kd, vd)]
            ref = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, w.block, scales=tuple(s for _, s in cs))
        hidx = torch.empty(idx.shape, dtype=torch.int32).pin_memory()
        out = sa.attention_host(q.pin_memory(), k.pin_memory(), v.pin_memory(), w.block, w.topk, dtype=dtype, kept_idx=hidx)
        assert torch.equal(out, ref.cpu())
        assert torch.equal(hidx, idx.cpu())


@pytest.mark.parametrize("B,H,block", [(2, 5, 128), (1, 20, 64), (3, 7, 128)])
def test_host_buffer_call_head_groups(B, H, block):
    """The host path runs groups of heads as a pipeline; groups never straddle a batch entry, the last group of a
    batch entry may be short, and with B*H > 16 groups the groups grow.  Result identical to the device calls."""
    g = torch.Generator().manual_seed(100 * B + H)
    N, d, topk = 700, 128, 3
    q, k, v = (torch.randn((B, H, N, d), generator=g).to(torch.bfloat16) for _ in range(3))
    qd, kd, vd = q.to(DEV), k.to(DEV), v.to(DEV)
    idx, cnt = sa.select(qd, kd, block, topk)
    ref = sa.fwd(qd, kd, vd, idx, cnt, block, check_status=True)
    hidx = torch.empty(idx.shape, dtype=torch.int32).pin_memory()
    out = sa.attention_host(q.pin_memory(), k.pin_memory(), v.pin_memory(), block, topk, kept_idx=hidx)
    assert torch.equal(hidx, idx.cpu())
    assert torch.equal(out, ref.cpu())
    out2 = sa.attention_host(q, k, v, block, topk)          # pageable host memory: same result
    assert torch.equal(out2, ref.cpu())


def test_fullsize_paper_block_size_64_bf16_and_fp8():
    """Wan2.1-14B-720P shape with the paper's trained 64x64 blocks (nb = 1182, 35 kept at 97 %)."""
    w64 = workloads.Workload("wan14b_b64", 3, 1, 40, 128, (21, 45, 80), 64, 0.97)
    assert w64.nb == 1182 and w64.topk == 35
    heads = [0, 21, 39]
    q, k, v = workloads.structured_qkv(w64, device=DEV)
    idx, cnt = sa.select(q, k, w64.block, w64.topk)
    out = sa.fwd(q, k, v, idx, cnt, w64.block, check_status=True)
    qh, kh, vh = (t[0, heads].cpu() for t in (q, k, v))
    ref_idx, ref_cnt = oracle.select(qh, kh, w64.block, w64.topk)
    assert torch.equal(idx[0, heads].cpu(), ref_idx)
    local = _sample_items(w64, range(len(heads)), 6, seed=17)
    items = [(heads[h], i) for h, i in local]
    ref_out, _ = oracle.attention(qh, kh, vh, ref_idx, ref_cnt, w64.block, items=local)
    rel, mx = _relrms(_gather(out[0], items, w64), _ref_rows(ref_out, local, w64))
    print(f"wan14b 64x64 bf16: {len(items)} work items, relRMS {rel:.3e}, max abs {mx:.3e}")
    assert rel <= 1e-2 and mx <= 3e-2
    cs = [sa.quant_fp8(t, w64.block) for t in (q, k, v)]
    out8 = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, w64.block, scales=tuple(s for _, s in cs), check_status=True)
    rc, rs = oracle.quant_fp8(kh, w64.block)
    assert torch.equal(cs[1][0][0, heads].cpu(), rc) and torch.equal(cs[1][1][0, heads].cpu().view(torch.int32), rs.view(torch.int32))
    local8 = local[:9]
    ref8, _ = oracle.attention(*(c[0, heads].cpu() for c, _ in cs), ref_idx, ref_cnt, w64.block, items=local8,
                               scales=tuple(s[0, heads].cpu() for _, s in cs))
    rel8, mx8 = _relrms(_gather(out8[0], [(heads[h], i) for h, i in local8], w64), _ref_rows(ref8, local8, w64))
    print(f"wan14b 64x64 fp8: {len(local8)} work items, relRMS {rel8:.3e}, max abs {mx8:.3e}")
    assert rel8 <= 5e-2


# ----------------------------------------------------------------------------- sparsity sweep on the 720P shape
SWEEP_HEADS = [0, 17, 39]
FP8_ROW_RELRMS = 1.5e-1     # guard beside the aggregate bound: one wrong row must not hide in the average


@pytest.fixture(scope="module")
def wan14b_inputs():
    w = workloads.WAN_14B_720P
    q, k, v = workloads.structured_qkv(w, device=DEV)
    cs = [sa.quant_fp8(t, w.block) for t in (q, k, v)]
    heads = SWEEP_HEADS
    host = {"bf16": tuple(t[0, heads].cpu() for t in (q, k, v)),
            "codes": tuple(c[0, heads].cpu() for c, _ in cs), "scales": tuple(s[0, heads].cpu() for _, s in cs)}
    yield w, (q, k, v), cs, host
    del q, k, v, cs
    torch.cuda.empty_cache()


def _row_relrms(got, ref):
    got, ref = got.double(), ref.double()
    return (((got - ref) ** 2).sum(-1) / (ref ** 2).sum(-1).clamp_min(1e-300)).sqrt()


@pytest.mark.parametrize("sparsity", [0.0, 0.5, 0.75, 0.9, 0.97])
def test_sparsity_sweep_points_bf16_and_fp8(wan14b_inputs, sparsity):
    """Every point of the sparsity sweep the benchmark reports (0 / 50 / 75 / 90 / 97 % on the 40-head
    75,600-token shape), bf16 and FP8, through the calls and launch configuration the benchmark times:
    selection in full on three heads against the oracle (bit-exact), then the forward on the whole tensors
    with a sample of work items (first block, ragged last block, two seeded random blocks per head) recomputed
    by the fp64 oracle.  The lists run from 18 to 591 tiles per query block."""
    w0, (q, k, v), cs, host = wan14b_inputs
    w = w0.with_sparsity(sparsity)
    heads = SWEEP_HEADS
    idx, cnt = sa.select(q, k, w.block, w.topk)
    qh, kh, vh = host["bf16"]
    ref_idx, ref_cnt = oracle.select(qh, kh, w.block, w.topk)
    assert torch.equal(idx[0, heads].cpu(), ref_idx), "kept-block lists differ from the oracle"
    assert torch.equal(cnt[0, heads].cpu(), ref_cnt)
    if sparsity == 0.0:
        assert w.topk == w.nb and torch.equal(ref_idx[0, 5], torch.arange(w.nb, dtype=torch.int32))
    local = _sample_items(w, range(len(heads)), 2, seed=int(1000 * sparsity) + 3)
    items = [(heads[h], i) for h, i in local]

    out, lse = sa.fwd(q, k, v, idx, cnt, w.block, return_lse=True, check_status=True)
    ref_out, ref_lse = oracle.attention(qh, kh, vh, ref_idx, ref_cnt, w.block, items=local)
    got, ref = _gather(out[0], items, w), _ref_rows(ref_out, local, w)
    rel, mx = _relrms(got, ref)
    dl = (_gather(lse[0][..., None], items, w)[:, 0].double() - _ref_rows(ref_lse[..., None], local, w)[:, 0]).abs().max().item()
    print(f"sweep s={sparsity} bf16: kept {w.topk}, {len(items)} items, relRMS {rel:.3e}, max abs {mx:.3e}, lse {dl:.3e}")
    assert rel <= 1e-2 and mx <= 3e-2 and dl <= 1e-2
    assert torch.isfinite(out.float()).all()
    del out, lse

    out8 = sa.fwd(cs[0][0], cs[1][0], cs[2][0], idx, cnt, w.block, scales=tuple(s for _, s in cs), check_status=True)
    ref8, _ = oracle.attention(*host["codes"], ref_idx, ref_cnt, w.block, items=local, scales=host["scales"])
    got8, r8 = _gather(out8[0], items, w), _ref_rows(ref8, local, w)
    rel8, mx8 = _relrms(got8, r8)
    rows8 = float(_row_relrms(got8, r8).max())
    print(f"sweep s={sparsity} fp8: relRMS {rel8:.3e}, max abs {mx8:.3e}, worst row relRMS {rows8:.3e}")
    assert rel8 <= 5e-2 and rows8 <= FP8_ROW_RELRMS
    assert torch.isfinite(out8.float()).all()
