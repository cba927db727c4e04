"""GPU parity of the low-rank compensation branch and gate fusion (Sec. 4.1) against the fp64 oracle.

Small cases are compared in full (several 128-token tiles, a ragged tail, batch > 1, strided
layouts); at the two benchmark shapes the state is compared for a sample of heads and the fused
output on sampled token rows (first tile, ragged last tile, seeded random rows).

Tolerances.  State: sums of bf16-rounded features times bf16 values in fp32, relative RMS error
<= 1e-2.  Fused output: relative RMS <= 1e-2; element-wise |err| <= 3e-2 + 2^-8 |ref| (the second
term is the bf16 rounding of the stored output, whose magnitude follows O_s)."""
import math

import pytest
import torch

import oracle
import paper_2609_23153_b200 as sa
import workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
RANK = 64


def _relrms(got, ref):
    got, ref = got.double(), ref.double()
    return math.sqrt(float(((got - ref) ** 2).sum()) / max(float((ref ** 2).sum()), 1e-300))


def _check_out(got, ref):
    got, ref = got.double(), ref.double()
    assert _relrms(got, ref) <= 1e-2
    assert bool(((got - ref).abs() <= 3e-2 + ref.abs() * 2.0 ** -8).all())


def _inputs(w, layout="bhnd"):
    q, k, v = workloads.structured_qkv(w, device=DEV)
    pq, pk, gate = workloads.compensation_params(w, RANK, device=DEV)
    axis, freq = workloads.rope_schedule(w.d, RANK)
    g = torch.Generator(device=DEV).manual_seed(w.cfg_id * 31 + 5)
    osp = torch.randn(q.shape, generator=g, device=DEV, dtype=torch.float32).to(torch.bfloat16)
    if layout == "bnhd":     # same logical tensors stored token-major
        q, k, v, osp = (t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v, osp))
    return q, k, v, osp, pq, pk, gate, axis, freq


@pytest.mark.parametrize("grid,H,B,layout", [((3, 10, 13), 2, 1, "bhnd"), ((2, 16, 40), 3, 1, "bnhd"),
                                             ((1, 9, 11), 2, 2, "bhnd"), ((5, 12, 16), 1, 1, "bhnd")])
def test_small_full(grid, H, B, layout):
    w = workloads.Workload("compsmall", 11 + H + B, B, H, 128, tuple(grid), 128, 0.5)
    q, k, v, osp, pq, pk, gate, axis, freq = _inputs(w, layout)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq, check_status=True)
    out = sa.comp_apply(q, pq, state, gate, osp, w.grid, axis, freq, check_status=True)
    torch.cuda.synchronize()
    rows = [(h, i) for h in range(H) for i in range(w.N)]
    for b in range(B):
        ref_state = oracle.comp_state(k[b].cpu().contiguous(), v[b].cpu().contiguous(), pk.cpu(), w.grid, axis, freq)
        assert _relrms(state[b].cpu(), ref_state) <= 1e-2
        ref = oracle.comp_apply(q[b].cpu().contiguous(), pq.cpu(), ref_state, gate[b].cpu(), osp[b].cpu().contiguous(),
                                w.grid, axis, freq, rows).reshape(H, w.N, w.d)
        _check_out(out[b].cpu(), ref)


def test_state_is_deterministic_and_apply_in_place():
    w = workloads.Workload("compdet", 17, 1, 2, 128, (4, 10, 16), 128, 0.5)
    q, k, v, osp, pq, pk, gate, axis, freq = _inputs(w)
    s1 = sa.comp_state(k, v, pk, w.grid, axis, freq)
    s2 = sa.comp_state(k, v, pk, w.grid, axis, freq)
    assert torch.equal(s1, s2)
    out = sa.comp_apply(q, pq, s1, gate, osp, w.grid, axis, freq)
    buf = osp.clone()
    sa.comp_apply(q, pq, s1, gate, buf, w.grid, axis, freq, out=buf)      # out aliases o_sparse
    assert torch.equal(out, buf)


def test_zero_gate_returns_sparse_output_bitwise():
    w = workloads.Workload("compzero", 19, 1, 2, 128, (2, 7, 19), 128, 0.5)
    q, k, v, osp, pq, pk, gate, axis, freq = _inputs(w)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq)
    out = sa.comp_apply(q, pq, state, torch.zeros_like(gate), osp, w.grid, axis, freq, check_status=True)
    assert torch.equal(out.view(torch.int16), osp.view(torch.int16))


def test_chain_with_sparse_branch():
    """select -> fwd -> compensation on one small structured workload, against the oracle chain."""
    w = workloads.small_structured(2, 128, (3, 16, 24), 128, 0.5, cfg_id=23)
    q, k, v = workloads.structured_qkv(w, device=DEV)
    pq, pk, gate = workloads.compensation_params(w, RANK, device=DEV)
    axis, freq = workloads.rope_schedule(w.d, RANK)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    o_s = sa.fwd(q, k, v, idx, cnt, w.block, check_status=True)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq, check_status=True)
    out = sa.comp_apply(q, pq, state, gate, o_s, w.grid, axis, freq, check_status=True)
    qc, kc, vc = q[0].cpu(), k[0].cpu(), v[0].cpu()
    ridx, rcnt = oracle.select(qc, kc, w.block, w.topk)
    assert torch.equal(ridx, idx[0].cpu())
    ref_os, _ = oracle.attention(qc, kc, vc, ridx, rcnt, w.block)
    ref_os = ref_os.reshape(w.H, w.nb * w.block, w.d)[:, : w.N]
    # the oracle's fusion starts from the bf16 sparse output the device branch produced (the
    # sparse branch itself is compared against ref_os here and in its own tests)
    assert _relrms(o_s[0].cpu(), ref_os) <= 1e-2
    ref_state = oracle.comp_state(kc, vc, pk.cpu(), w.grid, axis, freq)
    rows = [(h, i) for h in range(w.H) for i in range(w.N)]
    ref = oracle.comp_apply(qc, pq.cpu(), ref_state, gate[0].cpu(), o_s[0].cpu().contiguous(), w.grid, axis, freq,
                            rows).reshape(w.H, w.N, w.d)
    _check_out(out[0].cpu(), ref)


@pytest.mark.parametrize("name,heads", [("wan1p3b", [0, 5, 11]), ("wan14b", [0, 17, 39])])
def test_fullsize_sampled(name, heads):
    w = workloads.WORKLOADS[name]
    q, k, v, osp, pq, pk, gate, axis, freq = _inputs(w)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq, check_status=True)
    out = sa.comp_apply(q, pq, state, gate, osp, w.grid, axis, freq, check_status=True)
    torch.cuda.synchronize()
    g = torch.Generator().manual_seed(w.cfg_id)
    tail0 = (w.N // 128) * 128 if w.N % 128 else w.N - 128
    toks = sorted(set(range(0, 128, 9)) | set(range(tail0, w.N, 3)) |
                  {int(x) for x in torch.randint(0, w.N, (96,), generator=g)})
    sub = lambda t: t[0, heads].cpu().contiguous()
    ref_state = oracle.comp_state(sub(k), sub(v), pk[heads].cpu().contiguous(), w.grid, axis, freq)
    assert _relrms(state[0, heads].cpu(), ref_state) <= 1e-2
    rows = [(hi, i) for hi in range(len(heads)) for i in toks]
    ref = oracle.comp_apply(sub(q), pq[heads].cpu().contiguous(), ref_state, gate[0, heads].cpu().contiguous(), sub(osp),
                            w.grid, axis, freq, rows).reshape(len(heads), len(toks), w.d)
    got = out[0, heads][:, toks].cpu()
    _check_out(got, ref)


def test_argument_errors():
    w = workloads.Workload("comperr", 29, 1, 1, 128, (1, 8, 16), 128, 0.5)
    q, k, v, osp, pq, pk, gate, axis, freq = _inputs(w)
    with pytest.raises(sa.SparkAttnError) as e:
        sa.comp_state(k, v, pk, (1, 8, 15), axis, freq)              # grid does not cover N
    assert e.value.status == sa.E_INVALID_ARG
    with pytest.raises(sa.SparkAttnError) as e:
        sa.comp_state(k, v, pk[:, :32].contiguous(), w.grid, axis[:16], freq[:16])   # rank 32
    assert e.value.status == sa.E_UNSUPPORTED_SHAPE
    bad_axis = axis.clone()
    bad_axis[3] = 3
    with pytest.raises(sa.SparkAttnError) as e:
        sa.comp_state(k, v, pk, w.grid, bad_axis, freq)
    assert e.value.status == sa.E_INVALID_ARG
    state = torch.zeros((1, 1, RANK, 128), dtype=torch.float32, device=DEV)
    with pytest.raises(sa.SparkAttnError) as e:
        sa.comp_apply(q, pq, state, gate, osp, w.grid, axis, freq, eps=0.0)
    assert e.value.status == sa.E_INVALID_ARG
    with pytest.raises(sa.SparkAttnError) as e:
        sa.comp_state(k, v, pk, w.grid, axis, freq, workspace=torch.empty(256, dtype=torch.uint8, device=DEV))
    assert e.value.status == sa.E_WORKSPACE_TOO_SMALL
