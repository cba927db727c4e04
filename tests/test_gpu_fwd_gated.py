"""GPU parity of the forward with the fused gate epilogue (Sec. 4.1: O = O_s + g * r * O_lr).

Two comparisons.  (1) Against the fp64 oracle: oracle selection -> oracle attention gives O_s, which
is checked against the device's sparse branch; the oracle's fusion then starts from the bf16 O_s the
device's unfused forward produced (the fused kernel rounds O_s to bf16 exactly as that call stores
it), at the tolerances of the compensation tests: relative RMS <= 1e-2, |err| <= 3e-2 + 2^-8 |ref|.
(2) Against the two separate calls (fwd, then comp_apply): the fused kernel takes every step in
their arithmetic and order, so the outputs and the lse must be equal bit for bit."""
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


def _module_inputs(w, layout="bhnd"):
    q, k, v = workloads.structured_qkv(w, device=DEV)
    pq, pk, gate = workloads.compensation_params(w, RANK, device=DEV)
    axis, freq = workloads.rope_schedule(w.d, RANK)
    if layout == "bnhd":
        q, k, v = (t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) for t in (q, k, v))
    return q, k, v, pq, pk, gate, axis, freq


def _both(w, q, k, v, pq, pk, gate, axis, freq, idx, cnt):
    state = sa.comp_state(k, v, pk, w.grid, axis, freq, check_status=True)
    o_s, lse_s = sa.fwd(q, k, v, idx, cnt, w.block, return_lse=True, check_status=True)
    two = sa.comp_apply(q, pq, state, gate, o_s, w.grid, axis, freq, check_status=True)
    one, lse = sa.fwd_gated(q, k, v, idx, cnt, pq, state, gate, w.grid, axis, freq, return_lse=True, check_status=True)
    torch.cuda.synchronize()
    return state, o_s, lse_s, two, one, lse


@pytest.mark.parametrize("grid,H,B,sparsity,layout", [((3, 16, 24), 2, 1, 0.5, "bhnd"), ((5, 13, 17), 3, 2, 0.7, "bhnd"),
                                                     ((2, 20, 31), 2, 1, 0.0, "bnhd"), ((1, 9, 11), 1, 1, 0.5, "bhnd")])
def test_small_against_oracle_and_unfused(grid, H, B, sparsity, layout):
    w = workloads.Workload("gatedsmall", 41 + H + B, B, H, 128, tuple(grid), 128, sparsity)
    q, k, v, pq, pk, gate, axis, freq = _module_inputs(w, layout)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    state, o_s, lse_s, two, one, lse = _both(w, q, k, v, pq, pk, gate, axis, freq, idx, cnt)
    assert torch.equal(one.view(torch.int16), two.view(torch.int16))
    assert torch.equal(lse, lse_s)
    rows = [(h, i) for h in range(H) for i in range(w.N)]
    for b in range(B):
        qc, kc, vc = q[b].cpu().contiguous(), k[b].cpu().contiguous(), v[b].cpu().contiguous()
        ridx, rcnt = oracle.select(qc, kc, w.block, w.topk)
        assert torch.equal(ridx, idx[b].cpu())
        ref_os, _ = oracle.attention(qc, kc, vc, ridx, rcnt, w.block)
        ref_os = ref_os.reshape(H, w.nb * w.block, w.d)[:, : w.N]
        assert _relrms(o_s[b].cpu(), ref_os) <= 1e-2
        ref_state = oracle.comp_state(kc, vc, pk.cpu(), w.grid, axis, freq)
        ref = oracle.comp_apply(qc, pq.cpu(), ref_state, gate[b].cpu(), o_s[b].cpu().contiguous(), w.grid, axis, freq,
                                rows).reshape(H, w.N, w.d)
        _check_out(one[b].cpu(), ref)


def test_many_heads_per_cta_and_short_lists():
    """More (batch, head) pairs than a CTA sees in a row (the staged P_q / C change between items) and
    lists of one and two tiles (both warpgroups close in turn)."""
    w = workloads.Workload("gatedheads", 47, 2, 5, 128, (2, 16, 20), 128, 0.8)
    q, k, v, pq, pk, gate, axis, freq = _module_inputs(w)
    idx, cnt = sa.select(q, k, w.block, 2)
    cnt = cnt.clone()
    cnt[:, :, ::2] = 1                                        # every other query block keeps its first entry only
    _, _, lse_s, two, one, lse = _both(w, q, k, v, pq, pk, gate, axis, freq, idx, cnt)
    assert torch.equal(one.view(torch.int16), two.view(torch.int16))
    assert torch.equal(lse, lse_s)


def test_zero_gate_is_the_sparse_forward():
    w = workloads.Workload("gatedzero", 53, 1, 2, 128, (2, 12, 19), 128, 0.5)
    q, k, v, pq, pk, gate, axis, freq = _module_inputs(w)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq)
    o_s = sa.fwd(q, k, v, idx, cnt, w.block, check_status=True)
    one = sa.fwd_gated(q, k, v, idx, cnt, pq, state, torch.zeros_like(gate), w.grid, axis, freq, check_status=True)
    assert torch.equal(one.view(torch.int16), o_s.view(torch.int16))


@pytest.mark.parametrize("name,heads", [("wan1p3b", [0, 5, 11]), ("wan14b", [0, 17, 39])])
def test_fullsize_sampled(name, heads):
    """The benchmark shapes in the benchmark's launch configuration: bitwise against the two separate calls on
    the whole tensor, and against the oracle's fusion on sampled rows (first tile, ragged last tile, random)."""
    w = workloads.WORKLOADS[name]
    q, k, v, pq, pk, gate, axis, freq = _module_inputs(w)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    state, o_s, lse_s, two, one, lse = _both(w, q, k, v, pq, pk, gate, axis, freq, idx, cnt)
    assert torch.equal(one.view(torch.int16), two.view(torch.int16))
    assert torch.equal(lse, lse_s)
    g = torch.Generator().manual_seed(w.cfg_id + 7)
    tail0 = (w.N // 128) * 128 if w.N % 128 else w.N - 128
    toks = sorted(set(range(0, 128, 9)) | set(range(tail0, w.N, 3)) |
                  {int(x) for x in torch.randint(0, w.N, (96,), generator=g)})
    sub = lambda t: t[0, heads].cpu().contiguous()
    ref_state = oracle.comp_state(sub(k), sub(v), pk[heads].cpu().contiguous(), w.grid, axis, freq)
    rows = [(hi, i) for hi in range(len(heads)) for i in toks]
    ref = oracle.comp_apply(sub(q), pq[heads].cpu().contiguous(), ref_state, gate[0, heads].cpu().contiguous(), sub(o_s),
                            w.grid, axis, freq, rows).reshape(len(heads), len(toks), w.d)
    _check_out(one[0, heads][:, toks].cpu(), ref)


def test_argument_errors():
    w = workloads.Workload("gatederr", 59, 1, 1, 128, (1, 8, 32), 128, 0.5)
    q, k, v, pq, pk, gate, axis, freq = _module_inputs(w)
    idx, cnt = sa.select(q, k, w.block, w.topk)
    state = sa.comp_state(k, v, pk, w.grid, axis, freq)
    with pytest.raises(RuntimeError):                                     # grid does not multiply to N
        sa.fwd_gated(q, k, v, idx, cnt, pq, state, gate, (1, 8, 31), axis, freq)
    with pytest.raises(RuntimeError):                                     # eps must be positive
        sa.fwd_gated(q, k, v, idx, cnt, pq, state, gate, w.grid, axis, freq, eps=0.0)
    small = torch.empty(256, dtype=torch.uint8, device=DEV)
    with pytest.raises(RuntimeError):                                     # workspace too small
        sa.fwd_gated(q, k, v, idx, cnt, pq, state, gate, w.grid, axis, freq, workspace=small)
    shape64 = sa.make_shape(q, 64)
    assert sa.fwd_gated_workspace_bytes(shape64, 2, w.grid) == 0          # 64-token blocks: not offered
    assert sa.fwd_gated_workspace_bytes(sa.make_shape(q, 128), idx.shape[-1], w.grid) > 0
