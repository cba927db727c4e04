"""Pins for the compensation-branch oracle (CMP-0): an independent formulation with library
matmuls and complex rotations, closed forms and invariances."""
import math

import numpy as np
import pytest
import torch

import oracle
import workloads


def _positions(grid):
    T, Hg, Wg = grid
    n = np.arange(T * Hg * Wg)
    return np.stack([n // (Hg * Wg), (n // Wg) % Hg, n % Wg], axis=1)  # [N, 3]


def _features_numpy(x, P, grid, axis, freq):
    """x [N, d], P [r, d] float64 -> rotated features [N, r], via complex multiplication."""
    u = x @ P.T
    z = u / (1.0 + np.exp(-u))
    zc = z[:, 0::2] + 1j * z[:, 1::2]
    pos = _positions(grid)[:, axis]                      # [N, r/2]
    rot = np.exp(1j * pos * freq[None, :])
    zr = zc * rot
    out = np.empty_like(z)
    out[:, 0::2], out[:, 1::2] = zr.real, zr.imag
    return out


def _setup(H=2, d=16, r=8, grid=(2, 3, 5), seed=0):
    g = torch.Generator().manual_seed(seed)
    N = grid[0] * grid[1] * grid[2]
    mk = lambda *s: torch.randn(s, generator=g).to(torch.bfloat16)
    q, k, v, osp = mk(H, N, d), mk(H, N, d), mk(H, N, d), mk(H, N, d)
    pq, pk = (mk(H, r, d) * 0.5).to(torch.bfloat16), (mk(H, r, d) * 0.5).to(torch.bfloat16)
    gate = torch.rand((H, N), generator=g)
    axis = torch.tensor([0, 0, 1, 2][: r // 2] * (r // 8 or 1), dtype=torch.int32)[: r // 2]
    freq = torch.tensor([1.0, 0.3, 0.7, 0.11][: r // 2] * (r // 8 or 1), dtype=torch.float32)[: r // 2]
    return q, k, v, osp, pq, pk, gate, axis, freq, grid, N


def test_matches_library_formulation():
    q, k, v, osp, pq, pk, gate, axis, freq, grid, N = _setup()
    H, _, d = q.shape
    state = oracle.comp_state(k, v, pk, grid, axis, freq)
    rows = [(h, i) for h in range(H) for i in range(N)]
    out = oracle.comp_apply(q, pq, state, gate, osp, grid, axis, freq, rows, eps=1e-6).reshape(H, N, d).numpy()
    ax, fr = axis.numpy(), freq.double().numpy()
    for h in range(H):
        kt = _features_numpy(k[h].double().numpy(), pk[h].double().numpy(), grid, ax, fr)
        C = kt.T @ v[h].double().numpy()
        np.testing.assert_allclose(state[h].numpy(), C, atol=1e-11)
        qt = _features_numpy(q[h].double().numpy(), pq[h].double().numpy(), grid, ax, fr)
        y = qt @ C
        olr = y / np.sqrt((y ** 2).mean(axis=1, keepdims=True) + 1e-6)
        osn = osp[h].double().numpy()
        ref = osn + gate[h].double().numpy()[:, None] * np.sqrt((osn ** 2).mean(axis=1, keepdims=True)) * olr
        np.testing.assert_allclose(out[h], ref, atol=1e-11)


def test_zero_gate_returns_sparse_output_and_gate_is_linear():
    q, k, v, osp, pq, pk, gate, axis, freq, grid, N = _setup(seed=1)
    state = oracle.comp_state(k, v, pk, grid, axis, freq)
    rows = [(0, 3), (1, 7), (1, N - 1)]
    out0 = oracle.comp_apply(q, pq, state, torch.zeros_like(gate), osp, grid, axis, freq, rows)
    for n, (h, i) in enumerate(rows):
        np.testing.assert_array_equal(out0[n].numpy(), osp[h, i].double().numpy())
    out1 = oracle.comp_apply(q, pq, state, gate, osp, grid, axis, freq, rows)
    out2 = oracle.comp_apply(q, pq, state, 2 * gate, osp, grid, axis, freq, rows)
    np.testing.assert_allclose((out2 - out0).numpy(), 2 * (out1 - out0).numpy(), atol=1e-12)


def test_constant_value_rows_give_unit_rms_direction():
    # V = c for every token and channel: y_i = (q~_i . sum_j k~_j) c 1, so RMSNorm(y_i) = sign(.) 1 (eps = 0)
    q, k, v, osp, pq, pk, gate, axis, freq, grid, N = _setup(seed=2)
    vc = torch.full_like(v, 0.75)
    state = oracle.comp_state(k, vc, pk, grid, axis, freq)
    rows = [(0, i) for i in range(N)]
    out = oracle.comp_apply(q, pq, state, gate, osp, grid, axis, freq, rows, eps=0.0).numpy()
    osn = osp[0].double().numpy()
    delta = out - osn
    ri = np.sqrt((osn ** 2).mean(axis=1))
    expect = gate[0].double().numpy() * ri
    np.testing.assert_allclose(np.abs(delta), np.tile(expect[:, None], (1, osn.shape[1])), atol=1e-12)
    assert np.all(np.abs(np.sign(delta).sum(axis=1)) == osn.shape[1])      # one sign per row
    # scaling V by a positive factor changes nothing (RMSNorm, eps = 0)
    state2 = oracle.comp_state(k, (2 * v.float()).to(torch.bfloat16), pk, grid, axis, freq)
    state1 = oracle.comp_state(k, v, pk, grid, axis, freq)
    a = oracle.comp_apply(q, pq, state1, gate, osp, grid, axis, freq, rows[:5], eps=0.0)
    b = oracle.comp_apply(q, pq, state2, gate, osp, grid, axis, freq, rows[:5], eps=0.0)
    np.testing.assert_allclose(a.numpy(), b.numpy(), atol=1e-12)


def test_rotation_is_the_stated_one():
    # one head, P selects channels 0..3 (u = x[0:4]); freq pi/2 on axis t for pair 0, 0 for pair 1.
    d, r, grid = 4, 4, (2, 1, 1)
    P = torch.eye(4).to(torch.bfloat16)[None]
    axis = torch.tensor([0, 1], dtype=torch.int32)
    freq = torch.tensor([math.pi / 2, 0.0])
    k = torch.tensor([[[8.0, 16.0, 8.0, 16.0], [8.0, 16.0, 8.0, 16.0]]]).to(torch.bfloat16)   # silu(8) ~ 8, silu(16) ~ 16
    v = torch.zeros((1, 2, d), dtype=torch.bfloat16)
    v[0, 0, 0] = 1.0      # token 0 (t = 0) writes its feature into column 0
    v[0, 1, 1] = 1.0      # token 1 (t = 1) writes its rotated feature into column 1
    st = oracle.comp_state(k, v, P, grid, axis, freq)[0].numpy()
    s8, s16 = 8 / (1 + math.exp(-8)), 16 / (1 + math.exp(-16))
    np.testing.assert_allclose(st[:, 0], [s8, s16, s8, s16], atol=1e-12)        # t = 0: no rotation
    # t = 1, pair 0 turned by 90 degrees: (z0, z1) -> (-z1, z0); pair 1 (freq 0) unchanged
    np.testing.assert_allclose(st[:, 1], [-s16, s8, s8, s16], atol=2e-7)        # fp32 pi/2
    # the rotation preserves the norm of the feature
    q, kk, vv, osp, pq, pk, gate, ax, fr, g, N = _setup(seed=3)
    ident = oracle.comp_state(kk, vv, pk, g, ax, torch.zeros_like(fr))
    rot = oracle.comp_state(kk, vv, pk, g, ax, fr)
    assert not np.allclose(ident.numpy(), rot.numpy())


def test_relative_position_property():
    # q~_i . k~_j depends on positions only through their difference: rolling the whole sequence
    # by one frame (t -> t + 1 for queries and keys alike) leaves y unchanged for the frames that stay inside.
    H, d, r, grid = 1, 8, 4, (3, 2, 2)
    g = torch.Generator().manual_seed(5)
    N = 12
    frame = 4
    mk = lambda *s: torch.randn(s, generator=g).to(torch.bfloat16)
    q1, k1, v1 = mk(1, frame, d), mk(1, frame, d), mk(1, frame, d)
    pq, pk = mk(1, r, d), mk(1, r, d)
    axis = torch.tensor([0, 0], dtype=torch.int32)
    freq = torch.tensor([0.9, 0.2])
    zeros = torch.zeros((1, frame, d), dtype=torch.bfloat16)
    osp = torch.ones((1, N, d), dtype=torch.bfloat16)
    gate = torch.ones((1, N))
    outs = []
    for f in (0, 1):   # put the same content in frame f, zeros elsewhere (zero k rows give zero features)
        parts_q = [zeros] * 3; parts_k = [zeros] * 3; parts_v = [zeros] * 3
        parts_q[f], parts_k[f], parts_v[f] = q1, k1, v1
        qf, kf, vf = torch.cat(parts_q, 1), torch.cat(parts_k, 1), torch.cat(parts_v, 1)
        st = oracle.comp_state(kf, vf, pk, grid, axis, freq)
        rows = [(0, f * frame + i) for i in range(frame)]
        outs.append(oracle.comp_apply(qf, pq, st, gate, osp, grid, axis, freq, rows, eps=0.0).numpy())
    np.testing.assert_allclose(outs[0], outs[1], atol=1e-12)


def test_rope_schedule_generator():
    axis, freq = workloads.rope_schedule(128, 64)
    assert axis.tolist() == [0] * 22 + [1] * 10 and len(freq) == 32
    assert freq[0] == 1.0 and freq[22] == 1.0 and torch.all(freq[:22][1:] < freq[:22][:-1])
