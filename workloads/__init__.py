"""Seeded synthetic inputs for the block-sparse attention path.

This module only *draws inputs* (random tensors, a random block mask, the
integer kept-block budget for a sparsity level).  It holds none of the
method's arithmetic: no pooling, no scores, no softmax, no FP8 encode.  Both
the CPU oracle's tests and the CUDA path's tests/bench import it so that the
two sides always see the very same arrays.

Workload shapes
---------------
``tiny``        B=1 H=2  d=64  N=2048  (grid 2x32x32),  64x64 blocks, random 50 % mask
``wan1p3b``     B=1 H=12 d=128 N=32760 (grid 21x30x52), 128x128 blocks, 90 % sparsity
``wan14b``      B=1 H=40 d=128 N=75600 (grid 21x45x80), 128x128 blocks, 97 % sparsity

The two Wan shapes stand in for the self-attention activations of the video
DiT the paper evaluates (480x832 and 720x1280, 81 frames); those activations
need the trained model and are not available, so Q/K are a smooth
low-frequency field over the (t, y, x) latent grid plus white noise, which
gives the "few high-energy blocks over a flat background" structure that
makes block selection meaningful.  V is white noise.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Sequence, Tuple

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    cfg_id: int
    B: int
    H: int
    d: int
    grid: Tuple[int, int, int]  # (T, Hg, Wg), raster token order n = (t*Hg + y)*Wg + x
    block: int
    sparsity: float  # fraction of key blocks skipped per query block

    @property
    def N(self) -> int:
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def nb(self) -> int:
        return (self.N + self.block - 1) // self.block

    @property
    def tail(self) -> int:
        return self.N - (self.nb - 1) * self.block

    @property
    def topk(self) -> int:
        return kept_blocks_for_sparsity(self.sparsity, self.nb)

    def with_sparsity(self, s: float) -> "Workload":
        return replace(self, sparsity=s)

    def with_heads(self, H: int) -> "Workload":
        return replace(self, H=H)


TINY = Workload("tiny", 1, 1, 2, 64, (2, 32, 32), 64, 0.5)
WAN_1P3B_480P = Workload("wan1p3b", 2, 1, 12, 128, (21, 30, 52), 128, 0.90)
WAN_14B_720P = Workload("wan14b", 3, 1, 40, 128, (21, 45, 80), 128, 0.97)

WORKLOADS = {w.name: w for w in (TINY, WAN_1P3B_480P, WAN_14B_720P)}


def kept_blocks_for_sparsity(sparsity: float, nb: int) -> int:
    """Integer number of key blocks kept per query block for a block sparsity
    level: the nearest integer to (1 - s) * nb, at least one block."""
    return max(1, int(math.floor((1.0 - sparsity) * nb + 0.5)))


def tiny_inputs(w: Workload = TINY, seed: int = 0):
    """Q, K, V ~ N(0,1) iid drawn in fp32 in that order from one CPU
    generator, rounded to bf16.  Shapes [B, H, N, d]."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    shape = (w.B, w.H, w.N, w.d)
    q = torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    k = torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn(shape, generator=g, dtype=torch.float32).to(torch.bfloat16)
    return q, k, v


def random_block_mask(B: int, H: int, nb: int, keep: int, seed_base: int = 1000):
    """Random kept-block lists that always keep the diagonal block.

    For each (b, h, qb) the list is block ``qb`` plus ``keep - 1`` of the other
    blocks, taken from a permutation seeded with
    ``seed_base + (b*H + h)*nb + qb``, stored ascending.
    Returns (kept_idx int32 [B,H,nb,keep], kept_cnt int32 [B,H,nb])."""
    assert 1 <= keep <= nb
    idx = torch.empty((B, H, nb, keep), dtype=torch.int32)
    for b in range(B):
        for h in range(H):
            for qb in range(nb):
                g = torch.Generator(device="cpu")
                g.manual_seed(seed_base + (b * H + h) * nb + qb)
                others = torch.tensor([j for j in range(nb) if j != qb], dtype=torch.int64)
                perm = torch.randperm(nb - 1, generator=g)[: keep - 1]
                sel = torch.cat([others[perm], torch.tensor([qb])])
                idx[b, h, qb] = torch.sort(sel).values.to(torch.int32)
    cnt = torch.full((B, H, nb), keep, dtype=torch.int32)
    return idx, cnt


def _grid_coords(grid, device):
    T, Hg, Wg = grid
    n = torch.arange(T * Hg * Wg, device=device, dtype=torch.int64)
    x = n % Wg
    y = (n // Wg) % Hg
    t = n // (Wg * Hg)
    return t.double() / T, y.double() / Hg, x.double() / Wg


def structured_qkv(
    w: Workload,
    heads: Optional[Sequence[int]] = None,
    device: str = "cpu",
    noise: float = 0.5,
):
    """Q/K = smooth 3-D field (8 seeded sinusoids over t, y, x, amplitude 1/2
    each, shared between Q and K up to a small per-channel phase jitter on K)
    + ``noise`` * N(0,1); V ~ N(0,1).  Returns bf16 [B, len(heads), N, d].

    Per head h the generator seed is ``cfg_id * 100003 + b * 1009 + h``.  Four
    of the eight sinusoids have no x-frequency so that their energy survives
    pooling over a raster block (which spans at least one full grid row)."""
    heads = list(range(w.H)) if heads is None else list(heads)
    N, d = w.N, w.d
    tt, yy, xx = _grid_coords(w.grid, device)
    q = torch.empty((w.B, len(heads), N, d), dtype=torch.bfloat16, device=device)
    k = torch.empty_like(q)
    v = torch.empty_like(q)
    for b in range(w.B):
        for hi, h in enumerate(heads):
            seed = w.cfg_id * 100003 + b * 1009 + h
            gc = torch.Generator(device="cpu")
            gc.manual_seed(seed)
            M = 8
            ft = torch.randint(0, 3, (M,), generator=gc)
            fy = torch.randint(0, 4, (M,), generator=gc)
            fx = torch.randint(0, 4, (M,), generator=gc)
            fx[:4] = 0
            for m in range(M):  # no constant component
                if ft[m] == 0 and fy[m] == 0 and fx[m] == 0:
                    fy[m] = 1 + (m % 3)
            phi = torch.rand((M, d), generator=gc, dtype=torch.float64) * (2 * math.pi)
            delta = (torch.rand((M, d), generator=gc, dtype=torch.float64) - 0.5) * (math.pi / 2)
            ft, fy, fx = ft.to(device).double(), fy.to(device).double(), fx.to(device).double()
            theta = 2 * math.pi * (tt[:, None] * ft[None] + yy[:, None] * fy[None] + xx[:, None] * fx[None])
            sc = torch.cat([torch.sin(theta), torch.cos(theta)], dim=1).float()  # [N, 2M]
            phq = phi.to(device)
            phk = (phi + delta).to(device)
            wq = 0.5 * torch.cat([torch.cos(phq), torch.sin(phq)], dim=0).float()  # [2M, d]
            wk = 0.5 * torch.cat([torch.cos(phk), torch.sin(phk)], dim=0).float()
            gd = torch.Generator(device=device)
            gd.manual_seed(seed)
            eq = torch.randn((N, d), generator=gd, device=device, dtype=torch.float32)
            ek = torch.randn((N, d), generator=gd, device=device, dtype=torch.float32)
            ev = torch.randn((N, d), generator=gd, device=device, dtype=torch.float32)
            q[b, hi] = (sc @ wq + noise * eq).to(torch.bfloat16)
            k[b, hi] = (sc @ wk + noise * ek).to(torch.bfloat16)
            v[b, hi] = ev.to(torch.bfloat16)
    return q, k, v


def small_structured(H: int, d: int, grid, block: int, sparsity: float, cfg_id: int = 7) -> Workload:
    """A reduced workload of the same recipe, for cases the oracle finishes in seconds."""
    return Workload(f"small{cfg_id}", cfg_id, 1, H, d, tuple(grid), block, sparsity)


def shard_heads(H: int, world_size: int, rank: int) -> range:
    """Contiguous slice of heads owned by ``rank`` when H heads are split over
    ``world_size`` processes (no data-path exchange: heads are independent).
    The first ``H % world_size`` ranks take one extra head."""
    base, extra = divmod(H, world_size)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def rope_schedule(d: int, rank: int, theta: float = 10000.0):
    """Rank-truncated 3-D rotary schedule: the d/2 rotary pairs of a head are split over the axes
    (t, y, x) as (d/2 - 2*(d/6), d/6, d/6) pairs (22 / 21 / 21 for d = 128, the split video DiTs of
    this family use), pair p of an axis with n_a pairs has frequency theta^(-p / n_a); the
    compensation branch keeps the first rank/2 pairs.  Returns (axis int32 [rank/2], freq fp32 [rank/2])."""
    half = d // 2
    n_y = n_x = d // 6
    n_t = half - n_y - n_x
    axis, freq = [], []
    for a, n_a in enumerate((n_t, n_y, n_x)):
        for pidx in range(n_a):
            axis.append(a)
            freq.append(theta ** (-pidx / n_a))
    axis = torch.tensor(axis[: rank // 2], dtype=torch.int32)
    freq = torch.tensor(freq[: rank // 2], dtype=torch.float32)
    return axis, freq


def compensation_params(w: Workload, rank: int = 64, heads: Optional[Sequence[int]] = None, device: str = "cpu",
                        gate_scale: float = 0.3):
    """Seeded stand-ins for the trained parts of the compensation branch: low-rank projections
    P_q, P_k ~ N(0, 1/d) (bf16 [H, rank, d]) and a token-wise gate g ~ U(0, gate_scale) (fp32
    [B, H, N]; the trained gate starts near zero, a visible one is used so that the branch matters
    in parity tests)."""
    heads = list(range(w.H)) if heads is None else list(heads)
    g = torch.Generator(device="cpu")
    g.manual_seed(w.cfg_id * 7919 + 13)
    pq = (torch.randn((w.H, rank, w.d), generator=g) / math.sqrt(w.d)).to(torch.bfloat16)[heads]
    pk = (torch.randn((w.H, rank, w.d), generator=g) / math.sqrt(w.d)).to(torch.bfloat16)[heads]
    gd = torch.Generator(device=device)
    gd.manual_seed(w.cfg_id * 7919 + 14)
    gate = torch.rand((w.B, len(heads), w.N), generator=gd, device=device, dtype=torch.float32) * gate_scale
    return pq.to(device), pk.to(device), gate
