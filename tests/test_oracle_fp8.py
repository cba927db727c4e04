"""Pins for the FP8 oracle (QNT-1): the format's defining constants, a
brute-force nearest-value search over the decode table, every rounding
midpoint, saturation / underflow / signed zero, and a library cast."""
import math
import os

import numpy as np
import torch

import oracle


def _table():
    return np.array([oracle.e4m3_decode(c) for c in range(256)])


def test_decode_matches_format_constants():
    path = os.path.join(os.path.dirname(__file__), "golden", "e4m3_format_points.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        code, val = line.split()
        assert oracle.e4m3_decode(int(code, 16)) == float(val)
    t = _table()
    assert math.isnan(t[0x7F]) and math.isnan(t[0xFF])
    pos = t[:0x7F]
    assert np.all(np.diff(pos) > 0)            # strictly increasing in the code
    assert np.array_equal(t[0x80:0xFF], -pos)  # sign bit mirrors
    assert math.copysign(1.0, t[0x80]) == -1.0  # negative zero
    # decode agrees with a library table
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
    ok = ~np.isnan(lib)
    assert np.array_equal(lib[ok], t[ok]) and ok.sum() == 254


def test_encode_inverts_decode():
    t = _table()
    for c in range(256):
        if (c & 0x7F) == 0x7F:
            continue
        assert oracle.e4m3_encode(float(t[c])) == c


def _nearest_bruteforce(y: float) -> int:
    """Nearest finite code by exhaustive search; ties -> even mantissa bit; sign kept."""
    t = _table()
    sign = 0x80 if math.copysign(1.0, y) < 0 else 0
    a = abs(y)
    best, bestd = None, None
    for c in range(0x7F):
        dist = abs(t[c] - a)
        if best is None or dist < bestd or (dist == bestd and (c & 1) == 0):
            best, bestd = c, dist
    return sign | best


def test_encode_matches_bruteforce_search():
    rng = np.random.default_rng(1)
    ys = np.concatenate([
        rng.standard_normal(20000) * 100.0,
        rng.standard_normal(20000),
        rng.standard_normal(10000) * 0.01,
        rng.uniform(-450, 450, 10000),
    ]).astype(np.float32)
    ys = ys[np.abs(ys) <= 448.0]
    codes = oracle.e4m3_encode_array(ys)
    t = _table()
    # vectorised brute force with the same tie rule
    a = np.abs(ys.astype(np.float64))[:, None]
    dist = np.abs(t[None, :0x7F] - a)
    dmin = dist.min(axis=1, keepdims=True)
    cand = dist == dmin
    even = (np.arange(0x7F) % 2 == 0)[None, :]
    pick = np.where((cand & even).any(axis=1), (cand & even).argmax(axis=1), cand.argmax(axis=1))
    expect = pick.astype(np.uint8) | (np.signbit(ys).astype(np.uint8) << 7)
    assert np.array_equal(codes, expect)
    for y in ys[:300]:
        assert oracle.e4m3_encode(float(y)) == _nearest_bruteforce(float(y))


def test_every_midpoint_rounds_to_even_and_neighbours_round_to_nearest():
    t = _table()
    for c in range(0x7E):
        lo, hi = t[c], t[c + 1]
        mid = np.float32((lo + hi) / 2)
        assert float(mid) == (lo + hi) / 2  # midpoints are exact in fp32
        even = c if c % 2 == 0 else c + 1
        assert oracle.e4m3_encode(float(mid)) == even
        assert oracle.e4m3_encode(float(np.nextafter(mid, np.float32(0)))) == c
        assert oracle.e4m3_encode(float(np.nextafter(mid, np.float32(1e9)))) == c + 1
        assert oracle.e4m3_encode(-float(mid)) == (0x80 | even)


def test_saturation_underflow_signed_zero():
    assert oracle.e4m3_encode(449.0) == 0x7E
    assert oracle.e4m3_encode(464.0) == 0x7E
    assert oracle.e4m3_encode(1e9) == 0x7E
    assert oracle.e4m3_encode(-1e9) == 0xFE
    assert oracle.e4m3_encode(float("inf")) == 0x7E
    assert oracle.e4m3_encode(2.0 ** -10) == 0x00          # tie between 0 and 2^-9 -> even (0)
    assert oracle.e4m3_encode(float(np.nextafter(np.float32(2.0 ** -10), np.float32(1)))) == 0x01
    assert oracle.e4m3_encode(-(2.0 ** -10)) == 0x80
    assert oracle.e4m3_encode(0.0) == 0x00
    assert oracle.e4m3_encode(-0.0) == 0x80
    assert oracle.e4m3_encode(1e-30) == 0x00 and oracle.e4m3_encode(-1e-30) == 0x80
    assert oracle.e4m3_encode(2.0 ** -6) == 0x08
    assert oracle.e4m3_encode(float(np.float32(2.0 ** -6) * np.float32(1 - 2 ** -5))) == 0x08  # 7.75 * 2^-9 rounds up


def test_encode_matches_library_cast_in_range():
    g = torch.Generator().manual_seed(3)
    y = torch.cat([torch.randn(50000, generator=g) * s for s in (0.01, 1.0, 50.0, 150.0)])
    y = y[y.abs() <= 448.0]
    lib = y.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    mine = oracle.e4m3_encode_array(y.numpy())
    assert np.array_equal(lib, mine)


def test_block_quant_scales_and_codes():
    H, N, d, block = 2, 150, 16, 64   # tail block has 22 tokens
    g = torch.Generator().manual_seed(5)
    x = (torch.randn((H, N, d), generator=g) * 3).to(torch.bfloat16)
    x[1, 64:128] = 0                   # an all-zero block
    x[0, 3, 2] = -7.0                  # absmax element of block (0,0), negative
    x[0, :64].clamp_(-7, 7)
    codes, scales = oracle.quant_fp8(x, block)
    t = _table()
    nb = 3
    for h in range(H):
        for b in range(nb):
            blk = x[h, b * block:min(N, (b + 1) * block)].float()
            amax = max(float(blk.abs().max()), 1e-12)
            amax32 = np.float32(amax) if amax > 1e-12 else np.float32(1e-12)
            assert scales[h, b].item() == float(amax32 / np.float32(448.0))
            inv = np.float32(448.0) / amax32
            y = blk.numpy() * inv
            # library cast as the independent encoder (|y| <= 448 by construction)
            ref = torch.from_numpy(np.clip(y, -448, 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            got = codes[h, b * block:min(N, (b + 1) * block)].numpy()
            assert np.array_equal(ref, got)
    assert codes[0, 3, 2].item() == 0xFE                      # the absmax element maps to -448 exactly
    assert scales[1, 1].item() == float(np.float32(1e-12) / np.float32(448.0))
    assert set(np.unique(codes[1, 64:128].numpy()).tolist()) <= {0x00, 0x80}
    # dequantised values stay within half an e4m3 step of the input
    deq = torch.from_numpy(t[codes.long().numpy()]) * scales.double().repeat_interleave(block, 1)[:, :N, None]
    err = (deq - x.double()).abs()
    bound = scales.double().repeat_interleave(block, 1)[:, :N, None] * 16.0 + 1e-30  # half of the largest step (32)
    assert torch.all(err <= bound)


def test_per_token_quant_scales_and_codes():
    H, N, d = 2, 37, 32
    g = torch.Generator().manual_seed(8)
    x = (torch.randn((H, N, d), generator=g) * torch.logspace(-3, 2, N)[None, :, None]).to(torch.bfloat16)
    x[1, 5] = 0                         # an all-zero token
    x[0, 7, 3] = -9.0; x[0, 7].clamp_(-9, 9)
    codes, scales = oracle.quant_fp8_per_token(x)
    for h in range(H):
        for n in range(N):
            row = x[h, n].float().numpy()
            amax = np.float32(max(float(np.abs(row).max()), 1e-12))
            assert scales[h, n].item() == float(amax / np.float32(448.0))
            y = row * (np.float32(448.0) / amax)
            ref = torch.from_numpy(np.clip(y, -448, 448)).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
            assert np.array_equal(ref, codes[h, n].numpy())
    assert codes[0, 7, 3].item() == 0xFE
    assert set(np.unique(codes[1, 5].numpy()).tolist()) <= {0x00, 0x80}
    # a block of one token reproduces the block-wise routine
    c1, s1 = oracle.quant_fp8(x[:, :1].contiguous(), 64)
    assert torch.equal(c1, codes[:, :1]) and torch.equal(s1[:, 0], scales[:, 0])
