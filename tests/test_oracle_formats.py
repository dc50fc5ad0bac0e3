"""Pins for the oracle's element formats, encoder and block scale (no GPU).

Each check compares the oracle with something other than itself: the closed-form grids of the
OCP element formats, PyTorch's float8 casts (a library), explicit rounding thresholds, and the
closed form 2^(floor(log2 amax) - emax) of the E8M0 block scale.
"""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from oracle import E2M1, E2M3, E3M2, E4M3, E5M2

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FMT = {"E4M3": E4M3, "E5M2": E5M2, "E2M1": E2M1, "E3M2": E3M2, "E2M3": E2M3}


def test_e2m1_decode_grid():
    grid = [0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0]
    for c in range(8):
        assert oracle.decode_elem(E2M1, c) == grid[c]
        assert oracle.decode_elem(E2M1, c | 8) == -grid[c]
    assert math.copysign(1.0, oracle.decode_elem(E2M1, 8)) == -1.0  # 0x8 is -0


def test_fp6_decode_grids():
    """The 6-bit element formats of the OCP MX definition (the activations of MicroQonv+ and the "-6" variant,
    Sec. V), written out as explicit value grids: E3M2 bias 3 (subnormal step 2^-4, largest 28), E2M3 bias 1
    (subnormal step 2^-3, largest 7.5); no infinities or NaNs; the sign is bit 5."""
    e3m2 = [0.0, 0.0625, 0.125, 0.1875] + [(1 + m / 4) * 2.0 ** (e - 3) for e in range(1, 8) for m in range(4)]
    e2m3 = [k * 0.125 for k in range(8)] + [(1 + m / 8) * 2.0 ** (e - 1) for e in range(1, 4) for m in range(8)]
    assert len(e3m2) == 32 and len(e2m3) == 32
    assert e3m2[4] == 0.25 and e3m2[31] == 28.0 and e3m2[1] == 2.0 ** -4     # smallest normal, largest, smallest subnormal
    assert e2m3[8] == 1.0 and e2m3[31] == 7.5 and e2m3[1] == 2.0 ** -3
    for fmt, grid in ((E3M2, e3m2), (E2M3, e2m3)):
        for c in range(32):
            assert oracle.decode_elem(fmt, c) == grid[c], (fmt, c)
            assert oracle.decode_elem(fmt, c | 32) == -grid[c]
        assert math.copysign(1.0, oracle.decode_elem(fmt, 32)) == -1.0
        assert all(math.isfinite(oracle.decode_elem(fmt, c)) for c in range(64))


def test_fp6_encode_explicit_cases():
    # ties go to the code with an even low bit; magnitudes beyond the largest value saturate
    cases = {
        E2M3: [(1.0, 0x08), (1.0625, 0x08), (1.07, 0x09), (1.1875, 0x0A), (7.5, 0x1F), (7.75, 0x1F), (1e9, 0x1F), (0.0625, 0x00), (0.07, 0x01),
               (0.1875, 0x02), (3.75, 0x17), (3.875, 0x18)],
        E3M2: [(0.25, 0x04), (0.03125, 0x00), (0.04, 0x01), (0.09375, 0x02), (24.0, 0x1E), (26.0, 0x1E), (26.1, 0x1F), (28.0, 0x1F), (40.0, 0x1F),
               (1.125, 0x0C), (1.126, 0x0D), (1.375, 0x0E)],
    }
    for fmt, rows in cases.items():
        for v, code in rows:
            assert oracle.encode_elem(fmt, v) == code, (fmt, v)
            assert oracle.encode_elem(fmt, -v) == code | 32, (fmt, v)


@pytest.mark.parametrize("fmt,tdtype", [(E4M3, torch.float8_e4m3fn), (E5M2, torch.float8_e5m2)])
def test_fp8_decode_matches_library_view(fmt, tdtype):
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(tdtype).to(torch.float64).numpy()
    for c in range(256):
        v = oracle.decode_elem(fmt, c)
        if math.isnan(lib[c]):
            assert math.isnan(v)
        else:
            assert v == lib[c], (c, v, lib[c])


def test_fp8_landmarks():
    assert oracle.decode_elem(E4M3, 0x7E) == 448.0
    assert oracle.decode_elem(E4M3, 0x01) == 2.0 ** -9
    assert oracle.decode_elem(E4M3, 0x08) == 2.0 ** -6
    assert oracle.decode_elem(E5M2, 0x7B) == 57344.0
    assert oracle.decode_elem(E5M2, 0x01) == 2.0 ** -16
    assert oracle.decode_elem(E5M2, 0x04) == 2.0 ** -14
    assert math.isinf(oracle.decode_elem(E5M2, 0x7C))


@pytest.mark.parametrize("fmt,ncodes,maxc", [(E2M1, 16, 0x7), (E4M3, 256, 0x7E), (E5M2, 256, 0x7B), (E3M2, 64, 0x1F), (E2M3, 64, 0x1F)])
def test_encode_roundtrip_midpoints_saturation(fmt, ncodes, maxc):
    half = ncodes // 2
    for m in range(maxc + 1):
        for s in (0, half):
            assert oracle.encode_elem(fmt, oracle.decode_elem(fmt, m | s)) == (m | s)
    for m in range(maxc):
        lo, hi = oracle.decode_elem(fmt, m), oracle.decode_elem(fmt, m + 1)
        assert hi > lo  # monotone in code
        mid = (lo + hi) / 2
        even = m if m % 2 == 0 else m + 1
        assert oracle.encode_elem(fmt, mid) == even
        assert oracle.encode_elem(fmt, -mid) == (even | half)
        assert oracle.encode_elem(fmt, np.nextafter(mid, 0.0)) == m
        assert oracle.encode_elem(fmt, np.nextafter(mid, np.inf)) == m + 1
    top = oracle.decode_elem(fmt, maxc)
    for v in (top * 1.0001, top * 1.2, top * 2, 1e30):
        assert oracle.encode_elem(fmt, v) == maxc
        assert oracle.encode_elem(fmt, -v) == (maxc | half)
    assert oracle.encode_elem(fmt, 0.0) == 0
    assert oracle.encode_elem(fmt, -0.0) == half
    assert oracle.encode_elem(fmt, -1e-30) == half  # negative underflow keeps the sign


def test_e2m1_encode_explicit_thresholds():
    # (upper bound, inclusive?) -> code ; ties go to the code with an even low bit
    cases = [(0.2, 0), (0.25, 0), (0.26, 1), (0.74, 1), (0.75, 2), (1.2, 2), (1.25, 2), (1.3, 3), (1.74, 3),
             (1.75, 4), (2.4, 4), (2.5, 4), (2.6, 5), (3.4, 5), (3.5, 6), (4.9, 6), (5.0, 6), (5.1, 7), (100.0, 7)]
    for v, code in cases:
        assert oracle.encode_elem(E2M1, v) == code, v
        assert oracle.encode_elem(E2M1, -v) == code | 8, v


@pytest.mark.parametrize("fmt,tdtype,top", [(E4M3, torch.float8_e4m3fn, 448.0), (E5M2, torch.float8_e5m2, 57344.0)])
def test_fp8_encode_matches_library_cast(fmt, tdtype, top):
    rng = np.random.default_rng(7)
    v = np.concatenate([
        rng.standard_normal(4000) * rng.choice([1e-4, 1e-2, 1.0, 30.0, 400.0, 5e4], 4000),
        np.ldexp(rng.uniform(1, 2, 2000), rng.integers(-20, 17, 2000)) * rng.choice([-1, 1], 2000),
        [0.0, -0.0, top, -top, top * 1.5, -top * 3],
    ]).astype(np.float32)
    lib = torch.from_numpy(v).clamp(-top, top).to(tdtype).view(torch.uint8).numpy()
    for x, c in zip(v, lib):
        assert oracle.encode_elem(fmt, float(x)) == int(c), (x, c)


@pytest.mark.parametrize("fmt,emax", [(E2M1, 2), (E4M3, 8), (E5M2, 15), (E3M2, 4), (E2M3, 2)])
def test_scale_closed_form(fmt, emax):
    assert oracle.scale_code(fmt, 0.0) == 0
    for k in range(-140, 128):
        for amax in (2.0 ** k, 2.0 ** k * (1 + 2.0 ** -23), 2.0 ** k * (2 - 2.0 ** -22), 2.0 ** k * 1.5):
            want = min(max(k - emax + 127, 0), 254)
            assert oracle.scale_code(fmt, amax) == want, (k, amax)
    # the same through an independent route: integer exponent field of the fp32 encoding
    rng = np.random.default_rng(3)
    a = np.abs(rng.standard_normal(2000) * rng.choice([1e-30, 1e-6, 1.0, 1e5, 1e30], 2000)).astype(np.float32)
    a = a[a >= np.finfo(np.float32).tiny]
    expo = ((a.view(np.uint32) >> 23) & 0xFF).astype(np.int64)
    for x, e in zip(a, expo):
        assert oracle.scale_code(fmt, float(x)) == min(max(int(e) - emax, 0), 254)


def _golden_rows():
    rows = []
    with open(os.path.join(GOLD, "mx_block_vectors.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            fmt, vals, scale, codes, deq = [t.strip() for t in line.split(";")]
            rows.append((fmt, [float(t) for t in vals.split()], int(scale), [int(t, 16) for t in codes.split()],
                         [float(t) for t in deq.split()]))
    return rows


@pytest.mark.parametrize("row", _golden_rows(), ids=lambda r: f"{r[0]}-{r[1][0]}")
@pytest.mark.parametrize("block", [(1, 32), (32, 32)])
def test_hand_derived_block_vectors(row, block):
    fname, vals, scale, codes, deq = row
    fmt = FMT[fname]
    d = oracle.ConvDesc(1, 32, 1, 1, 32, 1, 1, 1, 1, 0, 0)
    x = np.zeros((1, 32, 1, 1), np.float32)
    x[0, : len(vals), 0, 0] = vals
    c, s = oracle.quantize(d, oracle.ROLE_X, fmt, x, block)
    assert s.tolist() == [scale]
    if fmt == E2M1:
        got = [(c[i // 2] >> (4 * (i % 2))) & 0xF for i in range(len(vals))]
        assert not c[2:].any()
    else:
        got = c[: len(vals)].tolist()
        assert not c[len(vals):].any()
    assert got == codes
    back = oracle.dequant(d, oracle.ROLE_X, fmt, c, s, block)[0, : len(vals), 0, 0]
    np.testing.assert_allclose(back, deq, rtol=1e-11, atol=0)


def test_paper_format_arithmetic():
    gold = {}
    with open(os.path.join(GOLD, "paper_format_arithmetic.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v, _ = [t.strip() for t in line.split(";", 2)]
                gold[k] = float(v)
    d = oracle.ConvDesc(32, 64, 16, 16, 64, 3, 3, 1, 1, 1, 1)
    fp32_bytes = 32 * 64 * 16 * 16 * 4
    cb, sb = oracle.qtensor_sizes(d, oracle.ROLE_X, E2M1, (1, 32))  # 4-bit + one 8-bit scale per 32
    assert round(fp32_bytes / (cb + sb), 2) == gold["backward_mem_move_fp32_over_4bit"]
    cb, sb = oracle.qtensor_sizes(d, oracle.ROLE_X, E2M1, (8, 8))  # the paper's 8x8 block
    elems = 32 * 64 * 16 * 16
    assert (cb * 8 - elems) / elems + sb * 8 / elems == gold["bits_per_unsigned_fp4_pixel_B64"]  # 3 + 8/64
    cb8, sb8 = oracle.qtensor_sizes(d, oracle.ROLE_X, E4M3, (8, 8))
    assert abs(fp32_bytes / (cb8 + sb8) - gold["fp8_gain_over_fp32_B64"]) < 0.01
    # storing the quantized im2col-expanded tensor instead costs Kh*Kw times more (stride 1, same-size output)
    icb, isb = oracle.im2col_sizes(d, E2M1, (8, 8))
    assert icb / cb == gold["act_quantizations_im2col_k3"] and isb / sb == gold["act_quantizations_im2col_k3"]


def test_packed_6bit_storage_layout():
    """pack6: code k of the array in bits 6k .. 6k+5 of one little-endian bit stream (16 codes in 12 bytes).  Checked against
    the same definition written with Python's unbounded integers, on explicit vectors and on random codes, and inverted by
    unpack6."""
    assert oracle.pack6(np.array([1, 0, 0, 0], dtype=np.uint8)).tolist() == [0x01, 0x00, 0x00]
    assert oracle.pack6(np.array([0, 1, 0, 0], dtype=np.uint8)).tolist() == [0x40, 0x00, 0x00]      # bit 6
    assert oracle.pack6(np.array([0, 0, 1, 0], dtype=np.uint8)).tolist() == [0x00, 0x10, 0x00]      # bit 12
    assert oracle.pack6(np.array([0, 0, 0, 63], dtype=np.uint8)).tolist() == [0x00, 0x00, 0xFC]     # bits 18 .. 23
    assert oracle.pack6(np.array([63, 63, 63, 63], dtype=np.uint8)).tolist() == [0xFF, 0xFF, 0xFF]
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 64, size=16 * 37, dtype=np.uint8)
    stream = 0
    for k, c in enumerate(codes.tolist()):
        stream |= c << (6 * k)
    want = np.frombuffer(stream.to_bytes(codes.size * 3 // 4, "little"), dtype=np.uint8)
    got = oracle.pack6(codes)
    assert got.size == codes.size * 3 // 4 and np.array_equal(got, want)
    assert np.array_equal(oracle.unpack6(got), codes)
    # a group of 16 codes is a 12-byte field of its own: packing commutes with any regrouping by 16
    perm = rng.permutation(37)
    assert np.array_equal(oracle.pack6(codes.reshape(37, 16)[perm]), got.reshape(37, 12)[perm].reshape(-1))
