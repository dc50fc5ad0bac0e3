"""Pins of the oracle's implementation of the paper's own number format (Sec. III-A, Eq. 4-6: fp32 scale per tensor,
E4M3 scale per block, E2M1 elements) - no GPU.  Hand-derived vectors, closed forms, a second derivation through library
casts, invariants and error bounds, chosen so that a dropped factor (the 6 of Eq. 5, the T_scale of Eq. 6), a wrong rounding
or a wrong block / scale index fails at least one of them."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "ts_block_vectors.txt")
E2M1_GRID = np.array([0, 0.5, 1, 1.5, 2, 3, 4, 6])


def unpack(codes):
    out = np.empty(codes.size * 2, dtype=np.uint8)
    out[0::2], out[1::2] = codes & 0xF, codes >> 4
    return out


def golden_blocks():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        vals, sc, bs, codes = [f.strip() for f in line.split("|")]
        rows.append(([float(v) for v in vals.split()], int(sc, 16), float(bs), [int(c, 16) for c in codes.split()]))
    return rows


def test_hand_derived_blocks():
    """Each vector becomes one 16 x 16 block (its own pixel) of a tensor whose maximum is 2688, so that T_scale = 1."""
    rows = golden_blocks()
    d = inputs.conv_desc(16, 16, 1, len(rows), 16, 1, 1, 0)
    x = np.zeros((16, 16, 1, len(rows)), dtype=np.float32)
    for p, (vals, _, _, _) in enumerate(rows):
        x[:len(vals), 0, 0, p] = vals            # down the sample axis of the block
    codes, scales, ts, amax = oracle.quantize_ts(d, oracle.ROLE_X, x)
    assert amax == 2688.0 and ts == 1.0          # Eq. 4: 2688 / (448 * 6)
    cc = unpack(codes).reshape(len(rows), 16, 32)
    sc = scales.reshape(len(rows), 1, 2)
    xh = oracle.dequant_ts(d, oracle.ROLE_X, codes, scales, ts)
    for p, (vals, want_sc, want_bs, want_codes) in enumerate(rows):
        assert sc[p, 0, 0] == want_sc, (p, hex(sc[p, 0, 0]))
        assert oracle.decode_elem(oracle.E4M3, want_sc) == want_bs
        assert list(cc[p, :len(vals), 0]) == want_codes, (p, list(cc[p, :len(vals), 0]))
        assert sc[p, 0, 1] == 0                   # the block of padded channels 16..31 is empty
        for i, c in enumerate(want_codes):        # fake quantization: element x block scale x tensor scale
            assert xh[i, 0, 0, p] == (-1.0 if c & 8 else 1.0) * E2M1_GRID[c & 7] * want_bs * ts


def test_eq5_closed_forms_and_the_factor_six():
    # a block maximum equal to the tensor maximum always gets the largest block scale, whatever the magnitude
    for amax in (2688.0, 1.0, 3e-5, 7e8, 0.3):
        t = np.float32(amax) / np.float32(448 * 6)
        assert oracle.block_scale_code(amax, t) == 0x7E
        assert oracle.ts_elem_code(amax, 448.0, t) == 7 and oracle.ts_elem_code(-amax, 448.0, t) == 15
    # block maxima that are exact E4M3 multiples of 6 T map to that E4M3 value
    for code in (0x01, 0x08, 0x30, 0x38, 0x45, 0x77, 0x7E):
        b = oracle.decode_elem(oracle.E4M3, code)
        assert oracle.block_scale_code(6.0 * b, 1.0) == code
        assert oracle.block_scale_code(6.0 * b * 0.25, 0.25) == code
    # midpoints between neighbouring E4M3 values go to the even code
    for code in range(1, 0x7E):
        lo, hi = oracle.decode_elem(oracle.E4M3, code), oracle.decode_elem(oracle.E4M3, code + 1)
        mid = 6.0 * (lo + hi) / 2          # exact in fp32: lo + hi has at most 5 significant bits
        assert oracle.block_scale_code(mid, 1.0) == (code if code % 2 == 0 else code + 1), code
    assert oracle.block_scale_code(0.0, 1.0) == 0 and oracle.block_scale_code(1.0, 0.0) == 0
    assert oracle.block_scale_code(1e9, 1.0) == 0x7E     # saturation (only reachable with an outside tensor maximum)


def test_second_derivation_through_library_casts():
    """The same three equations written with numpy float32 arithmetic, PyTorch's float8_e4m3fn cast for CastE4M3 (after
    clamping to 448, as that cast does not saturate) and a nearest-grid search for Round(.), on random data."""
    rng = np.random.default_rng(3)
    d = inputs.conv_desc(48, 40, 3, 5, 16, 1, 1, 0)
    x = (rng.standard_normal((48, 40, 3, 5)) * np.exp(rng.standard_normal((48, 40, 3, 5)))).astype(np.float32)
    codes, scales, ts, amax = oracle.quantize_ts(d, oracle.ROLE_X, x)
    assert amax == np.abs(x).max() and ts == np.float32(amax) / np.float32(2688.0)
    cc = unpack(codes).reshape(15, 48, 64)
    sc = scales.reshape(15, 3, 4)
    xs = x.transpose(2, 3, 0, 1).reshape(15, 48, 40)          # [pixel][n][c]
    for p in range(15):
        for rb in range(3):
            for cb in range(3):
                blk = xs[p, 16 * rb:16 * rb + 16, 16 * cb:min(16 * cb + 16, 40)]
                arg = np.float32(np.abs(blk).max()) / (np.float32(ts) * np.float32(6.0))
                b8 = torch.tensor([min(float(arg), 448.0)], dtype=torch.float32).to(torch.float8_e4m3fn)
                assert int(b8.view(torch.uint8)) == sc[p, rb, cb]
                bval = np.float32(float(b8.to(torch.float32)))
                if bval == 0:
                    continue
                v = blk / (bval * np.float32(ts))
                mag = np.minimum(np.abs(v).astype(np.float64), 6.0)
                dist = np.abs(mag[..., None] - E2M1_GRID)
                near = dist.argmin(-1)
                # ties: argmin takes the lower code; the even code is wanted
                tie = np.isclose(np.sort(dist, -1)[..., 0], np.sort(dist, -1)[..., 1], rtol=0, atol=0)
                near = np.where(tie & (near % 2 == 1), near + 1, near)
                want = near + 8 * np.signbit(v)
                got = cc[p, 16 * rb:16 * rb + 16, 16 * cb:16 * cb + blk.shape[1]]
                assert (got == want).all()


def test_scaling_by_a_power_of_two_changes_only_the_tensor_scale():
    rng = np.random.default_rng(4)
    d = inputs.conv_desc(32, 32, 4, 4, 32, 1, 1, 0)
    x = rng.standard_normal((32, 32, 4, 4)).astype(np.float32)
    c0, s0, t0, _ = oracle.quantize_ts(d, oracle.ROLE_X, x)
    for k in (-20, -3, 5, 30):
        c, s, t, _ = oracle.quantize_ts(d, oracle.ROLE_X, np.ldexp(x, k))
        assert np.array_equal(c, c0) and np.array_equal(s, s0) and t == np.ldexp(np.float32(t0), k)


@pytest.mark.parametrize("block", [(16, 16), (8, 8), (1, 16)], ids=["16x16", "8x8-paper", "1x16-line"])
@pytest.mark.parametrize("role", [oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY])
def test_error_bound_and_block_layout(role, block):
    """Every element is within half an E2M1 step (in units of its own block's scale) of its source value, with the block
    found by an index derivation written here independently (so a wrong block / scale index, or a dropped T_scale or
    B_scale in Eq. 6 or in the fake quantization, breaks the bound)."""
    rng = np.random.default_rng(5)
    d = inputs.conv_desc(40, 48, 3, 4, 56, 3, 1, 1)
    shape = oracle.logical_shape(d, role)
    x = (rng.standard_normal(shape) * np.exp(2 * rng.standard_normal(shape))).astype(np.float32)
    codes, scales, ts, _ = oracle.quantize_ts(d, role, x, block)
    xh = oracle.dequant_ts(d, role, codes, scales, ts, block)
    br, bc = block
    R, C = shape[0], shape[1]
    Cp = (C + 31) // 32 * 32
    P = shape[2] * shape[3]
    Rb, Cb = (R + br - 1) // br, Cp // bc
    sv = np.array([oracle.decode_elem(oracle.E4M3, c) for c in range(127)])[scales & 0x7F]
    sv = sv.reshape(Rb, P, Cb).transpose(1, 0, 2) if role == oracle.ROLE_W else sv.reshape(P, Rb, Cb)   # -> [p][rb][cb]
    xs = x.reshape(R, C, P).transpose(2, 0, 1)               # [p][r][c]
    xhs = xh.reshape(R, C, P).transpose(2, 0, 1)
    unit = np.repeat(np.repeat(sv, br, axis=1), bc, axis=2)[:, :R, :C] * ts
    ok = unit > 0
    v = np.abs(xs[ok] / unit[ok])
    err = np.abs(xhs[ok] - xs[ok]) / unit[ok]
    step = np.where(v < 2, 0.5, np.where(v < 4, 1.0, 2.0))
    assert (err <= step / 2 + 1e-6).all() or (v[err > step / 2 + 1e-6] > 6).all()
    assert (err[v > 6] <= v[v > 6] - 6 + 1e-6).all() and (v <= 6.0 / (1 - 2.0 ** -4) + 1e-3).all()   # Eq. 5 rounds B_scale down by at most 2^-4
    assert (xhs[~ok] == 0).all() and (np.abs(xs[~ok]) < unit.max()).all()


def test_zero_tensor_and_zero_blocks():
    d = inputs.conv_desc(32, 32, 2, 2, 32, 1, 1, 0)
    z = np.zeros((32, 32, 2, 2), dtype=np.float32)
    c, s, t, a = oracle.quantize_ts(d, oracle.ROLE_X, z)
    assert t == 0 and a == 0 and not c.any() and not s.any()
    z[3, 5, 1, 1] = -2.0
    c, s, t, a = oracle.quantize_ts(d, oracle.ROLE_X, z)
    assert a == 2.0 and np.count_nonzero(s) == 1 and np.count_nonzero(c) == 1
    assert np.allclose(oracle.dequant_ts(d, oracle.ROLE_X, c, s, t), z, rtol=1e-6, atol=0)      # T_scale = 2 / 2688 is rounded to fp32


def test_tensor_maximum_supplied_from_outside():
    """Statistics of earlier batches in place of the tensor's own maximum (Sec. VII-B): a larger value only coarsens the
    grid, a smaller one makes the top of the range saturate at 448 * 6 * T_scale = the supplied maximum."""
    rng = np.random.default_rng(6)
    d = inputs.conv_desc(32, 32, 3, 3, 32, 1, 1, 0)
    x = rng.standard_normal((32, 32, 3, 3)).astype(np.float32)
    amax = float(np.abs(x).max())
    c, s, t, a = oracle.quantize_ts(d, oracle.ROLE_X, x, amax=2 * amax)
    assert a == np.float32(amax) and t == np.float32(2 * amax) / np.float32(2688)
    xh = oracle.dequant_ts(d, oracle.ROLE_X, c, s, t)
    assert np.abs(xh - x).max() <= 0.25 * amax
    c, s, t, _ = oracle.quantize_ts(d, oracle.ROLE_X, x, amax=amax / 4)
    xh = oracle.dequant_ts(d, oracle.ROLE_X, c, s, t)
    assert np.abs(xh).max() == pytest.approx(amax / 4, rel=1e-6)
    big = np.abs(x) > amax / 4 * (1 + 2.0 ** -4)
    assert big.any() and (np.abs(xh[big]) == np.abs(xh).max()).all()


def test_stochastic_rounding_variant():
    """Same scales as round-to-nearest, codes at most one grid step away, unbiased on a constant field."""
    rng = np.random.default_rng(7)
    d = inputs.conv_desc(64, 32, 4, 4, 32, 1, 1, 0)
    x = rng.standard_normal((64, 32, 4, 4)).astype(np.float32)
    c0, s0, t0, _ = oracle.quantize_ts(d, oracle.ROLE_X, x)
    c1, s1, t1, _ = oracle.quantize_ts(d, oracle.ROLE_X, x, seed=9)
    assert np.array_equal(s0, s1) and t0 == t1 and not np.array_equal(c0, c1)
    u0, u1 = unpack(c0), unpack(c1)
    assert (np.abs((u0 & 7).astype(int) - (u1 & 7).astype(int)) <= 1).all() and ((u0 & 8) == (u1 & 8))[(u0 & 7) + (u1 & 7) > 0].all()
    # T_scale = 0.001 (one element of 2.688); every block holds 0.11 and 0.05: B_scale = CastE4M3(0.11 / 0.006 = 18.33) = 18,
    # so 0.05 / 0.018 = 2.78 sits between the grid values 2 and 3 and must average out to itself
    xc = np.full((64, 32, 4, 4), 0.11, dtype=np.float32)
    xc[0::2] = 0.05
    xc[0, 0, 0, 0] = 2.688
    c, s, t, _ = oracle.quantize_ts(d, oracle.ROLE_X, xc, seed=21)
    xh = oracle.dequant_ts(d, oracle.ROLE_X, c, s, t)
    sel = xc == np.float32(0.05)
    assert abs(xh[sel].mean() - 0.05) < 0.05 * 0.02
