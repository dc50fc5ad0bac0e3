"""Pins for the oracle's stochastic rounding (Eq. 6 with the stochastic Round(.), Sec. III-A) -- no GPU.

Checked against things other than the oracle itself: hand-derived threshold cases, the neighbours found by an
independent search over the closed-form grids, the expectation (an unbiased rounding reproduces the mean), the
deterministic quantizer (same scales, codes at most one grid step away), and the uniformity of the generator's draws.
"""
import os

import numpy as np
import pytest

import oracle
from oracle import E2M1, E2M3, E3M2, E4M3, E5M2
from paper_2609_28358_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")
FMT = {"E4M3": E4M3, "E5M2": E5M2, "E2M1": E2M1, "E3M2": E3M2, "E2M3": E2M3}
ALL = [E4M3, E5M2, E2M1, E3M2, E2M3]


def grid_of(fmt):
    """Non-negative finite values of a format from its closed form (exponent bits, mantissa bits, bias, number of magnitude codes)."""
    eb, mb, bias, ncodes = {E4M3: (4, 3, 7, 0x7F), E5M2: (5, 2, 15, 0x7C), E2M1: (2, 1, 1, 8), E3M2: (3, 2, 3, 32), E2M3: (2, 3, 1, 32)}[fmt]
    vals = []
    for m in range(ncodes):
        e, f = m >> mb, m & ((1 << mb) - 1)
        vals.append(f * 2.0 ** (1 - bias - mb) if e == 0 else (1 + f / (1 << mb)) * 2.0 ** (e - bias))
    return np.array(vals)


def mag_mask(fmt):
    return {E4M3: 0x7F, E5M2: 0x7F, E2M1: 0x7, E3M2: 0x1F, E2M3: 0x1F}[fmt]


def test_threshold_cases_from_golden_file():
    rows = 0
    for line in open(os.path.join(GOLD, "sr_threshold_vectors.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f, v, bits, code, _ = [t.strip() for t in line.split(";", 4)]
        assert oracle.encode_elem_sr(FMT[f], float(v), int(bits, 16)) == int(code, 16), line
        rows += 1
    assert rows >= 20


@pytest.mark.parametrize("fmt", ALL)
def test_result_is_a_neighbour_and_grid_values_do_not_move(fmt):
    grid = grid_of(fmt)
    rng = np.random.default_rng(11 + fmt)
    for v in grid:                                   # exact grid values: every draw returns them
        for bits in (0, 0xFFFFFFFF, 0x80000000, int(rng.integers(0, 2 ** 32))):
            assert oracle.decode_elem(fmt, oracle.encode_elem_sr(fmt, float(v), bits)) == v
    vals = np.concatenate([rng.uniform(0, grid[-1], 300), rng.uniform(0, grid[2], 100), -rng.uniform(0, grid[-1], 100)])
    for v in vals:
        a = abs(v)
        k = int(np.searchsorted(grid, a, side="right")) - 1     # grid[k] <= a < grid[k + 1]
        for bits in rng.integers(0, 2 ** 32, 4):
            code = oracle.encode_elem_sr(fmt, float(v), int(bits))
            got = oracle.decode_elem(fmt, code)
            assert abs(got) in (grid[k], grid[k + 1]), (fmt, v, bits)
            assert (got < 0 or (got == 0 and code > mag_mask(fmt))) == (v < 0) or got == 0 and v >= 0
            frac = (a - grid[k]) / (grid[k + 1] - grid[k])
            u = ((int(bits) >> 9) + 0.5) / 2 ** 23
            assert (abs(got) == grid[k + 1]) == (u < frac)


@pytest.mark.parametrize("fmt", ALL)
def test_saturation(fmt):
    top = grid_of(fmt)[-1]
    for v in (top, top * 1.01, top * 1e6):
        for bits in (0, 0xFFFFFFFF):
            assert oracle.decode_elem(fmt, oracle.encode_elem_sr(fmt, v, bits)) == top
            assert oracle.decode_elem(fmt, oracle.encode_elem_sr(fmt, -v, bits)) == -top


def test_generator_draws_are_uniform_and_distinct():
    n = 1 << 16
    for seed in (0, 1, 0xDEADBEEF12345678):
        r = np.array([oracle.sr_bits(seed, i) for i in range(n)], dtype=np.uint64)
        assert len(np.unique(r)) == n                                  # an invertible mix of the low index word: no repeats
        u = ((r >> np.uint64(9)).astype(np.float64) + 0.5) / 2 ** 23
        assert abs(u.mean() - 0.5) < 5 * (1 / 12 ** 0.5) / n ** 0.5
        hist = np.bincount((r >> np.uint64(24)).astype(np.int64), minlength=256)      # chi-square on the top byte, 255 d.o.f.
        chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 6 * (2 * 255) ** 0.5
        for b in range(32):                                            # every bit is balanced
            ones = int(((r >> np.uint64(b)) & np.uint64(1)).sum())
            assert abs(ones - n / 2) < 5 * (n / 4) ** 0.5, b
        lag = np.corrcoef(u[:-1], u[1:])[0, 1]                         # neighbouring elements are uncorrelated
        assert abs(lag) < 5 / n ** 0.5
    a = np.array([oracle.sr_bits(1, i) for i in range(4096)], dtype=np.int64)
    b = np.array([oracle.sr_bits(2, i) for i in range(4096)], dtype=np.int64)
    c = np.array([oracle.sr_bits(1, i + (1 << 32)) for i in range(4096)], dtype=np.int64)
    assert (a != b).mean() > 0.99 and (a != c).mean() > 0.99           # the seed and the high index word both re-key the stream


@pytest.mark.parametrize("fmt", ALL)
def test_tensor_quantizer_against_the_deterministic_one(fmt):
    d = inputs.conv_desc(40, 48, 5, 6, 70, 3, 1, 1)
    g = inputs.make_dy(d, 5, "gauss")
    c0, s0 = oracle.quantize(d, oracle.ROLE_DY, fmt, g)
    c1, s1 = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, seed=9)
    c2, s2 = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, seed=9)
    c3, _ = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, seed=10)
    assert (s0 == s1).all()                       # block scales do not depend on the rounding
    assert (c1 == c2).all() and (s1 == s2).all()  # a pure function of (input, seed)
    assert (c1 != c3).any() and (c1 != c0).any()
    x0 = oracle.dequant(d, oracle.ROLE_DY, fmt, c0, s0)
    x1 = oracle.dequant(d, oracle.ROLE_DY, fmt, c1, s1)
    # nearest rounding is never further from the input than stochastic rounding, the sign is kept, and the two codes are
    # the same or adjacent magnitudes (magnitude codes are ordered like the values)
    assert (np.abs(x0 - g) <= np.abs(x1 - g)).all()
    assert (np.sign(x1) * np.sign(g) >= 0).all()

    def mags(c):
        if fmt == E2M1:
            c = np.stack([c & 0xF, c >> 4], axis=-1).reshape(-1)
        return (c & mag_mask(fmt)).astype(np.int64)
    assert np.abs(mags(c1) - mags(c0)).max() == 1


@pytest.mark.parametrize("fmt", [E2M1, E4M3, E5M2])
def test_expectation_reproduces_the_input(fmt):
    """A tensor whose tiles hold one anchor value (fixing the scale) and otherwise a constant strictly between two grid
    values: the mean of the stochastic results approaches that constant (nearest rounding would sit on one neighbour)."""
    d = inputs.conv_desc(64, 32, 16, 16, 64, 1, 1, 0)
    g = np.full((64, 64, 16, 16), 0.3, dtype=np.float32)
    g[::32, ::32] = 1.0                            # tile maximum 1.0 -> scale 2^-emax; 0.3 is off-grid in every format
    c, s = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, seed=3)
    x = oracle.dequant(d, oracle.ROLE_DY, fmt, c, s)
    body = x[g != 1.0]
    vals = np.unique(body)
    assert len(vals) == 2 and vals[0] < np.float32(0.3) < vals[1]
    n = body.size
    sigma = (vals[1] - vals[0]) / 2 / n ** 0.5
    assert abs(body.mean() - float(np.float32(0.3))) < 5 * sigma
    c0, s0 = oracle.quantize(d, oracle.ROLE_DY, fmt, g)
    assert len(np.unique(oracle.dequant(d, oracle.ROLE_DY, fmt, c0, s0)[g != 1.0])) == 1
