"""Pins for the oracle's quantizer, channel-batch-first im2col and convolutions (no GPU).

Everything here compares the oracle with something it does not compute itself: invariants the
method guarantees (each tensor quantized once, blocks stay whole after im2col), index arithmetic
written a second way in numpy, the GEMM formulation of Sec. II-C, a float64 library convolution
with autograd, and exact integer arithmetic.
"""
import numpy as np
import pytest
import torch

import oracle
from oracle import E2M1, E4M3, E5M2, ROLE_DY, ROLE_W, ROLE_X
from paper_2609_28358_b200 import inputs

FMTS = [E4M3, E5M2, E2M1]
TILE, LINE = (32, 32), (1, 32)


def unpack(codes, fmt):
    if fmt == E2M1:
        return np.stack([codes & 0xF, codes >> 4], axis=-1).reshape(-1)
    return codes


def decode_table(fmt):
    n = 16 if fmt == E2M1 else 256
    return np.array([oracle.decode_elem(fmt, c) for c in range(n)])


# ---------------------------------------------------------------------------------- quantizer
@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("block", [TILE, LINE, (8, 8)])
def test_quantize_matches_numpy_restatement(fmt, block):
    """Second derivation of the whole quantizer in numpy: amax by reshape, scale by frexp,
    rounding by nearest-table lookup with explicit tie handling."""
    d = inputs.conv_desc(40, 48, 5, 6, 16, 3)  # ragged N (40) and C (48 -> Cp 64)
    x = inputs.make_x(d, 11, "gauss") * np.float32(3.0)
    codes, scales = oracle.quantize(d, ROLE_X, fmt, x, block)
    br, bc = block
    N, C, H, W = x.shape
    Cp, Rb = 64, -(-N // br)
    xs = np.zeros((H * W, Rb * br, Cp), np.float64)
    xs[:, :N, :C] = x.transpose(2, 3, 0, 1).reshape(H * W, N, C)
    blk = xs.reshape(H * W, Rb, br, Cp // bc, bc)
    amax = np.abs(blk).max(axis=(2, 4))
    _, e = np.frexp(amax)
    want_s = np.where(amax > 0, np.clip(e - 1 - oracle.FMT_EMAX[fmt] + 127, 0, 254), 0).astype(np.uint8)
    assert np.array_equal(scales.reshape(H * W, Rb, Cp // bc), want_s)
    v = blk * np.ldexp(1.0, 127 - want_s.astype(np.int64))[:, :, None, :, None]
    tab = decode_table(fmt)
    half = len(tab) // 2
    finite = np.array([c for c in range(half) if np.isfinite(tab[c])])
    mags = tab[finite]
    a = np.minimum(np.abs(v), mags.max())
    hi = np.searchsorted(mags, a, side="left").clip(1, len(mags) - 1)
    lo = hi - 1
    dl, dh = a - mags[lo], mags[hi] - a
    pick = np.where(dl < dh, lo, np.where(dh < dl, hi, np.where(finite[lo] % 2 == 0, lo, hi)))
    pick = np.where(a == 0, 0, pick)
    want_c = (finite[pick] | np.where(np.signbit(v), half, 0)).astype(np.uint8)
    want_c = want_c.reshape(H * W, Rb * br, Cp)[:, :N, :]
    want_c[:, :, C:] = 0  # padded channels hold code 0
    got = unpack(codes, fmt).reshape(H * W, N, Cp)
    assert np.array_equal(got, want_c)


@pytest.mark.parametrize("fmt", FMTS)
@pytest.mark.parametrize("role", [ROLE_X, ROLE_W, ROLE_DY])
def test_quantize_idempotent_and_error_bound(fmt, role):
    d = inputs.conv_desc(33, 40, 6, 6, 70, 3)
    src = {ROLE_X: inputs.make_x(d, 5, "relu"), ROLE_W: inputs.make_w(d, 5), ROLE_DY: inputs.make_dy(d, 5)}[role]
    c, s = oracle.quantize(d, role, fmt, src)
    back = oracle.dequant(d, role, fmt, c, s)
    c2, s2 = oracle.quantize(d, role, fmt, back.astype(np.float32))
    assert np.array_equal(c, c2) and np.array_equal(s, s2)  # Q(dequant(Q(x))) == Q(x)
    # no element moves by more than the worst case of its tile's top binade: half a step there, or
    # the saturation gap (2^(emax+1) - max) / max = 1/7 (FP8), 1/3 (FP4), relative to the tile maximum
    worst = {E4M3: 1 / 7, E5M2: 1 / 7, E2M1: 1 / 3}[fmt]
    assert np.abs(back - src).max() <= worst * np.abs(src).max()
    assert np.array_equal(np.signbit(back), np.signbit(src))


@pytest.mark.parametrize("fmt", FMTS)
def test_square_block_is_transpose_symmetric_line_block_is_not(fmt):
    """Sec. IV-B: a square block serves both contraction directions.  Swapping the two axes a
    square covers gives the transposed codes and the same scales; a line block does not."""
    d = inputs.conv_desc(64, 64, 3, 3, 8, 1, pad=0)
    x = inputs.make_x(d, 21, "gauss")
    xt = np.ascontiguousarray(x.transpose(1, 0, 2, 3))
    c, s = oracle.quantize(d, ROLE_X, fmt, x, TILE)
    ct, st = oracle.quantize(d, ROLE_X, fmt, xt, TILE)
    u = unpack(c, fmt).reshape(9, 64, 64)
    ut = unpack(ct, fmt).reshape(9, 64, 64)
    assert np.array_equal(u, ut.transpose(0, 2, 1))
    assert np.array_equal(s.reshape(9, 2, 2), st.reshape(9, 2, 2).transpose(0, 2, 1))
    cl, _ = oracle.quantize(d, ROLE_X, fmt, x, LINE)
    clt, _ = oracle.quantize(d, ROLE_X, fmt, xt, LINE)
    assert not np.array_equal(unpack(cl, fmt).reshape(9, 64, 64), unpack(clt, fmt).reshape(9, 64, 64).transpose(0, 2, 1))


@pytest.mark.parametrize("fmt", FMTS)
def test_special_tiles(fmt):
    d = inputs.conv_desc(32, 32, 1, 1, 32, 1, pad=0)
    emax = oracle.FMT_EMAX[fmt]
    # constant tile: every code equals the encoding of c / 2^(floor(log2 c) - emax)
    x = np.full((32, 32, 1, 1), 0.75, np.float32)
    c, s = oracle.quantize(d, ROLE_X, fmt, x)
    assert s.tolist() == [(-1) - emax + 127]
    assert np.all(unpack(c, fmt) == oracle.encode_elem(fmt, 0.75 * 2.0 ** (emax + 1)))
    assert np.array_equal(oracle.dequant(d, ROLE_X, fmt, c, s), x.astype(np.float64))
    # one-hot tile: the single element lands on 2^emax exactly, everything else is +0
    x = np.zeros((32, 32, 1, 1), np.float32)
    x[5, 17] = -3.0
    c, s = oracle.quantize(d, ROLE_X, fmt, x)
    u = unpack(c, fmt).reshape(32, 32)
    assert s.tolist() == [1 - emax + 127]
    assert u[5, 17] == oracle.encode_elem(fmt, -3.0 * 2.0 ** (emax - 1)) and np.count_nonzero(u) == 1
    # all-zero tile: scale code 0, codes 0 (sign kept for -0)
    x = np.zeros((32, 32, 1, 1), np.float32)
    x[0, 0] = -0.0
    c, s = oracle.quantize(d, ROLE_X, fmt, x)
    u = unpack(c, fmt).reshape(32, 32)
    assert s.tolist() == [0] and u[0, 0] == (8 if fmt == E2M1 else 0x80) and np.count_nonzero(u) == 1
    # line and square blocks agree when every line of the tile has its maximum in the same binade
    rng = np.random.default_rng(0)
    x = rng.uniform(-1, 1, (32, 32, 1, 1)).astype(np.float32)
    x[:, 0] = 1.5
    cl, sl = oracle.quantize(d, ROLE_X, fmt, x, LINE)
    ct, st = oracle.quantize(d, ROLE_X, fmt, x, TILE)
    assert np.array_equal(cl, ct) and np.all(sl == st[0])


def test_layouts_of_the_three_roles():
    """Stored order: X [H][W][N][Cp], W [Cout][Kh][Kw][Cinp], G_Y [Ho][Wo][N][Coutp] (Sec. IV-A/B),
    scales one per tile in the same order with the tiled axes divided by 32."""
    d = inputs.conv_desc(3, 5, 4, 6, 7, 3, stride=2)  # Ho=2, Wo=3
    tab = decode_table(E4M3)
    # values that are exactly representable with any scale the tile gets: powers of two tagged by index
    for role, shape in ((ROLE_X, (3, 5, 4, 6)), (ROLE_W, (7, 5, 3, 3)), (ROLE_DY, (3, 7, 2, 3))):
        src = np.arange(1, np.prod(shape) + 1, dtype=np.float32).reshape(shape) % 7 + 1  # 1..7, exact in E4M3
        c, s = oracle.quantize(d, role, E4M3, src)
        val = tab[c] * 2.0 ** (s.astype(np.float64).max() - 127)  # all tiles share a scale here (amax in [4,8))
        assert len(set(s.tolist())) == 1
        if role == ROLE_W:
            want = np.zeros((7, 3, 3, 32))
            want[..., :5] = src.transpose(0, 2, 3, 1)
        else:
            want = np.zeros(shape[2:] + (shape[0], 32))
            want[..., : shape[1]] = src.transpose(2, 3, 0, 1)
        assert np.array_equal(val.reshape(want.shape), want)


# ------------------------------------------------------------------------------------- im2col
@pytest.mark.parametrize("fmt", [E4M3, E2M1])
@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (3, 2, 1), (1, 1, 0), (1, 2, 0), (5, 2, 2), (3, 1, 0)])
def test_cbf_im2col_against_scatter_form(fmt, k, s, p):
    """Oracle gathers per tap; here every source pixel is scattered to the taps that see it."""
    d = inputs.conv_desc(37, 40, 7, 9, 8, k, s, p)
    x = inputs.make_x(d, 2, "relu")
    c, sc = oracle.quantize(d, ROLE_X, fmt, x)
    oc, osc = oracle.cbf_im2col(d, fmt, c, sc)
    Ho, Wo = inputs.out_hw(d)
    Cp, Nt = 64, 2
    rb = Cp * (4 if fmt == E2M1 else 8) // 8
    src = c.reshape(d.H, d.W, d.N, rb)
    ssrc = sc.reshape(d.H, d.W, Nt, Cp // 32)
    want = np.zeros((Ho, Wo, d.N, k, k, rb), np.uint8)
    wants = np.zeros((Ho, Wo, Nt, k, k, Cp // 32), np.uint8)
    taps = 0
    for h in range(d.H):
        for w in range(d.W):
            for kh in range(k):
                for kw in range(k):
                    a, b = h + p - kh, w + p - kw
                    if a % s or b % s or not (0 <= a // s < Ho) or not (0 <= b // s < Wo):
                        continue
                    want[a // s, b // s, :, kh, kw] = src[h, w]
                    wants[a // s, b // s, :, kh, kw] = ssrc[h, w]
                    taps += 1
    assert np.array_equal(oc.reshape(want.shape), want)
    assert np.array_equal(osc.reshape(wants.shape), wants)
    # every entry of X' decodes to the single quantized value of its source pixel (quantized once)
    xhat = oracle.dequant(d, ROLE_X, fmt, c, sc)
    tab = decode_table(fmt)
    u = unpack(oc, fmt).reshape(Ho, Wo, d.N, k, k, Cp)
    scale_full = np.repeat(np.repeat(osc.reshape(wants.shape), 32, axis=2)[:, :, : d.N], 32, axis=5)
    val = tab[u] * np.ldexp(1.0, scale_full.astype(np.int64) - 127)
    xpad = np.zeros((d.N, d.C_in, d.H + 2 * p, d.W + 2 * p))
    xpad[:, :, p:p + d.H, p:p + d.W] = xhat
    for kh in range(k):
        for kw in range(k):
            patch = xpad[:, :, kh:kh + s * Ho:s, kw:kw + s * Wo:s][:, :, :Ho, :Wo]
            assert np.array_equal(val[:, :, :, kh, kw, : d.C_in], patch.transpose(2, 3, 0, 1))
    assert taps > 0


def test_cbf_im2col_1x1_is_identity():
    d = inputs.conv_desc(32, 64, 6, 5, 8, 1, 1, 0)
    x = inputs.make_x(d, 4, "relu")
    c, s = oracle.quantize(d, ROLE_X, E2M1, x)
    oc, osc = oracle.cbf_im2col(d, E2M1, c, s)
    assert np.array_equal(oc, c) and np.array_equal(osc, s)


# ------------------------------------------------------------------------------- convolutions
def quantized_layer(d, fmts, seed, kinds=("relu", "kaiming", "small")):
    x = inputs.make_x(d, seed, kinds[0])
    w = inputs.make_w(d, seed, kinds[1])
    g = inputs.make_dy(d, seed, kinds[2])
    q = [oracle.quantize(d, r, f, t) for r, f, t in zip((ROLE_X, ROLE_W, ROLE_DY), fmts, (x, w, g))]
    hat = [oracle.dequant(d, r, f, c, s) for r, f, (c, s) in zip((ROLE_X, ROLE_W, ROLE_DY), fmts, q)]
    return q, hat


CONV_CASES = [(3, 1, 1), (3, 2, 1), (1, 1, 0), (1, 2, 0), (5, 1, 2), (3, 2, 0), (2, 2, 0)]


@pytest.mark.parametrize("k,s,p", CONV_CASES)
def test_convolutions_against_library_autograd(k, s, p):
    d = inputs.conv_desc(5, 6, 9, 8, 7, k, s, p)
    _, (xh, wh, gh) = quantized_layer(d, (E4M3, E4M3, E5M2), 9)
    xt = torch.tensor(xh, requires_grad=True)
    wt = torch.tensor(wh, requires_grad=True)
    yt = torch.nn.functional.conv2d(xt, wt, stride=s, padding=p)
    yt.backward(torch.tensor(gh))
    y, ya = oracle.conv_fwd(d, xh, wh)
    gx, gxa = oracle.conv_bwd_data(d, wh, gh)
    gw, gwa = oracle.conv_bwd_weight(d, gh, xh)
    for got, ref, ab in ((y, yt.detach().numpy(), ya), (gx, xt.grad.numpy(), gxa), (gw, wt.grad.numpy(), gwa)):
        assert got.shape == ref.shape
        assert (np.abs(got - ref) <= 1e-12 * ab + 1e-300).all()
        assert (ab >= np.abs(got) * (1 - 1e-12)).all()
    # sum|terms| against the same library routine on absolute values
    ya_ref = torch.nn.functional.conv2d(torch.tensor(np.abs(xh)), torch.tensor(np.abs(wh)), stride=s, padding=p).numpy()
    np.testing.assert_allclose(ya, ya_ref, rtol=1e-12, atol=1e-300)


@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (3, 2, 1), (1, 1, 0)])
def test_gemm_formulation_from_cbf_im2col(k, s, p):
    """Sec. II-C / IV-B: Y_f = W_f . X',  G_Wf = G_Yf . X'^T,  G_X' = W_f^T . G_Yf (+ col2im), with X'
    taken from the channel-batch-first im2col of the quantized activation and all three tensors
    in their stored 2-D views."""
    d = inputs.conv_desc(6, 40, 7, 6, 33, k, s, p)
    fm = (E4M3, E4M3, E5M2)
    (xq, wq, gq), (xh, wh, gh) = quantized_layer(d, fm, 13)
    Ho, Wo = inputs.out_hw(d)
    Cp, Cop = 64, 64
    oc, osc = oracle.cbf_im2col(d, E4M3, *xq)
    tab3, tab2 = decode_table(E4M3), decode_table(E5M2)
    sc = np.repeat(np.repeat(osc.reshape(Ho, Wo, 1, k, k, Cp // 32), 32, axis=2)[:, :, : d.N], 32, axis=5)
    Xp = (tab3[oc.reshape(Ho, Wo, d.N, k, k, Cp)] * np.ldexp(1.0, sc.astype(np.int64) - 127)).reshape(Ho * Wo * d.N, k * k * Cp)
    ws = np.repeat(np.repeat(wq[1].reshape(2, k, k, Cp // 32), 32, axis=0)[: d.C_out], 32, axis=3)
    Wf = (tab3[wq[0].reshape(d.C_out, k, k, Cp)] * np.ldexp(1.0, ws.astype(np.int64) - 127)).reshape(d.C_out, k * k * Cp)
    gs = np.repeat(np.repeat(gq[1].reshape(Ho, Wo, 1, Cop // 32), 32, axis=2)[:, :, : d.N], 32, axis=3)
    Gf = (tab2[gq[0].reshape(Ho, Wo, d.N, Cop)] * np.ldexp(1.0, gs.astype(np.int64) - 127)).reshape(Ho * Wo * d.N, Cop)[:, : d.C_out]
    y, ya = oracle.conv_fwd(d, xh, wh)
    Yf = Xp @ Wf.T  # [(ho,wo,n), co]
    assert (np.abs(Yf.reshape(Ho, Wo, d.N, d.C_out).transpose(2, 3, 0, 1) - y) <= 1e-12 * ya + 1e-300).all()
    gw, gwa = oracle.conv_bwd_weight(d, gh, xh)
    GWf = (Gf.T @ Xp).reshape(d.C_out, k, k, Cp)[..., : d.C_in].transpose(0, 3, 1, 2)
    assert (np.abs(GWf - gw) <= 1e-12 * gwa + 1e-300).all()
    gx, gxa = oracle.conv_bwd_data(d, wh, gh)
    GXp = (Gf @ Wf).reshape(Ho, Wo, d.N, k, k, Cp)  # G_X' in the layout of X'
    acc = np.zeros((d.N, d.C_in, d.H + 2 * p + s, d.W + 2 * p + s))
    for kh in range(k):
        for kw in range(k):
            acc[:, :, kh:kh + s * Ho:s, kw:kw + s * Wo:s] += GXp[:, :, :, kh, kw, : d.C_in].transpose(2, 3, 0, 1)
    assert (np.abs(acc[:, :, p:p + d.H, p:p + d.W] - gx) <= 1e-12 * gxa + 1e-300).all()


@pytest.mark.parametrize("fmts", [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1)])
@pytest.mark.parametrize("k,s,p", [(3, 1, 1), (3, 2, 1)])
def test_adjoint_identities_hold_because_each_tensor_is_quantized_once(fmts, k, s, p):
    d = inputs.conv_desc(34, 36, 8, 8, 40, k, s, p)
    _, (xh, wh, gh) = quantized_layer(d, fmts, 17, ("relu", "kaiming", "gauss"))
    y, _ = oracle.conv_fwd(d, xh, wh)
    gx, _ = oracle.conv_bwd_data(d, wh, gh)
    gw, _ = oracle.conv_bwd_weight(d, gh, xh)
    a, b, c = (y * gh).sum(), (xh * gx).sum(), (wh * gw).sum()
    scale = np.abs(y * gh).sum()
    assert abs(a - b) <= 1e-11 * scale and abs(a - c) <= 1e-11 * scale and scale > 0


def test_textbook_special_cases():
    d = inputs.conv_desc(3, 4, 6, 6, 4, 3)
    x = inputs.make_x(d, 1, "gauss").astype(np.float64)
    w = np.zeros((4, 4, 3, 3))
    w[np.arange(4), np.arange(4), 1, 1] = 1.0  # delta kernel
    y, _ = oracle.conv_fwd(d, x, w)
    assert np.array_equal(y, x)
    y, _ = oracle.conv_fwd(d, x, np.ones((4, 4, 3, 3)))  # box sum over channels and the 3x3 window
    xp = np.pad(x.sum(1), ((0, 0), (1, 1), (1, 1)))
    box = sum(xp[:, i:i + 6, j:j + 6] for i in range(3) for j in range(3))
    np.testing.assert_allclose(y, np.repeat(box[:, None], 4, 1), rtol=1e-13, atol=1e-13)
    d1 = inputs.conv_desc(3, 4, 6, 6, 5, 1, 1, 0)  # 1x1 conv is a matrix product over channels
    w1 = inputs.make_w(d1, 1).astype(np.float64)
    y, _ = oracle.conv_fwd(d1, x, w1)
    np.testing.assert_allclose(y, np.einsum("oc,nchw->nohw", w1[:, :, 0, 0], x), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("fmts", [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1)])
def test_small_integer_inputs_are_exact(fmts):
    """Values in {-2..2} survive every format whatever scale their tile gets, so every product and
    partial sum is an exactly representable integer: the quantized pipeline equals integer conv."""
    d = inputs.conv_desc(33, 35, 6, 7, 34, 3, 2, 1)
    (xq, wq, gq), (xh, wh, gh) = quantized_layer(d, fmts, 23, ("smallint",) * 3)
    x, w, g = inputs.make_x(d, 23, "smallint"), inputs.make_w(d, 23, "smallint"), inputs.make_dy(d, 23, "smallint")
    assert np.array_equal(xh, x) and np.array_equal(wh, w) and np.array_equal(gh, g)
    y, _ = oracle.conv_fwd(d, xh, wh)
    ref = torch.nn.functional.conv2d(torch.tensor(x, dtype=torch.int64), torch.tensor(w, dtype=torch.int64), stride=2, padding=1).numpy()
    assert np.array_equal(y, ref)


def test_sampled_outputs_equal_full_outputs():
    d = inputs.conv_desc(4, 5, 7, 7, 6, 3, 2, 1)
    _, (xh, wh, gh) = quantized_layer(d, (E4M3, E4M3, E5M2), 31)
    rng = np.random.default_rng(0)
    for full_fn, a, b in ((oracle.conv_fwd, xh, wh), (oracle.conv_bwd_data, wh, gh), (oracle.conv_bwd_weight, gh, xh)):
        y, ya = full_fn(d, a, b)
        idx = rng.choice(y.size, 50, replace=False)
        ys, yas = full_fn(d, a, b, idx)
        assert np.array_equal(ys, y.reshape(-1)[idx]) and np.array_equal(yas, ya.reshape(-1)[idx])
