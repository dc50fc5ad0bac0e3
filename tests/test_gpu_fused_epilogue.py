"""The quantizing producer epilogue (mq_conv_fwd_mx, mq_conv_bwd_data_mx) against the composition of pinned oracle
functions: convolution in float64 -> activation -> the oracle's quantizer (needs a B200).

The GPU quantizes its own fp32-accumulated result, which may differ from the float64 convolution by up to the GEMM bound
B = 1e-4 * sum|a*b| per element, and a code is a discontinuous function of its input.  Rule used here: the oracle
quantizes the two ends of each element's interval, act(y - B) and act(y + B) (the activations are monotone where it
matters: see _act_interval), as well as y itself.
  * A tile whose scale is the same at both ends has a determined scale: the GPU's must equal it.
  * In such a tile an element whose code is the same at both ends has a determined code: the GPU's must equal it.
  * Every other element must decode to a value between the two ends' decoded values (it sits at a rounding threshold).
  * Tiles whose amax straddles a power of two within B are counted and skipped.
The undetermined share is reported and bounded, so the rule cannot hide a broken kernel; in addition the GPU's codes must
agree with the oracle's codes of y itself on all but a small fraction of the elements."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import GEMM_TOL, dev, host

pytestmark = pytest.mark.gpu

E4M3, E5M2, E2M1, E3M2, E2M3 = mq.E4M3, mq.E5M2, mq.E2M1, mq.E3M2, mq.E2M3


def _act(y, act):
    if act == mq.ACT_RELU:
        return np.maximum(y, 0.0)
    if act == mq.ACT_SILU:
        return y / (1.0 + np.exp(-y))
    return y


def _act_interval(y, b, act):
    """[lo, hi] of act over [y - b, y + b], widened by the fp32 evaluation error of the activation."""
    lo, hi = _act(y - b, act), _act(y + b, act)
    if act == mq.ACT_SILU:
        # SiLU decreases below its minimum at y = -1.2785: take the envelope there (slope magnitude <= 0.1)
        lo, hi = np.minimum(lo, hi), np.maximum(lo, hi)
        near = np.abs(y + 1.2785) <= b + 1e-3
        lo = np.where(near, np.minimum(lo, -0.27847), lo)
        slack = 4e-6 * np.abs(_act(y, act)) + 1e-30
        lo, hi = lo - slack, hi + slack
    return lo, hi


def _decode_table(fmt):
    n = 16 if fmt == E2M1 else 256
    return np.array([oracle.decode_elem(fmt, c) if not np.isnan(oracle.decode_elem(fmt, c)) else 0.0 for c in range(n)])


def _unpack(codes, fmt):
    codes = np.asarray(codes)
    if fmt != E2M1:
        return codes
    out = np.empty(codes.size * 2, dtype=np.uint8)
    out[0::2] = codes & 0xF
    out[1::2] = codes >> 4
    return out


def check_emitted(name, d_out, role, fmt, y64, bound, act, got):
    """d_out: descriptor under which the emitted tensor is a role `role` tensor; y64 / bound in its logical NCHW order."""
    lo, hi = _act_interval(y64, bound, act)
    mid = _act(y64, act)
    q_lo, q_hi, q_mid = [oracle.quantize(d_out, role, fmt, a.astype(np.float32)) for a in (lo, hi, mid)]
    g_codes, g_scales = host(got.codes), host(got.scales)
    assert g_scales.shape == q_mid[1].shape and g_codes.shape == q_mid[0].shape
    # scales: view as [P][Nt][Ct]
    N = d_out.N
    C = d_out.C_in if role == oracle.ROLE_X else d_out.C_out
    Cp, Nt = (C + 31) // 32 * 32, (N + 31) // 32
    P = g_scales.size // (Nt * (Cp // 32))
    s_lo, s_hi = q_lo[1].reshape(P, Nt, Cp // 32), q_hi[1].reshape(P, Nt, Cp // 32)
    s_g = g_scales.reshape(P, Nt, Cp // 32)
    tile_fixed = s_lo == s_hi
    assert (s_g[tile_fixed] == s_lo[tile_fixed]).all(), f"{name}: a determined tile scale differs"
    # elements: [P][N][Cp] codes; tile of an element
    c_lo, c_hi, c_mid, c_g = [_unpack(c, fmt).reshape(P, N, Cp) for c in (q_lo[0], q_hi[0], q_mid[0], g_codes)]
    fixed_e = np.repeat(np.repeat(tile_fixed, 32, axis=2), 32, axis=1)[:, :N, :]
    det = fixed_e & (c_lo == c_hi)
    bad = det & (c_g != c_lo)
    assert not bad.any(), f"{name}: {int(bad.sum())} determined codes differ; first at {np.argwhere(bad)[0]}"
    tab = _decode_table(fmt)
    und = fixed_e & ~det
    v_g, v_lo, v_hi = tab[c_g[und]], tab[c_lo[und]], tab[c_hi[und]]
    assert ((v_g >= np.minimum(v_lo, v_hi)) & (v_g <= np.maximum(v_lo, v_hi))).all(), f"{name}: a code at a rounding threshold lies outside its interval"
    frac_und = 1.0 - det.mean()
    frac_diff = float((c_g != c_mid).mean())
    # the bound is loose (values near zero have sum|a*b| far above |y|), so a sizeable share sits "at a threshold"; what
    # makes the rule sharp is the second figure: the GPU agrees with the oracle's own codes of y on all but a sliver
    assert frac_und < 0.35, (name, frac_und)
    assert frac_diff < 0.01, (name, frac_diff)
    return frac_und, frac_diff


SHAPES = [
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),
    ("ragged", (40, 64, 6, 7, 70, 3, 1, 1)),            # ragged samples (two sample tiles), ragged output channels, odd width
    ("stride2", (33, 64, 9, 11, 40, 3, 2, 1)),
    ("k1_wide", (32, 256, 4, 8, 288, 1, 1, 0)),         # 256-channel tiles and a remainder tile
    ("deep_batch", (250, 128, 3, 4, 160, 3, 1, 1)),     # 8 sample tiles, the last ragged
    ("w14", (64, 64, 14, 14, 64, 3, 1, 1)),             # 14 columns: two-column tiles
    ("odd_channels", (36, 40, 6, 6, 72, 3, 1, 1)),      # 40 -> 72 channels (E2M1: 16-byte rows): not a tensor-core layer, the two-launch route
]


@pytest.mark.parametrize("act", [mq.ACT_NONE, mq.ACT_RELU, mq.ACT_SILU], ids=["none", "relu", "silu"])
@pytest.mark.parametrize("fmts,out_fmt", [((E4M3, E4M3, E5M2), E4M3), ((E2M1, E2M1, E2M1), E2M1), ((E4M3, E4M3, E5M2), E5M2), ((E3M2, E4M3, E5M2), E3M2)],
                         ids=["fp8", "fp4", "e5m2-out", "fp6"])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_forward_emits_next_layers_activation(name, shape, fmts, out_fmt, act):
    d = inputs.conv_desc(*shape)
    x, w = inputs.make_x(d, 61, "gauss"), inputs.make_w(d, 61)
    oq = [oracle.quantize(d, r, f, t) for r, f, t in zip((oracle.ROLE_X, oracle.ROLE_W), fmts, (x, w))]
    xh, wh = [oracle.dequant(d, r, f, *q) for r, f, q in zip((oracle.ROLE_X, oracle.ROLE_W), fmts, oq)]
    y64, ab = oracle.conv_fwd(d, xh, wh)
    gq = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip((mq.ROLE_X, mq.ROLE_W), fmts, (x, w))]
    yq = mq.conv_fwd_mx(d, gq[0], gq[1], out_fmt, act)
    assert mq.last_device_status() == 0
    ho, wo = inputs.out_hw(d)
    d_next = d._replace(C_in=d.C_out, H=ho, W=wo)      # the emitted tensor is the next layer's role-X tensor
    check_emitted(f"{name} fwd", d_next, oracle.ROLE_X, out_fmt, y64, GEMM_TOL * ab, act, yq)
    # feeding it to a following 1x1 layer works like any stored tensor
    d2 = inputs.conv_desc(d.N, d.C_out, ho, wo, 32, 1, 1, 0)
    w2q = mq.quantize(d2, mq.ROLE_W, E4M3 if out_fmt != E2M1 else E2M1, dev(inputs.make_w(d2, 62)))
    mq.conv_fwd(d2, yq, w2q)
    assert mq.last_device_status() == 0


@pytest.mark.parametrize("fmts,out_fmt", [((E4M3, E4M3, E5M2), E5M2), ((E2M1, E2M1, E2M1), E2M1)], ids=["fp8", "fp4"])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_input_gradient_emits_previous_layers_gradient(name, shape, fmts, out_fmt):
    d = inputs.conv_desc(*shape)
    w, g = inputs.make_w(d, 63), inputs.make_dy(d, 63, "gauss")
    oq = [oracle.quantize(d, r, f, t) for r, f, t in zip((oracle.ROLE_W, oracle.ROLE_DY), fmts[1:], (w, g))]
    wh, gh = [oracle.dequant(d, r, f, *q) for r, f, q in zip((oracle.ROLE_W, oracle.ROLE_DY), fmts[1:], oq)]
    gx64, ab = oracle.conv_bwd_data(d, wh, gh)
    gq = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip((mq.ROLE_W, mq.ROLE_DY), fmts[1:], (w, g))]
    dxq = mq.conv_bwd_data_mx(d, gq[0], gq[1], out_fmt)
    assert mq.last_device_status() == 0
    # G_X is N x C_in x H x W: the role-DY tensor of a layer whose output it is
    d_prev = inputs.conv_desc(d.N, 32, d.H, d.W, d.C_in, 1, 1, 0)
    check_emitted(f"{name} bwd_data", d_prev, oracle.ROLE_DY, out_fmt, gx64, GEMM_TOL * ab, mq.ACT_NONE, dxq)


@pytest.mark.parametrize("tw", [1, 2, 4])
@pytest.mark.parametrize("fmts,out_fmt", [((E4M3, E4M3, E5M2), E4M3), ((E2M1, E2M1, E2M1), E2M1)], ids=["fp8", "fp4"])
def test_every_tile_width(knobs, fmts, out_fmt, tw):
    """The epilogue's tiles are 1, 2 or 4 output columns wide (one column: a warp's rows are a whole sample tile; more: the
    warps of a tile exchange their maxima).  The library picks one per layer; here each is forced on the same ragged layer."""
    knobs(MQ_TC_MX_TW=tw)
    d = inputs.conv_desc(140, 64, 5, 6, 96, 3, 1, 1)
    x, w, g = inputs.make_x(d, 71, "gauss"), inputs.make_w(d, 71), inputs.make_dy(d, 71, "gauss")
    oq = [oracle.quantize(d, r, f, t) for r, f, t in zip((oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY), fmts, (x, w, g))]
    xh, wh, gh = [oracle.dequant(d, r, f, *q) for r, f, q in zip((oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY), fmts, oq)]
    gq = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip((mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY), fmts, (x, w, g))]
    y64, ab = oracle.conv_fwd(d, xh, wh)
    yq = mq.conv_fwd_mx(d, gq[0], gq[1], out_fmt, mq.ACT_RELU)
    assert mq.last_device_status() == 0
    ho, wo = inputs.out_hw(d)
    check_emitted(f"tw{tw} fwd", d._replace(C_in=d.C_out, H=ho, W=wo), oracle.ROLE_X, out_fmt, y64, GEMM_TOL * ab, mq.ACT_RELU, yq)
    gx64, ab = oracle.conv_bwd_data(d, wh, gh)
    dxq = mq.conv_bwd_data_mx(d, gq[1], gq[2], fmts[2])
    assert mq.last_device_status() == 0
    check_emitted(f"tw{tw} bwd_data", inputs.conv_desc(d.N, 32, d.H, d.W, d.C_in, 1, 1, 0), oracle.ROLE_DY, fmts[2], gx64, GEMM_TOL * ab,
                  mq.ACT_NONE, dxq)


def check_emitted_ts(name, d_out, role, y64, bound, act, amax_in, got):
    """check_emitted for the paper's own format (16 x 16 blocks, E4M3 block scales, the tensor maximum supplied)."""
    B16 = (16, 16)
    lo, hi = _act_interval(y64, bound, act)
    mid = _act(y64, act)
    q_lo, q_hi, q_mid = [oracle.quantize_ts(d_out, role, a.astype(np.float32), B16, amax=float(amax_in)) for a in (lo, hi, mid)]
    stats = host(got.tensor_scale)
    assert stats[0] == np.float32(amax_in) / (np.float32(448.0) * np.float32(6.0)), (name, stats)
    # the tensor's own maximum, left for the next step: that of the fp32 result, inside the bracket of the float64 one
    assert np.abs(lo).max() * (1 - 1e-6) <= stats[1] <= np.abs(hi).max() * (1 + 1e-6) or abs(stats[1] - np.abs(mid).max()) <= bound.max(), (name, stats)
    g_codes, g_scales = host(got.codes), host(got.scales)
    assert g_scales.shape == q_mid[1].shape and g_codes.shape == q_mid[0].shape
    N = d_out.N
    C = d_out.C_in if role == oracle.ROLE_X else d_out.C_out
    Cp, Nt = (C + 31) // 32 * 32, (N + 15) // 16
    P = g_scales.size // (Nt * (Cp // 16))
    s_lo, s_hi, s_g = [a.reshape(P, Nt, Cp // 16) for a in (q_lo[1], q_hi[1], g_scales)]
    tile_fixed = s_lo == s_hi
    assert (s_g[tile_fixed] == s_lo[tile_fixed]).all(), f"{name}: a determined block scale differs"
    c_lo, c_hi, c_mid, c_g = [_unpack(c, E2M1).reshape(P, N, Cp) for c in (q_lo[0], q_hi[0], q_mid[0], g_codes)]
    fixed_e = np.repeat(np.repeat(tile_fixed, 16, axis=2), 16, axis=1)[:, :N, :]
    det = fixed_e & (c_lo == c_hi)
    bad = det & (c_g != c_lo)
    assert not bad.any(), f"{name}: {int(bad.sum())} determined codes differ; first at {np.argwhere(bad)[0]}"
    tab = _decode_table(E2M1)
    und = fixed_e & ~det
    v_g, v_lo, v_hi = tab[c_g[und]], tab[c_lo[und]], tab[c_hi[und]]
    assert ((v_g >= np.minimum(v_lo, v_hi)) & (v_g <= np.maximum(v_lo, v_hi))).all(), f"{name}: a code at a rounding threshold lies outside its interval"
    frac_und = 1.0 - det.mean()
    frac_diff = float((c_g != c_mid).mean())
    assert frac_und < 0.45, (name, frac_und)
    assert frac_diff < 0.02, (name, frac_diff)
    return frac_und, frac_diff


TS_SHAPES = [
    ("c128", (140, 128, 6, 5, 128, 3, 1, 1)),          # one-column tiles (two sample tiles of 128, the second ragged), 64-byte chunks
    ("c256_n48", (48, 256, 5, 6, 256, 3, 1, 1)),       # two-column tiles (64 samples per tile), 256-channel tiles, three 16-sample blocks
    ("stride2", (64, 64, 9, 10, 192, 3, 2, 1)),        # 32-byte chunks; parity classes of the input gradient
    ("k1", (32, 512, 3, 4, 320, 1, 1, 0)),
    ("odd_channels", (36, 40, 6, 6, 72, 3, 1, 1)),     # not a tensor-core layer: the two-launch route
]


@pytest.mark.parametrize("act", [mq.ACT_NONE, mq.ACT_RELU, mq.ACT_SILU], ids=["none", "relu", "silu"])
@pytest.mark.parametrize("name,shape", TS_SHAPES, ids=[s[0] for s in TS_SHAPES])
def test_paper_format_in_and_out(name, shape, act):
    """mq_conv_fwd_ts / mq_conv_bwd_data_ts: operands and emitted tensor in the paper's own format (Eq. 4-6), the emitted
    tensor's maximum supplied (here: 0.8 x its true maximum, so the top saturates) - against conv in float64 ->
    activation -> oracle.quantize_ts with that maximum."""
    B16 = (16, 16)
    d = inputs.conv_desc(*shape)
    x, w, g = inputs.make_x(d, 91, "gauss"), inputs.make_w(d, 91), inputs.make_dy(d, 91, "gauss")
    roles = (oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY)
    oq = [oracle.quantize_ts(d, r, t, B16) for r, t in zip(roles, (x, w, g))]
    xh, wh, gh = [oracle.dequant_ts(d, r, o[0], o[1], o[2], B16) for r, o in zip(roles, oq)]
    gq = [mq.quantize_ts(d, r, dev(t)) for r, t in zip((mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY), (x, w, g))]
    ho, wo = inputs.out_hw(d)
    y64, ab = oracle.conv_fwd(d, xh, wh)
    amax = np.float32(0.8 * np.abs(_act(y64, act)).max())
    amax_dev = torch.tensor([amax], dtype=torch.float32, device="cuda")
    n0 = mq.kernel_launch_count()
    yq = mq.conv_fwd_ts(d, gq[0], gq[1], amax_dev, act)
    assert mq.last_device_status() == 0
    assert mq.kernel_launch_count() - n0 == 2      # tensor cores: scale expansion + the GEMM with the quantizing epilogue
    d_next = d._replace(C_in=d.C_out, H=ho, W=wo)
    check_emitted_ts(f"{name} fwd", d_next, oracle.ROLE_X, y64, GEMM_TOL * ab, act, amax, yq)
    # the emitted tensor feeds a following layer like any stored tensor of that format
    d2 = inputs.conv_desc(d.N, d.C_out, ho, wo, 64, 1, 1, 0)
    w2q = mq.quantize_ts(d2, mq.ROLE_W, dev(inputs.make_w(d2, 92)))
    mq.conv_fwd(d2, yq, w2q)
    assert mq.last_device_status() == 0
    if act == mq.ACT_NONE:
        gx64, ab = oracle.conv_bwd_data(d, wh, gh)
        amax = np.float32(0.8 * np.abs(gx64).max())
        amax_dev = torch.tensor([amax], dtype=torch.float32, device="cuda")
        n0 = mq.kernel_launch_count()
        dxq = mq.conv_bwd_data_ts(d, gq[1], gq[2], amax_dev)
        assert mq.last_device_status() == 0
        # 72 output channels are 48-byte rows of K: not a tensor-core layer - CUDA-core GEMM + the quantizer's two passes
        assert mq.kernel_launch_count() - n0 == (3 if name == "odd_channels" else 2)
        d_prev = inputs.conv_desc(d.N, 32, d.H, d.W, d.C_in, 1, 1, 0)
        check_emitted_ts(f"{name} bwd_data", d_prev, oracle.ROLE_DY, gx64, GEMM_TOL * ab, mq.ACT_NONE, amax, dxq)


def _tiles_of_slab(rng, n_pix, n_cb, border, count):
    """(pixel, channel block) pairs: the image's corner / edge pixels first, then random ones"""
    pix = list(border) + list(rng.integers(0, n_pix, count))
    return [(int(p), int(rng.integers(0, n_cb))) for p in pix[:count]]


@pytest.mark.parametrize("name,act", [("cfg5_e4m3_k3s1_c512_hw28", mq.ACT_RELU), ("cfg5_e4m3_k3s1_c512_hw56", mq.ACT_SILU),
                                      ("cfg5_e4m3_k1s1_c512_hw56", mq.ACT_RELU), ("cfg5_e4m3_k3s2_c512_hw28", mq.ACT_NONE),
                                      ("cfg5_e2m1_k3s1_c512_hw28", mq.ACT_RELU)],
                         ids=["3x3_hw28_relu", "3x3_hw56_silu", "1x1_hw56_relu", "3x3s2_hw28_none", "e2m1_hw28_relu"])
def test_bench_layers_full_size(name, act):
    """The layers `bench.py` times with the quantizing epilogue, on the GPU at full size (one-column tiles, 256-channel tiles,
    tensors beyond 2^31 elements).  The oracle checks whole sample tiles - (pixel, 32 samples, 32 channels), corner and edge
    pixels included, in the first and the last 32-sample slab - of the emitted activation tensor and of the emitted
    gradient tensor: the tile's 1024 sums in float64, then the bracket rule of check_emitted on the tiles laid side by side."""
    import types
    layer = {l.name: l for l in inputs.config5()}[name]
    d, (fx, fw, fg) = layer.desc, (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    x, w, g = inputs.layer_tensors(layer)
    ho, wo = inputs.out_hw(d)
    xq, wq, gq = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip((mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY), (fx, fw, fg), (x, w, g))]
    yq = mq.conv_fwd_mx(d, xq, wq, fx, act)
    dxq = mq.conv_bwd_data_mx(d, wq, gq, fg)
    assert mq.last_device_status() == 0
    wc, wsc = oracle.quantize(d, oracle.ROLE_W, fw, w)
    wh = oracle.dequant(d, oracle.ROLE_W, fw, wc, wsc)
    rng = np.random.default_rng(5)
    T = 24
    bpe = lambda f: 0.5 if f == E2M1 else 1.0
    for what, q_out, fmt_out, C, Hh, Ww, a in (("fwd", yq, fx, d.C_out, ho, wo, act), ("bwd_data", dxq, fg, d.C_in, d.H, d.W, mq.ACT_NONE)):
        Cp, Nt = (C + 31) // 32 * 32, (d.N + 31) // 32
        codes = q_out.codes.view(Hh * Ww, d.N, int(Cp * bpe(fmt_out)))
        scales = q_out.scales.view(Hh * Ww, Nt, Cp // 32)
        for slab in sorted({0, Nt - 1}):
            n0, n1 = 32 * slab, min(d.N, 32 * slab + 32)
            assert n1 - n0 == 32
            ds = d._replace(N=32)
            if what == "fwd":
                oc, osc = oracle.quantize(ds, oracle.ROLE_X, fx, x[n0:n1])
                ah = oracle.dequant(ds, oracle.ROLE_X, fx, oc, osc)
            else:
                oc, osc = oracle.quantize(ds, oracle.ROLE_DY, fg, g[n0:n1])
                ah = oracle.dequant(ds, oracle.ROLE_DY, fg, oc, osc)
            border = [0, Ww - 1, (Hh - 1) * Ww, Hh * Ww - 1, Ww // 2, (Hh // 2) * Ww]
            tiles = _tiles_of_slab(rng, Hh * Ww, Cp // 32, border, T)
            nn, cc = np.meshgrid(np.arange(32), np.arange(32), indexing="ij")
            idx = np.concatenate([((nn * C + 32 * cb + cc) * (Hh * Ww) + p).reshape(-1) for p, cb in tiles]).astype(np.int64)
            ref, ab = oracle.conv_fwd(ds, ah, wh, idx) if what == "fwd" else oracle.conv_bwd_data(ds, wh, ah, idx)
            # the tiles side by side as one pixel of a 32-sample tensor with 32 T channels
            y64 = ref.reshape(T, 32, 32).transpose(1, 0, 2).reshape(32, 32 * T, 1, 1)
            bnd = (GEMM_TOL * ab).reshape(T, 32, 32).transpose(1, 0, 2).reshape(32, 32 * T, 1, 1)
            bb = int(32 * bpe(fmt_out))
            got = types.SimpleNamespace(
                codes=torch.cat([codes[p, n0:n1, cb * bb:(cb + 1) * bb] for p, cb in tiles], dim=1).contiguous().reshape(-1),
                scales=torch.stack([scales[p, slab, cb] for p, cb in tiles]).contiguous())
            if what == "fwd":
                d_out, role = inputs.conv_desc(32, 32 * T, 1, 1, 32, 1, 1, 0), oracle.ROLE_X
            else:
                d_out, role = inputs.conv_desc(32, 32, 1, 1, 32 * T, 1, 1, 0), oracle.ROLE_DY
            check_emitted(f"{name} {what} slab {slab}", d_out, role, fmt_out, y64, bnd, a, got)


def test_bad_arguments():
    d = inputs.conv_desc(32, 64, 6, 6, 64, 3, 1, 1)
    xq, wq = mq.quantize(d, mq.ROLE_X, E4M3, dev(inputs.make_x(d, 1))), mq.quantize(d, mq.ROLE_W, E4M3, dev(inputs.make_w(d, 1)))
    with pytest.raises(mq.MqError) as e:
        mq.conv_fwd_mx(d, xq, wq, E4M3, act=7)
    assert e.value.status == 1
    small = mq.QTensor(torch.zeros(64, dtype=torch.uint8, device="cuda"), torch.zeros(64, dtype=torch.uint8, device="cuda"), E4M3, mq.ROLE_X)
    with pytest.raises(mq.MqError) as e:
        mq.conv_fwd_mx(d, xq, wq, E4M3, yq=small)
    assert e.value.status == 4
