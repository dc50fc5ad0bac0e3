"""Line blocks (the one-directional 1 x 32 block of Sec. III-A, MQ_BLOCK_LINE32) on the CUDA path against the CPU
oracle's block=(1, 32), through the C ABI (needs a B200): quantizer (every kernel variant, both source layouts,
stochastic rounding), channel-batch-first im2col and the forward GEMM (tensor-core and CUDA-core routes); and the
refusal of the two backward GEMMs, which is the limitation the paper's square blocks remove (Sec. III-B, III-C)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import assert_gemm_close, assert_same_bytes, border_indices, dev, host

pytestmark = pytest.mark.gpu

E4M3, E5M2, E2M1, E3M2, E2M3 = mq.E4M3, mq.E5M2, mq.E2M1, mq.E3M2, mq.E2M3
LINE = (1, 32)
SHAPES = [
    ("ragged", (40, 48, 5, 6, 70, 3, 1, 1)),          # 30 positions: the one-block-per-item kernel
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),
    ("stride2", (33, 64, 9, 11, 40, 3, 2, 1)),
    ("k1", (36, 40, 6, 8, 72, 1, 1, 0)),
    ("wide", (32, 256, 4, 8, 288, 3, 1, 1)),          # 128-byte K chunks, a remainder channel tile
    ("thin_n70", (70, 32, 6, 6, 40, 3, 1, 1)),        # thin layer (the whole-tile kernel in square mode; per-tap here)
    ("batch16", (16, 40, 10, 12, 72, 3, 1, 1)),
]


def line_case(name, shape, fmts, seed=51):
    d = inputs.conv_desc(*shape)
    x, w = inputs.make_x(d, seed, "relu"), inputs.make_w(d, seed)
    oq = [oracle.quantize(d, r, f, t, LINE) for r, f, t in zip((oracle.ROLE_X, oracle.ROLE_W), fmts, (x, w))]
    return d, x, w, oq


def check_fwd(d, fmts, oq, gq, samples=None, seed=0):
    xh = oracle.dequant(d, oracle.ROLE_X, fmts[0], *oq[0], LINE)
    wh = oracle.dequant(d, oracle.ROLE_W, fmts[1], *oq[1], LINE)
    shape = oracle.logical_shape(d, oracle.ROLE_DY)
    rng = np.random.default_rng(seed)
    idx = None
    if samples is not None and samples < int(np.prod(shape)):
        idx = np.unique(np.concatenate([rng.choice(int(np.prod(shape)), samples, replace=False), border_indices(shape, rng=rng)])).astype(np.int64)
    ref, ab = oracle.conv_fwd(d, xh, wh, idx)
    for layout in (mq.NCHW, mq.HWNC):
        y = mq.conv_fwd(d, gq[0], gq[1], layout=layout)
        yn = y if layout == mq.NCHW else y.permute(2, 3, 0, 1)
        got = host(yn.contiguous()).reshape(-1)
        assert_gemm_close(torch.from_numpy(got if idx is None else got[idx]), ref, ab, f"line-block fwd layout {layout}")
    assert mq.last_device_status() == 0


@pytest.mark.parametrize("route", ["tensor-cores", "cuda-cores", "whole-line-quantizer"])
@pytest.mark.parametrize("fmts", [(E4M3, E4M3), (E2M1, E2M1), (E5M2, E4M3), (E3M2, E2M3)], ids=lambda f: "-".join(map(str, f)))
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_line_blocks_quantize_im2col_forward(name, shape, fmts, route, knobs):
    if route == "cuda-cores":
        knobs(MQ_DISABLE_TC="1")
    if route == "whole-line-quantizer":
        knobs(MQ_QUANT_TMA="1")
    d, x, w, oq = line_case(name, shape, fmts)
    gq = [mq.quantize(d, r, f, dev(t), block=mq.LINE32) for r, f, t in zip((mq.ROLE_X, mq.ROLE_W), fmts, (x, w))]
    for what, g, (c, s) in zip(("X", "W"), gq, oq):
        assert_same_bytes(g.scales, s, f"{name} {what} line scales")
        assert_same_bytes(g.codes, c, f"{name} {what} line codes")
    # channel-fastest source, and the stochastic rounding: the same stored tensors
    xs, ws = np.ascontiguousarray(x.transpose(2, 3, 0, 1)), np.ascontiguousarray(w.transpose(0, 2, 3, 1))
    for what, role, f, src, (c, s) in (("X", mq.ROLE_X, fmts[0], xs, oq[0]), ("W", mq.ROLE_W, fmts[1], ws, oq[1])):
        g2 = mq.quantize(d, role, f, dev(src), src_layout=mq.HWNC, block=mq.LINE32)
        assert_same_bytes(g2.scales, s, f"{name} {what} line scales from channel-fastest source")
        assert_same_bytes(g2.codes, c, f"{name} {what} line codes from channel-fastest source")
    sc, ss = oracle.quantize_sr(d, oracle.ROLE_X, fmts[0], x, 17, LINE)
    for src, layout in ((x, mq.NCHW), (xs, mq.HWNC)):
        g3 = mq.quantize_sr(d, mq.ROLE_X, fmts[0], dev(src), 17, src_layout=layout, block=mq.LINE32)
        assert_same_bytes(g3.scales, ss, f"{name} stochastic line scales, layout {layout}")
        assert_same_bytes(g3.codes, sc, f"{name} stochastic line codes, layout {layout}")
    oc, osc = oracle.cbf_im2col(d, fmts[0], *oq[0], LINE)
    ic, isc = mq.cbf_im2col(d, gq[0])
    assert_same_bytes(isc, osc, f"{name} line im2col scales")
    assert_same_bytes(ic, oc, f"{name} line im2col codes")
    check_fwd(d, fmts, oq, gq)


def test_line_blocks_differ_from_square_blocks_and_cannot_run_backward():
    """A tile whose rows sit in different binades gets different scales per line; the two backward GEMMs refuse line
    blocks (their contraction runs across the lines), as does a mix of block shapes."""
    d = inputs.conv_desc(64, 64, 8, 8, 64, 3, 1, 1)
    x = inputs.make_x(d, 3, "gauss") * np.ldexp(1.0, np.arange(64) % 7 - 3).astype(np.float32)[:, None, None, None]
    w, g = inputs.make_w(d, 3), inputs.make_dy(d, 3, "gauss")
    xl = mq.quantize(d, mq.ROLE_X, E4M3, dev(x), block=mq.LINE32)
    xt = mq.quantize(d, mq.ROLE_X, E4M3, dev(x))
    assert xl.scales.numel() == 32 * xt.scales.numel()
    assert len(torch.unique(xl.scales)) > len(torch.unique(xt.scales))
    wl = mq.quantize(d, mq.ROLE_W, E4M3, dev(w), block=mq.LINE32)
    wt = mq.quantize(d, mq.ROLE_W, E4M3, dev(w))
    gl = mq.quantize(d, mq.ROLE_DY, E5M2, dev(g), block=mq.LINE32)
    for call in (lambda: mq.conv_bwd_data(d, wl, gl), lambda: mq.conv_bwd_weight(d, xl, gl), lambda: mq.conv_fwd(d, xl, wt),
                 lambda: mq.conv_fwd(d, xt, wl)):
        with pytest.raises(mq.MqError) as e:
            call()
        assert e.value.status == 2   # MQ_ERR_UNSUPPORTED


@pytest.mark.parametrize("name", ["cfg5_e4m3_k3s1_c256_hw28", "cfg5_e2m1_k3s2_c256_hw28", "config2"])
def test_line_blocks_at_workload_size(name):
    """Line-block quantizer, im2col and forward GEMM at the size of the benchmark's accounting run (every quantized byte,
    the whole im2col, sampled outputs)."""
    import bench
    layer = bench.workloads()[name]
    d = layer.desc
    fmts = (layer.fmt_x, layer.fmt_w)
    x, w, _ = inputs.layer_tensors(layer)
    oq = [oracle.quantize(d, r, f, t, LINE) for r, f, t in zip((oracle.ROLE_X, oracle.ROLE_W), fmts, (x, w))]
    gq = [mq.quantize(d, r, f, dev(t), block=mq.LINE32) for r, f, t in zip((mq.ROLE_X, mq.ROLE_W), fmts, (x, w))]
    for what, g, (c, s) in zip(("X", "W"), gq, oq):
        assert_same_bytes(g.scales, s, f"{name} {what} line scales")
        assert_same_bytes(g.codes, c, f"{name} {what} line codes")
    oc, osc = oracle.cbf_im2col(d, fmts[0], *oq[0], LINE)
    ic, isc = mq.cbf_im2col(d, gq[0])
    assert_same_bytes(isc, osc, f"{name} line im2col scales")
    assert_same_bytes(ic, oc, f"{name} line im2col codes")
    del oc, osc, ic, isc
    check_fwd(d, fmts, oq, gq, samples=5000)
