"""Packed 6-bit storage (MQ_E3M2_P6 / MQ_E2M3_P6): the 6-bit element formats at the six bits per element Sec. VI counts
for them - 16 codes in 12 bytes.  The stored tensor must be the packing (oracle.pack6: one little-endian bit stream) of
the oracle's one-code-per-byte tensor, from every quantizer kernel; im2col must gather the packed rows; the three GEMMs
must give, bit for bit, what they give on the one-code-per-byte tensors (same codes, same kernels), which in turn are
checked against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import GEMM_TOL, ROLES, assert_gemm_close, assert_same_bytes, dev, host

pytestmark = pytest.mark.gpu

PACKED = {mq.E3M2: mq.E3M2_P6, mq.E2M3: mq.E2M3_P6}

SHAPES = [
    ("ragged", (40, 48, 6, 6, 70, 3, 1, 1)),            # two channel tiles (rows of 48 bytes), ragged sample and channel tiles
    ("one_tile", (33, 20, 5, 7, 24, 3, 2, 1)),          # one channel tile: rows of 24 bytes (8-byte chunks in im2col), stride 2
    ("odd_tiles", (64, 96, 8, 8, 160, 1, 1, 0)),        # three / five channel tiles, 1x1
    ("tc_c256", (48, 256, 6, 7, 256, 3, 1, 1)),         # the tensor-core routes (forward, input gradient, weight gradient)
    ("tc_c128_s2", (40, 128, 9, 10, 128, 3, 2, 1)),     # stride 2: the weights of the input gradient are re-laid from a one-byte copy
]


def check_stored(name, g, codes, scales):
    assert_same_bytes(g.scales, scales, f"{name}: scales")
    assert g.codes.numel() == codes.size * 3 // 4, (name, g.codes.numel(), codes.size)
    assert_same_bytes(g.codes, oracle.pack6(codes), f"{name}: packed codes")


@pytest.mark.parametrize("fmt", [mq.E3M2, mq.E2M3], ids=["e3m2", "e2m3"])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_quantizers_and_im2col(knobs, name, shape, fmt):
    d = inputs.conv_desc(*shape)
    src = (inputs.make_x(d, 91, "relu"), inputs.make_w(d, 91), inputs.make_dy(d, 91, "small"))
    pf = PACKED[fmt]
    oq = [oracle.quantize(d, r, fmt, t) for r, t in zip(ROLES, src)]
    for what, r, t, o in zip(("X", "W", "dY"), ROLES, src, oq):
        check_stored(f"{name} {what}", mq.quantize(d, r, pf, dev(t)), *o)
    # channel-fastest source (the layout the convolution calls emit when layers chain)
    cl = (src[0].transpose(2, 3, 0, 1), src[1].transpose(0, 2, 3, 1), src[2].transpose(2, 3, 0, 1))
    for what, r, t, o in zip(("X", "W", "dY"), ROLES, cl, oq):
        check_stored(f"{name} {what} from channel-fastest source", mq.quantize(d, r, pf, dev(t), src_layout=mq.HWNC), *o)
    # the whole-line TMA kernel (large NCHW tensors), forced on this small one; line blocks; stochastic rounding
    knobs(MQ_QUANT_TMA=1)
    for what, r, t, o in zip(("X", "dY"), (mq.ROLE_X, mq.ROLE_DY), (src[0], src[2]), (oq[0], oq[2])):
        check_stored(f"{name} {what} whole-line kernel", mq.quantize(d, r, pf, dev(t)), *o)
    ol = oracle.quantize(d, oracle.ROLE_X, fmt, src[0], (1, 32))
    check_stored(f"{name} X line blocks, whole-line kernel", mq.quantize(d, mq.ROLE_X, pf, dev(src[0]), block=mq.LINE32), *ol)
    knobs(MQ_QUANT_TMA=0)
    check_stored(f"{name} X line blocks", mq.quantize(d, mq.ROLE_X, pf, dev(src[0]), block=mq.LINE32), *ol)
    osr = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, src[2], 77)
    check_stored(f"{name} dY stochastic", mq.quantize_sr(d, mq.ROLE_DY, pf, dev(src[2]), 77), *osr)
    # im2col gathers the packed rows
    xq = mq.quantize(d, mq.ROLE_X, pf, dev(src[0]))
    oc, osc = oracle.cbf_im2col(d, fmt, oq[0][0], oq[0][1])
    ic, isc = mq.cbf_im2col(d, xq)
    assert_same_bytes(isc, osc, f"{name} im2col scales")
    assert_same_bytes(ic, oracle.pack6(oc), f"{name} im2col packed codes")
    assert mq.last_device_status() == 0


@pytest.mark.parametrize("fmts", [(mq.E3M2, mq.E4M3, mq.E5M2), (mq.E2M3, mq.E2M3, mq.E2M3), (mq.E4M3, mq.E3M2, mq.E2M3)], ids=["plus", "six", "mixed"])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_gemms_match_the_one_code_per_byte_tensors(name, shape, fmts):
    d = inputs.conv_desc(*shape)
    src = (inputs.make_x(d, 92, "relu"), inputs.make_w(d, 92), inputs.make_dy(d, 92, "gauss"))
    pf = tuple(PACKED.get(f, f) for f in fmts)
    qu = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip(ROLES, fmts, src)]
    qp = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip(ROLES, pf, src)]
    for layout in (mq.NCHW, mq.HWNC):
        for what, fn, a, b in (("fwd", mq.conv_fwd, 0, 1), ("bwd_data", mq.conv_bwd_data, 1, 2), ("bwd_weight", mq.conv_bwd_weight, 0, 2)):
            want = fn(d, qu[a], qu[b], layout=layout)
            got = fn(d, qp[a], qp[b], layout=layout)
            assert torch.equal(got, want), (name, what, layout, float((got - want).abs().max()))
    # and against the oracle on the packed tensors, channel-first output
    oq = [oracle.quantize(d, r, f, t) for r, f, t in zip(ROLES, fmts, src)]
    xh, wh, gh = [oracle.dequant(d, r, f, o[0], o[1]) for r, f, o in zip(ROLES, fmts, oq)]
    ref, ab = oracle.conv_fwd(d, xh, wh)
    assert_gemm_close(mq.conv_fwd(d, qp[0], qp[1]), ref, ab, f"{name} fwd", GEMM_TOL)
    ref, ab = oracle.conv_bwd_data(d, wh, gh)
    assert_gemm_close(mq.conv_bwd_data(d, qp[1], qp[2]), ref, ab, f"{name} bwd_data", GEMM_TOL)
    ref, ab = oracle.conv_bwd_weight(d, gh, xh)
    assert_gemm_close(mq.conv_bwd_weight(d, qp[0], qp[2]), ref, ab, f"{name} bwd_weight", GEMM_TOL)
    assert mq.last_device_status() == 0


def test_cuda_core_routes_and_static_scratch(knobs):
    """Layers the tensor-core kernels do not take (forced here) read one-byte copies of packed operands from the call's scratch;
    the call on the library's static scratch accepts packed tensors like the ordinary one."""
    d = inputs.conv_desc(40, 48, 6, 6, 70, 3, 1, 1)
    src = (inputs.make_x(d, 94, "relu"), inputs.make_w(d, 94), inputs.make_dy(d, 94, "gauss"))
    fmts = (mq.E3M2, mq.E2M3, mq.E2M3)
    qu = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip(ROLES, fmts, src)]
    qp = [mq.quantize(d, r, PACKED[f], dev(t)) for r, f, t in zip(ROLES, fmts, src)]
    assert torch.equal(mq.conv_bwd_data_static(d, qp[1], qp[2]), mq.conv_bwd_data(d, qu[1], qu[2]))
    knobs(MQ_TC_NO_FP6=1)
    for what, fn, a, b in (("fwd", mq.conv_fwd, 0, 1), ("bwd_data", mq.conv_bwd_data, 1, 2), ("bwd_weight", mq.conv_bwd_weight, 0, 2)):
        n0 = mq.kernel_launch_count()
        want = fn(d, qu[a], qu[b])
        n1 = mq.kernel_launch_count()
        got = fn(d, qp[a], qp[b])
        n2 = mq.kernel_launch_count()
        assert torch.equal(got, want), (what, float((got - want).abs().max()))
        assert n2 - n1 == n1 - n0 + 2, (what, n1 - n0, n2 - n1)     # the two one-byte copies
    assert mq.last_device_status() == 0


def test_calls_that_do_not_take_packed_storage():
    d = inputs.conv_desc(32, 64, 6, 6, 64, 3, 1, 1)
    x, w = dev(inputs.make_x(d, 93, "relu")), dev(inputs.make_w(d, 93))
    xq, wq = mq.quantize(d, mq.ROLE_X, mq.E3M2_P6, x), mq.quantize(d, mq.ROLE_W, mq.E4M3, w)
    with pytest.raises(mq.MqError) as e:
        mq.conv_fwd_mx(d, xq, wq, mq.E4M3, mq.ACT_RELU)
    assert e.value.status == 2
    xu = mq.quantize(d, mq.ROLE_X, mq.E3M2, x)
    with pytest.raises(mq.MqError) as e:
        mq.conv_fwd_mx(d, xu, wq, mq.E3M2_P6, mq.ACT_RELU)
    assert e.value.status == 2
