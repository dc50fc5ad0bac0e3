"""The paper's own number format (Sec. III-A, Eq. 4-6: fp32 scale per tensor, E4M3 scale per 16 x 16 block, E2M1
elements; MQ_BLOCK_TS16) on the CUDA path against the CPU oracle, through the C ABI (needs a B200): quantizer (both source
layouts, own and supplied tensor maximum, stochastic rounding), im2col and the three GEMMs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import GEMM_TOL, assert_gemm_close, assert_same_bytes, check_large_layer, dev, host

pytestmark = pytest.mark.gpu

B16 = (16, 16)
ROLES = (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY)
SHAPES = [
    ("ragged", (40, 48, 5, 6, 70, 3, 1, 1)),          # 30 positions (scalar loads), ragged rows and channels
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),
    ("stride2", (33, 64, 9, 11, 40, 3, 2, 1)),
    ("k1", (36, 40, 6, 8, 72, 1, 1, 0)),
    ("few_samples", (5, 20, 8, 8, 24, 3, 1, 1)),
    ("wide", (32, 256, 4, 8, 288, 3, 1, 1)),
    # layers whose forward and input-gradient GEMMs run on the tensor cores (K a multiple of 64 elements)
    ("tc_c256", (48, 256, 6, 7, 256, 3, 1, 1)),       # 128-byte chunks, 256-channel tiles, three 16-sample blocks
    ("tc_c128_s2", (40, 128, 9, 10, 128, 3, 2, 1)),   # 64-byte chunks, stride 2 (parity classes of the input gradient)
    ("tc_c64_k1", (150, 64, 5, 4, 192, 1, 1, 0)),     # 32-byte chunks (four per stage), 1x1, ragged sample tile
    ("tc_c512_k1", (32, 512, 3, 4, 512, 1, 1, 0)),    # two 128-byte chunks per tap
    ("tc_n96", (96, 64, 6, 5, 128, 3, 1, 1)),         # three 32-sample tiles: the weight gradient's per-pixel mode (four K-blocks per pixel)
    ("tc_n24", (24, 128, 5, 5, 64, 3, 1, 1)),         # fewer than 32 samples: a half-empty sample tile
    ("tc_c512_pairs", (32, 512, 4, 8, 512, 3, 1, 1)), # 256-column tiles in pairs of blocks (each loads half of the weight tile)
]


def assert_ts_equal(name, g, o):
    codes, scales, ts, amax = o
    stats = host(g.tensor_scale)
    assert stats[1] == np.float32(amax), (name, stats, amax)
    assert stats[0] == np.float32(ts), (name, stats, ts)
    assert_same_bytes(g.scales, scales, f"{name} block scales")
    assert_same_bytes(g.codes, codes, f"{name} codes")


@pytest.mark.parametrize("kinds", [("relu", "small"), ("gauss", "gauss")], ids=["relu-small", "gauss"])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_quantizer_im2col_and_gemms(name, shape, kinds):
    d = inputs.conv_desc(*shape)
    src = (inputs.make_x(d, 71, kinds[0]), inputs.make_w(d, 71), inputs.make_dy(d, 71, kinds[1]))
    oq = [oracle.quantize_ts(d, r, t, B16) for r, t in zip(ROLES, src)]
    gq = [mq.quantize_ts(d, r, dev(t)) for r, t in zip(ROLES, src)]
    for what, g, o in zip(("X", "W", "dY"), gq, oq):
        assert_ts_equal(f"{name} {what}", g, o)
    # mq_quantize on such a destination is the same call; the channel-fastest source gives the same stored tensor
    g2 = mq.quantize(d, mq.ROLE_X, mq.E2M1, dev(src[0]), block=mq.TS16)
    assert_ts_equal(f"{name} X via mq_quantize", g2, oq[0])
    cl = (np.ascontiguousarray(src[0].transpose(2, 3, 0, 1)), np.ascontiguousarray(src[1].transpose(0, 2, 3, 1)), np.ascontiguousarray(src[2].transpose(2, 3, 0, 1)))
    for what, r, t, o in zip(("X", "W", "dY"), ROLES, cl, oq):
        assert_ts_equal(f"{name} {what} from channel-fastest source", mq.quantize_ts(d, r, dev(t), src_layout=mq.HWNC), o)
    # im2col: codes and block scales gathered; the tensor scale is the activation's
    oc, osc = oracle.cbf_im2col(d, oracle.E2M1, oq[0][0], oq[0][1], B16)
    ic, isc = mq.cbf_im2col(d, gq[0])
    assert_same_bytes(isc, osc, f"{name} im2col block scales")
    assert_same_bytes(ic, oc, f"{name} im2col codes")
    # the three GEMMs on the fake-quantized tensors
    xh, wh, gh = [oracle.dequant_ts(d, r, o[0], o[1], o[2], B16) for r, o in zip(ROLES, oq)]
    for layout in (mq.NCHW, mq.HWNC):
        y = mq.conv_fwd(d, gq[0], gq[1], layout=layout)
        ref, ab = oracle.conv_fwd(d, xh, wh)
        assert_gemm_close((y if layout == mq.NCHW else y.permute(2, 3, 0, 1)).contiguous(), ref, ab, f"{name} fwd layout {layout}", GEMM_TOL)
        dx = mq.conv_bwd_data(d, gq[1], gq[2], layout=layout)
        ref, ab = oracle.conv_bwd_data(d, wh, gh)
        assert_gemm_close((dx if layout == mq.NCHW else dx.permute(2, 3, 0, 1)).contiguous(), ref, ab, f"{name} bwd_data layout {layout}", GEMM_TOL)
        dw = mq.conv_bwd_weight(d, gq[0], gq[2], layout=layout)
        ref, ab = oracle.conv_bwd_weight(d, gh, xh)
        assert_gemm_close((dw if layout == mq.NCHW else dw.permute(0, 3, 1, 2)).contiguous(), ref, ab, f"{name} bwd_weight layout {layout}", GEMM_TOL)
    assert mq.last_device_status() == 0


@pytest.mark.parametrize("name,shape", [("aligned", (64, 96, 8, 8, 64, 3, 1, 1)), ("ragged", (40, 48, 6, 6, 70, 3, 1, 1)),
                                        ("few_samples", (5, 20, 8, 8, 24, 3, 1, 1)), ("wide", (33, 256, 4, 8, 288, 3, 1, 1))],
                         ids=["aligned", "ragged", "few_samples", "wide"])
def test_whole_line_quantizer(knobs, name, shape):
    """Large NCHW tensors take the second pass on the whole-line TMA kernel (items of 32 positions x 32 samples x 32
    channels, four 16 x 16 blocks per position); forced here on small shapes: same bytes as the oracle, own and
    supplied maximum, stochastic rounding."""
    knobs(MQ_QUANT_TMA=1)
    d = inputs.conv_desc(*shape)
    src = (inputs.make_x(d, 81, "relu"), inputs.make_dy(d, 81, "small"))
    for what, r, t in zip(("X", "dY"), (mq.ROLE_X, mq.ROLE_DY), src):
        o = oracle.quantize_ts(d, r, t, B16)
        assert_ts_equal(f"{name} {what}", mq.quantize_ts(d, r, dev(t)), o)
        amax = np.float32(1.7) * np.abs(t).max()
        o2 = oracle.quantize_ts(d, r, t, B16, amax=float(amax))
        amax_dev, t_dev = torch.tensor([amax], dtype=torch.float32, device="cuda"), dev(t)
        n0 = mq.kernel_launch_count()
        g2 = mq.quantize_ts(d, r, t_dev, amax_in=amax_dev)
        n1 = mq.kernel_launch_count()
        assert_same_bytes(g2.scales, o2[1], f"{name} {what} supplied maximum: block scales")
        assert_same_bytes(g2.codes, o2[0], f"{name} {what} supplied maximum: codes")
        # a supplied maximum makes it ONE launch that still records the tensor's own maximum for the next step
        assert n1 - n0 == 1, (name, what, n1 - n0)
        st = host(g2.tensor_scale)
        assert st[1] == np.abs(t).max() and st[0] == np.float32(o2[2]), (name, what, st)
        o3 = oracle.quantize_ts(d, r, t, B16, seed=99)
        g3 = mq.quantize_ts(d, r, dev(t), seed=99)
        assert_same_bytes(g3.scales, o3[1], f"{name} {what} stochastic: block scales")
        assert_same_bytes(g3.codes, o3[0], f"{name} {what} stochastic: codes")
    assert mq.last_device_status() == 0


@pytest.mark.parametrize("name", ["cfg5_e2m1_k3s1_c512_hw28", "cfg5_e2m1_k3s2_c512_hw28", "cfg5_e2m1_k1s1_c512_hw28", "cfg5_e2m1_k3s1_c256_hw56",
                                  "cfg5_e2m1_k3s1_c512_hw56"])
def test_config5_points_full_size(name):
    """The points `bench.py` times in this format ('<layer>+ts16'), on the GPU at full size; the oracle checks sample slabs,
    channel blocks and W with the whole tensor's maximum supplied (see check_large_layer)."""
    check_large_layer({l.name: l for l in inputs.config5()}[name], block=mq.TS16)


def test_tensor_core_and_cuda_core_routes_agree(knobs):
    """The forward and input-gradient GEMMs of this format run on the tensor cores where the layer allows it
    (kind::mxf4nvf4: E4M3 scales per 16 elements in tensor memory, the tensors' fp32 scales applied to the accumulator)
    and on the CUDA-core kernels elsewhere; the same layer through both routes."""
    d = inputs.conv_desc(48, 128, 7, 6, 192, 3, 1, 1)
    src = (inputs.make_x(d, 75, "gauss"), inputs.make_w(d, 75), inputs.make_dy(d, 75, "gauss"))
    gq = [mq.quantize_ts(d, r, dev(t)) for r, t in zip(ROLES, src)]
    n0 = mq.kernel_launch_count()
    y_tc, dx_tc = mq.conv_fwd(d, gq[0], gq[1]), mq.conv_bwd_data(d, gq[1], gq[2])
    n_tc = mq.kernel_launch_count() - n0
    knobs(MQ_TC_NO_TS16=1)
    n0 = mq.kernel_launch_count()
    y_cc, dx_cc = mq.conv_fwd(d, gq[0], gq[1]), mq.conv_bwd_data(d, gq[1], gq[2])
    n_cc = mq.kernel_launch_count() - n0
    assert mq.last_device_status() == 0
    assert n_tc == 4 and n_cc == 2, (n_tc, n_cc)      # scale expansion + GEMM per call against one CUDA-core kernel per call
    oq = [oracle.quantize_ts(d, r, t, B16) for r, t in zip(ROLES, src)]
    xh, wh, gh = [oracle.dequant_ts(d, r, o[0], o[1], o[2], B16) for r, o in zip(ROLES, oq)]
    ref, ab = oracle.conv_fwd(d, xh, wh)
    assert_gemm_close(y_tc, ref, ab, "fwd tensor cores", GEMM_TOL)
    assert_gemm_close(y_cc, ref, ab, "fwd CUDA cores", GEMM_TOL)
    ref, ab = oracle.conv_bwd_data(d, wh, gh)
    assert_gemm_close(dx_tc, ref, ab, "bwd_data tensor cores", GEMM_TOL)
    assert_gemm_close(dx_cc, ref, ab, "bwd_data CUDA cores", GEMM_TOL)
    # the weight gradient: contraction over the samples, the second direction of the same 16 x 16 blocks
    n0 = mq.kernel_launch_count()
    dw_cc = mq.conv_bwd_weight(d, gq[0], gq[2])
    n_cc = mq.kernel_launch_count() - n0
    knobs(MQ_TC_NO_TS16=0)
    n0 = mq.kernel_launch_count()
    dw_tc = mq.conv_bwd_weight(d, gq[0], gq[2])
    n_tc = mq.kernel_launch_count() - n0
    assert mq.last_device_status() == 0
    assert n_cc == 2 and n_tc > 2, (n_cc, n_tc)       # CUDA cores: GEMM + reduction; tensor cores: re-layout / scale expansion launches as well
    ref, ab = oracle.conv_bwd_weight(d, gh, xh)
    assert_gemm_close(dw_tc, ref, ab, "bwd_weight tensor cores", GEMM_TOL)
    assert_gemm_close(dw_cc, ref, ab, "bwd_weight CUDA cores", GEMM_TOL)


def test_tensor_maximum_from_an_earlier_step_and_stochastic_rounding():
    d = inputs.conv_desc(64, 96, 8, 8, 64, 3, 1, 1)
    g0, g1 = inputs.make_dy(d, 81, "gauss"), inputs.make_dy(d, 82, "gauss") * np.float32(1.7)
    q0 = mq.quantize_ts(d, mq.ROLE_DY, dev(g0))
    # step 2 quantizes with step 1's maximum (smaller than its own: the top saturates) and leaves its own maximum behind
    q1 = mq.quantize_ts(d, mq.ROLE_DY, dev(g1), amax_in=q0.tensor_scale[1:2])
    o1 = oracle.quantize_ts(d, oracle.ROLE_DY, g1, B16, amax=float(np.abs(g0).max()))
    assert_ts_equal("supplied maximum", q1, o1)
    assert host(q1.tensor_scale)[1] == np.abs(g1).max()
    # stochastic Round(.), same draws on both sides
    for seed in (3, 0xABCDEF0123456789):
        qs = mq.quantize_ts(d, mq.ROLE_DY, dev(g0), seed=seed)
        assert_ts_equal(f"stochastic seed {seed}", qs, oracle.quantize_ts(d, oracle.ROLE_DY, g0, B16, seed=seed))


def test_edge_values_and_argument_checks():
    d = inputs.conv_desc(32, 32, 4, 4, 32, 1, 1, 0)
    rng = np.random.default_rng(9)
    x = rng.standard_normal((32, 32, 4, 4)).astype(np.float32)
    x[:16, :16, 0, 0] = 0.0                       # an empty block
    x[0, 0, 0, 0] = -0.0
    x[:16, 16:, 0, 1] *= np.float32(1e-6)         # a block whose scale rounds to zero
    x[16:, :16, 0, 2] = np.float32(0.75) * rng.choice([0.5, 1.5, 2.5, 3.5, 5.0, -5.0], (16, 16)).astype(np.float32)   # ties
    x[5, 7, 3, 3] = 900.0                         # the tensor maximum
    assert_ts_equal("edge values", mq.quantize_ts(d, mq.ROLE_X, dev(x)), oracle.quantize_ts(d, oracle.ROLE_X, x, B16))
    z = np.zeros_like(x)
    assert_ts_equal("zero tensor", mq.quantize_ts(d, mq.ROLE_X, dev(z)), oracle.quantize_ts(d, oracle.ROLE_X, z, B16))
    # element format must be E2M1 and a tensor-scale buffer must be given; operands of a GEMM must share the block type
    bad = mq.empty_qtensor(d, mq.ROLE_X, mq.E2M1, block=mq.TS16)
    bad.fmt = mq.E4M3
    with pytest.raises(mq.MqError) as e:
        mq.quantize(d, mq.ROLE_X, mq.E4M3, dev(x), out=bad)
    assert e.value.status == 1
    nots = mq.empty_qtensor(d, mq.ROLE_X, mq.E2M1, block=mq.TS16)
    nots.tensor_scale = None
    with pytest.raises(mq.MqError) as e:
        mq.quantize(d, mq.ROLE_X, mq.E2M1, dev(x), out=nots)
    assert e.value.status == 1
    xq = mq.quantize_ts(d, mq.ROLE_X, dev(x))
    wq = mq.quantize(d, mq.ROLE_W, mq.E2M1, dev(inputs.make_w(d, 1)))
    with pytest.raises(mq.MqError) as e:
        mq.conv_fwd(d, xq, wq)
    assert e.value.status == 2
