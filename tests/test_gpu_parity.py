"""Parity of the CUDA path with the CPU oracle, through the C ABI (needs a B200).

Small cases span several tiles and ragged tails in every dimension; the workload cases run the
benchmark's configurations at full size and compare every quantized byte and sampled GEMM
outputs (all outputs where the oracle finishes in seconds)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import (OracleLayer, assert_gemm_close, assert_same_bytes, check_convs, check_im2col, check_large_layer, check_quantize, dev,
                         gpu_quantize_layer)

pytestmark = pytest.mark.gpu

E4M3, E5M2, E2M1, E3M2, E2M3 = mq.E4M3, mq.E5M2, mq.E2M1, mq.E3M2, mq.E2M3
FMT_SETS = [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1), (E5M2, E4M3, E4M3), (E2M1, E4M3, E5M2),
            (E3M2, E4M3, E5M2), (E2M3, E2M3, E2M3), (E3M2, E2M3, E3M2)]   # the 6-bit formats: MicroQonv+ activations, "-6", mixed


def make_layer(name, desc, fmts, seed, kinds=("relu", "kaiming", "small")):
    return inputs.Layer(name, desc, fmts[0], fmts[1], fmts[2], kinds[0], kinds[1], kinds[2], seed)


SMALL_SHAPES = [
    # N, C_in, H, W, C_out, K, stride, pad
    ("ragged", (40, 48, 5, 6, 70, 3, 1, 1)),       # P = 30 (scalar loads), ragged N, C_in, C_out
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),      # vector loads, whole tiles
    ("stride2", (33, 64, 9, 11, 40, 3, 2, 1)),     # odd image, stride 2
    ("k1", (36, 40, 6, 6, 72, 1, 1, 0)),           # 1x1
    ("k1s2", (32, 32, 8, 8, 32, 1, 2, 0)),         # 1x1 stride 2
    ("k1_w8", (40, 128, 6, 8, 160, 1, 1, 0)),      # 1x1 with rows of whole 16-byte units: staged stores, clipped channel tile and samples
    ("k5", (8, 16, 12, 12, 24, 5, 2, 2)),          # 5x5, C < 32
    ("nopad", (16, 32, 7, 7, 32, 3, 1, 0)),        # no padding
    ("rect", (4, 35, 6, 10, 33, 3, 1, 1)),
    ("thin_wide", (16, 32, 6, 8, 160, 3, 1, 1)),   # thin contraction, two output-channel tiles (weight tile reloaded) in fwd
    ("wide_thin", (16, 160, 6, 8, 32, 3, 1, 1)),   # the same situation in the input gradient
    ("wide", (32, 256, 4, 8, 288, 3, 1, 1)),       # 256-channel MMAs (8-bit) and a remainder channel tile
    ("deep_batch", (250, 320, 3, 4, 288, 3, 1, 1)),  # 8 sample tiles (ragged): E2M1 whole-line re-layout with partial channel groups, block pairs
    ("thin_n70", (70, 48, 5, 6, 40, 3, 1, 1)),       # thin layer, three sample tiles in one four-block K stage (one pixel per stage)
    ("stem7", (8, 3, 20, 20, 24, 7, 2, 3)),          # 7x7 stride-2 stem on 3 channels: seven taps of 32 bytes as one weight-gradient operand
    ("batch16", (16, 40, 10, 12, 72, 3, 1, 1)),      # at most 16 samples: quantizer items of 16 positions (120 positions: partial last item)
    ("shared_rows", (70, 128, 5, 6, 256, 3, 1, 1)),  # 128-byte K chunks, unit strides: activation-side scale chunks shared across output rows (ragged N, W)
]


@pytest.mark.parametrize("fmts", FMT_SETS, ids=lambda f: "-".join(map(str, f)))
@pytest.mark.parametrize("name,shape", SMALL_SHAPES, ids=[s[0] for s in SMALL_SHAPES])
def test_small_layers_all_steps(name, shape, fmts):
    d = inputs.conv_desc(*shape)
    ol = OracleLayer(make_layer(name, d, fmts, seed=100 + len(name), kinds=("relu", "kaiming", "gauss")))
    qs = check_quantize(ol)
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=None, layouts=(mq.NCHW, mq.HWNC))


@pytest.mark.parametrize("fmt", [E4M3, E5M2, E2M1])
@pytest.mark.parametrize("shape", [(40, 48, 5, 6, 70, 3, 1, 1), (64, 96, 8, 8, 64, 3, 1, 1), (33, 35, 6, 7, 34, 3, 2, 1)],
                         ids=["ragged", "aligned", "odd-channels"])
def test_quantize_channel_fastest_source(shape, fmt):
    """The same logical tensors handed over as fp32 [H][W][N][C] / [Cout][Kh][Kw][Cin] give the oracle's stored bytes."""
    d = inputs.conv_desc(*shape)
    ol = OracleLayer(make_layer("hwnc_src", d, (fmt, fmt, fmt), seed=7, kinds=("relu", "kaiming", "gauss")))
    x, w, g = ol.src
    srcs = (np.ascontiguousarray(x.transpose(2, 3, 0, 1)), np.ascontiguousarray(w.transpose(0, 2, 3, 1)), np.ascontiguousarray(g.transpose(2, 3, 0, 1)))
    for role, name, src, (c, s_) in zip((0, 1, 2), ("X", "W", "dY"), srcs, ol.q):
        q = mq.quantize(d, role, fmt, torch.from_numpy(src).cuda(), src_layout=mq.HWNC)
        assert_same_bytes(q.scales, s_, f"{name} scales from channel-fastest source")
        assert_same_bytes(q.codes, c, f"{name} codes from channel-fastest source")


@pytest.mark.parametrize("fmt", [E4M3, E5M2, E2M1])
def test_quantize_edge_values(fmt):
    """Zero tiles, -0, ties, saturation, huge and tiny magnitudes, fp32 subnormals."""
    d = inputs.conv_desc(64, 64, 4, 4, 32, 1, 1, 0)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((64, 64, 4, 4)).astype(np.float32)
    x[:32, :32, 0, 0] = 0.0
    x[0, 0, 0, 0] = -0.0
    x[:32, 32:, 0, 1] = np.float32(1.5) * rng.choice([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 7.0, -7.9], (32, 32)).astype(np.float32)
    x[32:, :32, 0, 2] *= np.float32(1e30)
    x[32:, 32:, 0, 3] *= np.float32(1e-30)
    x[:32, :32, 1, 0] = rng.standard_normal((32, 32)).astype(np.float32) * np.float32(1e-41)  # subnormal inputs
    x[:32, :32, 1, 1] = np.ldexp(rng.standard_normal((32, 32)), rng.integers(-20, 20, (32, 32))).astype(np.float32)
    x[:32, :32, 1, 2] = np.float32(3.4e38)
    x[:32, 32:, 1, 3] = np.float32(448.0)
    oc, osc = oracle.quantize(d, oracle.ROLE_X, fmt, x)
    q = mq.quantize(d, mq.ROLE_X, fmt, dev(x))
    assert_same_bytes(q.scales, osc, "scales")
    assert_same_bytes(q.codes, oc, "codes")


@pytest.mark.parametrize("fmts", [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1)], ids=["fp8", "fp4"])
def test_small_integer_inputs_are_exact_on_gpu(fmts):
    """Integers in {-2..2} are exact in every format: the GPU GEMMs must equal the oracle exactly,
    which isolates indexing and scale routing from rounding."""
    d = inputs.conv_desc(33, 35, 6, 7, 34, 3, 2, 1)
    ol = OracleLayer(make_layer("smallint", d, fmts, 23, ("smallint",) * 3))
    qs = check_quantize(ol)
    xh, wh, gh = ol.hat
    y, _ = oracle.conv_fwd(d, xh, wh)
    gx, _ = oracle.conv_bwd_data(d, wh, gh)
    gw, _ = oracle.conv_bwd_weight(d, gh, xh)
    assert np.array_equal(mq.conv_fwd(d, qs[0], qs[1]).cpu().numpy().astype(np.float64), y)
    assert np.array_equal(mq.conv_bwd_data(d, qs[1], qs[2]).cpu().numpy().astype(np.float64), gx)
    assert np.array_equal(mq.conv_bwd_weight(d, qs[0], qs[2]).cpu().numpy().astype(np.float64), gw)


def test_config1_full_parity():
    (layer,) = inputs.config1()
    ol = OracleLayer(layer)
    qs = check_quantize(ol)
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=None)


def test_config2_full_size():
    """The benchmark's workload: every quantized byte, the whole im2col, sampled GEMM outputs."""
    (layer,) = inputs.config2()
    ol = OracleLayer(layer)
    qs = check_quantize(ol)
    # what the square-tile reading does to this workload: most tiles hold an outlier, so most
    # ordinary activations round to zero -- the fraction must be what the oracle predicts
    codes = ol.q[0][0]
    nz_oracle = np.count_nonzero(codes & 0x7) + np.count_nonzero((codes >> 4) & 0x7)
    g = qs[0].codes
    nz_gpu = int(torch.count_nonzero(g & 0x7)) + int(torch.count_nonzero((g >> 4) & 0x7))
    assert nz_gpu == nz_oracle
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=20000)


@pytest.mark.parametrize("idx", [0, 1], ids=["3x3", "1x1"])
def test_config4_full_size(idx):
    layer = inputs.config4()[idx]
    ol = OracleLayer(layer)
    qs = check_quantize(ol)
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=8000)


def _cfg3_layers():
    return inputs.config3()


@pytest.mark.parametrize("li", range(24))
def test_config3_layers_full_size(li):
    layer = _cfg3_layers()[li]
    ol = OracleLayer(layer)
    qs = check_quantize(ol)
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=6000)


CFG5_POINTS = ["cfg5_e4m3_k3s1_c64_hw14", "cfg5_e4m3_k3s2_c128_hw28", "cfg5_e4m3_k1s1_c256_hw14", "cfg5_e2m1_k3s1_c128_hw14",
               "cfg5_e2m1_k1s2_c64_hw28", "cfg5_e2m1_k3s2_c256_hw14", "cfg5_e4m3_k3s1_c512_hw14", "cfg5_e4m3_k3s1_c64_hw56",
               "cfg5_e2m1_k3s1_c256_hw14", "cfg5_e4m3_k1s1_c256_hw28"]


@pytest.mark.parametrize("name", CFG5_POINTS)
def test_config5_points_full_size(name):
    layer = {l.name: l for l in inputs.config5()}[name]
    ol = OracleLayer(layer)
    qs = check_quantize(ol)
    check_im2col(ol, qs[0])
    check_convs(ol, qs, samples=4000)


# The large points of the sweep: every (format, kernel, stride) family at 512 channels on 56x56 and 28x28 images, the
# 3x3 families at 256 channels on 56x56.  Tensors reach 1.6 GB of fp32 and 3.7 GB of X' (offsets beyond 2^31 bytes).
CFG5_LARGE = [f"cfg5_{f}_k{k}s{s}_c512_hw{hw}" for f in ("e4m3", "e2m1") for k in (3, 1) for s in (1, 2) for hw in (56, 28)] + \
             [f"cfg5_{f}_k3s{s}_c256_hw56" for f in ("e4m3", "e2m1") for s in (1, 2)]


@pytest.mark.parametrize("name", CFG5_LARGE)
def test_config5_large_points_full_size(name):
    """The GPU runs the point at full size; the oracle checks sample slabs, channel blocks and W (see check_large_layer)."""
    layer = {l.name: l for l in inputs.config5()}[name]
    check_large_layer(layer)


@pytest.mark.parametrize("packed6", [False, True], ids=["one-per-byte", "packed"])
@pytest.mark.parametrize("idx", [0, 1], ids=["e3m2-act", "e2m3"])
def test_fp6_layers_full_size(idx, packed6):
    """The two 6-bit layers the benchmark reports (256 channels, 28x28, N = 256), in both storages of the 6-bit codes."""
    check_large_layer(inputs.fp6_layers()[idx], packed6=packed6)


@pytest.mark.parametrize("slabs", [8, 1, 3], ids=["slabs8", "one_slab", "slabs3"])
@pytest.mark.parametrize("fmts", [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1), (mq.E3M2_P6, E4M3, mq.E2M3_P6)], ids=["fp8", "fp4", "fp6-packed"])
def test_layer_from_host_buffers_matches_the_device_calls(fmts, slabs, knobs):
    """mq_conv_layer_host (pinned host tensors in, host results out, copies overlapped with the kernels, the step run slab by
    slab along the batch) gives, twice in a row, exactly the Y and G_X of the separate device-side calls; G_W is the sum of
    the slabs' weight gradients - exactly the device call's with one slab, within the GEMM bound of the oracle otherwise."""
    knobs(MQ_HOST_SLABS=slabs)
    d = inputs.conv_desc(150, 64, 12, 16, 96, 3, 1, 1)        # five sample tiles, the last ragged
    layer = make_layer("host", d, fmts, seed=11, kinds=("relu", "kaiming", "gauss"))
    x, w, g = inputs.layer_tensors(layer)
    q = [mq.quantize(d, r, f, torch.from_numpy(t).cuda()) for r, f, t in zip((0, 1, 2), fmts, (x, w, g))]
    want = (mq.conv_fwd(d, q[0], q[1]).cpu(), mq.conv_bwd_data(d, q[1], q[2]).cpu(), mq.conv_bwd_weight(d, q[0], q[2]).cpu())
    hx, hw, hg = [torch.from_numpy(t).pin_memory() for t in (x, w, g)]
    outs = [torch.empty(t.shape, dtype=torch.float32).pin_memory() for t in want]
    arena = torch.empty(mq.conv_layer_host_arena_size(d, *fmts), dtype=torch.uint8, device="cuda")
    for _ in range(2):
        for o in outs:
            o.fill_(float("nan"))
        mq.conv_layer_host(d, fmts, hx, hw, hg, outs[0], outs[1], outs[2], arena)
        torch.cuda.synchronize()
        for name, got, exp in zip(("Y", "dX", "dW"), outs, want):
            if name != "dW" or slabs == 1:
                assert torch.equal(got, exp), f"{name} from host buffers differs from the device call"
    if slabs != 1:
        fmts = tuple({mq.E3M2_P6: E3M2, mq.E2M3_P6: E2M3}.get(f, f) for f in fmts)   # (packed storage: the same codes)
        oq = [oracle.quantize(d, r, f, t) for r, f, t in zip((oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY), fmts, (x, w, g))]
        xh, gh = oracle.dequant(d, oracle.ROLE_X, fmts[0], *oq[0]), oracle.dequant(d, oracle.ROLE_DY, fmts[2], *oq[2])
        ref, ab = oracle.conv_bwd_weight(d, gh, xh)
        assert_gemm_close(outs[2], ref, ab, "dW summed over slabs")
    assert mq.last_device_status() == 0


def test_6bit_gemms_on_cuda_cores(knobs):
    """The CUDA-core route of 6-bit operands (the default packs them for the tensor cores; the weight gradient always
    takes this route)."""
    knobs(MQ_TC_NO_FP6="1")
    d = inputs.conv_desc(64, 96, 8, 8, 64, 3, 1, 1)
    for fmts in ((E3M2, E4M3, E5M2), (E2M3, E2M3, E2M3)):
        ol = OracleLayer(make_layer("fp6_cuda_cores", d, fmts, seed=31, kinds=("relu", "kaiming", "gauss")))
        qs = check_quantize(ol)
        check_convs(ol, qs, samples=20000, layouts=(mq.NCHW, mq.HWNC))


ALT_PATHS = [("MQ_TC_NO_HALO", "1"), ("MQ_TC_NO_FUSED", "1"), ("MQ_TC_NO_TMA_STORE", "1"), ("MQ_TC_TMA_STORE", "1"), ("MQ_TC_NO_PAIR", "1"),
             ("MQ_TC_BN", "256"), ("MQ_TC_TW", "4"), ("MQ_TC_TW", "16"), ("MQ_TC_TW", "32"), ("MQ_WGRAD_NO_FLAT", "1"),
             ("MQ_WGRAD_NO_GROUP", "1"), ("MQ_WGRAD_NO_GROUP8", "1"), ("MQ_WGRAD_N128", "1"), ("MQ_WGRAD_NO_CTA2", "1"), ("MQ_TC_NO_MMA_CP", "1"), ("MQ_WGRAD_MMA_CP", "1"), ("MQ_TC_FP4_BN128", "1"), ("MQ_TC_NO_SFA_DEDUP", "1"), ("MQ_TC_NO_WT_FUSED", "1"), ("MQ_WGRAD_FP4_PIXEL", "1"), ("MQ_WGRAD_SPLITS", "3"), ("MQ_DISABLE_TC_WGRAD", "1"), ("MQ_DISABLE_TC", "1"),
             ("MQ_NO_PDL", "1"), ("MQ_QUANT_NO_R16", "1"), ("MQ_QUANT_TMA", "0"), ("MQ_WGRAD_NO_WIDE_PREP", "1"), ("MQ_WGRAD_NO_SFB_DEDUP", "1"), ("MQ_TC_NO_SNAP", "1"), ("MQ_TC_NO_DUO", "1")]
ALT_SHAPES = [("thin", (32, 64, 8, 16, 96, 3, 1, 1)), ("wide_s2", (32, 256, 8, 12, 288, 3, 2, 1)), ("wide_s1", (32, 256, 4, 8, 288, 3, 1, 1)),
              ("thin32_s2", (40, 20, 9, 10, 48, 3, 2, 1))]
# knobs that act on other shapes: at most 16 samples (quantizer items of 16 positions), 256 samples x 256 channels (the wide E2M1
# weight-gradient preparation)
ALT_EXTRA = {"MQ_QUANT_NO_R16": [("batch16", (16, 40, 10, 12, 72, 3, 1, 1))], "MQ_WGRAD_NO_WIDE_PREP": [("n256_c256", (256, 256, 4, 4, 256, 3, 1, 1))],
             "MQ_TC_NO_SNAP": [("c512_bn256", (40, 512, 6, 7, 500, 3, 1, 1))],
             "MQ_TC_NO_DUO": [("c512_pairs", (32, 512, 8, 8, 512, 3, 1, 1))]}


@pytest.mark.parametrize("fmts", [(E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1)], ids=["fp8", "fp4"])
@pytest.mark.parametrize("name,shape", [("c512", (32, 512, 8, 8, 512, 3, 1, 1)), ("c256_ragged", (48, 256, 6, 12, 300, 3, 1, 1))], ids=["c512", "c256_ragged"])
def test_block_pairs_on_256_column_tiles(name, shape, fmts):
    """Forward and input gradient of layers with 256-column tiles, unit strides and an even tile count run as pairs of blocks
    on 256 x 256 tiles (each block loads half of the weight tile): same parity bar, both output layouts."""
    d = inputs.conv_desc(*shape)
    ol = OracleLayer(make_layer(name, d, fmts, seed=29, kinds=("relu", "kaiming", "gauss")))
    qs = check_quantize(ol)
    check_convs(ol, qs, samples=30000, layouts=(mq.NCHW, mq.HWNC), ops=("fwd", "dx"))


@pytest.mark.parametrize("knob", ALT_PATHS, ids=[f"{k}={v}" for k, v in ALT_PATHS])
def test_alternate_kernel_paths(knob, knobs):
    """Every switchable kernel path (per-tap instead of whole-tile, unfused preparation, plain stores, other tile
    shapes, the other weight-gradient modes incl. single blocks where pairs are the default, the CUDA-core kernels) meets the same parity bar."""
    knobs(**{knob[0]: knob[1]})
    for name, shape in ALT_SHAPES + ALT_EXTRA.get(knob[0], []):
        d = inputs.conv_desc(*shape)
        for fmts in ((E4M3, E4M3, E5M2), (E2M1, E2M1, E2M1)):
            ol = OracleLayer(make_layer(name, d, fmts, seed=23, kinds=("relu", "kaiming", "gauss")))
            qs = check_quantize(ol)
            check_convs(ol, qs, samples=20000, layouts=(mq.NCHW, mq.HWNC))


TMA_Q_SHAPES = [
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),          # whole tiles, two strips of 32 positions
    ("ragged_n_c", (40, 48, 6, 6, 70, 3, 1, 1)),       # 36 positions: a partial second strip; ragged rows and channels
    ("few_positions", (250, 320, 3, 4, 288, 3, 1, 1)),  # 12 positions: a box wider than the tensor; 8 row tiles, the last ragged
    ("batch16", (16, 40, 10, 12, 72, 3, 1, 1)),        # two boxes per item
    ("batch5", (5, 16, 10, 10, 24, 3, 1, 1)),          # one box per item, 16 channels, 100 positions
    ("odd_rows", (77, 35, 8, 8, 34, 3, 1, 1)),         # three row tiles, the last of 13 rows (two boxes)
]


@pytest.mark.parametrize("fmt", [E4M3, E5M2, E2M1, E3M2, E2M3])
@pytest.mark.parametrize("name,shape", TMA_Q_SHAPES, ids=[s[0] for s in TMA_Q_SHAPES])
def test_quantize_whole_line_kernel_on_small_shapes(name, shape, fmt, knobs):
    """The whole-line (TMA) quantizer that large NCHW tensors take, forced onto small ragged ones: the oracle's bytes,
    with round-to-nearest and with the stochastic rounding."""
    knobs(MQ_QUANT_TMA="1")
    d = inputs.conv_desc(*shape)
    ol = OracleLayer(make_layer(name, d, (fmt, fmt, fmt), seed=41, kinds=("relu", "kaiming", "gauss")))
    check_quantize(ol)
    g = ol.src[2]
    oc, osc = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, 99)
    q = mq.quantize_sr(d, mq.ROLE_DY, fmt, dev(g), 99)
    assert_same_bytes(q.scales, osc, f"{name} stochastic scales")
    assert_same_bytes(q.codes, oc, f"{name} stochastic codes")
    assert mq.last_device_status() == 0


def test_bounded_waits_give_up_and_the_context_stays_usable():
    """Every device-side wait of the library is bounded.  Here the quantizer's TMA pipeline runs with its loader switched
    off and a limit of a few thousand polls, so each wait runs out: the kernel must return normally with
    MQ_ERR_TIMEOUT in the device status word (read once, then cleared), and the next ordinary call must be correct."""
    d = inputs.conv_desc(64, 96, 8, 8, 64, 3, 1, 1)
    ol = OracleLayer(make_layer("timeout", d, (E4M3, E4M3, E5M2), seed=43, kinds=("relu", "kaiming", "gauss")))
    assert mq.last_device_status() == 0
    mq.selftest_wait_timeout(d, mq.ROLE_X, E4M3, dev(ol.src[0]), polls=2000)
    torch.cuda.synchronize()                      # the kernel has returned: nothing hangs
    assert mq.last_device_status() == 6           # MQ_ERR_TIMEOUT
    assert mq.last_device_status() == 0           # reading it cleared it
    qs = check_quantize(ol)                       # the context is intact
    check_convs(ol, qs, samples=None)
