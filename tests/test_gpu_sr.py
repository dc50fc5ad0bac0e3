"""Parity of the CUDA quantizer's stochastic rounding (the gradient's Round(.) of Eq. 6, Sec. III-A) with the CPU
oracle, through the C ABI (needs a B200).  Both sides implement the same counter-based per-element draw, so codes and
scales must agree bit for bit -- for every kernel variant (16-byte rows, scalar fallback, channel-fastest source),
every element format, edge values, and the benchmark's gradient tensor at full size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import assert_same_bytes, dev

pytestmark = pytest.mark.gpu

E4M3, E5M2, E2M1, E3M2, E2M3 = mq.E4M3, mq.E5M2, mq.E2M1, mq.E3M2, mq.E2M3
SHAPES = [
    ("ragged", (40, 48, 5, 6, 70, 3, 1, 1)),       # 30 positions: scalar-load kernel
    ("aligned", (64, 96, 8, 8, 64, 3, 1, 1)),      # 64 positions: the pipelined kernel, several tiles
    ("stride2", (33, 64, 9, 11, 40, 3, 2, 1)),     # ragged N and C_out
    ("small_batch", (16, 48, 6, 8, 40, 3, 1, 1)),  # at most 16 samples: the 16-positions-per-item variant of the pipelined kernel
    ("tiny_batch", (5, 20, 8, 8, 24, 3, 1, 1)),    # the same with ragged rows, channels and a partial last item
]


@pytest.mark.parametrize("fmt", [E4M3, E5M2, E2M1, E3M2, E2M3])
@pytest.mark.parametrize("name,shape", SHAPES, ids=[s[0] for s in SHAPES])
def test_gradient_codes_match_the_oracle(name, shape, fmt):
    d = inputs.conv_desc(*shape)
    g = inputs.make_dy(d, 31, "gauss")
    for seed in (0, 7, 0xFEDCBA9876543210):
        oc, osc = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, seed)
        q = mq.quantize_sr(d, mq.ROLE_DY, fmt, dev(g), seed)
        assert_same_bytes(q.scales, osc, f"{name} scales seed {seed}")
        assert_same_bytes(q.codes, oc, f"{name} codes seed {seed}")
        # the channel-fastest source gives the same stored tensor: the draw is keyed by the logical index
        q2 = mq.quantize_sr(d, mq.ROLE_DY, fmt, dev(np.ascontiguousarray(g.transpose(2, 3, 0, 1))), seed, src_layout=mq.HWNC)
        assert_same_bytes(q2.codes, oc, f"{name} codes from channel-fastest source seed {seed}")
        assert_same_bytes(q2.scales, osc, f"{name} scales from channel-fastest source seed {seed}")


@pytest.mark.parametrize("fmt", [E4M3, E2M1])
def test_per_element_key_path(fmt, knobs):
    """Tensors of 2^32 elements or more derive the stream key from the index's high word per element; forced here on a
    small tensor (high word 0), where it must give the same bytes."""
    knobs(MQ_SR_WIDE="1")
    d = inputs.conv_desc(64, 96, 8, 8, 64, 3, 1, 1)
    g = inputs.make_dy(d, 8, "gauss")
    oc, osc = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, g, 77)
    for src, layout in ((g, mq.NCHW), (np.ascontiguousarray(g.transpose(2, 3, 0, 1)), mq.HWNC)):
        q = mq.quantize_sr(d, mq.ROLE_DY, fmt, dev(src), 77, src_layout=layout)
        assert_same_bytes(q.codes, oc, "codes")
        assert_same_bytes(q.scales, osc, "scales")


@pytest.mark.parametrize("fmt", [E4M3, E2M1])
def test_every_role_accepts_it(fmt):
    d = inputs.conv_desc(36, 40, 6, 6, 72, 3, 1, 1)
    x, w, g = inputs.make_x(d, 3, "gauss"), inputs.make_w(d, 3), inputs.make_dy(d, 3, "small")
    for role, t in ((mq.ROLE_X, x), (mq.ROLE_W, w), (mq.ROLE_DY, g)):
        oc, osc = oracle.quantize_sr(d, role, fmt, t, 5)
        q = mq.quantize_sr(d, role, fmt, dev(t), 5)
        assert_same_bytes(q.scales, osc, f"role {role} scales")
        assert_same_bytes(q.codes, oc, f"role {role} codes")


@pytest.mark.parametrize("fmt", [E4M3, E5M2, E2M1])
def test_edge_values(fmt):
    """Zero tiles, -0, exact grid values, saturation, huge and tiny magnitudes, fp32 subnormals."""
    d = inputs.conv_desc(64, 32, 4, 4, 64, 1, 1, 0)
    rng = np.random.default_rng(5)
    x = rng.standard_normal((64, 64, 4, 4)).astype(np.float32)
    x[:32, :32, 0, 0] = 0.0
    x[0, 0, 0, 0] = -0.0
    x[:32, 32:, 0, 1] = np.float32(1.5) * rng.choice([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0, 7.0, -7.9], (32, 32)).astype(np.float32)
    x[32:, :32, 0, 2] *= np.float32(1e30)
    x[32:, 32:, 0, 3] *= np.float32(1e-30)
    x[:32, :32, 1, 0] = rng.standard_normal((32, 32)).astype(np.float32) * np.float32(1e-41)
    x[:32, :32, 1, 1] = np.ldexp(rng.standard_normal((32, 32)), rng.integers(-20, 20, (32, 32))).astype(np.float32)
    x[:32, :32, 1, 2] = np.float32(3.4e38)
    x[:32, 32:, 1, 3] = np.float32(448.0)
    oc, osc = oracle.quantize_sr(d, oracle.ROLE_DY, fmt, x, 11)
    q = mq.quantize_sr(d, mq.ROLE_DY, fmt, dev(x), 11)
    assert_same_bytes(q.scales, osc, "scales")
    assert_same_bytes(q.codes, oc, "codes")


def test_config2_gradient_full_size_and_its_gemms():
    """The benchmark's gradient tensor, every byte; the stochastic codes then feed the input- and weight-gradient GEMMs
    like any stored tensor (sampled outputs against the oracle's convolutions of the oracle's stochastic tensor)."""
    from parity_util import OracleLayer, check_convs, gpu_quantize_layer
    (layer,) = inputs.config2()
    ol = OracleLayer(layer)
    seed = 2024
    ol.q[2] = oracle.quantize_sr(ol.desc, oracle.ROLE_DY, layer.fmt_dy, ol.src[2], seed)
    qs = gpu_quantize_layer(ol)
    qs[2] = mq.quantize_sr(ol.desc, mq.ROLE_DY, layer.fmt_dy, dev(ol.src[2]), seed)
    assert_same_bytes(qs[2].scales, ol.q[2][1], "dY scales")
    assert_same_bytes(qs[2].codes, ol.q[2][0], "dY codes")
    rne = oracle.quantize(ol.desc, oracle.ROLE_DY, layer.fmt_dy, ol.src[2])[0]
    assert (rne != ol.q[2][0]).mean() > 0.05          # it is a different tensor from the nearest-rounded one
    check_convs(ol, qs, samples=5000)
