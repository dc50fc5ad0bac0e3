"""Host-side checks of the C-ABI library (no GPU, no compute calls): it loads, exports every
symbol the header declares, answers size queries like the oracle, and rejects bad arguments on
the host before touching the device."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2609_28358_b200 import inputs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mq():
    from paper_2609_28358_b200 import build, mq as _mq

    build.build()
    return _mq


def declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(mq_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(mq):
    syms = declared_symbols()
    assert {"mq_quantize", "mq_cbf_im2col", "mq_conv_fwd", "mq_conv_bwd_data", "mq_conv_bwd_weight"} <= set(syms)
    for s in syms:
        assert hasattr(mq.lib(), s), s


def test_status_strings(mq):
    assert mq.status_string(0) == "MQ_OK"
    assert mq.status_string(6) == "MQ_ERR_TIMEOUT"
    assert len({mq.status_string(i) for i in range(7)}) == 7


@pytest.mark.parametrize("desc", [inputs.conv_desc(8, 32, 32, 32, 64, 3), inputs.conv_desc(37, 48, 9, 7, 70, 3, 2),
                                  inputs.conv_desc(256, 512, 14, 14, 512, 1, 1, 0)])
def test_size_queries_match_oracle(mq, desc):
    for fmt in (mq.E4M3, mq.E5M2, mq.E2M1, mq.E3M2, mq.E2M3):
        for role in (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY):
            assert mq.qtensor_sizes(desc, role, fmt) == oracle.qtensor_sizes(desc, role, fmt)
            assert mq.qtensor_sizes(desc, role, fmt, mq.LINE32) == oracle.qtensor_sizes(desc, role, fmt, (1, 32))
        assert mq.im2col_sizes(desc, fmt) == oracle.im2col_sizes(desc, fmt)
        assert mq.im2col_sizes(desc, fmt, mq.LINE32) == oracle.im2col_sizes(desc, fmt, (1, 32))
        for op in (mq.OP_FWD, mq.OP_BWD_DATA, mq.OP_BWD_WEIGHT):
            assert mq.workspace_size(desc, op, fmt, fmt) >= 0
        assert mq.workspace_size(desc, mq.OP_FWD, fmt, fmt, mq.LINE32) >= 0
        for op in (mq.OP_BWD_DATA, mq.OP_BWD_WEIGHT):      # a line-quantized tensor cannot feed the other contraction direction
            with pytest.raises(mq.MqError) as e:
                mq.workspace_size(desc, op, fmt, fmt, mq.LINE32)
            assert e.value.status == 2
    # packed 6-bit storage: three quarters of the one-code-per-byte tensor, the same scales; never less scratch
    for fmt, pf in ((mq.E3M2, mq.E3M2_P6), (mq.E2M3, mq.E2M3_P6)):
        for role in (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY):
            cb, sb = mq.qtensor_sizes(desc, role, fmt)
            assert mq.qtensor_sizes(desc, role, pf) == (cb * 3 // 4, sb)
        cb, sb = mq.im2col_sizes(desc, fmt)
        assert mq.im2col_sizes(desc, pf) == (cb * 3 // 4, sb)
        for op in (mq.OP_FWD, mq.OP_BWD_DATA, mq.OP_BWD_WEIGHT):
            assert mq.workspace_size(desc, op, pf, pf) >= mq.workspace_size(desc, op, fmt, fmt)
            assert mq.workspace_size(desc, op, pf, mq.E4M3 if op != mq.OP_BWD_DATA else mq.E5M2) >= 0
        for op in (mq.OP_FWD, mq.OP_BWD_DATA):             # the quantizing epilogue does not take it
            with pytest.raises(mq.MqError) as e:
                mq.conv_mx_workspace_size(desc, op, pf, mq.E4M3)
            assert e.value.status == 2


def test_bad_arguments_are_rejected_on_the_host(mq):
    L = mq.lib()
    good = mq._d(inputs.conv_desc(8, 32, 8, 8, 32, 3))
    cb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    assert L.mq_qtensor_sizes(None, 0, 0, 0, ctypes.byref(cb), ctypes.byref(sb)) == 1
    assert L.mq_qtensor_sizes(ctypes.byref(good), 7, 0, 0, ctypes.byref(cb), ctypes.byref(sb)) == 1
    assert L.mq_qtensor_sizes(ctypes.byref(good), 0, 9, 0, ctypes.byref(cb), ctypes.byref(sb)) == 1
    assert L.mq_qtensor_sizes(ctypes.byref(good), 0, 0, 5, ctypes.byref(cb), ctypes.byref(sb)) == 1   # no such block shape
    bad = mq._d(inputs.conv_desc(8, 32, 8, 8, 32, 3), block_size=16)
    assert L.mq_qtensor_sizes(ctypes.byref(bad), 0, 0, 0, ctypes.byref(cb), ctypes.byref(sb)) == 2  # unsupported block length
    neg = mq._d(inputs.conv_desc(0, 32, 8, 8, 32, 3))
    assert L.mq_qtensor_sizes(ctypes.byref(neg), 0, 0, 0, ctypes.byref(cb), ctypes.byref(sb)) == 1
    big_k = mq._d(inputs.conv_desc(1, 32, 2, 2, 32, 7, 1, 0))
    assert L.mq_qtensor_sizes(ctypes.byref(big_k), 0, 0, 0, ctypes.byref(cb), ctypes.byref(sb)) == 1
    # entry points: null / misaligned / undersized buffers never reach a launch
    F32, BF16, NCHW = mq.F32, mq.BF16, mq.NCHW
    q = mq._QTensor(None, None, 0, 0, 0, 0, 0, None)
    assert L.mq_quantize(ctypes.byref(good), None, F32, NCHW, ctypes.byref(q), None) == 1
    q = mq._QTensor(0x1000, 0x2000, 16, 16, 0, 0, 0, None)
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, NCHW, ctypes.byref(q), None) == 4  # too small
    q = mq._QTensor(0x1008, 0x2000, 1 << 30, 1 << 30, 0, 0, 0, None)
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, NCHW, ctypes.byref(q), None) == 3  # alignment
    q = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 0, 0, None)
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, 7, ctypes.byref(q), None) == 1  # no such source layout
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), 9, NCHW, ctypes.byref(q), None) == 1  # no such element type
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), BF16, NCHW, ctypes.byref(q), None) == 2  # bf16 source: not in this build
    qbad = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 0, 3, None)
    assert L.mq_quantize(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, NCHW, ctypes.byref(qbad), None) == 1  # no such block shape
    # the stochastic-rounding entry point validates the same way (the seed is any 64-bit value)
    seed = ctypes.c_uint64(0xFFFFFFFFFFFFFFFF)
    assert L.mq_quantize_sr(ctypes.byref(good), None, F32, NCHW, ctypes.byref(q), seed, None) == 1
    assert L.mq_quantize_sr(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, 7, ctypes.byref(q), seed, None) == 1
    assert L.mq_quantize_sr(ctypes.byref(good), ctypes.c_void_p(0x3004), F32, NCHW, ctypes.byref(q), seed, None) == 3
    small = mq._QTensor(0x1000, 0x2000, 16, 16, 0, 2, 0, None)
    assert L.mq_quantize_sr(ctypes.byref(good), ctypes.c_void_p(0x3000), F32, NCHW, ctypes.byref(small), seed, None) == 4
    assert L.mq_cbf_im2col(ctypes.byref(good), ctypes.byref(q), None, None, None) == 1
    qw = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 1, 0, None)
    out = ctypes.c_void_p(0x4000)
    assert L.mq_conv_fwd(ctypes.byref(good), ctypes.byref(qw), ctypes.byref(qw), out, F32, NCHW, None, 0, None) == 1  # wrong role
    assert L.mq_conv_fwd(ctypes.byref(good), ctypes.byref(q), ctypes.byref(qw), out, F32, 5, None, 0, None) == 1  # layout
    assert L.mq_conv_fwd(ctypes.byref(good), ctypes.byref(q), ctypes.byref(qw), out, 9, NCHW, None, 0, None) == 1  # element type
    assert L.mq_conv_fwd(ctypes.byref(good), ctypes.byref(q), ctypes.byref(qw), out, BF16, NCHW, None, 0, None) == 2  # bf16 output: not in this build
    need = mq.workspace_size(inputs.conv_desc(8, 32, 8, 8, 32, 3), mq.OP_BWD_WEIGHT, 0, 0)
    qg = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 2, 0, None)
    if need:
        assert L.mq_conv_bwd_weight(ctypes.byref(good), ctypes.byref(q), ctypes.byref(qg), out, F32, NCHW, None, 0, None) == 4
    # line blocks: accepted by the forward GEMM only; operands must agree on the block shape
    ql = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 0, 1, None)
    qwl = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 1, 1, None)
    qgl = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, 0, 2, 1, None)
    assert L.mq_conv_fwd(ctypes.byref(good), ctypes.byref(ql), ctypes.byref(qw), out, F32, NCHW, None, 0, None) == 2  # mixed block shapes
    assert L.mq_conv_bwd_data(ctypes.byref(good), ctypes.byref(qwl), ctypes.byref(qgl), out, F32, NCHW, None, 0, None) == 2
    assert L.mq_conv_bwd_weight(ctypes.byref(good), ctypes.byref(ql), ctypes.byref(qgl), out, F32, NCHW, None, 0, None) == 2
    # the quantizing epilogue in the paper's own format: all three tensors in that format, a supplied maximum
    E2M1, TS16 = mq.E2M1, mq.TS16
    ts_x = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, E2M1, 0, TS16, 0x5000)
    ts_w = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, E2M1, 1, TS16, 0x5000)
    ts_y = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, E2M1, 0, TS16, 0x5000)
    amax = ctypes.c_void_p(0x6000)
    assert L.mq_conv_ts_workspace_size(ctypes.byref(good), 0, None) == 1
    assert L.mq_conv_ts_workspace_size(ctypes.byref(good), 2, ctypes.byref(cb)) == 1           # no weight-gradient variant
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(ts_x), ctypes.byref(ts_w), 0, None, ctypes.byref(ts_y), None, 0, None) == 1   # no maximum
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(ts_x), ctypes.byref(ts_w), 7, amax, ctypes.byref(ts_y), None, 0, None) == 1   # no such activation
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(q), ctypes.byref(qw), 0, amax, ctypes.byref(ts_y), None, 0, None) == 2        # MX operands
    mx_y = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, E2M1, 0, 0, 0x5000)
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(ts_x), ctypes.byref(ts_w), 0, amax, ctypes.byref(mx_y), None, 0, None) == 2   # MX output
    small_y = mq._QTensor(0x1000, 0x2000, 16, 16, E2M1, 0, TS16, 0x5000)
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(ts_x), ctypes.byref(ts_w), 0, amax, ctypes.byref(small_y), None, 0, None) == 4
    assert L.mq_conv_fwd_ts(ctypes.byref(good), ctypes.byref(ts_x), ctypes.byref(ts_w), 0, ctypes.c_void_p(0x6002), ctypes.byref(ts_y), None, 0, None) == 3
    ts_g = mq._QTensor(0x1000, 0x2000, 1 << 30, 1 << 30, E2M1, 2, TS16, 0x5000)
    assert L.mq_conv_bwd_data_ts(ctypes.byref(good), ctypes.byref(ts_w), ctypes.byref(ts_g), None, ctypes.byref(ts_g), None, 0, None) == 1
    # the quantizer of that format: the supplied maximum may not live in the words the call rewrites, and must be 4-byte aligned
    src = ctypes.c_void_p(0x7000)
    assert L.mq_quantize_ts(ctypes.byref(good), src, F32, NCHW, ctypes.byref(ts_x), ctypes.c_void_p(0x5004), None, None) == 1
    assert L.mq_quantize_ts(ctypes.byref(good), src, F32, NCHW, ctypes.byref(ts_x), ctypes.c_void_p(0x6002), None, None) == 3
    assert L.mq_quantize_ts(ctypes.byref(good), src, F32, NCHW, ctypes.byref(mx_y), amax, None, None) == 1   # not that format
