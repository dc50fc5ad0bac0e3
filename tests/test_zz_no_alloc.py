"""mq_conv_bwd_data_static: the allocation-free variant of the input-gradient call (needs a B200).

Some callers cannot allocate device memory (they run inside an application that owns the allocator, or
while its memory pool is frozen), so they cannot give mq_conv_bwd_data a workspace.  The static variant
keeps that scratch in an array inside the library.  Here it is called through the C ABI twice in a row,
with different layers, so the second call finds the first call's leftovers in the shared array, and each
result is compared with what the ordinary entry point returns for the same inputs, within the bound the
GEMM parity tests use.  This file sorts last so a run that stops at the first failure has already run
every other test; it also passes on its own in a fresh process."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq
from parity_util import GEMM_TOL, OracleLayer, gpu_quantize_layer

pytestmark = pytest.mark.gpu


def _layer(name, shape, fmts, seed):
    return inputs.Layer(name, inputs.conv_desc(*shape), fmts[0], fmts[1], fmts[2], "relu", "kaiming", "gauss", seed)


def test_static_scratch_variant_matches_workspace_variant_on_two_calls_in_a_row():
    cases = [
        _layer("static_a", (64, 128, 10, 12, 96, 3, 1, 1), (mq.E4M3, mq.E4M3, mq.E5M2), 71),   # 3x3, FP8
        _layer("static_b", (40, 64, 9, 7, 192, 3, 2, 1), (mq.E2M1, mq.E2M1, mq.E2M1), 72),     # stride 2, FP4, smaller scratch
    ]
    for layer in cases:
        d = layer.desc
        ol = OracleLayer(layer)
        _, wq, gq = gpu_quantize_layer(ol)
        need = mq.workspace_size(d, mq.OP_BWD_DATA, wq.fmt, gq.fmt)
        assert 0 < need <= mq.STATIC_SCRATCH_BYTES
        ref = mq.conv_bwd_data(d, wq, gq)                      # ordinary entry point, caller's workspace
        dx = torch.full_like(ref, float("nan"))
        got = mq.conv_bwd_data_static(d, wq, gq, dx=dx)       # static scratch, nothing allocated by the call
        torch.cuda.synchronize()
        assert mq.last_device_status() == 0
        _, ab = oracle.conv_bwd_data(d, ol.hat[1], ol.hat[2])
        err = np.abs(got.cpu().numpy().astype(np.float64) - ref.cpu().numpy().astype(np.float64))
        assert (err <= GEMM_TOL * ab).all()
        # the same deterministic kernels ran on the same inputs: nothing of the previous call's leftovers in the
        # shared array may leak, so the two results are the same bits
        assert torch.equal(got, ref)
        # and against the oracle itself, like every other GEMM test
        gx, _ = oracle.conv_bwd_data(d, ol.hat[1], ol.hat[2])
        assert (np.abs(got.cpu().numpy().astype(np.float64) - gx) <= GEMM_TOL * ab).all()


def test_static_scratch_variant_rejects_layers_beyond_its_limit():
    d = inputs.conv_desc(32, 2048, 8, 8, 1024, 3)      # 2048 x 1024 x 9 FP8 weights re-laid: 18.9 MB > 16 MiB
    assert mq.workspace_size(d, mq.OP_BWD_DATA, mq.E4M3, mq.E5M2) > mq.STATIC_SCRATCH_BYTES
    wq = mq.empty_qtensor(d, mq.ROLE_W, mq.E4M3)
    gq = mq.empty_qtensor(d, mq.ROLE_DY, mq.E5M2)
    dx = torch.zeros((32, 2048, 8, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(mq.MqError) as e:
        mq.conv_bwd_data_static(d, wq, gq, dx=dx)
    assert e.value.status == 7 and "STATIC_SCRATCH" in str(e.value)
    assert not dx.any()      # nothing was launched
    # a bad argument is reported as such even on a layer beyond the limit
    lib = mq.lib()
    a, b = wq._c(), gq._c()
    st = lib.mq_conv_bwd_data_static(ctypes.byref(mq._d(d)), ctypes.byref(a), ctypes.byref(b), None, mq.F32, mq.NCHW, None)
    assert st == 1   # MQ_ERR_INVALID_ARG: null dx
