"""Shared helpers of the GPU parity tests: run the oracle and the CUDA path on the same seeded
inputs and compare.  Codes, scales and layouts must be bit-exact; GEMM outputs must satisfy
|gpu - oracle| <= 1e-4 * sum_i |a_i * b_i| per output element (fp32 accumulation on the GPU,
float64 in the oracle)."""
import numpy as np
import torch

import oracle
from paper_2609_28358_b200 import inputs, mq

GEMM_TOL = 1e-4
ROLES = (mq.ROLE_X, mq.ROLE_W, mq.ROLE_DY)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t):
    return t.detach().cpu().numpy()


def assert_same_bytes(got, want, what):
    got = host(got).reshape(-1)
    want = np.asarray(want).reshape(-1)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    if not np.array_equal(got, want):
        bad = np.flatnonzero(got != want)
        raise AssertionError(f"{what}: {bad.size} of {got.size} bytes differ; first at {bad[0]}: gpu {got[bad[0]]:#x} oracle {want[bad[0]]:#x}")


def assert_gemm_close(got, ref, ref_abs, what, tol=GEMM_TOL):
    got = host(got).astype(np.float64).reshape(-1)
    ref = np.asarray(ref).reshape(-1)
    ref_abs = np.asarray(ref_abs).reshape(-1)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    err = np.abs(got - ref)
    bound = tol * ref_abs
    bad = np.flatnonzero(~(err <= bound))
    if bad.size:
        i = bad[np.argmax((err - bound)[bad])]
        raise AssertionError(f"{what}: {bad.size} of {got.size} outputs outside {tol}*sum|ab|; worst at {i}: "
                             f"gpu {got[i]!r} oracle {ref[i]!r} bound {bound[i]!r}")
    return float((err / np.maximum(bound, 1e-300)).max()) if got.size else 0.0


class OracleLayer:
    """Oracle results for one layer: quantized tensors, their dequantized values."""

    def __init__(self, layer, tensors=None):
        self.layer = layer
        self.desc = layer.desc
        self.fmts = (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
        self.src = tensors if tensors is not None else inputs.layer_tensors(layer)
        self.q = [oracle.quantize(self.desc, r, f, t) for r, f, t in zip(ROLES, self.fmts, self.src)]
        self._hat = None

    @property
    def hat(self):
        if self._hat is None:
            self._hat = [oracle.dequant(self.desc, r, f, c, s) for r, f, (c, s) in zip(ROLES, self.fmts, self.q)]
        return self._hat


def gpu_quantize_layer(ol):
    """Quantize the layer's three tensors on the GPU; returns [xq, wq, dyq]."""
    return [mq.quantize(ol.desc, r, f, dev(t)) for r, f, t in zip(ROLES, ol.fmts, ol.src)]


def check_quantize(ol, qs=None):
    qs = qs or gpu_quantize_layer(ol)
    for name, q, (c, s) in zip(("X", "W", "dY"), qs, ol.q):
        assert_same_bytes(q.scales, s, f"{ol.layer.name} {name} scales")
        assert_same_bytes(q.codes, c, f"{ol.layer.name} {name} codes")
    return qs


def check_im2col(ol, xq):
    oc, osc = oracle.cbf_im2col(ol.desc, ol.fmts[0], *ol.q[0])
    gc, gs = mq.cbf_im2col(ol.desc, xq)
    assert_same_bytes(gs, osc, f"{ol.layer.name} im2col scales")
    assert_same_bytes(gc, oc, f"{ol.layer.name} im2col codes")


def _sample(size, count, rng, always=()):
    if count is None or count >= size:
        return None
    idx = np.unique(np.concatenate([rng.choice(size, count, replace=False), np.asarray(always, dtype=np.int64)]))
    return idx.astype(np.int64)


def border_indices(shape, per_edge=64, rng=None):
    """Flat indices on the spatial border of an [A][B][H][W] tensor (first/last rows and columns)."""
    A, B, H, W = shape
    rng = rng or np.random.default_rng(0)
    out = []
    for _ in range(per_edge):
        a, b = rng.integers(A), rng.integers(B)
        for h, w in ((0, rng.integers(W)), (H - 1, rng.integers(W)), (rng.integers(H), 0), (rng.integers(H), W - 1)):
            out.append(((a * B + b) * H + h) * W + w)
    return np.asarray(out, dtype=np.int64)


def check_convs(ol, qs, samples=None, layouts=(mq.NCHW,), seed=0, ops=("fwd", "dx", "dw")):
    """Run the three GEMMs on the GPU from the GPU-quantized tensors and compare with the oracle's
    convolutions of the dequantized tensors (all outputs, or `samples` outputs per tensor plus
    border pixels)."""
    d = ol.desc
    xq, wq, gq = qs
    xh, wh, gh = ol.hat
    rng = np.random.default_rng(seed)
    worst = {}
    for layout in layouts:
        if "fwd" in ops:
            y = mq.conv_fwd(d, xq, wq, layout=layout)
            yn = y if layout == mq.NCHW else y.permute(2, 3, 0, 1)
            shape = oracle.logical_shape(d, oracle.ROLE_DY)
            idx = _sample(int(np.prod(shape)), samples, rng, border_indices(shape, rng=rng) if samples else ())
            ref, ab = oracle.conv_fwd(d, xh, wh, idx)
            got = host(yn.contiguous()).reshape(-1)
            worst["fwd"] = assert_gemm_close(torch.from_numpy(got if idx is None else got[idx]), ref, ab, f"{ol.layer.name} fwd layout {layout}")
        if "dx" in ops:
            dx = mq.conv_bwd_data(d, wq, gq, layout=layout)
            dxn = dx if layout == mq.NCHW else dx.permute(2, 3, 0, 1)
            shape = oracle.logical_shape(d, oracle.ROLE_X)
            idx = _sample(int(np.prod(shape)), samples, rng, border_indices(shape, rng=rng) if samples else ())
            ref, ab = oracle.conv_bwd_data(d, wh, gh, idx)
            got = host(dxn.contiguous()).reshape(-1)
            worst["dx"] = assert_gemm_close(torch.from_numpy(got if idx is None else got[idx]), ref, ab, f"{ol.layer.name} bwd_data layout {layout}")
        if "dw" in ops:
            dw = mq.conv_bwd_weight(d, xq, gq, layout=layout)
            dwn = dw if layout == mq.NCHW else dw.permute(0, 3, 1, 2)
            shape = oracle.logical_shape(d, oracle.ROLE_W)
            idx = _sample(int(np.prod(shape)), samples if samples is None else max(samples // 16, 256), rng)
            ref, ab = oracle.conv_bwd_weight(d, gh, xh, idx)
            got = host(dwn.contiguous()).reshape(-1)
            worst["dw"] = assert_gemm_close(torch.from_numpy(got if idx is None else got[idx]), ref, ab, f"{ol.layer.name} bwd_weight layout {layout}")
    return worst
