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

# every output buffer the binding creates for these tests starts as NaN (fp32) / 0xA5 (bytes): an element a kernel
# fails to write cannot pass by holding what an earlier call left in recycled memory
mq.DEBUG_FILL = True


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
    assert mq.last_device_status() == 0, "a bounded device-side wait gave up"
    return worst


def _pick_blocks(nblocks, want, rng):
    """`want` of the `nblocks` 32-channel blocks: the first, the last and random ones in between."""
    if nblocks <= want:
        return list(range(nblocks))
    mid = rng.choice(np.arange(1, nblocks - 1), want - 2, replace=False)
    return sorted({0, nblocks - 1, *map(int, mid)})


def check_large_layer(layer, samples=3000, dw_mac_budget=3e10, seed=0, block=None, packed6=False):
    """Parity of a layer too large for the oracle to process whole.  The GPU runs the whole layer at full size; the
    oracle checks it on pieces that are independent of the rest of the tensor:
      * the first and the last 32-sample slab (tiles never span slabs; Y and G_X of a sample depend on that sample
        only): every quantized byte and scale of X and G_Y, the im2col of the slab, sampled Y and G_X outputs with the
        image border included;
      * a subset of 32-channel blocks over ALL samples (tiles never span channel blocks; G_W[co, ci] depends on channels
        co and ci only): every quantized byte of those blocks - which reaches the far end of tensors beyond 2^31
        bytes - and the weight gradient of (chosen output blocks) x (chosen input blocks), every tap: in full while
        that fits `dw_mac_budget` multiply-adds of the oracle, else samples stratified over (output block, tap, input block);
      * W in full.
    block=mq.TS16: the paper's own format (E2M1 elements whatever the layer names).  Its blocks are 16 x 16, so the same
    pieces are independent once the oracle is given the whole tensor's maximum (Eq. 4), which is computed here with numpy
    and also compared with what the GPU's first pass found.
    packed6: the GPU keeps the layer's 6-bit tensors in packed storage (16 codes in 12 bytes); the oracle's one-code-per-byte
    pieces are packed (oracle.pack6) before the comparison - every piece is whole 32-channel rows, hence whole groups."""
    d = layer.desc
    ts = block == mq.TS16
    fx, fw, fg = (mq.E2M1,) * 3 if ts else (layer.fmt_x, layer.fmt_w, layer.fmt_dy)
    P6 = {mq.E3M2: mq.E3M2_P6, mq.E2M3: mq.E2M3_P6}
    gx, gw, gg = [P6.get(f, f) if packed6 else f for f in (fx, fw, fg)]        # the GPU's storage of each tensor
    enc = lambda f, c: oracle.pack6(c) if f in P6.values() else c
    bs = 16 if ts else 32                       # side of a scale block
    name = layer.name + (" (paper's format)" if ts else "")
    rng = np.random.default_rng(seed)
    x, w, g = inputs.layer_tensors(layer)
    ho, wo = inputs.out_hw(d)
    N, Nt = d.N, (d.N + bs - 1) // bs
    cp, cop = (d.C_in + 31) // 32 * 32, (d.C_out + 31) // 32 * 32
    bpe = lambda f: 0.5 if f == mq.E2M1 else (0.75 if f in P6.values() else 1.0)
    OR = (oracle.ROLE_X, oracle.ROLE_W, oracle.ROLE_DY)
    amax = [float(np.abs(t).max()) for t in (x, w, g)] if ts else None

    def oq(dsub, r, f, t):          # oracle: (codes, scales, tensor scale)
        if ts:
            o = oracle.quantize_ts(dsub, OR[r], t, (16, 16), amax=amax[r])
            return o[0], o[1], o[2]
        return oracle.quantize(dsub, OR[r], f, t) + (None,)

    def odq(dsub, r, f, c, sc, t):
        return oracle.dequant_ts(dsub, OR[r], c, sc, t, (16, 16)) if ts else oracle.dequant(dsub, OR[r], f, c, sc)

    if ts:
        xq, wq, gq = [mq.quantize_ts(d, r, dev(t)) for r, t in zip(ROLES, (x, w, g))]
        for q, a in zip((xq, wq, gq), amax):
            st = host(q.tensor_scale)
            assert st[1] == np.float32(a) and st[0] == np.float32(a) / (np.float32(448.0) * np.float32(6.0)), (name, st, a)
    else:
        xq, wq, gq = [mq.quantize(d, r, f, dev(t)) for r, f, t in zip(ROLES, (gx, gw, gg), (x, w, g))]
    wc, wsc, wt = oq(d, 1, fw, w)
    assert_same_bytes(wq.scales, wsc, f"{name} W scales")
    assert_same_bytes(wq.codes, enc(gw, wc), f"{name} W codes")
    wh = odq(d, 1, fw, wc, wsc, wt)
    ic, isc = mq.cbf_im2col(d, xq)
    y = mq.conv_fwd(d, xq, wq)
    dx = mq.conv_bwd_data(d, wq, gq)
    dw = mq.conv_bwd_weight(d, xq, gq)
    P, Po, taps = d.H * d.W, ho * wo, d.Kh * d.Kw
    xcodes = xq.codes.view(P, N, int(cp * bpe(gx)))
    gcodes = gq.codes.view(Po, N, int(cop * bpe(gg)))
    xscales = xq.scales.view(P, Nt, cp // bs)
    gscales = gq.scales.view(Po, Nt, cop // bs)
    icodes = ic.view(Po, N, int(taps * cp * bpe(gx)))
    iscales = isc.view(Po, Nt, taps * (cp // bs))
    worst = {}
    for slab in sorted({0, (N + 31) // 32 - 1}):
        n0, n1 = 32 * slab, min(N, 32 * slab + 32)
        b0, b1 = n0 // bs, (n1 + bs - 1) // bs          # scale rows of the slab
        ds = d._replace(N=n1 - n0)
        xc, xsc, xt = oq(ds, 0, fx, x[n0:n1])
        gc, gsc, gt = oq(ds, 2, fg, g[n0:n1])
        assert_same_bytes(xscales[:, b0:b1].contiguous(), xsc, f"{name} X scales, samples {n0}..{n1}")
        assert_same_bytes(xcodes[:, n0:n1].contiguous(), enc(gx, xc), f"{name} X codes, samples {n0}..{n1}")
        assert_same_bytes(gscales[:, b0:b1].contiguous(), gsc, f"{name} dY scales, samples {n0}..{n1}")
        assert_same_bytes(gcodes[:, n0:n1].contiguous(), enc(gg, gc), f"{name} dY codes, samples {n0}..{n1}")
        oc, osc = oracle.cbf_im2col(ds, fx, xc, xsc, (16, 16)) if ts else oracle.cbf_im2col(ds, fx, xc, xsc)
        assert_same_bytes(iscales[:, b0:b1].contiguous(), osc, f"{name} im2col scales, samples {n0}..{n1}")
        assert_same_bytes(icodes[:, n0:n1].contiguous(), enc(gx, oc), f"{name} im2col codes, samples {n0}..{n1}")
        del oc, osc
        xh = odq(ds, 0, fx, xc, xsc, xt)
        gh = odq(ds, 2, fg, gc, gsc, gt)
        shape = (n1 - n0, d.C_out, ho, wo)
        idx = _sample(int(np.prod(shape)), samples, rng, border_indices(shape, rng=rng))
        ref, ab = oracle.conv_fwd(ds, xh, wh, idx)
        got = host(y[n0:n1].contiguous()).reshape(-1)[idx]
        worst["fwd"] = max(worst.get("fwd", 0.0), assert_gemm_close(torch.from_numpy(got), ref, ab, f"{name} fwd, samples {n0}..{n1}"))
        shape = (n1 - n0, d.C_in, d.H, d.W)
        idx = _sample(int(np.prod(shape)), samples, rng, border_indices(shape, rng=rng))
        ref, ab = oracle.conv_bwd_data(ds, wh, gh, idx)
        got = host(dx[n0:n1].contiguous()).reshape(-1)[idx]
        worst["dx"] = max(worst.get("dx", 0.0), assert_gemm_close(torch.from_numpy(got), ref, ab, f"{name} bwd_data, samples {n0}..{n1}"))
        del xh, gh
    del ic, isc, icodes, iscales, y, dx
    # channel blocks over all samples
    assert d.C_in % 32 == 0 and d.C_out % 32 == 0
    bi, bo = _pick_blocks(cp // 32, 4, rng), _pick_blocks(cop // 32, 4, rng)
    if cop // 32 >= 16:   # one output block in each 128-row tile of the weight gradient, at a different place in each
        bo = [4 * t + (t % 4) for t in range(4)] if cop // 32 == 16 else bo
    ci = np.concatenate([np.arange(32 * b, 32 * b + 32) for b in bi])
    co = np.concatenate([np.arange(32 * b, 32 * b + 32) for b in bo])
    dsel = d._replace(C_in=ci.size, C_out=co.size)
    xs = np.ascontiguousarray(x[:, ci])
    gs = np.ascontiguousarray(g[:, co])
    del x, g
    xc, xsc, xt = oq(dsel, 0, fx, xs)
    gc, gsc, gt = oq(dsel, 2, fg, gs)
    del xs, gs
    bx, bg = int(32 * bpe(gx)), int(32 * bpe(gg))
    tb = lambda blocks: torch.as_tensor(blocks, device="cuda")
    sb = lambda blocks: tb([(32 // bs) * b + k for b in blocks for k in range(32 // bs)])      # scale columns of 32-channel blocks
    assert_same_bytes(xscales[:, :, sb(bi)].contiguous(), xsc, f"{name} X scales, channel blocks {bi}")
    assert_same_bytes(xcodes.view(P, N, cp // 32, bx)[:, :, tb(bi)].contiguous(), enc(gx, xc), f"{name} X codes, channel blocks {bi}")
    assert_same_bytes(gscales[:, :, sb(bo)].contiguous(), gsc, f"{name} dY scales, channel blocks {bo}")
    assert_same_bytes(gcodes.view(Po, N, cop // 32, bg)[:, :, tb(bo)].contiguous(), enc(gg, gc), f"{name} dY codes, channel blocks {bo}")
    xh = odq(dsel, 0, fx, xc, xsc, xt)
    gh = odq(dsel, 2, fg, gc, gsc, gt)
    got = host(dw[tb(co)][:, tb(ci)].contiguous()).reshape(-1)
    per_out = float(N) * ho * wo
    if co.size * ci.size * taps * per_out <= dw_mac_budget:
        idx = None
    else:
        per = max(1, int(dw_mac_budget / per_out / (len(bo) * taps * len(bi))))
        o, i, t = np.meshgrid(np.arange(len(bo)), np.arange(len(bi)), np.arange(taps), indexing="ij")
        o, i, t = [np.repeat(a.reshape(-1), per) for a in (o, i, t)]
        idx = np.unique(((32 * o + rng.integers(0, 32, o.size)) * ci.size + 32 * i + rng.integers(0, 32, o.size)) * taps + t).astype(np.int64)
    ref, ab = oracle.conv_bwd_weight(dsel, gh, xh, idx)
    worst["dw"] = assert_gemm_close(torch.from_numpy(got if idx is None else got[idx]), ref, ab, f"{name} bwd_weight, blocks {bo} x {bi}")
    assert mq.last_device_status() == 0, "a bounded device-side wait gave up"
    return worst
