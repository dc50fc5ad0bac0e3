"""Python binding of ``libmq.so``: the same names as the C ABI (``include/mq.h``), argument
marshalling only.  PyTorch supplies device memory and the current CUDA stream; every step of the
path runs in the library's kernels.  There is no fallback: if the library is missing or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from collections import namedtuple

import torch

ConvDesc = namedtuple("ConvDesc", "N C_in H W C_out Kh Kw stride_h stride_w pad_h pad_w")

E4M3, E5M2, E2M1, E3M2, E2M3 = 0, 1, 2, 3, 4
E3M2_P6, E2M3_P6 = 5, 6          # the 6-bit formats in packed storage: 16 codes in 12 bytes instead of one code per byte
ROLE_X, ROLE_W, ROLE_DY = 0, 1, 2
NCHW, HWNC = 0, 1
TILE32, LINE32, TS16 = 0, 1, 2   # 32 x 32 squares (default) / 1 x 32 lines along the channel axis / the paper's own format: 16 x 16
                                 # squares with an E4M3 block scale and an fp32 tensor scale (E2M1 elements)
F32, BF16 = 0, 1
OP_FWD, OP_BWD_DATA, OP_BWD_WEIGHT = 0, 1, 2
OK = 0

# When true, every output buffer this module creates is pre-filled (fp32 with NaN, bytes with 0xA5) instead of left
# uninitialised, so that an element a kernel fails to write cannot pass a comparison by holding an earlier result.
DEBUG_FILL = False

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmq.so")
_lib = None


class MqError(RuntimeError):
    def __init__(self, call, status):
        self.status = status
        super().__init__(f"{call} failed: {status_string(status)} ({status})")


class _Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in
                ("N", "C_in", "H", "W", "C_out", "Kh", "Kw", "stride_h", "stride_w", "pad_h", "pad_w", "block_size")]


class _QTensor(ctypes.Structure):
    _fields_ = [("codes", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("codes_bytes", ctypes.c_size_t),
                ("scales_bytes", ctypes.c_size_t), ("fmt", ctypes.c_int), ("role", ctypes.c_int), ("block", ctypes.c_int), ("tensor_scale", ctypes.c_void_p)]


def lib():
    """The loaded C-ABI library.  Raises if it has not been built (python -m paper_2609_28358_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_28358_b200.build`; "
                               "there is no fallback path")
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.mq_status_string.restype = ctypes.c_char_p
        _lib.mq_kernel_launch_count.restype = ctypes.c_ulonglong
        _lib.mq_reload_env.restype = None
    return _lib


def status_string(status):
    return lib().mq_status_string(int(status)).decode()


def _d(desc, block_size=32):
    return _Desc(*[int(v) for v in desc], block_size)


def _check(call, st):
    if st != OK:
        raise MqError(call, st)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


class QTensor:
    """A stored MX tensor: device uint8 buffers for codes and tile scales."""

    def __init__(self, codes, scales, fmt, role, block=TILE32, tensor_scale=None):
        self.codes, self.scales, self.fmt, self.role, self.block = codes, scales, fmt, role, block
        self.tensor_scale = tensor_scale      # TS16: two device floats (T_scale, max|X|)

    def _c(self):
        return _QTensor(self.codes.data_ptr(), self.scales.data_ptr(), self.codes.numel(), self.scales.numel(), self.fmt, self.role, self.block,
                        self.tensor_scale.data_ptr() if self.tensor_scale is not None else None)


def _new(shape, dtype, device):
    t = torch.empty(shape, dtype=dtype, device=device)
    if DEBUG_FILL:
        t.fill_(float("nan") if dtype.is_floating_point else 0xA5)
    return t


def qtensor_sizes(desc, role, fmt, block=TILE32):
    cb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    _check("mq_qtensor_sizes", lib().mq_qtensor_sizes(ctypes.byref(_d(desc)), role, fmt, block, ctypes.byref(cb), ctypes.byref(sb)))
    return cb.value, sb.value


def im2col_sizes(desc, fmt, block=TILE32):
    cb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    _check("mq_im2col_sizes", lib().mq_im2col_sizes(ctypes.byref(_d(desc)), fmt, block, ctypes.byref(cb), ctypes.byref(sb)))
    return cb.value, sb.value


def workspace_size(desc, op, fmt_a, fmt_b, block=TILE32):
    b = ctypes.c_size_t()
    _check("mq_workspace_size", lib().mq_workspace_size(ctypes.byref(_d(desc)), op, fmt_a, fmt_b, block, ctypes.byref(b)))
    return b.value


def empty_qtensor(desc, role, fmt, device="cuda", block=TILE32):
    cb, sb = qtensor_sizes(desc, role, fmt, block)
    ts = _new(2, torch.float32, device) if block == TS16 else None
    return QTensor(_new(cb, torch.uint8, device), _new(sb, torch.uint8, device), fmt, role, block, ts)


_DTYPES = {torch.float32: F32, torch.bfloat16: BF16}


def quantize(desc, role, fmt, src, out=None, src_layout=NCHW, stream=None, block=TILE32):
    """mq_quantize: device tensor (NCHW / OIHW, or channel-fastest with src_layout=HWNC) -> stored MX tensor."""
    assert src.is_cuda and src.dtype in _DTYPES and src.is_contiguous()
    if out is None:
        out = empty_qtensor(desc, role, fmt, src.device, block)
    q = out._c()
    _check("mq_quantize", lib().mq_quantize(ctypes.byref(_d(desc)), ctypes.c_void_p(src.data_ptr()), _DTYPES[src.dtype], src_layout, ctypes.byref(q),
                                           _stream(stream)))
    return out


def quantize_sr(desc, role, fmt, src, seed, out=None, src_layout=NCHW, stream=None, block=TILE32):
    """mq_quantize_sr: as quantize(), with stochastic rounding of the elements (the gradient's rounding); `seed` is a 64-bit integer."""
    assert src.is_cuda and src.dtype in _DTYPES and src.is_contiguous()
    if out is None:
        out = empty_qtensor(desc, role, fmt, src.device, block)
    q = out._c()
    _check("mq_quantize_sr", lib().mq_quantize_sr(ctypes.byref(_d(desc)), ctypes.c_void_p(src.data_ptr()), _DTYPES[src.dtype], src_layout, ctypes.byref(q),
                                                 ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF), _stream(stream)))
    return out


def quantize_ts(desc, role, src, out=None, src_layout=NCHW, amax_in=None, seed=None, stream=None):
    """mq_quantize_ts: the paper's own format (fp32 tensor scale, E4M3 scale per 16 x 16 block, E2M1 elements).  amax_in: a
    device float tensor holding the maximum Eq. 4 should use (e.g. an earlier tensor's tensor_scale[1:2]); None = this
    tensor's own (two passes).  seed: stochastic rounding with that 64-bit seed."""
    assert src.is_cuda and src.dtype in _DTYPES and src.is_contiguous()
    if out is None:
        out = empty_qtensor(desc, role, E2M1, src.device, TS16)
    q = out._c()
    sd = ctypes.c_uint64(int(seed) & 0xFFFFFFFFFFFFFFFF) if seed is not None else None
    _check("mq_quantize_ts", lib().mq_quantize_ts(ctypes.byref(_d(desc)), ctypes.c_void_p(src.data_ptr()), _DTYPES[src.dtype], src_layout, ctypes.byref(q),
                                                 ctypes.c_void_p(amax_in.data_ptr()) if amax_in is not None else None,
                                                 ctypes.byref(sd) if sd is not None else None, _stream(stream)))
    return out


def selftest_wait_timeout(desc, role, fmt, src, polls=2000, stream=None):
    """mq_selftest_wait_timeout: runs the quantizer's TMA pipeline with its loader off and short wait limits, so every
    bounded wait gives up; the kernel must return normally with the device status word set."""
    out = empty_qtensor(desc, role, fmt, src.device)
    q = out._c()
    _check("mq_selftest_wait_timeout", lib().mq_selftest_wait_timeout(ctypes.byref(_d(desc)), ctypes.c_void_p(src.data_ptr()), ctypes.byref(q),
                                                                    ctypes.c_uint(polls), _stream(stream)))
    return out


def cbf_im2col(desc, xq, out_codes=None, out_scales=None, stream=None):
    """mq_cbf_im2col: stored quantized activation -> (codes, scales) of X'."""
    cb, sb = im2col_sizes(desc, xq.fmt, xq.block)
    if out_codes is None:
        out_codes = _new(cb, torch.uint8, xq.codes.device)
    if out_scales is None:
        out_scales = _new(sb, torch.uint8, xq.codes.device)
    q = xq._c()
    _check("mq_cbf_im2col", lib().mq_cbf_im2col(ctypes.byref(_d(desc)), ctypes.byref(q), ctypes.c_void_p(out_codes.data_ptr()),
                                               ctypes.c_void_p(out_scales.data_ptr()), _stream(stream)))
    return out_codes, out_scales


def _out_hw(desc):
    d = ConvDesc(*desc)
    return ((d.H + 2 * d.pad_h - d.Kh) // d.stride_h + 1, (d.W + 2 * d.pad_w - d.Kw) // d.stride_w + 1)


def _conv(name, op, desc, qa, qb, out, shape_nchw, shape_hwnc, layout, workspace, stream, dtype=torch.float32):
    dev = qa.codes.device
    if out is None:
        out = _new(shape_nchw if layout == NCHW else shape_hwnc, dtype, dev)
    need = workspace_size(desc, op, qa.fmt, qb.fmt, qa.block)
    if workspace is None and need > 0:
        workspace = _new(need, torch.uint8, dev)
    wp = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    wn = workspace.numel() * workspace.element_size() if workspace is not None else 0
    a, b = qa._c(), qb._c()
    fn = getattr(lib(), name)
    _check(name, fn(ctypes.byref(_d(desc)), ctypes.byref(a), ctypes.byref(b), ctypes.c_void_p(out.data_ptr()), _DTYPES[out.dtype], layout, wp,
                    ctypes.c_size_t(wn), _stream(stream)))
    return out


def conv_fwd(desc, xq, wq, y=None, layout=NCHW, workspace=None, stream=None, dtype=torch.float32):
    d = ConvDesc(*desc)
    ho, wo = _out_hw(d)
    return _conv("mq_conv_fwd", OP_FWD, desc, xq, wq, y, (d.N, d.C_out, ho, wo), (ho, wo, d.N, d.C_out), layout, workspace, stream, dtype)


def conv_bwd_data(desc, wq, dyq, dx=None, layout=NCHW, workspace=None, stream=None, dtype=torch.float32):
    d = ConvDesc(*desc)
    return _conv("mq_conv_bwd_data", OP_BWD_DATA, desc, wq, dyq, dx, (d.N, d.C_in, d.H, d.W), (d.H, d.W, d.N, d.C_in), layout, workspace, stream, dtype)


ACT_NONE, ACT_RELU, ACT_SILU = 0, 1, 2


def conv_mx_workspace_size(desc, op, fmt_a, fmt_b):
    b = ctypes.c_size_t()
    _check("mq_conv_mx_workspace_size", lib().mq_conv_mx_workspace_size(ctypes.byref(_d(desc)), op, fmt_a, fmt_b, ctypes.byref(b)))
    return b.value


def _mx_out(desc, op, fmt, role, device):
    """An empty stored tensor of what the quantizing epilogue emits: the forward result as a role-X tensor of
    N x C_out x Ho x Wo, the input gradient as a role-DY tensor of N x C_in x H x W."""
    d = ConvDesc(*desc)
    ho, wo = _out_hw(d)
    c, h, w = (d.C_out, ho, wo) if op == OP_FWD else (d.C_in, d.H, d.W)
    cp = (c + 31) // 32 * 32
    cb = h * w * d.N * cp * (4 if fmt == E2M1 else 8) // 8
    sb = h * w * ((d.N + 31) // 32) * (cp // 32)
    return QTensor(_new(cb, torch.uint8, device), _new(sb, torch.uint8, device), fmt, role)


def _conv_mx(name, op, desc, qa, qb, out, extra, workspace, stream):
    need = conv_mx_workspace_size(desc, op, qa.fmt, qb.fmt)
    if workspace is None and need > 0:
        workspace = _new(need, torch.uint8, qa.codes.device)
    wp = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    wn = workspace.numel() * workspace.element_size() if workspace is not None else 0
    a, b, o = qa._c(), qb._c(), out._c()
    _check(name, getattr(lib(), name)(ctypes.byref(_d(desc)), ctypes.byref(a), ctypes.byref(b), *extra, ctypes.byref(o), wp, ctypes.c_size_t(wn), _stream(stream)))
    return out


def conv_fwd_mx(desc, xq, wq, fmt, act=ACT_NONE, yq=None, workspace=None, stream=None):
    """mq_conv_fwd_mx: act(conv(X, W)) emitted as the next layer's stored activation (element format `fmt`)."""
    if yq is None:
        yq = _mx_out(desc, OP_FWD, fmt, ROLE_X, xq.codes.device)
    return _conv_mx("mq_conv_fwd_mx", OP_FWD, desc, xq, wq, yq, (ctypes.c_int(act),), workspace, stream)


def conv_bwd_data_mx(desc, wq, dyq, fmt, dxq=None, workspace=None, stream=None):
    """mq_conv_bwd_data_mx: the input gradient emitted as the previous layer's stored output gradient."""
    if dxq is None:
        dxq = _mx_out(desc, OP_BWD_DATA, fmt, ROLE_DY, wq.codes.device)
    return _conv_mx("mq_conv_bwd_data_mx", OP_BWD_DATA, desc, wq, dyq, dxq, (), workspace, stream)


def conv_ts_workspace_size(desc, op):
    b = ctypes.c_size_t()
    _check("mq_conv_ts_workspace_size", lib().mq_conv_ts_workspace_size(ctypes.byref(_d(desc)), op, ctypes.byref(b)))
    return b.value


def _ts_out(desc, op, role, device):
    """An empty stored tensor in the paper's own format of what the quantizing epilogue emits (see _mx_out)."""
    d = ConvDesc(*desc)
    ho, wo = _out_hw(d)
    c, h, w = (d.C_out, ho, wo) if op == OP_FWD else (d.C_in, d.H, d.W)
    cp = (c + 31) // 32 * 32
    return QTensor(_new(h * w * d.N * cp // 2, torch.uint8, device), _new(h * w * ((d.N + 15) // 16) * (cp // 16), torch.uint8, device), E2M1, role, TS16,
                   _new(2, torch.float32, device))


def _conv_ts(name, op, desc, qa, qb, out, extra, workspace, stream):
    need = conv_ts_workspace_size(desc, op)
    if workspace is None and need > 0:
        workspace = _new(need, torch.uint8, qa.codes.device)
    wp = ctypes.c_void_p(workspace.data_ptr()) if workspace is not None else None
    wn = workspace.numel() * workspace.element_size() if workspace is not None else 0
    a, b, o = qa._c(), qb._c(), out._c()
    _check(name, getattr(lib(), name)(ctypes.byref(_d(desc)), ctypes.byref(a), ctypes.byref(b), *extra, ctypes.byref(o), wp, ctypes.c_size_t(wn), _stream(stream)))
    return out


def conv_fwd_ts(desc, xq, wq, amax_in, act=ACT_NONE, yq=None, workspace=None, stream=None):
    """mq_conv_fwd_ts: act(conv(X, W)) emitted as the next layer's stored activation in the paper's own format; amax_in: a
    device float tensor holding the maximum Eq. 4 uses (an earlier step's tensor_scale[1:2])."""
    assert amax_in.is_cuda and amax_in.dtype == torch.float32 and amax_in.numel() >= 1
    if yq is None:
        yq = _ts_out(desc, OP_FWD, ROLE_X, xq.codes.device)
    return _conv_ts("mq_conv_fwd_ts", OP_FWD, desc, xq, wq, yq, (ctypes.c_int(act), ctypes.c_void_p(amax_in.data_ptr())), workspace, stream)


def conv_bwd_data_ts(desc, wq, dyq, amax_in, dxq=None, workspace=None, stream=None):
    """mq_conv_bwd_data_ts: the input gradient emitted as the previous layer's stored output gradient in the paper's own format."""
    assert amax_in.is_cuda and amax_in.dtype == torch.float32 and amax_in.numel() >= 1
    if dxq is None:
        dxq = _ts_out(desc, OP_BWD_DATA, ROLE_DY, wq.codes.device)
    return _conv_ts("mq_conv_bwd_data_ts", OP_BWD_DATA, desc, wq, dyq, dxq, (ctypes.c_void_p(amax_in.data_ptr()),), workspace, stream)


STATIC_SCRATCH_BYTES = 16 << 20


def conv_bwd_data_static(desc, wq, dyq, dx=None, layout=NCHW, stream=None):
    """mq_conv_bwd_data_static: the input gradient for callers that cannot allocate device memory (a plug-in
    inside an application that owns the allocator, a frozen memory pool).  The library's own static device
    array serves as scratch; layers needing more than STATIC_SCRATCH_BYTES raise MqError(MQ_ERR_STATIC_SCRATCH).
    `dx` should be passed in by such callers; it is only created here for convenience when omitted."""
    d = ConvDesc(*desc)
    if dx is None:
        dx = _new((d.N, d.C_in, d.H, d.W) if layout == NCHW else (d.H, d.W, d.N, d.C_in), torch.float32, wq.codes.device)
    a, b = wq._c(), dyq._c()
    _check("mq_conv_bwd_data_static", lib().mq_conv_bwd_data_static(ctypes.byref(_d(desc)), ctypes.byref(a), ctypes.byref(b),
                                                                  ctypes.c_void_p(dx.data_ptr()), _DTYPES[dx.dtype], layout, _stream(stream)))
    return dx


def conv_bwd_weight(desc, xq, dyq, dw=None, layout=NCHW, workspace=None, stream=None):
    d = ConvDesc(*desc)
    return _conv("mq_conv_bwd_weight", OP_BWD_WEIGHT, desc, xq, dyq, dw, (d.C_out, d.C_in, d.Kh, d.Kw), (d.C_out, d.Kh, d.Kw, d.C_in), layout, workspace, stream)


def reload_env():
    """mq_reload_env: the MQ_* environment knobs are read once each; call this after changing one."""
    lib().mq_reload_env()


def kernel_launch_count():
    return int(lib().mq_kernel_launch_count())


def last_device_status(stream=None):
    return int(lib().mq_last_device_status(_stream(stream)))


def conv_layer_host_arena_size(desc, fmt_x, fmt_w, fmt_dy):
    b = ctypes.c_size_t()
    _check("mq_conv_layer_host_arena_size", lib().mq_conv_layer_host_arena_size(ctypes.byref(_d(desc)), fmt_x, fmt_w, fmt_dy, ctypes.byref(b)))
    return b.value


def conv_layer_host(desc, fmts, x, w, dy, y, dx, dw, arena, stream=None):
    """mq_conv_layer_host: host fp32 tensors in (pinned for asynchronous copies), host fp32 results out."""
    for t in (x, w, dy, y, dx, dw):
        assert not t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
    assert arena.is_cuda
    _check("mq_conv_layer_host", lib().mq_conv_layer_host(
        ctypes.byref(_d(desc)), fmts[0], fmts[1], fmts[2], ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(w.data_ptr()),
        ctypes.c_void_p(dy.data_ptr()), ctypes.c_void_p(y.data_ptr()), ctypes.c_void_p(dx.data_ptr()), ctypes.c_void_p(dw.data_ptr()),
        ctypes.c_void_p(arena.data_ptr()), ctypes.c_size_t(arena.numel() * arena.element_size()), _stream(stream)))
