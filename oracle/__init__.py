"""CPU oracle for the MicroQonv hot path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes/numpy wrapper around ``mq_oracle.cpp`` (plain C++, compiled with g++).  Only the
tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the CUDA
library and its Python binding never do, and nothing here imports them.

All arrays are host numpy arrays.  Conventions (Sec. II-A, IV-A, IV-B of the paper):
  * ``desc`` = ConvDesc(N, C_in, H, W, C_out, Kh, Kw, stride_h, stride_w, pad_h, pad_w)
  * roles: X (activations, NCHW), W (weights, OIHW), DY (output gradient, N.Cout.Ho.Wo)
  * element formats: E4M3, E5M2, E3M2, E2M3 (one byte per code), E2M1 (two codes per byte, lower index in
    the low nibble); block scale E8M0; pack6 / unpack6 give the packed storage of the 6-bit codes (16 in 12 bytes)
  * block shape (br, bc): br along N (X, DY) or Cout (W); bc along the channel axis that is
    stored fastest.  (32, 32) is the square block, (1, 32) the line block.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from collections import namedtuple

import numpy as np

E4M3, E5M2, E2M1, E3M2, E2M3 = 0, 1, 2, 3, 4
ROLE_X, ROLE_W, ROLE_DY = 0, 1, 2
FMT_BITS = {E4M3: 8, E5M2: 8, E2M1: 4, E3M2: 8, E2M3: 8}   # stored bits per code (6-bit codes: one per byte)
FMT_EMAX = {E4M3: 8, E5M2: 15, E2M1: 2, E3M2: 4, E2M3: 2}

ConvDesc = namedtuple("ConvDesc", "N C_in H W C_out Kh Kw stride_h stride_w pad_h pad_w")

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mq_oracle.cpp")
_LIB = os.path.join(_HERE, "libmq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (g++ -O2 -fopenmp).  Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _l():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.orc_decode_elem.restype = ctypes.c_double
        lib.orc_decode_elem.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.orc_encode_elem.restype = ctypes.c_int
        lib.orc_encode_elem.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.orc_scale_code.restype = ctypes.c_int
        lib.orc_scale_code.argtypes = [ctypes.c_int, ctypes.c_double]
        lib.orc_encode_elem_sr.restype = ctypes.c_int
        lib.orc_encode_elem_sr.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_uint32]
        lib.orc_sr_bits.restype = ctypes.c_uint32
        lib.orc_sr_bits.argtypes = [ctypes.c_uint64, ctypes.c_uint64]
        lib.orc_quantize_sr.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_uint64,
                                        ctypes.c_void_p, ctypes.c_void_p]
        lib.orc_quantize_ts.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_float, ctypes.c_int, ctypes.c_uint64,
                                        ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        lib.orc_dequant_ts.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_float, ctypes.c_void_p]
        lib.orc_block_scale_code.argtypes = [ctypes.c_float, ctypes.c_float]
        lib.orc_ts_elem_code.argtypes = [ctypes.c_float, ctypes.c_float, ctypes.c_float]
        _lib = lib
    return _lib


def _desc(desc) -> np.ndarray:
    return np.asarray(list(desc), dtype=np.int32)


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def num_threads() -> int:
    return int(_l().orc_num_threads())


def decode_elem(fmt: int, code: int) -> float:
    return float(_l().orc_decode_elem(fmt, int(code)))


def encode_elem(fmt: int, v: float) -> int:
    return int(_l().orc_encode_elem(fmt, float(v)))


def encode_elem_sr(fmt: int, v: float, bits: int) -> int:
    """Stochastic Round(.) of Eq. 6 for one scaled value, given the element's 32 random bits."""
    return int(_l().orc_encode_elem_sr(fmt, float(v), int(bits) & 0xFFFFFFFF))


def sr_bits(seed: int, index: int) -> int:
    """The 32 random bits of element `index` (position in the logical NCHW / OIHW tensor) under `seed`."""
    return int(_l().orc_sr_bits(int(seed), int(index)))


def scale_code(fmt: int, amax: float) -> int:
    return int(_l().orc_scale_code(fmt, float(amax)))


def out_hw(desc):
    d = ConvDesc(*desc)
    return ((d.H + 2 * d.pad_h - d.Kh) // d.stride_h + 1, (d.W + 2 * d.pad_w - d.Kw) // d.stride_w + 1)


def logical_shape(desc, role):
    d = ConvDesc(*desc)
    if role == ROLE_X:
        return (d.N, d.C_in, d.H, d.W)
    if role == ROLE_W:
        return (d.C_out, d.C_in, d.Kh, d.Kw)
    ho, wo = out_hw(d)
    return (d.N, d.C_out, ho, wo)


def qtensor_sizes(desc, role, fmt, block=(32, 32)):
    cb, sb = ctypes.c_int64(), ctypes.c_int64()
    _l().orc_qtensor_sizes(_p(_desc(desc)), role, fmt, block[0], block[1], ctypes.byref(cb), ctypes.byref(sb))
    return cb.value, sb.value


def quantize(desc, role, fmt, src, block=(32, 32)):
    """fp32 logical tensor -> (codes uint8[...], scales uint8[...]) in the stored order."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    assert src.shape == logical_shape(desc, role), (src.shape, logical_shape(desc, role))
    assert np.isfinite(src).all(), "non-finite inputs are outside the contract"
    cb, sb = qtensor_sizes(desc, role, fmt, block)
    codes = np.zeros(cb, dtype=np.uint8)
    scales = np.zeros(sb, dtype=np.uint8)
    rc = _l().orc_quantize(_p(_desc(desc)), role, fmt, block[0], block[1], _p(src), _p(codes), _p(scales))
    assert rc == 0
    return codes, scales


def quantize_sr(desc, role, fmt, src, seed, block=(32, 32)):
    """As quantize(), with the stochastic Round(.) of Eq. 6 (Sec. III-A: the gradient's rounding)."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    assert src.shape == logical_shape(desc, role), (src.shape, logical_shape(desc, role))
    assert np.isfinite(src).all(), "non-finite inputs are outside the contract"
    cb, sb = qtensor_sizes(desc, role, fmt, block)
    codes = np.zeros(cb, dtype=np.uint8)
    scales = np.zeros(sb, dtype=np.uint8)
    rc = _l().orc_quantize_sr(_p(_desc(desc)), role, fmt, block[0], block[1], _p(src), int(seed), _p(codes), _p(scales))
    assert rc == 0
    return codes, scales


def quantize_ts(desc, role, src, block=(16, 16), amax=None, seed=None):
    """The paper's own number format (Sec. III-A, Eq. 4-6): fp32 scale per tensor, E4M3 scale per block, E2M1 elements.
    Returns (codes, block scales as E4M3 bytes, T_scale, max|X|).  amax: take T_scale from this value instead of the
    tensor's own maximum (statistics of earlier batches, Sec. VII-B).  seed: stochastic Round(.) with that seed."""
    src = np.ascontiguousarray(src, dtype=np.float32)
    assert src.shape == logical_shape(desc, role), (src.shape, logical_shape(desc, role))
    assert np.isfinite(src).all(), "non-finite inputs are outside the contract"
    cb, sb = qtensor_sizes(desc, role, E2M1, block)
    codes = np.zeros(cb, dtype=np.uint8)
    scales = np.zeros(sb, dtype=np.uint8)
    ts, am = np.zeros(1, dtype=np.float32), np.zeros(1, dtype=np.float32)
    rc = _l().orc_quantize_ts(_p(_desc(desc)), role, block[0], block[1], _p(src), ctypes.c_float(-1.0 if amax is None else float(amax)),
                              0 if seed is None else 1, 0 if seed is None else int(seed), _p(codes), _p(scales), _p(ts), _p(am))
    assert rc == 0
    return codes, scales, float(ts[0]), float(am[0])


def dequant_ts(desc, role, codes, scales, tensor_scale, block=(16, 16)):
    """Fake quantization of the paper's own format: element x block scale x tensor scale, float64, logical order."""
    out = np.zeros(logical_shape(desc, role), dtype=np.float64)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    _l().orc_dequant_ts(_p(_desc(desc)), role, block[0], block[1], _p(codes), _p(scales), ctypes.c_float(tensor_scale), _p(out))
    return out


def block_scale_code(block_amax, tensor_scale):
    """Eq. 5 for one block: the E4M3 code of max|X_i| / (T_scale * 6)."""
    return int(_l().orc_block_scale_code(ctypes.c_float(block_amax), ctypes.c_float(tensor_scale)))


def ts_elem_code(x, block_scale, tensor_scale):
    """Eq. 6 for one element (round to nearest): the E2M1 code of x / (B_scale * T_scale)."""
    return int(_l().orc_ts_elem_code(ctypes.c_float(x), ctypes.c_float(block_scale), ctypes.c_float(tensor_scale)))


def dequant(desc, role, fmt, codes, scales, block=(32, 32)):
    """stored MX tensor -> float64 logical tensor (fake quantization)."""
    out = np.zeros(logical_shape(desc, role), dtype=np.float64)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    _l().orc_dequant(_p(_desc(desc)), role, fmt, block[0], block[1], _p(codes), _p(scales), _p(out))
    return out


def pack6(codes):
    """Packed storage of a tensor of 6-bit codes (Sec. VI counts six bits per element for the 6-bit formats): the low six
    bits of every code as one little-endian bit stream - code k of the flat array occupies bits 6k .. 6k+5 - so that 16
    codes take 12 bytes.  Layout only: no arithmetic of the method."""
    c = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    assert c.size % 4 == 0 and int(c.max(initial=0)) < 64
    bits = np.unpackbits(c[:, None], axis=1, bitorder="little")[:, :6]
    return np.packbits(bits.reshape(-1), bitorder="little")


def unpack6(packed):
    """Inverse of pack6: one code per byte."""
    b = np.ascontiguousarray(packed, dtype=np.uint8).reshape(-1)
    assert b.size % 3 == 0
    bits = np.unpackbits(b, bitorder="little").reshape(-1, 6)
    return np.packbits(np.pad(bits, ((0, 0), (0, 2))), axis=1, bitorder="little").reshape(-1)


def im2col_sizes(desc, fmt, block=(32, 32)):
    cb, sb = ctypes.c_int64(), ctypes.c_int64()
    _l().orc_im2col_sizes(_p(_desc(desc)), fmt, block[0], block[1], ctypes.byref(cb), ctypes.byref(sb))
    return cb.value, sb.value


def cbf_im2col(desc, fmt, codes, scales, block=(32, 32)):
    cb, sb = im2col_sizes(desc, fmt, block)
    oc = np.zeros(cb, dtype=np.uint8)
    osc = np.zeros(sb, dtype=np.uint8)
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    scales = np.ascontiguousarray(scales, dtype=np.uint8)
    _l().orc_cbf_im2col(_p(_desc(desc)), fmt, block[0], block[1], _p(codes), _p(scales), _p(oc), _p(osc))
    return oc, osc


def _conv(fn, desc, a, b, out_shape, idx):
    a = np.ascontiguousarray(a, dtype=np.float64)
    b = np.ascontiguousarray(b, dtype=np.float64)
    if idx is None:
        count = int(np.prod(out_shape))
        y = np.zeros(out_shape, dtype=np.float64)
        ya = np.zeros(out_shape, dtype=np.float64)
        ip = None
    else:
        idx = np.ascontiguousarray(idx, dtype=np.int64)
        count = idx.size
        y = np.zeros(count, dtype=np.float64)
        ya = np.zeros(count, dtype=np.float64)
        ip = idx
    fn(_p(_desc(desc)), _p(a), _p(b), _p(ip), ctypes.c_int64(count), _p(y), _p(ya))
    return y, ya


def conv_fwd(desc, x, w, idx=None):
    """Y = W * X (Eq. 1) on float64 tensors; returns (Y, sum|terms|).  idx: flat output indices."""
    return _conv(_l().orc_conv_fwd, desc, x, w, logical_shape(desc, ROLE_DY), idx)


def conv_bwd_data(desc, w, g, idx=None):
    """G_X (Eq. 2, the adjoint of Eq. 1 in X); returns (G_X, sum|terms|)."""
    return _conv(_l().orc_conv_bwd_data, desc, w, g, logical_shape(desc, ROLE_X), idx)


def conv_bwd_weight(desc, g, x, idx=None):
    """G_W (Eq. 3); returns (G_W, sum|terms|)."""
    return _conv(_l().orc_conv_bwd_weight, desc, g, x, logical_shape(desc, ROLE_W), idx)
