// Internal declarations shared by the library's translation units (not part of the ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_fp4.h>
#include <cuda_fp6.h>
#include <stdint.h>

#include "mq.h"

namespace mq {

// Derived geometry of one layer (Sec. II-A) and of its stored tensors (Sec. IV-A/B).
struct Geom {
  int N, Cin, H, W, Cout, Kh, Kw, sh, sw, ph, pw;
  int Ho, Wo;
  int Cp, Cop;  // channels rounded up to 32
  int Nt;       // ceil(N / 32)
  int Ct, Cot;  // Cp / 32, Cop / 32
};

inline Geom make_geom(const mq_conv_desc& d) {
  Geom g;
  g.N = d.N; g.Cin = d.C_in; g.H = d.H; g.W = d.W; g.Cout = d.C_out; g.Kh = d.Kh; g.Kw = d.Kw;
  g.sh = d.stride_h; g.sw = d.stride_w; g.ph = d.pad_h; g.pw = d.pad_w;
  g.Ho = (d.H + 2 * d.pad_h - d.Kh) / d.stride_h + 1;
  g.Wo = (d.W + 2 * d.pad_w - d.Kw) / d.stride_w + 1;
  g.Cp = (d.C_in + 31) / 32 * 32;
  g.Cop = (d.C_out + 31) / 32 * 32;
  g.Nt = (d.N + 31) / 32;
  g.Ct = g.Cp / 32;
  g.Cot = g.Cop / 32;
  return g;
}

__host__ __device__ inline int fmt_bits(int fmt) { return fmt == MQ_E2M1 ? 4 : 8; }
__host__ __device__ inline int fmt_emax(int fmt) { return fmt == MQ_E4M3 ? 8 : (fmt == MQ_E5M2 ? 15 : (fmt == MQ_E3M2 ? 4 : 2)); }
__host__ __device__ inline bool fmt_is_6bit(int fmt) { return fmt == MQ_E3M2 || fmt == MQ_E2M3; }
// packed 6-bit storage: the same element formats, 16 codes in 12 bytes
__host__ __device__ inline bool fmt_is_packed6(int fmt) { return fmt == MQ_E3M2_P6 || fmt == MQ_E2M3_P6; }
__host__ __device__ inline int fmt_base(int fmt) { return fmt == MQ_E3M2_P6 ? MQ_E3M2 : (fmt == MQ_E2M3_P6 ? MQ_E2M3 : fmt); }
__host__ __device__ inline int fmt_store_bits(int fmt) { return fmt_is_packed6(fmt) ? 6 : fmt_bits(fmt); }
// 16 one-byte 6-bit codes (four words) -> the 96-bit field of the packed storage: code k in bits 6k .. 6k+5
__host__ __device__ inline void pack6x16(const uint32_t w[4], uint32_t out[3]) {
  uint32_t t[4];
  for (int i = 0; i < 4; ++i) t[i] = (w[i] & 0x3Fu) | ((w[i] >> 2) & 0xFC0u) | ((w[i] >> 4) & 0x3F000u) | ((w[i] >> 6) & 0xFC0000u);
  out[0] = t[0] | (t[1] << 24);
  out[1] = (t[1] >> 8) | (t[2] << 16);
  out[2] = (t[2] >> 16) | (t[3] << 8);
}
// and back: the field's three words -> 16 one-byte codes
__host__ __device__ inline void unpack6x16(const uint32_t in[3], uint32_t w[4]) {
  uint32_t t[4];
  t[0] = in[0] & 0xFFFFFFu;
  t[1] = ((in[0] >> 24) | (in[1] << 8)) & 0xFFFFFFu;
  t[2] = ((in[1] >> 16) | (in[2] << 16)) & 0xFFFFFFu;
  t[3] = in[2] >> 8;
  for (int i = 0; i < 4; ++i) w[i] = (t[i] & 0x3Fu) | ((t[i] & 0xFC0u) << 2) | ((t[i] & 0x3F000u) << 4) | ((t[i] & 0xFC0000u) << 6);
}
// format field of the tcgen05 instruction descriptor (kind::mxf8f6f4)
__host__ __device__ inline unsigned fmt_mma_code(int fmt) { return fmt == MQ_E4M3 ? 0u : (fmt == MQ_E5M2 ? 1u : (fmt == MQ_E2M3 ? 3u : (fmt == MQ_E3M2 ? 4u : 5u))); }

// Number of kernels the library has launched in this process (diagnostic; see mq_kernel_launch_count).
void count_launches(int n);

// Streaming multiprocessors of the current device (148 on a B200); grids are sized in multiples of it.
inline int sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return 148;
  return sms;
}

// Integer value of an MQ_* environment knob.  Each knob is read from the environment ONCE, on its first use in the
// process, and answered from a table afterwards, so that a size query and the call it sizes always see the same plan;
// mq_reload_env() (a diagnostic entry point) empties the table.
int env_int(const char* name, int dflt);

// ---- launchers (defined in the .cu files) ---------------------------------------------------
struct QuantArgs {
  const float* src;
  uint8_t* codes;
  uint8_t* scales;
  int P, R, C, Cp;                 // positions, rows of the 2-D view, channels, padded channels
  long long out_stride_p, out_stride_r;  // in elements of the codes tensor
  long long sc_stride_p, sc_stride_r;    // in scale bytes
  int fmt;
  // source strides in floats when the source has the channel axis fastest (fp32 [H][W][N][C] / [Cout][Kh][Kw][Cin]):
  // element (p, r, c) at p * src_stride_p + r * src_stride_r + c; both zero for the NCHW / OIHW source
  long long src_stride_p, src_stride_r;
  // stochastic rounding (Eq. 6 with the stochastic Round(.), Sec. III-A): 0 = round to nearest even
  int sr;
  unsigned sr_seed_lo, sr_seed_hi;   // the 64-bit seed
  unsigned sr_key0;                  // stream key of elements whose index is below 2^32 (computed on the host)
  int sr_wide;                       // 1: the tensor has 2^32 elements or more (keys are derived per element)
  int act;                           // mq_act applied to every element before quantization (channel-fastest source only; 0: none)
  int line;                          // 1: line blocks (one scale per row and 32 channels; the sc strides are per row), 0: 32 x 32 tiles
  unsigned int* status;              // device status word: set when a bounded wait gives up
  // test hooks of the TMA kernel's abort path: polls a barrier wait may take (0: the default limit), and 1 = the loader
  // issues no copies, so that every wait on them runs out
  unsigned wait_limit;
  int debug_skip_loads;
  // the paper's own format on the whole-line kernel (launch_quantize_ts_tma): where Eq. 4 takes max|X| from, and the
  // tensor's statistics buffer (T_scale is written to [0])
  const float* ts_amax;
  float* ts_stats;
  int packed6;        // 1: 6-bit codes leave packed, 16 codes in 12 bytes (out strides stay in elements)
  int ts_track_max;   // 1: the kernel also collects max|X| into ts_stats[1] (maximum supplied from outside: the tensor is read once)
};
// invertible 32-bit mixer (xor-shift, odd multiply, twice, xor-shift) behind the per-element draws
__host__ __device__ __forceinline__ unsigned sr_mix32(unsigned x) {
  x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15; x *= 0x846CA68Bu; x ^= x >> 16;
  return x;
}
cudaError_t launch_quantize(const QuantArgs& a, cudaStream_t s);
// The paper's own format (fp32 tensor scale, E4M3 scale per 16 x 16 block, E2M1 elements; mq_quantize_ts.cu).  stats: device, two
// floats (T_scale, max|X|); amax_in: device fp32 that Eq. 4 takes its maximum from, or null for the tensor's own.
cudaError_t launch_quantize_ts(const QuantArgs& a, const float* amax_in, float* stats, cudaStream_t s);
// Second pass of that quantizer on the whole-line TMA kernel (NCHW / OIHW source with 16-byte rows): true if the tensor qualifies
bool quantize_ts_tma_eligible(const QuantArgs& a);
cudaError_t launch_quantize_ts_tma(const QuantArgs& a, const float* amax_src, float* stats, cudaStream_t s, bool track_max = false);

struct Im2colArgs {
  const uint8_t* codes;
  const uint8_t* scales;
  uint8_t* out_codes;
  uint8_t* out_scales;
  Geom g;
  int fmt;
  int line;   // 1: line blocks (scales per sample instead of per 32 samples)
  int ts16;   // 1: 16 x 16 blocks (scales per 16 samples and 16 channels)
};
cudaError_t launch_im2col(const Im2colArgs& a, cudaStream_t s);

struct ConvArgs {
  Geom g;
  const uint8_t* a_codes;  // first operand of the call (fwd: X, bwd_data: W, bwd_weight: X)
  const uint8_t* a_scales;
  const uint8_t* b_codes;  // second operand (fwd: W, bwd_data: G_Y, bwd_weight: G_Y)
  const uint8_t* b_scales;
  int fmt_a, fmt_b;
  float* out;
  int out_layout;
  void* workspace;
  size_t ws_bytes;
  int line;   // 1: both operands carry line-block scales (one per row), forward GEMM only
  int ts16;   // 1: both operands are in the paper's own format: E4M3 scales per 16 x 16 block and a tensor scale each
  const float* a_tscale;   // device: T_scale of the first / second operand (ts16)
  const float* b_tscale;
};
// CUDA-core implicit-GEMM kernels: every shape, every format pair.
cudaError_t launch_conv_generic(int op, const ConvArgs& a, cudaStream_t s);
size_t conv_generic_workspace(int op, const Geom& g);
int conv_generic_bwd_weight_splits(const Geom& g);

// ---- device helpers --------------------------------------------------------------------------
#ifdef __CUDACC__

// 2^(code-127) as fp32 (code 0 gives the subnormal 2^-127)
__device__ __forceinline__ float e8m0_to_float(unsigned code) {
  return code == 0 ? __uint_as_float(0x00400000u) : __uint_as_float(code << 23);
}

// Exact decode of 8 consecutive codes (K- or MN-contiguous in memory) to fp32, times `scale`.
template <int FMT>
__device__ __forceinline__ void decode8(const uint8_t* codes_base, long long elem_off, float scale, float* out, int fmt8 = FMT) {
  // FMT: MQ_E2M1 (packed nibbles) or any other value for the one-byte-per-code formats, whose actual format is fmt8
  if (FMT == MQ_E2M1) {
    uint32_t v = *reinterpret_cast<const uint32_t*>(codes_base + (elem_off >> 1));
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __half2_raw h = __nv_cvt_fp4x2_to_halfraw2((__nv_fp4x2_storage_t)((v >> (8 * i)) & 0xFF), __NV_E2M1);
      float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
      out[2 * i] = f.x * scale;
      out[2 * i + 1] = f.y * scale;
    }
  } else {
    uint2 v = *reinterpret_cast<const uint2*>(codes_base + elem_off);
    uint32_t w[2] = {v.x, v.y};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      unsigned short pair = (unsigned short)((w[i >> 1] >> (16 * (i & 1))) & 0xFFFF);
      __half2_raw h;
      if (fmt8 == MQ_E4M3) h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)pair, __NV_E4M3);
      else if (fmt8 == MQ_E5M2) h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)pair, __NV_E5M2);
      else if (fmt8 == MQ_E3M2) h = __nv_cvt_fp6x2_to_halfraw2((__nv_fp6x2_storage_t)pair, __NV_E3M2);
      else h = __nv_cvt_fp6x2_to_halfraw2((__nv_fp6x2_storage_t)pair, __NV_E2M3);
      float2 f = __half22float2(*reinterpret_cast<__half2*>(&h));
      out[2 * i] = f.x * scale;
      out[2 * i + 1] = f.y * scale;
    }
  }
}

// ---- quantization arithmetic shared by the quantizer kernels and the quantizing GEMM epilogue (Eq. 5-6, E8M0 form) ----
template <int FMT>
__device__ __forceinline__ unsigned encode2(float lo, float hi) {
  // two elements -> two codes (lo in the low byte / nibble), round-to-nearest-even, saturating
  if (FMT == MQ_E2M1) {
    return (unsigned)__nv_cvt_float2_to_fp4x2(make_float2(lo, hi), __NV_E2M1, cudaRoundNearest);
  } else if (FMT == MQ_E3M2 || FMT == MQ_E2M3) {
    // two 6-bit codes, each in the low six bits of its byte (the container the tensor core reads)
    return (unsigned)__nv_cvt_float2_to_fp6x2(make_float2(lo, hi), FMT == MQ_E3M2 ? __NV_E3M2 : __NV_E2M3, cudaRoundNearest);
  } else {
    return (unsigned)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, FMT == MQ_E4M3 ? __NV_E4M3 : __NV_E5M2);
  }
}

// x / den of Eq. 6 (den = Scale_b x T_scale, or 0 for an all-zero block / tensor: the element is then a signed zero).  A zero
// numerator would send __fdiv_rn down its slow path (a call that the whole warp waits for - post-ReLU tensors are half
// zeros: measured 2x on the quantizing epilogue), so zeros divide a stand-in and keep their sign; the quotient of every
// other value is the IEEE one.
__device__ __forceinline__ float ts_div(float x, float den) {
  const bool z = x == 0.f || !(den > 0.f);
  const float q = __fdiv_rn(z ? 1.f : x, z ? 1.f : den);
  return z ? copysignf(0.f, x) : q;
}

// activation of the quantizing producer epilogue (mq_act), evaluated in fp32
__device__ __forceinline__ float mx_activation(float y, int act) {
  if (act == MQ_ACT_RELU) return fmaxf(y, 0.f);
  if (act == MQ_ACT_SILU) return __fdividef(y, 1.f + __expf(-y));
  return y;
}

__device__ __forceinline__ int scale_code_of(unsigned amax_bits, int emax) {
  // floor(log2 amax) = biased exponent - 127 for normal amax; subnormal / zero amax clamps to 0
  const int e = (int)(amax_bits >> 23) - emax;
  return min(max(e, 0), 254);
}

// 2^(127 - code) as a normal fp32 number: code = clamp(E - emax, 0, 254) with E <= 254 and emax >= 2, so
// 127 - code lies in [-125, 127].  x * 2^(127 - code) is then exact (|result| < 2^(emax + 1)) except where it
// underflows below 2^-126, far under half of the smallest element step, where it rounds to zero either way.
__device__ __forceinline__ float scale_factor(int code) { return __uint_as_float((unsigned)(254 - code) << 23); }

// Stochastic Round(.) of Eq. 6 (Sec. III-A: the gradient's rounding).  x is the scaled element, idx its index in the
// logical NCHW / OIHW tensor.  The element's draw is 32 bits of a counter-based generator keyed by (seed, idx);
// u = (top 23 bits + 1/2) / 2^23.  With lo <= |x| < hi neighbours on the format's grid, the result is hi when
// u < (|x| - lo) / (hi - lo), else lo -- returned as a float that lies on the grid, so the round-to-nearest
// conversion that follows is exact.  Everything below is exact in fp32: |x| / step has at most 24 significant bits,
// its fractional part and (23-bit draw + 1/2) likewise.  Magnitudes at or beyond the largest one are left to the
// conversion's saturation.
// lo: low word of the element's index; key: the stream key of its high word (sr_key)
template <int FMT>
__device__ __forceinline__ float sr_value(float x, unsigned lo, unsigned key) {
  constexpr int M = (FMT == MQ_E4M3 || FMT == MQ_E2M3) ? 3 : (FMT == MQ_E2M1 ? 1 : 2);                      // mantissa bits
  constexpr int EMIN = FMT == MQ_E4M3 ? -6 : (FMT == MQ_E5M2 ? -14 : (FMT == MQ_E3M2 ? -2 : 0));           // smallest normal exponent
  // fp32 pattern of the largest magnitude: 448, 57344, 6, 28, 7.5
  constexpr unsigned MAXBITS = FMT == MQ_E4M3 ? 0x43E00000u : (FMT == MQ_E5M2 ? 0x47600000u : (FMT == MQ_E2M1 ? 0x40C00000u : (FMT == MQ_E3M2 ? 0x41E00000u : 0x40F00000u)));
  const unsigned b = __float_as_uint(x) & 0x7fffffffu;       // |x|; patterns of non-negative floats order like their values
  const unsigned r23 = sr_mix32(lo ^ key) >> 9;
  // normal range of the format: the grid keeps M mantissa bits of the fp32 pattern.  The dropped field f (23 - M bits)
  // is the fraction of a step in units of 2^-(23 - M): f * 2^M > draw + 1/2 is an integer comparison, and stepping up
  // is an integer addition on the pattern (the carry walks into the exponent at a binade's end).
  constexpr unsigned MASK = (1u << (23 - M)) - 1u;
  const unsigned f = b & MASK;
  const unsigned q_norm = (b - f) + (((f << M) > r23) ? MASK + 1u : 0u);
  // below it the step is the constant 2^(EMIN - M): t = |x| / step < 2^M, floor through a round-down addition of 2^23,
  // draw + 1/2 as (2^23 + draw) - (2^23 - 1/2); all exact
  const float t = __uint_as_float(b) * __uint_as_float((unsigned)(127 + M - EMIN) << 23);
  const float fl = __fadd_rd(t, 8388608.f) - 8388608.f;
  const float u = __uint_as_float(0x4B000000u | r23) - 8388607.5f;
  const float up = (t - fl) * 8388608.f > u ? 1.f : 0.f;
  const unsigned q_sub = __float_as_uint((fl + up) * __uint_as_float((unsigned)(127 + EMIN - M) << 23));
  unsigned q = b >= ((unsigned)(127 + EMIN) << 23) ? q_norm : q_sub;
  q = b < MAXBITS ? q : b;      // at or beyond the largest magnitude: left to the conversion's saturation
  return __uint_as_float(q | (__float_as_uint(x) & 0x80000000u));
}
// Stream key of an element from the high word of its index; tensors below 2^32 elements (a.sr_wide == 0, uniform)
// take the key computed on the host.
__device__ __forceinline__ unsigned sr_key(const QuantArgs& a, long long idx) {
  if (!a.sr_wide) return a.sr_key0;
  return sr_mix32(a.sr_seed_lo ^ sr_mix32(a.sr_seed_hi ^ sr_mix32((unsigned)((unsigned long long)idx >> 32))));
}

#endif  // __CUDACC__

// ---- programmatic dependent launch --------------------------------------------------------------------------
// Kernels of this library are launched with programmatic stream serialization: a kernel may be scheduled while its
// predecessor in the stream is still draining, and executes pdl_wait() (griddepcontrol.wait: returns once the
// predecessor grid has completed and its writes are visible) before its first access to global memory.  Every
// kernel waits, so completion is transitive along the stream.  MQ_NO_PDL=1 launches them plainly.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
bool pdl_enabled();
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// the same with thread-block clusters of `cluster_x` consecutive blocks (grid.x a multiple of it)
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, unsigned cluster_x, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_x; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace mq
