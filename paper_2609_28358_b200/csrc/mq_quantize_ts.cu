// Quantizer of the paper's own number format (Sec. III-A): an fp32 scale per tensor (Eq. 4), an E4M3 scale per block
// (Eq. 5), E2M1 elements (Eq. 6), on 16 x 16 square blocks over the two axes Sec. IV-B names for each tensor - the
// square's side set to the tensor core's finest scale granularity (16 elements), the paper's own 8 x 8 being below it.
//
// Two passes when the tensor's own maximum is wanted (Eq. 4 needs max|X| before any element can be scaled):
// tensor_amax_kernel reduces max|X| into the tensor's statistics buffer, quantize_ts_kernel then reads it.  With the
// maximum supplied from outside (statistics of earlier batches, Sec. VII-B) nothing has to wait for this tensor's maximum:
// large NCHW / OIHW tensors then take ONE pass, the whole-line quantizer collecting max|X| for the next step from the block
// maxima it forms anyway; the others keep the separate reduction, which the quantizer does not wait for.
//
// Every operation of Eq. 4-6 is one IEEE single-precision operation, in the order written (division = __fdiv_rn,
// products = __fmul_rn): the roundings decide integer codes, so nothing here may be contracted or approximated.
// CastE4M3 and Round(.) are the hardware's round-to-nearest-even, saturating conversions.
//
// quantize_ts_kernel: one warp per (16 x 16 block, 8 consecutive positions).  Lane (r, h) = (lane >> 1, lane & 1) owns
// row r, channels 8 h .. 8 h + 7 of the block at the 8 positions: 64 values.  From an NCHW source the 8 positions of a
// (row, channel) are 32 contiguous bytes (two 128-bit loads); from a channel-fastest source the 8 channels are.  Block
// maxima are warp reductions (one per position), a lane's 8 codes leave as one 32-bit store, lane 0 writes the block's
// scale bytes.
#include "mq_internal.cuh"

namespace mq {
namespace {

// act: mq_act applied to every element first (the two-launch route of the quantizing epilogue), 0 = none
__global__ void __launch_bounds__(256) tensor_amax_kernel(const float* __restrict__ src, long long n, unsigned* __restrict__ amax_bits, int act) {
  pdl_wait();
  float m = 0.f;
  const long long n4 = (reinterpret_cast<uintptr_t>(src) & 15) == 0 ? n >> 2 : 0;
  const long long stride = (long long)gridDim.x * blockDim.x, t0 = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (long long i = t0; i < n4; i += stride) {
    float4 v = __ldg(reinterpret_cast<const float4*>(src) + i);
    if (act) { v.x = mx_activation(v.x, act); v.y = mx_activation(v.y, act); v.z = mx_activation(v.z, act); v.w = mx_activation(v.w, act); }
    m = fmaxf(fmaxf(m, fmaxf(fabsf(v.x), fabsf(v.y))), fmaxf(fabsf(v.z), fabsf(v.w)));
  }
  for (long long i = 4 * n4 + t0; i < n; i += stride) m = fmaxf(m, fabsf(act ? mx_activation(__ldg(src + i), act) : __ldg(src + i)));
  const unsigned w = __reduce_max_sync(0xffffffffu, __float_as_uint(m));    // bit patterns of non-negative floats order like the values
  if ((threadIdx.x & 31) == 0 && w != 0) atomicMax(amax_bits, w);
}

__device__ __forceinline__ float e4m3_value(unsigned code) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)code, __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half*>(&h));
}

// stats: [0] T_scale (written here), [1] max|X| of this tensor (written by the first pass); amax_src: where Eq. 4 takes
// its maximum from: &stats[1], or the caller's value
template <bool SR>
__global__ void __launch_bounds__(256) quantize_ts_kernel(QuantArgs a, const float* __restrict__ amax_src, float* __restrict__ stats, int Rb, int Cb,
                                                          unsigned n_pstrips, unsigned n_items, int vec) {
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int r_l = lane >> 1, h = lane & 1;
  const float tscale = __fdiv_rn(*amax_src, __fmul_rn(448.0f, 6.0f));                        // Eq. 4
  if (blockIdx.x == 0 && threadIdx.x == 0) stats[0] = tscale;
  const float t6 = __fmul_rn(tscale, 6.0f);
#pragma unroll 1
  for (unsigned it = blockIdx.x * 8u + (threadIdx.x >> 5); it < n_items; it += gridDim.x * 8u) {
    // position strip fastest, then channel block, then row block
    const unsigned ps = it % n_pstrips; const unsigned u = it / n_pstrips;
    const int cb = (int)(u % (unsigned)Cb), rb = (int)(u / (unsigned)Cb);
    const int p0 = (int)ps * 8, r = rb * 16 + r_l, c0 = cb * 16 + 8 * h;
    float v[8][8];   // [channel][position]
#pragma unroll
    for (int k = 0; k < 8; ++k)
#pragma unroll
      for (int j = 0; j < 8; ++j) v[k][j] = 0.f;
    if (r < a.R) {
      if (a.src_stride_r == 0) {   // NCHW / OIHW: element (p, r, c) at (r C + c) P + p
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (c0 + k < a.C) {
            const float* q = a.src + ((long long)r * a.C + c0 + k) * a.P + p0;
            if (vec && p0 + 8 <= a.P) {
              const float4 lo = __ldg(reinterpret_cast<const float4*>(q)), hi = __ldg(reinterpret_cast<const float4*>(q) + 1);
              v[k][0] = lo.x; v[k][1] = lo.y; v[k][2] = lo.z; v[k][3] = lo.w; v[k][4] = hi.x; v[k][5] = hi.y; v[k][6] = hi.z; v[k][7] = hi.w;
            } else {
#pragma unroll
              for (int j = 0; j < 8; ++j) if (p0 + j < a.P) v[k][j] = __ldg(q + j);
            }
          }
        }
      } else {                     // channel-fastest: element (p, r, c) at p stride_p + r stride_r + c
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (p0 + j < a.P) {
            const float* q = a.src + (long long)(p0 + j) * a.src_stride_p + (long long)r * a.src_stride_r + c0;
#pragma unroll
            for (int k = 0; k < 8; ++k) if (c0 + k < a.C) v[k][j] = a.act ? mx_activation(__ldg(q + k), a.act) : __ldg(q + k);
          }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      float m = 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) m = fmaxf(m, fabsf(v[k][j]));
      const float bmax = __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(m)));
      unsigned sc = 0;
      if (bmax > 0.f && tscale > 0.f) sc = (unsigned)__nv_cvt_float_to_fp8(__fdiv_rn(bmax, t6), __NV_SATFINITE, __NV_E4M3) & 0x7Fu;   // Eq. 5
      const float bscale = e4m3_value(sc);
      const bool live = bscale > 0.f && tscale > 0.f;
      const float den = __fmul_rn(bscale, tscale);
      const bool p_ok = p0 + j < a.P;
      if (lane == 0 && p_ok) a.scales[(long long)(p0 + j) * a.sc_stride_p + (long long)rb * a.sc_stride_r + cb] = (uint8_t)sc;
      unsigned word = 0;
#pragma unroll
      for (int k = 0; k < 8; k += 2) {
        float x0 = ts_div(v[k][j], live ? den : 0.f);                                         // Eq. 6
        float x1 = ts_div(v[k + 1][j], live ? den : 0.f);
        if (SR && live) {
          const long long e0 = ((long long)r * a.C + c0 + k) * a.P + p0 + j;
          x0 = sr_value<MQ_E2M1>(x0, (unsigned)e0, sr_key(a, e0));
          x1 = sr_value<MQ_E2M1>(x1, (unsigned)(e0 + a.P), sr_key(a, e0 + a.P));
        }
        word |= encode2<MQ_E2M1>(x0, x1) << (4 * k);
      }
      if (p_ok && r < a.R) {
        const long long e = (long long)(p0 + j) * a.out_stride_p + (long long)r * a.out_stride_r + c0;
        *reinterpret_cast<unsigned*>(a.codes + (e >> 1)) = word;
      }
    }
  }
}

}  // namespace

// stats: device, two floats (T_scale, max|X|).  amax_in: device fp32 to take Eq. 4's maximum from, or null for the
// tensor's own.
cudaError_t launch_quantize_ts(const QuantArgs& a, const float* amax_in, float* stats, cudaStream_t s) {
  const long long n = (long long)a.P * a.R * a.C;
  cudaError_t e = cudaMemsetAsync(stats + 1, 0, sizeof(float), s);
  if (e != cudaSuccess) return e;
  long long blocks = (n / 4 + 255) / 256;
  if (blocks > (long long)sm_count() * 8) blocks = (long long)sm_count() * 8;
  if (blocks < 1) blocks = 1;
  if (a.act && a.src_stride_r == 0) return cudaErrorInvalidValue;   // the activation rides on the channel-fastest source only
  // maximum supplied from outside and the whole-line kernel applies: ONE pass - the quantizer collects this tensor's own
  // maximum for the next step while it works (MQ_QUANT_TS_TWO_PASS=1 keeps the separate reduction)
  if (amax_in && quantize_ts_tma_eligible(a) && !env_int("MQ_QUANT_TS_TWO_PASS", 0)) {
    count_launches(1);
    return launch_quantize_ts_tma(a, amax_in, stats, s, true);
  }
  // the source of either layout is a dense array of n floats
  e = launch_pdl(tensor_amax_kernel, dim3((unsigned)blocks), dim3(256), 0, s, a.src, n, reinterpret_cast<unsigned*>(stats + 1), a.act);
  if (e != cudaSuccess) return e;
  const int Rb = (a.R + 15) / 16, Cb = a.Cp / 16;
  const long long n_pstrips = (a.P + 7) / 8, n_items = n_pstrips * Rb * Cb;
  if (n_items <= 0 || n_items > 0xffffffffLL) return cudaErrorInvalidValue;
  long long qb = (n_items + 7) / 8;
  if (qb > (long long)sm_count() * 32) qb = (long long)sm_count() * 32;
  const int vec = (a.P % 4 == 0 && (reinterpret_cast<uintptr_t>(a.src) & 15) == 0) ? 1 : 0;
  const float* amax_src = amax_in ? amax_in : stats + 1;
  count_launches(2);
  // large NCHW / OIHW tensors with 16-byte rows: the whole-line TMA kernel (items of 32 positions x 32 rows x 32 channels = 4 blocks per position)
  if (quantize_ts_tma_eligible(a)) return launch_quantize_ts_tma(a, amax_src, stats, s);
  if (a.sr) return launch_pdl(quantize_ts_kernel<true>, dim3((unsigned)qb), dim3(256), 0, s, a, amax_src, stats, Rb, Cb, (unsigned)n_pstrips, (unsigned)n_items, vec);
  return launch_pdl(quantize_ts_kernel<false>, dim3((unsigned)qb), dim3(256), 0, s, a, amax_src, stats, Rb, Cb, (unsigned)n_pstrips, (unsigned)n_items, vec);
}

}  // namespace mq
