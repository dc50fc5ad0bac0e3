// Single-pass MX quantizer (Sec. III-A, Eq. 5-6 in the E8M0 form; square blocks of Sec. IV-B) that
// also re-lays the tensor into its channel-batch-first stored order (Sec. IV-A).
//
// The logical source (NCHW / OIHW fp32) is seen as R x C matrices at P positions with the position
// axis fastest in memory: element (p, r, c) lives at (r*C + c)*P + p.  One thread block owns one
// 32(r) x 32(c) tile at PS = 8 consecutive positions: 1024 source rows x 32 bytes, every 32-byte
// sector read exactly once with 128-bit loads.  Per position it reduces |x| over the tile
// (per-thread max, warp shuffles, one shared-memory exchange), derives the E8M0 code from the
// exponent field of the maximum, converts with the hardware RNE+saturate conversions and stages
// the codes in shared memory so the [n][c] slab of each position leaves as 16-byte stores.
#include <cstdlib>

#include "mq_internal.cuh"

namespace mq {
namespace {

constexpr int PS = 8;           // positions per block
constexpr int QT_THREADS = 256;

template <int FMT>
__device__ __forceinline__ unsigned encode2(float lo, float hi) {
  // two elements -> two codes (lo in the low byte / nibble), round-to-nearest-even, saturating
  if (FMT == MQ_E2M1) {
    return (unsigned)__nv_cvt_float2_to_fp4x2(make_float2(lo, hi), __NV_E2M1, cudaRoundNearest);
  } else {
    return (unsigned)__nv_cvt_float2_to_fp8x2(make_float2(lo, hi), __NV_SATFINITE, FMT == MQ_E4M3 ? __NV_E4M3 : __NV_E5M2);
  }
}

// 128-bit read-only load that asks L2 to bring in the whole 128-byte line (the other sectors of the
// line are read next, by this block's following sub-strips)
__device__ __forceinline__ float4 ldg128_l2_128(const float* p) {
  float4 v;
  asm volatile("ld.global.nc.L2::128B.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

template <int FMT, bool VEC>
__global__ void __launch_bounds__(QT_THREADS) quantize_kernel(QuantArgs a, int n_pstrips, int Rt, int Ct, int loops, int hint) {
  __shared__ __align__(16) unsigned red[8][2][4];          // per-warp, per-quad partial maxima
  __shared__ __align__(16) uint8_t stage[PS][32][32];       // codes, one byte each, [p][r][c]

  const int t = threadIdx.x;
  const int lane = t & 31, warp = t >> 5;
  long long bid = blockIdx.x;
  const int n_groups = (n_pstrips + loops - 1) / loops;
  const int psg = (int)(bid % n_groups); bid /= n_groups;
  const int ct = (int)(bid % Ct);
  const int rt = (int)(bid / Ct);
  const int r0 = rt * 32, c0 = ct * 32;
  for (int sub = 0; sub < loops; ++sub) {
  const int ps = psg * loops + sub;
  if (ps >= n_pstrips) break;
  const int p0 = ps * PS;
  if (sub > 0) __syncthreads();   // previous sub-strip's copy-out has finished reading `stage` / `red`

  // thread -> (channel, position quad); 8 rows of the tile: r = 4*i + t/64
  const int quad = t & 1;
  const int c = (t >> 1) & 31;
  const int rsub = t >> 6;
  const int pq = p0 + 4 * quad;

  float v[8][4];
  const bool c_ok = (c0 + c) < a.C;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = r0 + 4 * i + rsub;
    const bool ok = c_ok && r < a.R;
    const float* row = a.src + ((long long)r * a.C + (c0 + c)) * a.P;
    if (VEC) {
      float4 f = make_float4(0.f, 0.f, 0.f, 0.f);
      if (ok && pq < a.P) f = hint ? ldg128_l2_128(row + pq) : __ldg(reinterpret_cast<const float4*>(row + pq));  // P % 4 == 0: whole quad valid
      v[i][0] = f.x; v[i][1] = f.y; v[i][2] = f.z; v[i][3] = f.w;
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) v[i][j] = (ok && pq + j < a.P) ? __ldg(row + pq + j) : 0.f;
    }
  }

  // amax per position over the 32 x 32 tile, on the bit patterns of |x| (order-preserving)
  unsigned m[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    unsigned mm = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) mm = max(mm, __float_as_uint(v[i][j]) & 0x7fffffffu);
#pragma unroll
    for (int off = 2; off < 32; off <<= 1) mm = max(mm, __shfl_xor_sync(0xffffffffu, mm, off));
    m[j] = mm;
  }
  if (lane < 2) {
#pragma unroll
    for (int j = 0; j < 4; ++j) red[warp][lane][j] = m[j];
  }
  __syncthreads();
  unsigned code[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    unsigned mm = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) mm = max(mm, red[w][quad][j]);
    // floor(log2 amax) = biased exponent - 127 for normal amax; subnormal / zero amax clamps to 0
    int e = (int)(mm >> 23) - fmt_emax(FMT);
    code[j] = (unsigned)min(max(e, 0), 254);
  }
  if (t < PS) {  // thread t holds position p0 + t in quad t/4 only if its own quad matches: recompute
    unsigned mm = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) mm = max(mm, red[w][t >> 2][t & 3]);
    int e = (int)(mm >> 23) - fmt_emax(FMT);
    if (p0 + t < a.P) a.scales[(long long)(p0 + t) * a.sc_stride_p + (long long)rt * a.sc_stride_r + ct] = (uint8_t)min(max(e, 0), 254);
  }

  // x * 2^(127 - code), exact: split the power of two so both factors are normal numbers
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int ex = 127 - (int)code[j];       // in [-127, 127]
    const int e1 = ex / 2, e2 = ex - e1;      // |e1|, |e2| <= 64
    const float f1 = __uint_as_float((unsigned)(e1 + 127) << 23);
    const float f2 = __uint_as_float((unsigned)(e2 + 127) << 23);
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      unsigned two = encode2<FMT>(v[i][j] * f1 * f2, v[i + 1][j] * f1 * f2);
      unsigned lo, hi;
      if (FMT == MQ_E2M1) { lo = two & 0xF; hi = (two >> 4) & 0xF; }
      else { lo = two & 0xFF; hi = (two >> 8) & 0xFF; }
      stage[4 * quad + j][4 * i + rsub][c] = (uint8_t)lo;
      stage[4 * quad + j][4 * (i + 1) + rsub][c] = (uint8_t)hi;
    }
  }
  __syncthreads();

  // copy out: per position a 32(r) x 32(c) slab; rows are contiguous runs of the stored tensor
  if (FMT == MQ_E2M1) {
    // 256 rows (p, r), 16 bytes each after packing two codes per byte
    const int p = t >> 5, r = t & 31;
    if (p0 + p < a.P && r0 + r < a.R) {
      const uint4* srcw = reinterpret_cast<const uint4*>(&stage[p][r][0]);
      uint4 lo = srcw[0], hi = srcw[1];
      uint32_t in[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
      uint32_t outw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        // 8 one-byte codes (two words) -> one word of 8 nibbles, lower index in the lower nibble
        uint32_t w0 = in[2 * k], w1 = in[2 * k + 1];
        uint32_t b0 = (w0 & 0xF) | ((w0 >> 4) & 0xF0) | ((w0 >> 8) & 0xF00) | ((w0 >> 12) & 0xF000);
        uint32_t b1 = (w1 & 0xF) | ((w1 >> 4) & 0xF0) | ((w1 >> 8) & 0xF00) | ((w1 >> 12) & 0xF000);
        outw[k] = b0 | (b1 << 16);
      }
      long long e = (long long)(p0 + p) * a.out_stride_p + (long long)(r0 + r) * a.out_stride_r + c0;
      *reinterpret_cast<uint4*>(a.codes + (e >> 1)) = make_uint4(outw[0], outw[1], outw[2], outw[3]);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int id = t + QT_THREADS * k;  // 512 chunks of 16 bytes
      const int p = id >> 6, r = (id >> 1) & 31, half = id & 1;
      if (p0 + p < a.P && r0 + r < a.R) {
        uint4 val = *reinterpret_cast<const uint4*>(&stage[p][r][16 * half]);
        long long e = (long long)(p0 + p) * a.out_stride_p + (long long)(r0 + r) * a.out_stride_r + c0 + 16 * half;
        *reinterpret_cast<uint4*>(a.codes + e) = val;
      }
    }
  }
  }  // sub-strips
}

}  // namespace

cudaError_t launch_quantize(const QuantArgs& a, cudaStream_t s) {
  const int n_pstrips = (a.P + PS - 1) / PS;
  const int Rt = (a.R + 31) / 32, Ct = a.Cp / 32;
  static int variant = -1;
  if (variant < 0) { const char* v = std::getenv("MQ_QUANT_VARIANT"); variant = v ? std::atoi(v) : 0; }
  const int hint = variant >= 1 ? 1 : 0;
  int loops = variant >= 2 ? 4 : 1;
  if (variant == 3) loops = 2;
  const long long blocks = (long long)((n_pstrips + loops - 1) / loops) * Rt * Ct;
  if (blocks <= 0 || blocks > 0x7fffffffLL) return cudaErrorInvalidValue;
  const bool vec = (a.P % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.src) & 15) == 0);
#define MQ_LAUNCH_Q(F)                                                                                  \
  do {                                                                                                  \
    if (vec) quantize_kernel<F, true><<<(unsigned)blocks, QT_THREADS, 0, s>>>(a, n_pstrips, Rt, Ct, loops, hint);    \
    else     quantize_kernel<F, false><<<(unsigned)blocks, QT_THREADS, 0, s>>>(a, n_pstrips, Rt, Ct, loops, hint);   \
  } while (0)
  switch (a.fmt) {
    case MQ_E4M3: MQ_LAUNCH_Q(MQ_E4M3); break;
    case MQ_E5M2: MQ_LAUNCH_Q(MQ_E5M2); break;
    case MQ_E2M1: MQ_LAUNCH_Q(MQ_E2M1); break;
    default: return cudaErrorInvalidValue;
  }
#undef MQ_LAUNCH_Q
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace mq
