// CUDA-core implicit-GEMM kernels for the three block-scaled convolution GEMMs (Sec. II-C, IV-B,
// Eq. 7).  They accept every shape and every element-format pair and serve the shapes the
// tensor-core kernels do not cover (thin channel counts, odd geometry).  Operands are decoded
// exactly (code -> fp16 -> fp32, times the tile's power-of-two scale) into shared memory, one
// 32-element MX block of K per step, and accumulated in fp32.
//
//   fwd        : M = (ho,wo,n)   N = co           K = (kh,kw | ci)   A = X gathered, B = W     both K-contiguous
//   bwd_data   : M = (h,w,n)     N = ci           K = (kh,kw | co)   A = G_Y gathered (K-contiguous), B = W (N-contiguous)
//   bwd_weight : M = co          N = (kh,kw,ci)   K = (ho,wo | n)    A = G_Y, B = X gathered   both MN-contiguous
#include "mq_conv_tc.cuh"

namespace mq {
namespace {

constexpr int TM = 64, TN = 64, TK = 32, GT = 256, PADF = 4;

struct Tiles {
  alignas(16) float As[TK][TM + PADF];
  alignas(16) float Bs[TK][TN + PADF];
};

__device__ __forceinline__ void store_kmajor(float (*S)[TM + PADF], int row, int kq, const float* v) {
#pragma unroll
  for (int j = 0; j < 8; ++j) S[kq * 8 + j][row] = v[j];
}
__device__ __forceinline__ void store_mnmajor(float (*S)[TM + PADF], int k, int mq, const float* v) {
  *reinterpret_cast<float4*>(&S[k][mq * 8]) = make_float4(v[0], v[1], v[2], v[3]);
  *reinterpret_cast<float4*>(&S[k][mq * 8 + 4]) = make_float4(v[4], v[5], v[6], v[7]);
}
__device__ __forceinline__ void zero8(float* v) {
#pragma unroll
  for (int j = 0; j < 8; ++j) v[j] = 0.f;
}

// Scale of the 8 consecutive channels starting at channel c of row `row` at position `pos` of a stored tensor:
//   activation-like tensors ([pos][row][c], R rows): sc[(pos * RB + row_block) * CB + channel_block]
//   weights ([row][pos][c], P positions):            sc[(row_block * P + pos) * CB + channel_block]
// with 32 x 32 tiles (E8M0), line blocks (one row per block) or, ts16, 16 x 16 blocks whose E4M3 scale is multiplied by the
// tensor's fp32 scale t.
__device__ __forceinline__ float e4m3_to_float(unsigned code) {
  const __half_raw h = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)code, __NV_E4M3);
  return __half2float(*reinterpret_cast<const __half*>(&h));
}
__device__ __forceinline__ float act_scale(const ConvArgs& a, const uint8_t* sc, float t, long long pos, int row, int c, int R, int Cp) {
  if (a.ts16) return e4m3_to_float(sc[(pos * ((R + 15) >> 4) + (row >> 4)) * (Cp >> 4) + (c >> 4)]) * t;
  if (a.line) return e8m0_to_float(sc[(pos * R + row) * (Cp >> 5) + (c >> 5)]);
  return e8m0_to_float(sc[(pos * ((R + 31) >> 5) + (row >> 5)) * (Cp >> 5) + (c >> 5)]);
}
__device__ __forceinline__ float w_scale(const ConvArgs& a, const uint8_t* sc, float t, int row, int taps, int tap, int c, int Cp) {
  if (a.ts16) return e4m3_to_float(sc[((long long)(row >> 4) * taps + tap) * (Cp >> 4) + (c >> 4)]) * t;
  if (a.line) return e8m0_to_float(sc[((long long)row * taps + tap) * (Cp >> 5) + (c >> 5)]);
  return e8m0_to_float(sc[((long long)(row >> 5) * taps + tap) * (Cp >> 5) + (c >> 5)]);
}

__device__ __forceinline__ void mma_tile(const Tiles& sm, int ty, int tx, float acc[4][4]) {
#pragma unroll
  for (int k = 0; k < TK; ++k) {
    float4 a = *reinterpret_cast<const float4*>(&sm.As[k][ty * 4]);
    float4 b = *reinterpret_cast<const float4*>(&sm.Bs[k][tx * 4]);
    float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
  }
}

// ------------------------------------------------------------------------------------ forward
template <int FX, int FW>
__global__ void __launch_bounds__(GT) fwd_generic(ConvArgs a) {
  __shared__ Tiles sm;
  const Geom& g = a.g;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int row_l = tid >> 2, kq = tid & 3;
  const long long M = (long long)g.Ho * g.Wo * g.N;
  const long long m0 = (long long)blockIdx.x * TM;
  const int n0 = blockIdx.y * TN;
  const int taps = g.Kh * g.Kw;

  const long long m = m0 + row_l;
  const bool m_ok = m < M;
  int n = 0, wo = 0, ho = 0;
  if (m_ok) { n = (int)(m % g.N); long long q = m / g.N; wo = (int)(q % g.Wo); ho = (int)(q / g.Wo); }
  const int co = n0 + row_l;
  const bool co_ok = co < g.Cout;
  const float ta = a.ts16 ? *a.a_tscale : 1.f, tb = a.ts16 ? *a.b_tscale : 1.f;

  float acc[4][4] = {};
  for (int tap = 0; tap < taps; ++tap) {
    const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
    const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
    const bool pix_ok = m_ok && h >= 0 && h < g.H && w >= 0 && w < g.W;
    const long long pix = (long long)h * g.W + w;
    for (int kb = 0; kb < g.Ct; ++kb) {
      float va[8], vb[8];
      if (pix_ok) {
        const float s = act_scale(a, a.a_scales, ta, pix, n, kb * 32 + kq * 8, g.N, g.Cp);
        decode8<FX>(a.a_codes, (pix * g.N + n) * g.Cp + kb * 32 + kq * 8, s, va, a.fmt_a);
      } else zero8(va);
      if (co_ok) {
        const float s = w_scale(a, a.b_scales, tb, co, taps, tap, kb * 32 + kq * 8, g.Cp);
        decode8<FW>(a.b_codes, ((long long)co * taps + tap) * g.Cp + kb * 32 + kq * 8, s, vb, a.fmt_b);
      } else zero8(vb);
      __syncthreads();
      store_kmajor(sm.As, row_l, kq, va);
      store_kmajor(sm.Bs, row_l, kq, vb);
      __syncthreads();
      mma_tile(sm, ty, tx, acc);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long mm = m0 + ty * 4 + i;
    if (mm >= M) continue;
    const int nn = (int)(mm % g.N); const long long q = mm / g.N;
    const int wwo = (int)(q % g.Wo), hho = (int)(q / g.Wo);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c >= g.Cout) continue;
      if (a.out_layout == MQ_NCHW) a.out[(((long long)nn * g.Cout + c) * g.Ho + hho) * g.Wo + wwo] = acc[i][j];
      else a.out[mm * g.Cout + c] = acc[i][j];
    }
  }
}

// --------------------------------------------------------------------------------- input gradient
template <int FW, int FG>
__global__ void __launch_bounds__(GT) bwd_data_generic(ConvArgs a) {
  __shared__ Tiles sm;
  const Geom& g = a.g;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int row_l = tid >> 2, kq = tid & 3;   // A units: (row, 8 consecutive k)
  const int k_l = tid >> 3, nq = tid & 7;     // B units: (k, 8 consecutive ci)
  const long long M = (long long)g.H * g.W * g.N;
  const long long m0 = (long long)blockIdx.x * TM;
  const int n0 = blockIdx.y * TN;
  const int taps = g.Kh * g.Kw;

  const long long m = m0 + row_l;
  const bool m_ok = m < M;
  int n = 0, w = 0, h = 0;
  if (m_ok) { n = (int)(m % g.N); long long q = m / g.N; w = (int)(q % g.W); h = (int)(q / g.W); }
  const int ci0 = n0 + nq * 8;
  const bool ci_ok = ci0 < g.Cp;
  const float ta = a.ts16 ? *a.a_tscale : 1.f, tb = a.ts16 ? *a.b_tscale : 1.f;

  float acc[4][4] = {};
  for (int tap = 0; tap < taps; ++tap) {
    const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
    const int hn = h + g.ph - kh, wn = w + g.pw - kw;
    bool pix_ok = m_ok && hn >= 0 && wn >= 0 && (hn % g.sh) == 0 && (wn % g.sw) == 0;
    const int ho = hn / g.sh, wo = wn / g.sw;
    pix_ok = pix_ok && ho < g.Ho && wo < g.Wo;
    const long long pix = (long long)ho * g.Wo + wo;
    for (int kb = 0; kb < g.Cot; ++kb) {
      float va[8], vb[8];
      if (pix_ok) {
        const float s = act_scale(a, a.b_scales, tb, pix, n, kb * 32 + kq * 8, g.N, g.Cop);
        decode8<FG>(a.b_codes, (pix * g.N + n) * g.Cop + kb * 32 + kq * 8, s, va, a.fmt_b);
      } else zero8(va);
      const int co = kb * 32 + k_l;
      if (ci_ok && co < g.Cout) {
        const float s = w_scale(a, a.a_scales, ta, co, taps, tap, ci0, g.Cp);
        decode8<FW>(a.a_codes, ((long long)co * taps + tap) * g.Cp + ci0, s, vb, a.fmt_a);
      } else zero8(vb);
      __syncthreads();
      store_kmajor(sm.As, row_l, kq, va);
      store_mnmajor(sm.Bs, k_l, nq, vb);
      __syncthreads();
      mma_tile(sm, ty, tx, acc);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long mm = m0 + ty * 4 + i;
    if (mm >= M) continue;
    const int nn = (int)(mm % g.N); const long long q = mm / g.N;
    const int ww = (int)(q % g.W), hh = (int)(q / g.W);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = n0 + tx * 4 + j;
      if (c >= g.Cin) continue;
      if (a.out_layout == MQ_NCHW) a.out[(((long long)nn * g.Cin + c) * g.H + hh) * g.W + ww] = acc[i][j];
      else a.out[mm * g.Cin + c] = acc[i][j];
    }
  }
}

// -------------------------------------------------------------------------------- weight gradient
// Partial sums over a slice of output pixels go to workspace [split][C_out][taps*Cp]; a second
// kernel adds the slices in a fixed order and writes G_W in its final layout.
template <int FX, int FG>
__global__ void __launch_bounds__(GT) bwd_weight_generic(ConvArgs a, int splits) {
  __shared__ Tiles sm;
  const Geom& g = a.g;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const int k_l = tid >> 3, q8 = tid & 7;
  const int m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int taps = g.Kh * g.Kw;
  const int J = taps * g.Cp;
  const int npix = g.Ho * g.Wo;
  const int split = blockIdx.z;
  const int pix_begin = (int)((long long)npix * split / splits), pix_end = (int)((long long)npix * (split + 1) / splits);

  const int co0 = m0 + q8 * 8;
  const bool co_ok = co0 < g.Cop;
  const int j0 = n0 + q8 * 8;
  const bool j_ok = j0 < J;
  const int tap = j_ok ? j0 / g.Cp : 0, ci0 = j_ok ? j0 - tap * g.Cp : 0;
  const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
  const float ta = a.ts16 ? *a.a_tscale : 1.f, tb = a.ts16 ? *a.b_tscale : 1.f;

  float acc[4][4] = {};
  for (int pix = pix_begin; pix < pix_end; ++pix) {
    const int ho = pix / g.Wo, wo = pix - ho * g.Wo;
    const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
    const bool x_ok = j_ok && h >= 0 && h < g.H && w >= 0 && w < g.W;
    const long long xpix = (long long)h * g.W + w;
    for (int kb = 0; kb < g.Nt; ++kb) {
      const int n = kb * 32 + k_l;
      float va[8], vb[8];
      if (co_ok && n < g.N) {
        const float s = act_scale(a, a.b_scales, tb, pix, n, co0, g.N, g.Cop);
        decode8<FG>(a.b_codes, ((long long)pix * g.N + n) * g.Cop + co0, s, va, a.fmt_b);
      } else zero8(va);
      if (x_ok && n < g.N) {
        const float s = act_scale(a, a.a_scales, ta, xpix, n, ci0, g.N, g.Cp);
        decode8<FX>(a.a_codes, (xpix * g.N + n) * g.Cp + ci0, s, vb, a.fmt_a);
      } else zero8(vb);
      __syncthreads();
      store_mnmajor(sm.As, k_l, q8, va);
      store_mnmajor(sm.Bs, k_l, q8, vb);
      __syncthreads();
      mma_tile(sm, ty, tx, acc);
    }
  }
  float* part = reinterpret_cast<float*>(a.workspace) + (long long)split * g.Cout * J;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int co = m0 + ty * 4 + i;
    if (co >= g.Cout) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int jj = n0 + tx * 4 + j;
      if (jj < J) part[(long long)co * J + jj] = acc[i][j];
    }
  }
}

// Adds the split-K partial sums [split][Cout][taps][Cp] in a fixed order and writes G_W in its final layout.
// The reads are `splits` times the writes, so threads follow the partials' own order (4 consecutive input
// channels per thread, 16-byte loads); a block's four thread groups take every fourth split each and are
// combined through shared memory in group order, so the result does not depend on scheduling.
// ta, tb: the two tensors' fp32 scales when the partial sums still lack them (tensor-core GEMM on E4M3-scaled blocks, Eq. 4), else null
__global__ void __launch_bounds__(256) bwd_weight_reduce(const float* __restrict__ part, float* __restrict__ out, Geom g, int splits, int layout,
                                                         const float* __restrict__ ta, const float* __restrict__ tb) {
  pdl_wait();
  const float os = ta ? __ldg(ta) * __ldg(tb) : 1.f;
  __shared__ float4 sh[3][64];
  const int taps = g.Kh * g.Kw;
  const int cq = g.Cp >> 2;                                   // float4 columns per (co, tap)
  const long long quads = (long long)g.Cout * taps * cq;
  const long long slab = (long long)g.Cout * taps * g.Cp;     // floats per split
  const int col = threadIdx.x & 63, grp = threadIdx.x >> 6;
  for (long long base = (long long)blockIdx.x * 64; base < quads; base += (long long)gridDim.x * 64) {
    const long long qd = base + col;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    if (qd < quads) {
      const float4* p = reinterpret_cast<const float4*>(part) + qd;
#pragma unroll 4
      for (int k = grp; k < splits; k += 4) {
        const float4 v = __ldg(p + (long long)k * (slab >> 2));
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      }
    }
    if (grp > 0) sh[grp - 1][col] = s;
    __syncthreads();
    if (grp == 0 && qd < quads) {
#pragma unroll
      for (int q = 0; q < 3; ++q) { const float4 v = sh[q][col]; s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
      const int c4 = (int)(qd % cq); const long long r = qd / cq;
      const int tap = (int)(r % taps), co = (int)(r / taps);
      const float vals[4] = {s.x * os, s.y * os, s.z * os, s.w * os};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int ci = 4 * c4 + e;
        if (ci < g.Cin) {
          if (layout == MQ_NCHW) out[((long long)co * g.Cin + ci) * taps + tap] = vals[e];
          else out[((long long)co * taps + tap) * g.Cin + ci] = vals[e];
        }
      }
    }
    __syncthreads();
  }
}

}  // namespace

int conv_generic_bwd_weight_splits(const Geom& g) {
  const int taps = g.Kh * g.Kw;
  const long long tiles = (long long)((g.Cop + TM - 1) / TM) * ((taps * g.Cp + TN - 1) / TN);
  long long splits = ((long long)sm_count() * 4 + tiles - 1) / tiles;
  const long long npix = (long long)g.Ho * g.Wo;
  if (splits > npix) splits = npix;
  if (splits > 256) splits = 256;
  if (splits < 1) splits = 1;
  return (int)splits;
}

size_t conv_generic_workspace(int op, const Geom& g) {
  if (op != MQ_OP_BWD_WEIGHT) return 0;
  return (size_t)conv_generic_bwd_weight_splits(g) * g.Cout * g.Kh * g.Kw * g.Cp * sizeof(float);
}

cudaError_t launch_bwd_weight_reduce(const float* partial, float* out, const Geom& g, int splits, int layout, cudaStream_t s, const float* ta,
                                     const float* tb) {
  const long long quads = (long long)g.Cout * g.Kh * g.Kw * (g.Cp / 4);
  unsigned blocks = (unsigned)((quads + 63) / 64);
  if (blocks > (unsigned)sm_count() * 16) blocks = (unsigned)sm_count() * 16;
  count_launches(1);
  return launch_pdl(bwd_weight_reduce, dim3(blocks), dim3(256), 0, s, partial, out, g, splits, layout, ta, tb);
}

// Two template classes per operand: packed E2M1 (2) or one byte per code (0; the format itself is read at run time)
#define MQ_DISPATCH2(FA, FB, CALL)                                                         \
  switch (((FA) == MQ_E2M1 ? 2 : 0) + ((FB) == MQ_E2M1 ? 1 : 0)) {                            \
    case 0: { constexpr int A_ = 0, B_ = 0; CALL; } break;                                 \
    case 1: { constexpr int A_ = 0, B_ = 2; CALL; } break;                                 \
    case 2: { constexpr int A_ = 2, B_ = 0; CALL; } break;                                 \
    case 3: { constexpr int A_ = 2, B_ = 2; CALL; } break;                                 \
    default: return cudaErrorInvalidValue;                                                 \
  }

cudaError_t launch_conv_generic(int op, const ConvArgs& a, cudaStream_t s) {
  const Geom& g = a.g;
  if (op == MQ_OP_FWD) {
    const long long M = (long long)g.Ho * g.Wo * g.N;
    dim3 grid((unsigned)((M + TM - 1) / TM), (unsigned)((g.Cout + TN - 1) / TN));
    MQ_DISPATCH2(a.fmt_a, a.fmt_b, (fwd_generic<A_, B_><<<grid, GT, 0, s>>>(a)));
  } else if (op == MQ_OP_BWD_DATA) {
    const long long M = (long long)g.H * g.W * g.N;
    dim3 grid((unsigned)((M + TM - 1) / TM), (unsigned)((g.Cin + TN - 1) / TN));
    MQ_DISPATCH2(a.fmt_a, a.fmt_b, (bwd_data_generic<A_, B_><<<grid, GT, 0, s>>>(a)));
  } else {
    const int splits = conv_generic_bwd_weight_splits(g);
    const int J = g.Kh * g.Kw * g.Cp;
    dim3 grid((unsigned)((g.Cop + TM - 1) / TM), (unsigned)((J + TN - 1) / TN), (unsigned)splits);
    MQ_DISPATCH2(a.fmt_a, a.fmt_b, (bwd_weight_generic<A_, B_><<<grid, GT, 0, s>>>(a, splits)));
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long quads = (long long)g.Cout * g.Kh * g.Kw * (g.Cp / 4);
    unsigned blocks = (unsigned)((quads + 63) / 64);
    if (blocks > (unsigned)sm_count() * 16) blocks = (unsigned)sm_count() * 16;
    bwd_weight_reduce<<<blocks, 256, 0, s>>>(reinterpret_cast<const float*>(a.workspace), a.out, g, splits, a.out_layout, nullptr, nullptr);
    count_launches(1);
  }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace mq
