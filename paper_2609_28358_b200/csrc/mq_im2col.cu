// Channel-batch-first im2col of the already-quantized activation (Sec. IV-A): a pure gather of MX
// element bytes and of the tile scales that belong to them.  A thread block produces the X' rows of one
// output pixel for 32 consecutive samples -- a contiguous run of 32 * Kh*Kw * row bytes -- so consecutive
// threads write consecutive 16-byte chunks (the write stream is Kh*Kw/s^2 times the read stream and sets
// the cost); the reads revisit each stored pixel Kh*Kw times and are served by L2.  Out-of-image taps are
// written as zero bytes.  Index arithmetic is done once per block (a table of source offsets per chunk of
// a row) and advanced incrementally, never per chunk.
#include "mq_internal.cuh"

namespace mq {
namespace {

constexpr int IC_THREADS = 256;
constexpr int IC_MAX_J = 1024;   // chunks per X' row held in the offset table
constexpr int IC_TABLE = 2048;   // table entries per block: PX pixels x J chunks

__device__ __forceinline__ void zero_chunk(uint4& v) { v = make_uint4(0, 0, 0, 0); }
__device__ __forceinline__ void zero_chunk(uint2& v) { v = make_uint2(0, 0); }

// PX consecutive output pixels per block amortise the block's fixed cost (launch, offset table, barrier) over
// PX * 32 rows of X'.  V: the chunk - 16 bytes, or 8 where a row is no multiple of 16 bytes (packed 6-bit codes, 24 bytes per
// 32 channels, with an odd number of channel tiles).
template <typename V>
__global__ void __launch_bounds__(IC_THREADS) im2col_kernel(Im2colArgs a, int rc, int J, int PX, unsigned n_main) {
  pdl_wait();
  const Geom& g = a.g;
  __shared__ int soff[IC_TABLE];   // source chunk offset of row chunk j of pixel px relative to sample 0, -1: zero
  const int taps = g.Kh * g.Kw;
  if (blockIdx.x < n_main) {
    const unsigned pg = blockIdx.x / (unsigned)g.Nt;
    const int nt = (int)(blockIdx.x - pg * (unsigned)g.Nt);
    const unsigned pix0 = pg * (unsigned)PX;
    const unsigned npix = (unsigned)(g.Ho * g.Wo);
    const int px_n = (int)min((unsigned)PX, npix - pix0);
    for (int e = threadIdx.x; e < px_n * J; e += IC_THREADS) {
      const int px = e / J, j = e - px * J;
      const unsigned pix = pix0 + px;
      const int ho = (int)(pix / (unsigned)g.Wo), wo = (int)(pix - (unsigned)ho * (unsigned)g.Wo);
      const int tap = j / rc, ch = j - tap * rc;
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      soff[e] = (h >= 0 && h < g.H && w >= 0 && w < g.W) ? ((h * g.W + w) * g.N) * rc + ch : -1;   // < 2^31 chunks checked on the host
    }
    __syncthreads();
    const int n0 = nt * 32;
    const int rows = min(32, g.N - n0);
    const int total = rows * J;
    const V* src = reinterpret_cast<const V*>(a.codes) + (long long)n0 * rc;
    const int dn = IC_THREADS / J, dj = IC_THREADS - dn * J;
    V* dst0 = reinterpret_cast<V*>(a.out_codes) + ((long long)pix0 * g.N + n0) * J;
    const long long px_stride = (long long)g.N * J;      // chunks between the rows of consecutive pixels
    // chunk i = n * J + j of every pixel of the block, advanced by IC_THREADS per step without divisions; the loads of
    // four pixels are issued before their stores (the kernel waits on L2 latency, not on bandwidth)
    int n = threadIdx.x / J, j = threadIdx.x - n * J;
#pragma unroll 1
    for (int i = threadIdx.x; i < total; i += IC_THREADS) {
      const V* s_n = src + n * rc;
#pragma unroll 1
      for (int px0 = 0; px0 < px_n; px0 += 4) {
        V v[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          zero_chunk(v[q]);
          if (px0 + q < px_n) {
            const int so = soff[(px0 + q) * J + j];
            if (so >= 0) v[q] = __ldg(s_n + so);
          }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (px0 + q < px_n) __stcs(dst0 + (px0 + q) * px_stride + i, v[q]);
      }
      n += dn; j += dj;
      if (j >= J) { j -= J; ++n; }
    }
  } else {
    // scales [ho][wo][nt][kh][kw][ct]; with line blocks one entry per sample: [ho][wo][n][kh][kw][ct]
    const int Rt = a.line ? g.N : (a.ts16 ? (g.N + 15) / 16 : g.Nt), Cb = a.ts16 ? g.Cp / 16 : g.Ct;
    const long long n_scales = (long long)g.Ho * g.Wo * Rt * taps * Cb;
    for (long long id = (long long)(blockIdx.x - n_main) * IC_THREADS + threadIdx.x; id < n_scales; id += (long long)(gridDim.x - n_main) * IC_THREADS) {
      long long q = id;
      const int ct = (int)(q % Cb); q /= Cb;
      const int tap = (int)(q % taps); q /= taps;
      const int nt = (int)(q % Rt); q /= Rt;
      const int wo = (int)(q % g.Wo);
      const int ho = (int)(q / g.Wo);
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      uint8_t sc = 0;
      if (h >= 0 && h < g.H && w >= 0 && w < g.W) sc = a.scales[(((long long)h * g.W + w) * Rt + nt) * Cb + ct];
      a.out_scales[id] = sc;
    }
  }
}

// General fallback (rows longer than the offset table, or tensors beyond 2^31 chunks): one thread per chunk.
template <typename V>
__global__ void __launch_bounds__(IC_THREADS) im2col_generic_kernel(Im2colArgs a, int row_chunks, long long code_chunks, long long n_scales) {
  const Geom& g = a.g;
  const long long stride = (long long)gridDim.x * IC_THREADS;
  const int taps = g.Kh * g.Kw;
  for (long long id = (long long)blockIdx.x * IC_THREADS + threadIdx.x; id < code_chunks + n_scales; id += stride) {
    if (id < code_chunks) {
      long long q = id;
      const int ch = (int)(q % row_chunks); q /= row_chunks;
      const int tap = (int)(q % taps); q /= taps;
      const int n = (int)(q % g.N); q /= g.N;
      const int wo = (int)(q % g.Wo);
      const int ho = (int)(q / g.Wo);
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      V v;
      zero_chunk(v);
      if (h >= 0 && h < g.H && w >= 0 && w < g.W) v = __ldg(reinterpret_cast<const V*>(a.codes) + (((long long)h * g.W + w) * g.N + n) * row_chunks + ch);
      __stcs(reinterpret_cast<V*>(a.out_codes) + id, v);
    } else {
      long long q = id - code_chunks;
      const int Rt = a.line ? g.N : (a.ts16 ? (g.N + 15) / 16 : g.Nt), Cb = a.ts16 ? g.Cp / 16 : g.Ct;
      const int ct = (int)(q % Cb); q /= Cb;
      const int tap = (int)(q % taps); q /= taps;
      const int nt = (int)(q % Rt); q /= Rt;
      const int wo = (int)(q % g.Wo);
      const int ho = (int)(q / g.Wo);
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      uint8_t sc = 0;
      if (h >= 0 && h < g.H && w >= 0 && w < g.W) sc = a.scales[(((long long)h * g.W + w) * Rt + nt) * Cb + ct];
      a.out_scales[id - code_chunks] = sc;
    }
  }
}

}  // namespace

template <typename V>
cudaError_t launch_im2col_v(const Im2colArgs& a, cudaStream_t s) {
  const Geom& g = a.g;
  const int rc = g.Cp * fmt_store_bits(a.fmt) / 8 / (int)sizeof(V);  // chunks per (pixel, sample) row
  const int taps = g.Kh * g.Kw;
  const long long J = (long long)taps * rc;
  const long long src_chunks = (long long)g.H * g.W * g.N * rc;
  int PX = (int)(IC_TABLE / (J > 0 ? J : 1));
  if (PX > 8) PX = 8;
  if (PX < 1) PX = 1;
  const long long n_main = (((long long)g.Ho * g.Wo + PX - 1) / PX) * g.Nt;
  const long long n_scales = (long long)g.Ho * g.Wo * (a.line ? g.N : (a.ts16 ? (g.N + 15) / 16 : g.Nt)) * taps * (a.ts16 ? g.Cp / 16 : g.Ct);
  count_launches(1);
  if (J <= IC_MAX_J && src_chunks < 0x7fffffffLL && n_main < 0x7fff0000LL) {
    long long sc_blocks = (n_scales + IC_THREADS - 1) / IC_THREADS;
    if (sc_blocks > sm_count() * 4) sc_blocks = sm_count() * 4;
    if (sc_blocks < 1) sc_blocks = 1;
    return launch_pdl(im2col_kernel<V>, dim3((unsigned)(n_main + sc_blocks)), dim3(IC_THREADS), 0, s, a, rc, (int)J, PX, (unsigned)n_main);
  }
  const long long code_chunks = (long long)g.Ho * g.Wo * g.N * J;
  const long long total = code_chunks + n_scales;
  long long blocks = (total + IC_THREADS - 1) / IC_THREADS;
  const long long cap = (long long)sm_count() * 8 * 16;  // grid-stride beyond this
  if (blocks > cap) blocks = cap;
  if (blocks <= 0) return cudaErrorInvalidValue;
  im2col_generic_kernel<V><<<(unsigned)blocks, IC_THREADS, 0, s>>>(a, rc, code_chunks, n_scales);
  return cudaGetLastError();
}

cudaError_t launch_im2col(const Im2colArgs& a, cudaStream_t s) {
  if ((a.g.Cp * fmt_store_bits(a.fmt) / 8) % 16 != 0) return launch_im2col_v<uint2>(a, s);
  return launch_im2col_v<uint4>(a, s);
}

}  // namespace mq
