// Channel-batch-first im2col of the already-quantized activation (Sec. IV-A): a pure gather of MX
// element bytes and of the tile scales that belong to them.  One thread moves one 16-byte chunk of
// the output, so consecutive threads write consecutive bytes of X' (the write stream is Kh*Kw/s^2
// times the read stream and sets the cost); the reads revisit each stored pixel Kh*Kw times and are
// served by L2.  Out-of-image taps are written as zero bytes.
#include "mq_internal.cuh"

namespace mq {
namespace {

constexpr int IC_THREADS = 256;

__global__ void __launch_bounds__(IC_THREADS) im2col_kernel(Im2colArgs a, int row_chunks, long long code_chunks, long long n_scales) {
  const Geom& g = a.g;
  const long long stride = (long long)gridDim.x * IC_THREADS;
  const int taps = g.Kh * g.Kw;
  for (long long id = (long long)blockIdx.x * IC_THREADS + threadIdx.x; id < code_chunks + n_scales; id += stride) {
    if (id < code_chunks) {
      // output order [ho][wo][n][kh][kw][chunk]
      long long q = id;
      const int ch = (int)(q % row_chunks); q /= row_chunks;
      const int tap = (int)(q % taps); q /= taps;
      const int n = (int)(q % g.N); q /= g.N;
      const int wo = (int)(q % g.Wo);
      const int ho = (int)(q / g.Wo);
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (h >= 0 && h < g.H && w >= 0 && w < g.W) {
        const long long src = (((long long)h * g.W + w) * g.N + n) * row_chunks + ch;
        v = __ldg(reinterpret_cast<const uint4*>(a.codes) + src);
      }
      __stcs(reinterpret_cast<uint4*>(a.out_codes) + id, v);
    } else {
      // scales [ho][wo][nt][kh][kw][ct]
      long long q = id - code_chunks;
      const int ct = (int)(q % g.Ct); q /= g.Ct;
      const int tap = (int)(q % taps); q /= taps;
      const int nt = (int)(q % g.Nt); q /= g.Nt;
      const int wo = (int)(q % g.Wo);
      const int ho = (int)(q / g.Wo);
      const int kh = tap / g.Kw, kw = tap - kh * g.Kw;
      const int h = ho * g.sh + kh - g.ph, w = wo * g.sw + kw - g.pw;
      uint8_t sc = 0;
      if (h >= 0 && h < g.H && w >= 0 && w < g.W) sc = a.scales[(((long long)h * g.W + w) * g.Nt + nt) * g.Ct + ct];
      a.out_scales[id - code_chunks] = sc;
    }
  }
}

}  // namespace

cudaError_t launch_im2col(const Im2colArgs& a, cudaStream_t s) {
  const Geom& g = a.g;
  const int row_chunks = g.Cp * fmt_bits(a.fmt) / 8 / 16;  // 16-byte chunks per (pixel, sample) row
  const long long code_chunks = (long long)g.Ho * g.Wo * g.N * g.Kh * g.Kw * row_chunks;
  const long long n_scales = (long long)g.Ho * g.Wo * g.Nt * g.Kh * g.Kw * g.Ct;
  const long long total = code_chunks + n_scales;
  long long blocks = (total + IC_THREADS - 1) / IC_THREADS;
  const long long cap = 148LL * 8 * 16;  // grid-stride beyond this
  if (blocks > cap) blocks = cap;
  if (blocks <= 0) return cudaErrorInvalidValue;
  im2col_kernel<<<(unsigned)blocks, IC_THREADS, 0, s>>>(a, row_chunks, code_chunks, n_scales);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace mq
