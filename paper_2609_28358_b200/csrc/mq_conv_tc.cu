// Tensor-core implicit-GEMM kernel for mq_conv_fwd and mq_conv_bwd_data (Sec. II-C / IV-B GEMMs,
// block-scaled as Eq. 7) on sm_100a: tcgen05 block-scaled MMA with accumulators and scale vectors
// in tensor memory, operands brought by TMA straight from the stored channel-batch-first tensors
// (the im2col of Sec. IV-A is implicit: every tap is a shifted TMA box, out-of-image taps are the
// TMA zero fill).
//
// A small kernel first expands the compact tile scales (one E8M0 byte per 32x32 tile) into the per-row
// scale-vector chunks the MMA reads, one chunk per (tile, pipeline stage), in scratch.
//
// One persistent thread block per SM, 16 warps, every role loop run by its whole warp with only the asynchronous
// instruction itself under an elected lane:
//   warps 0, 12   loaders of the activation boxes (even / odd stages)
//   warps 3, 13   loaders of the weight boxes (even / odd stages)
//   warps 14, 15  loaders of the stage's two scale-vector chunks (even / odd stages)
//   warp 1        MMA issuer: the stage's scale copies smem -> TMEM (tcgen05.cp), then its MMAs
//   warp 2        scale copier (E2M1 with the separate-copier option only)
//   warps 4-11    epilogue: TMEM -> registers -> global (fp32) or a staged TMA store, overlapped with the next tile's
//                 main loop: a second accumulator where it fits; 256-column tiles (one accumulator) are copied whole into
//                 registers and handed back before the stores (fp32 output: these two warpgroups take registers from the
//                 other two with setmaxnreg); two warps per TMEM lane quadrant, half of the columns each
// Wide layers run the DUO instance: clusters of two blocks on 256 x 256 tiles (cta_group::2), see conv_tc_kernel.
// A pipeline stage holds 128 bytes of K per row (four MMAs): one 128-byte box, or 128/KB boxes of KB
// bytes when a tap has fewer than 128 bytes of channels (then several taps share a stage).
// Every wait is bounded; on expiry the kernel records MQ_ERR_TIMEOUT in the status word and drains.
#include <cstdlib>
#include "mq_conv_tc.cuh"
#include "mq_tcgen05.cuh"

namespace mq {
namespace {
using namespace tc;

constexpr int TC_THREADS = 512;   // 16 warps: MMA, scale copier, scale expander / loader, 8 epilogue, 5 more loaders
// The quantizing epilogue of the paper's own format (emitted format 5) runs with 16 epilogue warps (8 more, warps 16-23): a block
// of it is a chain of latencies (tensor-memory load, warp reductions, IEEE divisions, conversions, stores) that two warps
// per scheduler do not hide; four do better, at 80 registers per thread (measured, 512 channels 28x28 3x3: 320 -> 278 us).
// The MX formats' epilogue (multiplications instead of divisions) was measured the other way: 345 -> 384 us, 1x1 323 -> 404 us;
// the fp32 direct-store epilogue does not change with 16 warps (445 -> 456 us: its stores are the bound).
constexpr int TC_THREADS_MX = 768;
__host__ __device__ constexpr int tc_threads_of(int epi) { return epi == 5 ? TC_THREADS_MX : TC_THREADS; }
constexpr int A_STAGE_BYTES = 128 * 128;
constexpr int SFA_BYTES = 1024;   // up to 2 groups of 4 scale bytes per row
constexpr int SFB_BYTES = 2048;   // up to 2 groups x 2 atoms of 128 rows
constexpr int SF_COLS = 24;       // TMEM columns of one scale buffer: 8 (A) + 16 (B)
// The same three for kind 2 (four scale bytes per row and MMA instead of at most two)
constexpr int SFA_BYTES_NV = 2048, SFB_BYTES_NV = 4096, SF_COLS_NV = 48;
__host__ __device__ constexpr int spa_of_kind(int kind) { return kind == 2 ? 4 : (kind == 1 ? 2 : 1); }


struct Tile { int c0, w0, n0, h, cls, ct; };

// Tile order: stride class fastest (the classes of an input gradient interleave inside the same 32-byte
// sectors), then output column tile, output row, channel tile, sample tile.  Tiles that run at the same time
// then complete whole (n, c) planes of an NCHW output quickly, so partially written lines do not linger in
// L2, and they share input rows between neighbouring taps.
// Division by a launch constant: d == 1 costs nothing, otherwise one multiply-high with m = ceil(2^32 / d)
// (exact while t * d < 2^32; the host refuses to plan a launch for which that does not hold).
__device__ __forceinline__ unsigned fdiv(unsigned t, int d, uint32_t m) { return d == 1 ? t : __umulhi(t, m); }

__device__ __forceinline__ Tile decode_tile(const ConvTcParams& p, unsigned t) {
  Tile q;
  unsigned u = fdiv(t, p.classes, p.m_classes);
  q.cls = (int)(t - u * p.classes); t = u;
  u = fdiv(t, p.tiles_w, p.m_tiles_w); q.w0 = (int)(t - u * p.tiles_w) * p.TW; t = u;
  u = fdiv(t, p.tiles_h, p.m_tiles_h); q.h = (int)(t - u * p.tiles_h); t = u;
  u = fdiv(t, p.tiles_c, p.m_tiles_c); q.ct = (int)(t - u * p.tiles_c); q.c0 = q.ct * p.BN;
  q.n0 = (int)u * p.TN;
  return q;
}
// number of A-side scale chunks of a launch
__host__ __device__ __forceinline__ unsigned conv_tc_sfa_chunks(const ConvTcParams& p) {
  const unsigned tiles_m = (unsigned)(p.total_tiles / p.tiles_c);
  if (p.sfa_dedup) return tiles_m / (unsigned)(p.tiles_h * p.classes) * (unsigned)p.sfa_hk * (unsigned)(p.Kw * p.cpt);
  return tiles_m * (unsigned)p.max_stages;
}
// index of a tile among the tiles that differ in anything but the channel tile (A-side scale chunks)
__device__ __forceinline__ unsigned tile_m_index(const ConvTcParams& p, const Tile& q) {
  return (((unsigned)(q.n0 >> p.lgTN) * p.tiles_h + q.h) * p.tiles_w + (q.w0 >> p.lgTW)) * p.classes + q.cls;
}
__device__ __forceinline__ Tile tile_of_m_index(const ConvTcParams& p, unsigned tm) {
  Tile q;
  unsigned u = fdiv(tm, p.classes, p.m_classes);
  q.cls = (int)(tm - u * p.classes); tm = u;
  u = fdiv(tm, p.tiles_w, p.m_tiles_w); q.w0 = (int)(tm - u * p.tiles_w) * p.TW; tm = u;
  u = fdiv(tm, p.tiles_h, p.m_tiles_h); q.h = (int)(tm - u * p.tiles_h);
  q.n0 = (int)u * p.TN; q.c0 = 0; q.ct = 0;
  return q;
}

// The i-th tile of this block.  Plain mode: round robin over the blocks.  Pair mode (input gradient with a column
// stride of 2, NCHW output): tiles 2k and 2k + 1 are the two column-parity classes of the same output positions
// (the class is the fastest tile index) and go to the same block back to back, into the two accumulators, so
// that the epilogue can interleave them into contiguous stores.
__device__ __forceinline__ unsigned tile_of_iter(const ConvTcParams& p, unsigned i) {
  return p.pair ? 2u * (blockIdx.x + (i >> 1) * gridDim.x) + (i & 1u) : blockIdx.x + i * gridDim.x;
}

// The taps that contribute to a tile, as a small 2-D range walked without divisions.
// Forward: all (kh, kw); source pixel = (ho*sh - ph + kh, wo*sw - pw + kw).
// Input gradient: the taps whose offset has the parity of the tile's class (h + ph - kh and w + pw - kw
// divisible by the stride): kh = kh0 + sh*ia, kw = kw0 + sw*ib; source pixel = (hi + dh0 - ia, wi + dw0 - ib).
template <int MODE>
struct TapWalk {
  int nkh, nkw;      // tap counts along h and w
  int hs0, ws0;      // source row / first source column of tap (0, 0)
  int tap0;          // weight tap index of tap (0, 0)
  int tap_dh, tap_dw;  // weight tap index increments per ia / ib
  __device__ __forceinline__ void init(const ConvTcParams& p, const Tile& t) {
    if (MODE == MQ_OP_FWD) {
      nkh = p.Kh; nkw = p.Kw;
      hs0 = t.h * p.sh - p.ph; ws0 = t.w0 * p.sw - p.pw;
      tap0 = 0; tap_dh = p.Kw; tap_dw = 1;
    } else {
      const int ch = (int)fdiv((unsigned)t.cls, p.sw, p.m_sw), cw = t.cls - ch * p.sw;
      const int kh0 = (ch + p.ph) - (int)fdiv((unsigned)(ch + p.ph), p.sh, p.m_sh) * p.sh;
      const int kw0 = (cw + p.pw) - (int)fdiv((unsigned)(cw + p.pw), p.sw, p.m_sw) * p.sw;
      nkh = kh0 < p.Kh ? (int)fdiv((unsigned)(p.Kh - kh0 + p.sh - 1), p.sh, p.m_sh) : 0;
      nkw = kw0 < p.Kw ? (int)fdiv((unsigned)(p.Kw - kw0 + p.sw - 1), p.sw, p.m_sw) : 0;
      hs0 = t.h + (int)fdiv((unsigned)(ch + p.ph - kh0), p.sh, p.m_sh); ws0 = t.w0 + (int)fdiv((unsigned)(cw + p.pw - kw0), p.sw, p.m_sw);
      tap0 = kh0 * p.Kw + kw0; tap_dh = p.sh * p.Kw; tap_dw = p.sw;
    }
  }
  __device__ __forceinline__ int chunks(const ConvTcParams& p) const { return nkh * nkw * p.cpt; }
};
// position inside a TapWalk: (ia, ib, cc) with cc the chunk of the tap's channel row
struct ChunkPos {
  int ia, ib, cc;
  __device__ __forceinline__ void reset() { ia = 0; ib = 0; cc = 0; }
  template <int MODE>
  __device__ __forceinline__ void advance(const TapWalk<MODE>& w, int cpt) {
    if (++cc == cpt) { cc = 0; if (++ib == w.nkw) { ib = 0; ++ia; } }
  }
};
template <int MODE>
__device__ __forceinline__ int src_h(const TapWalk<MODE>& w, const ChunkPos& c) { return MODE == MQ_OP_FWD ? w.hs0 + c.ia : w.hs0 - c.ia; }
template <int MODE>
__device__ __forceinline__ int src_w0(const TapWalk<MODE>& w, const ChunkPos& c) { return MODE == MQ_OP_FWD ? w.ws0 + c.ib : w.ws0 - c.ib; }
template <int MODE>
__device__ __forceinline__ int tap_index(const TapWalk<MODE>& w, const ChunkPos& c) { return w.tap0 + c.ia * w.tap_dh + c.ib * w.tap_dw; }

// Product of the two tensors' fp32 scales (Eq. 4) that the accumulator of kind 2 is multiplied by; 1 for the other kinds
__device__ __forceinline__ float out_scale_of(const ConvTcParams& p) { return p.kind_fp4 == 2 ? __ldg(p.a_tscale) * __ldg(p.b_tscale) : 1.f; }
__device__ __forceinline__ void scale16(uint32_t* v, float os) {
#pragma unroll
  for (int j = 0; j < 16; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * os);
}
// An epilogue warp hands its accumulator back: to this block's barrier, or (a pair of blocks: the peer's warps) to the
// leader's, whose MMA warp waits for the epilogues of both blocks.
// Accumulator buffer of a block's tcount-th tile and the parity of that buffer's barriers (1 or 2 buffers; a third
// buffer of 128 columns was measured on stride-2 and 1x1 layers: no change)
__device__ __forceinline__ int acc_index(const ConvTcParams& p, uint32_t tcount) { return (int)(tcount & (uint32_t)(p.n_acc - 1)); }
__device__ __forceinline__ uint32_t acc_phase(const ConvTcParams& p, uint32_t tcount) { return (tcount >> (p.n_acc - 1)) & 1u; }
__device__ __forceinline__ void release_acc(uint64_t* bar, int leader_remote) {
  if (leader_remote) mbar_arrive_remote(bar, 0); else mbar_arrive(bar);
}

// Epilogue role (warps 4-11): TMEM -> registers -> global (fp32), two warps per TMEM lane quadrant, each
// taking half of the tile's columns.
template <int MODE>
__device__ __forceinline__ void epilogue_role(const ConvTcParams& p, uint32_t tmem, uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag,
                                              int warp, int lane, unsigned total, int leader_remote = 0) {
    const int quad = warp & 3;           // TMEM lane quadrant this warp may read
    const int half = (warp - 4) >> 2;    // warps 4-7 take the first half of the tile's columns, 8-11 the second
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int cbeg = half == 0 ? 0 : ((p.BN / 2 + 15) & ~15);
    const int cend = half == 0 ? ((p.BN / 2 + 15) & ~15) : p.BN;
    const long long cs = (long long)p.Hd * p.Wd;
    const float os = out_scale_of(p);
    uint32_t tcount = 0;
    for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = acc_index(p, tcount);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[acc], acc_phase(p, tcount), p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      int yo, xo;
      if (MODE == MQ_OP_FWD) { yo = tile.h; xo = tile.w0 + tw_; }
      else {
        const int ch = (int)fdiv((unsigned)tile.cls, p.sw, p.m_sw);
        yo = ch + p.sh * tile.h; xo = tile.cls - ch * p.sw + p.sw * (tile.w0 + tw_);
      }
      const int n = tile.n0 + tn;
      const bool row_ok = yo < p.Hd && xo < p.Wd && n < p.N;
      const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16);
      const bool full_cols = tile.c0 + p.BN <= p.Cd;
      float* o_nchw = p.out + (((long long)n * p.Cd + tile.c0 + cbeg) * p.Hd + yo) * p.Wd + xo;
      float* o_hwnc = p.out + (((long long)yo * p.Wd + xo) * p.N + n) * p.Cd + tile.c0 + cbeg;
      // one 16-column chunk at a time and no unrolling over chunks: its code size matters more (instruction-cache
      // misses stall every role) than its latency (double-buffering the TMEM loads was measured: no change - the
      // NCHW stores themselves are the bound)
#pragma unroll 1
      for (int c = cbeg; c < cend; c += 16) {
        uint32_t v[16];
        if (Q > 0) {
          tmem_ld_32x32b_x16(taddr + c, v);
          tmem_ld_wait();
          if (p.kind_fp4 == 2) scale16(v, os);
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
        if (row_ok) {
          if (p.out_layout == MQ_NCHW) {
#pragma unroll
            for (int j = 0; j < 16; ++j) { if (full_cols || tile.c0 + c + j < p.Cd) *o_nchw = __uint_as_float(v[j]); o_nchw += cs; }
          } else {
            if (full_cols && (p.Cd & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<float4*>(o_hwnc + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (tile.c0 + c + j < p.Cd) o_hwnc[j] = __uint_as_float(v[j]);
            }
            o_hwnc += 16;
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) release_acc(&tempty[acc], leader_remote);
    }
}

// Epilogue role for 256-column tiles (ONE accumulator: the MMA lane cannot start the next tile before this one has left
// tensor memory).  Each of the eight warps copies its 32 rows x 128 columns into REGISTERS, hands the accumulator back at
// once and only then stores - so the stores of a tile (request-bound: 128 KB through 4-byte rows) overlap the next tile's
// MMAs instead of holding them up.  The registers come from the loader / MMA warpgroups (warpgroup_regs_inc / _dec).
template <int MODE>
__device__ __forceinline__ void epilogue_snap_role(const ConvTcParams& p, uint32_t tmem, uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag,
                                                   int warp, int lane, unsigned total, int leader_remote = 0) {
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int cbeg = 128 * half;
    const long long cs = (long long)p.Hd * p.Wd;
    const float os = out_scale_of(p);
    uint32_t tcount = 0;
    for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = acc_index(p, tcount);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[acc], acc_phase(p, tcount), p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      uint32_t v[128];
      if (Q > 0) {
        const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16) + cbeg;
#pragma unroll
        for (int k = 0; k < 8; ++k) tmem_ld_32x32b_x16(taddr + 16 * k, v + 16 * k);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 128; ++j) v[j] = 0u;
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) release_acc(&tempty[acc], leader_remote);      // the accumulator is free: the next tile's MMAs may start
      int yo, xo;
      if (MODE == MQ_OP_FWD) { yo = tile.h; xo = tile.w0 + tw_; }
      else {
        const int ch = (int)fdiv((unsigned)tile.cls, p.sw, p.m_sw);
        yo = ch + p.sh * tile.h; xo = tile.cls - ch * p.sw + p.sw * (tile.w0 + tw_);
      }
      const int n = tile.n0 + tn;
      if (!(yo < p.Hd && xo < p.Wd && n < p.N)) continue;
      const int ncols = min(128, p.Cd - tile.c0 - cbeg);     // columns of this half inside the tensor (may be <= 0)
      if (p.kind_fp4 == 2) {
#pragma unroll
        for (int j = 0; j < 128; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * os);
      }
      if (p.out_layout == MQ_NCHW) {
        float* o = p.out + (((long long)n * p.Cd + tile.c0 + cbeg) * p.Hd + yo) * p.Wd + xo;
#pragma unroll
        for (int j = 0; j < 128; ++j) { if (j < ncols) *o = __uint_as_float(v[j]); o += cs; }
      } else {
        float* o = p.out + (((long long)yo * p.Wd + xo) * p.N + n) * p.Cd + tile.c0 + cbeg;
        if (ncols == 128 && (p.Cd & 3) == 0) {
#pragma unroll
          for (int j = 0; j < 128; j += 4)
            *reinterpret_cast<float4*>(o + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
        } else {
#pragma unroll
          for (int j = 0; j < 128; ++j) if (j < ncols) o[j] = __uint_as_float(v[j]);
        }
      }
    }
}

// Epilogue role of the pair mode (see tile_of_iter): both accumulators hold the same output rows and channels for the
// even and the odd output columns; a thread writes them as float2 (x = 2 (w0 + tw), x + 1), so a warp's store covers
// 64-byte runs per sample instead of every other float.
template <int MODE>
__device__ __forceinline__ void epilogue_pair_role(const ConvTcParams& p, uint32_t tmem, uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag,
                                                   int warp, int lane, unsigned total) {
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int cbeg = half == 0 ? 0 : ((p.BN / 2 + 15) & ~15);
    const int cend = half == 0 ? ((p.BN / 2 + 15) & ~15) : p.BN;
    const long long cs = (long long)p.Hd * p.Wd;
    const float os = out_scale_of(p);
#pragma unroll 1
    for (unsigned j = 0, t; (t = tile_of_iter(p, 2 * j)) < total && !*abort_flag; ++j) {
      const Tile t0 = decode_tile(p, t), t1 = decode_tile(p, t + 1);
      TapWalk<MODE> w0, w1;
      w0.init(p, t0); w1.init(p, t1);
      const int Q0 = w0.chunks(p), Q1 = w1.chunks(p);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[0], j & 1, p.status, MQ_ERR_TIMEOUT) && mbar_wait(&tfull[1], j & 1, p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      const int ch = (int)fdiv((unsigned)t0.cls, p.sw, p.m_sw);
      const int yo = ch + p.sh * t0.h, xo = p.sw * (t0.w0 + tw_);     // even column; the odd class writes xo + 1
      const int n = t0.n0 + tn;
      const bool row_ok = yo < p.Hd && xo < p.Wd && n < p.N;          // Wd is even in this mode: xo + 1 < Wd as well
      const uint32_t taddr = tmem + ((uint32_t)(32 * quad) << 16);
      float* o = p.out + (((long long)n * p.Cd + t0.c0 + cbeg) * p.Hd + yo) * p.Wd + xo;
#pragma unroll 1
      for (int c = cbeg; c < cend; c += 16) {
        uint32_t v0[16], v1[16];
        if (Q0 > 0) tmem_ld_32x32b_x16(taddr + c, v0);
        if (Q1 > 0) tmem_ld_32x32b_x16(taddr + p.BN + c, v1);
        tmem_ld_wait();
        if (p.kind_fp4 == 2) { scale16(v0, os); scale16(v1, os); }   // (accumulators without taps are zeroed below)
        if (Q0 == 0) {
#pragma unroll
          for (int q = 0; q < 16; ++q) v0[q] = 0u;
        }
        if (Q1 == 0) {
#pragma unroll
          for (int q = 0; q < 16; ++q) v1[q] = 0u;
        }
        if (row_ok) {
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            if (t0.c0 + c + q < p.Cd) *reinterpret_cast<float2*>(o) = make_float2(__uint_as_float(v0[q]), __uint_as_float(v1[q]));
            o += cs;
          }
        } else {
          o += 16 * cs;
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&tempty[0]); mbar_arrive(&tempty[1]); }
    }
}

// The same with the accumulators copied into registers first (128-column tiles: 2 x 64 columns per warp = 128 registers, see
// epilogue_snap_role): both accumulators are handed back before the stores, which then run under the next pair's MMAs.
template <int MODE>
__device__ __forceinline__ void epilogue_pair_snap_role(const ConvTcParams& p, uint32_t tmem, uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag,
                                                        int warp, int lane, unsigned total) {
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int cbeg = 64 * half;
    const long long cs = (long long)p.Hd * p.Wd;
    const float os = out_scale_of(p);
#pragma unroll 1
    for (unsigned j = 0, t; (t = tile_of_iter(p, 2 * j)) < total && !*abort_flag; ++j) {
      const Tile t0 = decode_tile(p, t), t1 = decode_tile(p, t + 1);
      TapWalk<MODE> w0, w1;
      w0.init(p, t0); w1.init(p, t1);
      const int Q0 = w0.chunks(p), Q1 = w1.chunks(p);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[0], j & 1, p.status, MQ_ERR_TIMEOUT) && mbar_wait(&tfull[1], j & 1, p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      uint32_t v0[64], v1[64];
      const uint32_t taddr = tmem + ((uint32_t)(32 * quad) << 16) + cbeg;
      if (Q0 > 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) tmem_ld_32x32b_x16(taddr + 16 * k, v0 + 16 * k);
      }
      if (Q1 > 0) {
#pragma unroll
        for (int k = 0; k < 4; ++k) tmem_ld_32x32b_x16(taddr + 128 + 16 * k, v1 + 16 * k);
      }
      tmem_ld_wait();
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&tempty[0]); mbar_arrive(&tempty[1]); }
      const float s0 = Q0 > 0 ? os : 0.f, s1 = Q1 > 0 ? os : 0.f;     // (an accumulator without taps holds nothing of this tile)
      const int ch = (int)fdiv((unsigned)t0.cls, p.sw, p.m_sw);
      const int yo = ch + p.sh * t0.h, xo = p.sw * (t0.w0 + tw_);     // even column; the odd class writes xo + 1
      const int n = t0.n0 + tn;
      if (!(yo < p.Hd && xo < p.Wd && n < p.N)) continue;            // Wd is even in this mode: xo + 1 < Wd as well
      const int ncols = min(64, p.Cd - t0.c0 - cbeg);
      float* o = p.out + (((long long)n * p.Cd + t0.c0 + cbeg) * p.Hd + yo) * p.Wd + xo;
      const bool plain = p.kind_fp4 != 2 && Q0 > 0 && Q1 > 0;
#pragma unroll
      for (int q = 0; q < 64; ++q) {
        if (q < ncols) {
          if (plain) *reinterpret_cast<float2*>(o) = make_float2(__uint_as_float(v0[q]), __uint_as_float(v1[q]));
          else *reinterpret_cast<float2*>(o) = make_float2(Q0 > 0 ? __uint_as_float(v0[q]) * s0 : 0.f, Q1 > 0 ? __uint_as_float(v1[q]) * s1 : 0.f);
        }
        o += cs;
      }
    }
}

// Quantizing epilogue (warps 4-11): the producer applies the activation and emits the NEXT tensor's stored MX form -
// codes [Hd][Wd][N][Cp] and one E8M0 byte per 32-sample x 32-channel tile at a pixel - instead of fp32, i.e. the
// tensor is quantized on chip before it is stored and the fp32 round trip through HBM disappears.  Tiles are TW <= 4
// output columns x 128 / TW >= 32 samples, so a quantization tile (one pixel, 32 samples, 32 channels) lies inside one
// GEMM tile: its 32 samples sit in TW consecutive TMEM lane quadrants (8, 16 or 32 lanes each), its channels in 32
// accumulator columns.  Per 32-channel block a warp loads its 32 x 32 values, applies the activation, takes the
// per-lane maximum and reduces it over the lanes of the same output column (one integer warp reduction).  With
// one-column tiles (the host's choice whenever the batch fills them) a warp's 32 rows ARE a sample tile and that is
// the tile's maximum; with 2 or 4 columns the TW warps of a tile combine their maxima through shared memory (one
// named barrier per block among the four warps of a column half).  Scale and codes then follow exactly the
// quantizer's arithmetic.  A lane writes its row's 32 codes as two stores (a row of the emitted tensor is
// channel-contiguous), and the accumulator goes back to the MMA warp right after the warp's last TMEM load.
// Measured (N = 256, 512 channels, 56 x 56, 1x1, E4M3 -> E4M3 with ReLU, us): one kernel for all formats with a switch per
// block 602; an instance per format 461 (a non-inlined role per format: 785); 256-channel tiles 410; one-column tiles
// 368, without the exchange 323.  Fewer ALU instructions (three-input maxima, ReLU by clearing negative codes after
// packing instead of a maximum per element) or the warp reduction left out: no change - a block takes about 1100
// cycles of its warp for some 150 instructions, i.e. the epilogue waits on latencies (TMEM load, reduction,
// conversion chains) that two warps per scheduler cannot hide, and a second register buffer to overlap two blocks
// does not fit in 128 registers (spills: 538).  Dropped earlier: staging the codes in shared memory for 64-byte
// store runs (slower: the stores are not what the epilogue waits for); two passes over the columns (all maxima
// first, one barrier per tile), which read tensor memory twice and return the accumulator late (slower).
__device__ __forceinline__ void half_sync(int half) { asm volatile("bar.sync %0, 128;" ::"r"(2 + half) : "memory"); }
__device__ __forceinline__ bool half_any(int half, bool pred) {
  int r;
  asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %2, 0;\n\tbar.red.or.pred q, %1, 128, p;\n\tselp.b32 %0, 1, 0, q;\n\t}\n" : "=r"(r) : "r"(2 + half), "r"(pred ? 1 : 0) : "memory");
  return r != 0;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float r;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
// 16 values of a row x f -> 16 codes, stored as one 16-byte (E2M1: 8-byte) word.  RELU: the codes of negative values
// are cleared afterwards, four (E2M1: eight) codes per 32-bit operation - quantize(max(x, 0)) = quantize(x) with the
// negative codes set to zero, and the clearing costs a fifth of a maximum per element.
template <int FMT, bool RELU>
__device__ __forceinline__ void mx_encode_half(const uint32_t* v, float f, uint8_t* dst) {
  unsigned w[4];
#pragma unroll
  for (int k = 0; k < 16; k += 4) {
    const unsigned lo = encode2<FMT>(__uint_as_float(v[k]) * f, __uint_as_float(v[k + 1]) * f);
    const unsigned hi = encode2<FMT>(__uint_as_float(v[k + 2]) * f, __uint_as_float(v[k + 3]) * f);
    w[k >> 2] = FMT == MQ_E2M1 ? (lo | (hi << 8)) : (lo | (hi << 16));
  }
  if (FMT == MQ_E2M1) {
    unsigned q0 = w[0] | (w[1] << 16), q1 = w[2] | (w[3] << 16);
    if (RELU) {
      q0 &= ~(((q0 >> 3) & 0x11111111u) * 0xFu);
      q1 &= ~(((q1 >> 3) & 0x11111111u) * 0xFu);
    }
    *reinterpret_cast<uint2*>(dst) = make_uint2(q0, q1);
  } else {
    if (RELU) {
      constexpr int S = (FMT == MQ_E4M3 || FMT == MQ_E5M2) ? 7 : 5;   // sign bit of a code in its byte
#pragma unroll
      for (int j = 0; j < 4; ++j) w[j] &= ~(((w[j] >> S) & 0x01010101u) * 0xFFu);
    }
    *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
struct MxBlockCtx {
  int Q, bend, half, quad, grp0, tw_, lane, c0;
  uint32_t taddr;
  bool row_ok;
  unsigned col_mask;
  unsigned* my_red;
  uint8_t* o_codes;
  uint8_t* o_scale;
  uint64_t* tempty_acc;
  // the paper's own format (FMT 5): product of the operands' tensor scales (applied to the accumulator first), T_scale of the
  // emitted tensor and 6 T_scale (Eq. 4-5), the running maximum of this warp's emitted values
  float in_scale, tscale, t6;
  unsigned* own_max;
};
// The paper's own format as the emitted one (FMT 5; Eq. 4-6 with the tensor maximum supplied from an earlier step, Sec. VII-B):
// E2M1 elements, one E4M3 scale per 16 samples x 16 channels, written [pixel][ceil(N/16)][C_p/16].  A warp's 32 rows are
// 32 samples of one pixel (one-column tiles: two 16-sample blocks, lanes 0-15 and 16-31) or 16 samples of each of two
// pixels (two-column tiles: even and odd lanes); a 32-channel block of the accumulator is two 16-channel blocks.  Every
// operation of Eq. 5-6 is one IEEE single-precision operation in the order written, as in the quantizer.
template <int ACT>
__device__ __forceinline__ void ts_block(const ConvTcParams& p, MxBlockCtx& c, int b, uint32_t* v) {
  float m[2] = {0.f, 0.f};
  if (c.Q > 0) {
    tmem_ld_wait();
#pragma unroll
    for (int k = 0; k < 32; ++k) {
      float x = __uint_as_float(v[k]) * c.in_scale;
      if (ACT != MQ_ACT_NONE) x = mx_activation(x, ACT);
      v[k] = __float_as_uint(x);
      m[k >> 4] = fmaxf(m[k >> 4], fabsf(x));
    }
  } else {
#pragma unroll
    for (int k = 0; k < 32; ++k) v[k] = 0u;
  }
  const bool more = c.Q > 0 && b + 1 < c.bend;
  if (b + 1 == c.bend) {      // the accumulator has been read: hand it back before the arithmetic and the stores
    tc_fence_before_sync();
    __syncwarp();
    if (c.lane == 0) mbar_arrive(c.tempty_acc);
  }
  const bool blk_ok = c.row_ok && c.c0 + 32 * b < p.mx_Cp;
  float den[2];
  unsigned sc2 = 0;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const unsigned mb = __reduce_max_sync(c.col_mask, c.row_ok ? __float_as_uint(m[h]) : 0u);
    const float bmax = __uint_as_float(mb);
    *c.own_max = max(*c.own_max, mb);
    unsigned sc = 0;
    if (bmax > 0.f && c.tscale > 0.f) sc = (unsigned)__nv_cvt_float_to_fp8(__fdiv_rn(bmax, c.t6), __NV_SATFINITE, __NV_E4M3) & 0x7Fu;   // Eq. 5
    const __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)sc, __NV_E4M3);
    const float bscale = __half2float(*reinterpret_cast<const __half*>(&hr));
    den[h] = (bscale > 0.f && c.tscale > 0.f) ? __fmul_rn(bscale, c.tscale) : 0.f;
    sc2 |= sc << (8 * h);
  }
  // the first lane of each 16-sample block writes the two scale bytes of its 32 channels
  if (blk_ok && c.lane == __ffs(c.col_mask) - 1) *reinterpret_cast<unsigned short*>(c.o_scale + 2 * b) = (unsigned short)sc2;
  uint8_t* dst = c.o_codes + 16 * b;
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    unsigned w[2] = {0u, 0u};
#pragma unroll
    for (int k = 0; k < 16; k += 2) {
      const float x0 = __uint_as_float(v[16 * h + k]), x1 = __uint_as_float(v[16 * h + k + 1]);
      const float q0 = ts_div(x0, den[h]), q1 = ts_div(x1, den[h]);                                   // Eq. 6
      w[k >> 3] |= encode2<MQ_E2M1>(q0, q1) << (4 * (k & 7));
    }
    if (blk_ok) *reinterpret_cast<uint2*>(dst + 8 * h) = make_uint2(w[0], w[1]);
    if (more) tmem_ld_32x32b_x16(c.taddr + 32 * (b + 1) + 16 * h, v + 16 * h);
  }
}

// One 32-channel block of a warp's 32 rows.  v holds (or is about to hold) the block's accumulator values; each half of
// the next block's load is issued as soon as its 16 registers have been converted, so it is in flight during the rest of
// the conversion, the stores and the loop's bookkeeping (a second register buffer, which would put the whole of the next
// load behind this block's arithmetic, does not fit in 128 registers: measured with spills, 1.6x slower).
template <int FMT, int ACT>
__device__ __forceinline__ void mx_block(const ConvTcParams& p, const MxBlockCtx& c, int b, uint32_t* v) {
  constexpr int emax = FMT == MQ_E4M3 ? 8 : (FMT == MQ_E5M2 ? 15 : (FMT == MQ_E3M2 ? 4 : 2));
  constexpr int bpe4 = FMT == MQ_E2M1 ? 1 : 2;
  float m = 0.f;
  if (c.Q > 0) {
    tmem_ld_wait();
    float m0 = 0.f, m1 = 0.f;
    if (ACT == MQ_ACT_SILU) {
#pragma unroll
      for (int k = 0; k < 32; ++k) v[k] = __float_as_uint(mx_activation(__uint_as_float(v[k]), MQ_ACT_SILU));
    }
#pragma unroll
    for (int k = 0; k < 32; k += 4) {
      if (ACT == MQ_ACT_RELU) {
        m0 = fmax3(m0, __uint_as_float(v[k]), __uint_as_float(v[k + 1]));
        m1 = fmax3(m1, __uint_as_float(v[k + 2]), __uint_as_float(v[k + 3]));
      } else {
        m0 = fmax3(m0, fabsf(__uint_as_float(v[k])), fabsf(__uint_as_float(v[k + 1])));
        m1 = fmax3(m1, fabsf(__uint_as_float(v[k + 2])), fabsf(__uint_as_float(v[k + 3])));
      }
    }
    m = fmaxf(m0, m1);
  } else {
#pragma unroll
    for (int k = 0; k < 32; ++k) v[k] = 0u;
  }
  const bool more = c.Q > 0 && b + 1 < c.bend;
  if (b + 1 == c.bend) {      // the accumulator has been read: hand it back before the arithmetic and the stores
    tc_fence_before_sync();
    __syncwarp();
    if (c.lane == 0) mbar_arrive(c.tempty_acc);
  }
  // maximum over the lanes of the same output column: non-negative floats order like their bit patterns, so one
  // integer warp reduction per column group replaces a chain of shuffles
  const unsigned mb = __reduce_max_sync(c.col_mask, c.row_ok ? __float_as_uint(m) : 0u);
  unsigned mx = mb;
  if (p.TW > 1) {     // the sample tile spans TW warps: exchange the maxima through shared memory
    unsigned* rb = c.my_red + (b & 1) * 16;
    if (c.lane < p.TW) rb[c.quad * 4 + c.lane] = mb;
    half_sync(c.half);
    mx = 0;
    for (int g = 0; g < p.TW; ++g) mx = max(mx, rb[(c.grp0 + g) * 4 + c.tw_]);
  }
  const int code = scale_code_of(mx, emax);
  const bool blk_ok = c.row_ok && c.c0 + 32 * b < p.mx_Cp;
  if (c.quad == c.grp0 && c.lane < p.TW && blk_ok) c.o_scale[b] = (uint8_t)code;
  const float f = scale_factor(code);
  uint8_t* dst = c.o_codes + ((32 * b * bpe4) >> 1);
  if (blk_ok) mx_encode_half<FMT, ACT == MQ_ACT_RELU>(v, f, dst);
  if (more) tmem_ld_32x32b_x16(c.taddr + 32 * (b + 1), v);
  if (blk_ok) mx_encode_half<FMT, ACT == MQ_ACT_RELU>(v + 16, f, dst + 8 * bpe4);   // 16 codes further: 16 bytes (E2M1: 8)
  if (more) tmem_ld_32x32b_x16(c.taddr + 32 * (b + 1) + 16, v + 16);
}
// FMT: element format of the emitted tensor.  The role is compiled into kernel instances of its own (conv_tc_kernel's EPI
// parameter), one per format, and the activation is chosen outside the block loop.
template <int MODE, int FMT>
__device__ __forceinline__ void epilogue_mx_role(const ConvTcParams& p, unsigned* red, uint32_t tmem, uint64_t* tfull, uint64_t* tempty,
                                                 volatile int* abort_flag, int warp, int lane, unsigned total) {
    const int quad = warp & 3;
    const int half = warp < 12 ? (warp - 4) >> 2 : 2 + ((warp - 16) >> 2);   // column group 0..3 of this warp (four warps each, one per lane quadrant)
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int nblk = p.BN >> 5;                         // 32-channel blocks of a tile
    constexpr int NG = FMT == 5 ? 4 : 2;                // column groups: 16 epilogue warps for the paper's format, else 8
    const int per = (nblk + NG - 1) / NG;
    const int bbeg = min(nblk, half * per), bend = min(nblk, bbeg + per);
    const int grp0 = quad & ~(p.TW - 1);                // first quadrant of the TW quadrants that hold this sample tile
    constexpr bool TS = FMT == 5;                       // the paper's own format (16 x 16 blocks; TW is 1 or 2)
    constexpr int bpe4 = (FMT == MQ_E2M1 || TS) ? 1 : 2;        // bytes per element x 2
    const int Ct = TS ? p.mx_Cp >> 4 : p.mx_Cp >> 5;
    unsigned* my_red = red + half * 32;                 // [parity][quadrant][column]
    // lanes of this lane's column (TS: of its 16-sample block - half a warp with one-column tiles)
    const unsigned col_mask = TS ? (p.TW == 1 ? 0xffffu << (lane & 16) : 0x55555555u << (lane & 1))
                                 : (p.TW == 1 ? 0xffffffffu : (p.TW == 2 ? 0x55555555u : 0x11111111u)) << (lane & (p.TW - 1));
    unsigned own_max = 0;
    float ts_in = 1.f, ts_t = 0.f, ts_t6 = 0.f;
    if (TS) {
      ts_in = out_scale_of(p);
      ts_t = __fdiv_rn(__ldg(p.mx_ts_amax), __fmul_rn(448.0f, 6.0f));                       // Eq. 4
      ts_t6 = __fmul_rn(ts_t, 6.0f);
      if (blockIdx.x == 0 && warp == 4 && lane == 0) p.mx_ts_stats[0] = ts_t;
    }
    uint32_t tcount = 0;
    for (unsigned t = blockIdx.x; t < total; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = acc_index(p, tcount);
      bool ok = true;
      if (lane == 0) ok = !*abort_flag && mbar_wait(&tfull[acc], acc_phase(p, tcount), p.status, MQ_ERR_TIMEOUT);
      // the four warps of a half leave together or not at all: they meet at barriers inside the tile
      // (one-column tiles have no barriers inside: each warp decides for itself)
      if (p.TW > 1 ? half_any(half, !ok) : __shfl_sync(0xffffffffu, ok ? 0 : 1, 0) != 0) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      int yo, xo;
      if (MODE == MQ_OP_FWD) { yo = tile.h; xo = tile.w0 + tw_; }
      else {
        const int ch = (int)fdiv((unsigned)tile.cls, p.sw, p.m_sw);
        yo = ch + p.sh * tile.h; xo = tile.cls - ch * p.sw + p.sw * (tile.w0 + tw_);
      }
      const int n = tile.n0 + tn;
      const bool row_ok = yo < p.Hd && xo < p.Wd && n < p.N;
      const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16);
      const long long pix = (long long)yo * p.Wd + xo;
      uint8_t* o_codes = p.mx_codes + (((pix * p.N + n) * p.mx_Cp + tile.c0) * bpe4 >> 1);
      uint8_t* o_scale = TS ? p.mx_scales + (pix * ((p.N + 15) >> 4) + (n >> 4)) * Ct + (tile.c0 >> 4)
                            : p.mx_scales + (pix * p.Nt + (n >> 5)) * Ct + (tile.c0 >> 5);
      // no separate activation pass for none / ReLU: the maximum of max(x, 0) is the maximum of x and 0, and negative
      // codes are cleared after packing
      MxBlockCtx c;
      c.Q = Q; c.bend = bend; c.taddr = taddr; c.row_ok = row_ok; c.col_mask = col_mask; c.my_red = my_red; c.half = half; c.quad = quad;
      c.grp0 = grp0; c.tw_ = tw_; c.lane = lane; c.o_codes = o_codes; c.o_scale = o_scale; c.c0 = tile.c0; c.tempty_acc = &tempty[acc];
      c.in_scale = ts_in; c.tscale = ts_t; c.t6 = ts_t6; c.own_max = &own_max;
      uint32_t v[32];
      if (Q > 0 && bbeg < bend) {
        tmem_ld_32x32b_x16(taddr + 32 * bbeg, v);
        tmem_ld_32x32b_x16(taddr + 32 * bbeg + 16, v + 16);
      }
      // the activation is chosen outside the block loop: three straight-line copies instead of a test per element
      if constexpr (TS) {
        if (p.mx_act == MQ_ACT_RELU) {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) ts_block<MQ_ACT_RELU>(p, c, b, v);
        } else if (p.mx_act == MQ_ACT_SILU) {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) ts_block<MQ_ACT_SILU>(p, c, b, v);
        } else {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) ts_block<MQ_ACT_NONE>(p, c, b, v);
        }
      } else {
        if (p.mx_act == MQ_ACT_RELU) {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) mx_block<FMT, MQ_ACT_RELU>(p, c, b, v);
        } else if (p.mx_act == MQ_ACT_SILU) {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) mx_block<FMT, MQ_ACT_SILU>(p, c, b, v);
        } else {
#pragma unroll 1
          for (int b = bbeg; b < bend; ++b) mx_block<FMT, MQ_ACT_NONE>(p, c, b, v);
        }
      }
      if (bbeg >= bend) {      // a tile of 32 channels leaves the second half without a block
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[acc]);
      }
    }
    if (TS) {   // this tensor's own maximum, for the next step's Eq. 4: one atomic per warp
      const unsigned wmax = __reduce_max_sync(0xffffffffu, own_max);
      if (lane == 0 && wmax != 0) atomicMax(reinterpret_cast<unsigned*>(p.mx_ts_stats + 1), wmax);
    }
}

// Epilogue role with TMA stores, NCHW output (warps 4-11).  Each warp moves its 32 rows x up to 64 channels on
// its own: TMEM -> registers -> a private [channel][row] staging slice (row index fastest, so the writes are
// conflict-free), then one lane stores the slice as a box of the output seen as (W, N, C, H): TW columns x
// 32/TW samples x the channels.  The store engine clips the box at the tensor's edges and keeps the store
// instructions out of the load/store pipe that the MMA issue shares.  The slice is reused only after the
// previous tile's store has read it, which by then is long done.
constexpr int EPI_STAGING_BYTES = 8 * 64 * 32 * 4;   // warps x [64 channels][32 rows] floats
template <int MODE>
__device__ __forceinline__ void epilogue_tma_role(const ConvTcParams& p, const CUtensorMap* map_out, float* staging, uint32_t tmem,
                                                  uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag, int warp, int lane, unsigned total,
                                                  int leader_remote = 0) {
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int cbeg = half == 0 ? 0 : ((p.BN / 2 + 15) & ~15);
    const int cend = half == 0 ? ((p.BN / 2 + 15) & ~15) : p.BN;
    float* buf = staging + (warp - 4) * (64 * 32);
    const int n_off = quad * (32 >> p.lgTW);          // first sample of this warp's rows inside the tile
    const bool hwnc = p.out_layout == MQ_HWNC;
    const int hrow = lane;   // the [H][W][N][C] store's box walks (sample, column) in the rows' own order
    const float os = out_scale_of(p);
    uint32_t tcount = 0;
    for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = acc_index(p, tcount);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[acc], acc_phase(p, tcount), p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      const int cls_h = MODE == MQ_OP_FWD ? 0 : (int)fdiv((unsigned)tile.cls, p.sw, p.m_sw);
      const int yo = MODE == MQ_OP_FWD ? tile.h : cls_h + p.sh * tile.h;
      const int xo0 = MODE == MQ_OP_FWD ? tile.w0 : (tile.cls - cls_h * p.sw) + p.sw * tile.w0;   // first output column (a parity class's columns are sw apart)
      const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16);
      if (cbeg >= cend) {      // a tile of 16 channels leaves the second half without columns
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) release_acc(&tempty[acc], leader_remote);
      }
#pragma unroll 1
      for (int c0 = cbeg; c0 < cend; c0 += 64) {
        const int nch = min(4, (cend - c0) >> 4);
        if (lane == 0) bulk_wait_group_read<0>();      // the previous store has read the slice
        __syncwarp();
        // chunk by chunk, rolled: the hot loop stays small in the instruction cache
#pragma unroll 1
        for (int i = 0; i < nch; ++i) {
          uint32_t v[16];
          if (Q > 0) {
            tmem_ld_32x32b_x16(taddr + c0 + 16 * i, v);
            tmem_ld_wait();
            if (p.kind_fp4 == 2) scale16(v, os);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0u;
          }
          if (!hwnc) {
            float* bi = buf + (16 * i) * 32 + lane;
#pragma unroll
            for (int j = 0; j < 16; ++j) bi[j * 32] = __uint_as_float(v[j]);
          } else {
            // [Ho][Wo][N][C] output: rows of 32 channels (128 bytes, 128-byte swizzle: consecutive lanes hit different
            // bank groups); chunk i is the 16-byte units 4 (i & 1) .. + 3 of 32-channel group i >> 1
            uint8_t* bg = reinterpret_cast<uint8_t*>(buf) + (i >> 1) * 4096 + hrow * 128;
#pragma unroll
            for (int u = 0; u < 4; ++u)
              *reinterpret_cast<uint4*>(bg + ((((i & 1) * 4 + u) ^ (hrow & 7)) << 4)) = make_uint4(v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
          }
        }
        if (c0 + 64 >= cend) {   // the accumulator has been read: hand it back before the store
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) release_acc(&tempty[acc], leader_remote);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (!hwnc) tma_store_4d(map_out, buf, xo0, tile.n0 + n_off, tile.c0 + c0, yo);
          else {
            tma_store_4d(map_out, buf, tile.c0 + c0, xo0, tile.n0 + n_off, yo);
            if (nch > 2) tma_store_4d(map_out, buf + 1024, tile.c0 + c0 + 32, xo0, tile.n0 + n_off, yo);
          }
          bulk_commit_group();
        }
      }
    }
    if (lane == 0) bulk_wait_group_all();
}

// The same for 256-column tiles with ONE accumulator: the warp first copies its 32 rows x 128 columns into registers and hands
// the accumulator back (see epilogue_snap_role), then stages and stores its two 64-channel slices from the registers.
template <int MODE>
__device__ __forceinline__ void epilogue_tma_snap_role(const ConvTcParams& p, const CUtensorMap* map_out, float* staging, uint32_t tmem,
                                                       uint64_t* tfull, uint64_t* tempty, volatile int* abort_flag, int warp, int lane, unsigned total,
                                                       int leader_remote = 0) {
    const int quad = warp & 3;
    const int half = (warp - 4) >> 2;
    const int cbeg = 128 * half;
    float* buf = staging + (warp - 4) * (64 * 32);
    const int n_off = quad * (32 >> p.lgTW);
    const bool hwnc = p.out_layout == MQ_HWNC;
    const int hrow = lane;
    const float os = out_scale_of(p);
    uint32_t tcount = 0;
    for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = acc_index(p, tcount);
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[acc], acc_phase(p, tcount), p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      uint32_t v[128];
      if (Q > 0) {
        const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16) + cbeg;
#pragma unroll
        for (int k = 0; k < 8; ++k) tmem_ld_32x32b_x16(taddr + 16 * k, v + 16 * k);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 128; ++j) v[j] = 0u;
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) release_acc(&tempty[acc], leader_remote);      // the accumulator is free: the next tile's MMAs may start
      if (p.kind_fp4 == 2) {
#pragma unroll
        for (int j = 0; j < 128; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * os);
      }
      const int cls_h = MODE == MQ_OP_FWD ? 0 : (int)fdiv((unsigned)tile.cls, p.sw, p.m_sw);
      const int yo = MODE == MQ_OP_FWD ? tile.h : cls_h + p.sh * tile.h;
      const int xo0 = MODE == MQ_OP_FWD ? tile.w0 : (tile.cls - cls_h * p.sw) + p.sw * tile.w0;
#pragma unroll
      for (int rd = 0; rd < 2; ++rd) {
        const int c0 = cbeg + 64 * rd;
        if (tile.c0 + c0 >= p.Cd) break;              // (a ragged last channel tile: nothing of this slice is inside the tensor)
        if (lane == 0) bulk_wait_group_read<0>();      // the previous store has read the slice
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t* vv = v + 64 * rd + 16 * i;
          if (!hwnc) {
            float* bi = buf + (16 * i) * 32 + lane;
#pragma unroll
            for (int j = 0; j < 16; ++j) bi[j * 32] = __uint_as_float(vv[j]);
          } else {
            uint8_t* bg = reinterpret_cast<uint8_t*>(buf) + (i >> 1) * 4096 + hrow * 128;
#pragma unroll
            for (int u = 0; u < 4; ++u)
              *reinterpret_cast<uint4*>(bg + ((((i & 1) * 4 + u) ^ (hrow & 7)) << 4)) = make_uint4(vv[4 * u], vv[4 * u + 1], vv[4 * u + 2], vv[4 * u + 3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (!hwnc) tma_store_4d(map_out, buf, xo0, tile.n0 + n_off, tile.c0 + c0, yo);
          else {
            tma_store_4d(map_out, buf, tile.c0 + c0, xo0, tile.n0 + n_off, yo);
            tma_store_4d(map_out, buf + 1024, tile.c0 + c0 + 32, xo0, tile.n0 + n_off, yo);
          }
          bulk_commit_group();
        }
      }
    }
    if (lane == 0) bulk_wait_group_all();
}

// EPI: -1 = fp32 output (the three fp32 epilogue roles, chosen at run time: an instance per role was measured, no
// change); 0..4 = quantizing epilogue emitting element format EPI
// registers per thread of the epilogue warpgroups / of the others in the fp32-output kernels (16 warps, 128 per thread at launch)
#ifndef MQ_EPI_REGS
#define MQ_EPI_REGS 192
#endif
constexpr uint32_t EPI_REGS = MQ_EPI_REGS, OTHER_REGS = 256 - MQ_EPI_REGS;
static_assert(2 * (EPI_REGS + OTHER_REGS) * 128 == 512 * 128, "the warpgroups' register budgets must add up to the launch's");

// DUO: the two blocks of a cluster work on ONE 256 x 256 tile (cta_group::2): each loads the activation rows of its own
// 128-row tile (tiles 2k and 2k + 1 of the round robin: same channel tile, neighbouring positions) and HALF of the weight
// tile's 256 rows, so a stage brings 32 KB instead of 48 KB of operands into a block's shared memory - these GEMMs wait for
// operands (E2M1) or run at the power cap (E4M3).  The leader's lane issues the scale copies, MMAs and commits for both
// blocks; every copy of either block counts on the LEADER's stage barrier (its loaders announce both blocks' bytes); the
// commits free the stage and publish the accumulator in both blocks; the peer's epilogue warps hand the accumulator back
// on the leader's barrier.  map_sfa / map_sfb: the scale images as rows of 256 bytes (tiled copies can count on a barrier
// of the other block, plain bulk copies cannot).
template <int MODE, int KB, int KIND, int EPI = -1, bool DUO = false>
__global__ void __launch_bounds__(tc_threads_of(EPI), 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_out,
               const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb, const ConvTcParams p) {
  constexpr int G = 128 / KB;          // chunks per stage
  constexpr int APC = KB / 32;         // MMA K-atoms (32 bytes) per chunk
  constexpr bool FP4 = KIND != 0;
  constexpr int SPA = spa_of_kind(KIND);     // scale bytes per atom
  constexpr int SFA_B = KIND == 2 ? SFA_BYTES_NV : SFA_BYTES, SFB_B = KIND == 2 ? SFB_BYTES_NV : SFB_BYTES;
  constexpr int SFC = KIND == 2 ? SF_COLS_NV : SF_COLS, SFB_OFF = KIND == 2 ? 16 : 8;   // TMEM columns per stage; B-side offset in them
  constexpr int BPC = APC * SPA;       // scale bytes per chunk: 1, 2, 4 or 8
  constexpr int LAYOUT = KB == 128 ? 2 : (KB == 64 ? 4 : 6);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int b_stage_bytes = (DUO ? p.BN / 2 : p.BN) * 128;    // (a pair of blocks: each holds half of the weight tile's rows)
  const int stage_bytes = A_STAGE_BYTES + b_stage_bytes + SFA_B + SFB_B;
  float* staging = reinterpret_cast<float*>(smem + (size_t)p.stages * stage_bytes);   // TMA-store epilogue only
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes + (p.tma_store ? EPI_STAGING_BYTES : 0));
  uint64_t* empty = full + p.stages;
  uint64_t* sffull = empty + p.stages;     // scale vectors of the stage have landed in TMEM
  uint64_t* tfull = sffull + p.stages;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  unsigned* mx_red = reinterpret_cast<unsigned*>((reinterpret_cast<uintptr_t>(tmem_slot + 2) + 15) & ~static_cast<uintptr_t>(15));   // quantizing epilogue only

  // The warp index goes through a shuffle so that the compiler knows it to be warp-uniform: the role loops below are
  // run by whole warps, their arithmetic stays in the uniform datapath, and only the copy / MMA / commit instructions
  // are issued by one elected lane (around `if (lane == 0)` every operand of those instructions would first be moved
  // out of a per-thread register, which more than doubles the issuing thread's cycles per instruction).
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const uint32_t rank = DUO ? __shfl_sync(0xffffffffu, cluster_ctarank(), 0) : 0u;   // 0: the pair's leader
  const int atoms_b = (p.BN + 127) / 128;
  const unsigned total = (unsigned)p.total_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 3); mbar_init(&empty[s], 1); mbar_init(&sffull[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], (EPI == 5 || DUO) ? 16 : 8); }
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
    if (p.tma_store) prefetch_tensormap(&map_out);
  }
  if (warp == 1) {
    if (DUO) { tmem_alloc_2(tmem_slot, 512); tmem_relinquish_2(); }
    else { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (DUO) cluster_sync_all();   // both blocks' barriers and tensor memory exist before anything crosses over
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();   // set-up above touched only shared memory, tensor memory and the kernel parameters

  // loader warps: (kind, parity of the stages it serves)
  const int lkind = (warp == 0 || warp == 12) ? 0 : ((warp == 3 || warp == 13) ? 1 : ((warp == 14 || warp == 15) ? 2 : -1));
  const int lhalf = (warp == 12 || warp == 13 || warp == 15) ? 1 : 0;
  // The epilogue warps are whole warpgroups (4-7, 8-11; with 24 warps also 16-23), the other roles share groups 0-3 and 12-15.
  // fp32 output: the epilogue groups take registers from the other two for their copy of a 256-column accumulator
  // (epilogue_snap_role): (2 x OTHER_REGS + 2 x EPI_REGS) x 128 threads = the 512 x 128 registers of the launch bound.
  if ((warp >= 4 && warp < 12) || warp >= 16) {
    if (EPI < 0) warpgroup_regs_inc<EPI_REGS>();
    if (EPI >= 0) epilogue_mx_role<MODE, EPI < 0 ? 0 : EPI>(p, mx_red, tmem, tfull, tempty, abort_flag, warp, lane, total);
    else if (p.pair && p.BN == 128 && p.snap) epilogue_pair_snap_role<MODE>(p, tmem, tfull, tempty, abort_flag, warp, lane, total);
    else if (p.pair) epilogue_pair_role<MODE>(p, tmem, tfull, tempty, abort_flag, warp, lane, total);
    else if (p.tma_store && p.BN == 256 && p.snap) epilogue_tma_snap_role<MODE>(p, &map_out, staging, tmem, tfull, tempty, abort_flag, warp, lane, total, DUO && rank != 0);
    else if (p.tma_store) epilogue_tma_role<MODE>(p, &map_out, staging, tmem, tfull, tempty, abort_flag, warp, lane, total);
    else if (p.BN == 256 && p.snap) epilogue_snap_role<MODE>(p, tmem, tfull, tempty, abort_flag, warp, lane, total, DUO && rank != 0);
    else epilogue_role<MODE>(p, tmem, tfull, tempty, abort_flag, warp, lane, total);
  } else {
  if (EPI < 0) warpgroup_regs_dec<OTHER_REGS>();
  if (lkind >= 0) {
    // ------------------------------------------------------------------ TMA loaders
    // A warp gets one bulk copy accepted per ~170 cycles whatever its size, and the loop around it is a chain of
    // dependent instructions, so a stage's copies are spread over warps: one KIND of copy (activation boxes, weight
    // boxes, the two scale chunks) per pair of warps, which take even and odd stages.  Every warp walks all stages
    // (the walk is a few additions) but waits and issues only for its own; each kind arrives once per stage on the
    // stage's barrier with its own byte count.
    {
      uint32_t s = 0, phase = 0, gi = 0;
      const uint32_t row_bytes = lkind == 1 ? (uint32_t)(DUO ? p.BN / 2 : p.BN) * KB : (p.a_tx34 ? 96u * KB : 128u * KB);
      for (unsigned i = 0, t; (t = tile_of_iter(p, i)) < total && !*abort_flag; ++i) {
        const Tile tile = decode_tile(p, t);
        TapWalk<MODE> tw;
        tw.init(p, tile);
        const int Q = tw.chunks(p);
        ChunkPos pos;
        pos.reset();
        const uint8_t* sfa_src = p.sfa_img + (size_t)tile_m_index(p, tile) * p.max_stages * (512 * SPA);
        const uint8_t* sfb_src = p.sfb_img + ((size_t)tile.cls * p.tiles_c + tile.ct) * p.max_stages * (512 * SPA * atoms_b);
        // shared A-side chunks: keyed by the source row (output row + kh, or + Kh-1-kh for the input gradient)
        const int dd_row = p.tiles_w * tw.nkw * p.cpt;
        const uint8_t* sfa_dd = p.sfa_img + ((size_t)(((tile.n0 >> p.lgTN) * p.sfa_hk + tile.h + (MODE == MQ_OP_FWD ? 0 : p.Kh - 1)) * p.tiles_w +
                                                      (tile.w0 >> p.lgTW)) * (tw.nkw * p.cpt)) * (512 * SPA);
        for (int q0 = 0; q0 < Q; q0 += G, ++gi) {
          const int nch = min(G, Q - q0);
          const bool mine = (gi & 1u) == (uint32_t)lhalf;
          if (G == 1 && p.sfa_dedup)
            sfa_src = sfa_dd + (long long)((MODE == MQ_OP_FWD ? pos.ia : -pos.ia) * dd_row + pos.ib * p.cpt + pos.cc) * (512 * SPA);
          // coordinates of the stage's boxes, before the wait
          int c0[G], c1[G], c2[G];
#pragma unroll
          for (int c = 0; c < G; ++c) {
            if (c < nch) {
              c0[c] = pos.cc * KB;
              c1[c] = lkind == 1 ? tap_index(tw, pos) : src_w0(tw, pos);
              c2[c] = src_h(tw, pos);
              pos.advance(tw, p.cpt);
            }
          }
          if (mine) {
            uint8_t* sa = smem + (size_t)s * stage_bytes;
            uint8_t* sb = sa + A_STAGE_BYTES;
            if (!mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
            if (DUO) {
              // both blocks' copies count on the leader's barrier; its loaders announce the bytes of both
              if (elect_one()) {
                const uint32_t lbar = cluster_addr_of(&full[s], 0);
                if (lkind == 2) {
                  if (rank == 0) mbar_arrive_expect_tx(&full[s], 2u * 512u * SPA * (1 + atoms_b));
                  tma_load_2d_pair(sb + b_stage_bytes, &map_sfa, lbar, 0, (int)((sfa_src - p.sfa_img) >> 8));
                  tma_load_2d_pair(sb + b_stage_bytes + SFA_B, &map_sfb, lbar, 0, (int)((sfb_src - p.sfb_img) >> 8));
                } else {
                  if (rank == 0) mbar_arrive_expect_tx(&full[s], 2u * row_bytes);
                  if (lkind == 1) tma_load_3d_pair(sb, &map_b, lbar, c0[0], c1[0], tile.c0 + (int)rank * (p.BN / 2));
                  else tma_load_4d_pair(sa, &map_a, lbar, c0[0], c1[0], tile.n0, c2[0]);
                }
              }
            } else
            if (elect_one()) {
              if (lkind == 2) {
                mbar_arrive_expect_tx(&full[s], 512u * SPA * (1 + atoms_b));
                bulk_load(sb + b_stage_bytes, sfa_src, 512 * SPA, &full[s]);
                bulk_load(sb + b_stage_bytes + SFA_B, sfb_src, 512 * SPA * atoms_b, &full[s]);
              } else {
                mbar_arrive_expect_tx(&full[s], (uint32_t)nch * row_bytes);
#pragma unroll
                for (int c = 0; c < G; ++c) {
                  if (c < nch) {
                    if (lkind == 1) tma_load_3d(sb + c * p.BN * KB, &map_b, &full[s], c0[c], c1[c], tile.c0);
                    else tma_load_4d(sa + c * 128 * KB, &map_a, &full[s], c0[c], c1[c], tile.n0, c2[c]);
                  }
                }
              }
            }
            __syncwarp();
          }
          sfa_src += 512 * SPA;
          sfb_src += 512 * SPA * atoms_b;
          if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (a pair of blocks: the leader's)
    if (!DUO || rank == 0) {
      const uint64_t op_desc = smem_desc_base(16, 8 * KB, LAYOUT);
      const uint32_t sf_base = tmem + p.n_acc * p.BN;
      const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
      const uint64_t a_desc0 = smem_desc(op_desc, smem_u32(smem));
      const uint64_t b_desc0 = smem_desc(op_desc, smem_u32(smem + A_STAGE_BYTES));
      const uint32_t b_chunk16 = (uint32_t)(p.BN * KB) >> 4;
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint64_t sfa_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes));
      const uint64_t sfb_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes + SFA_B));
      uint32_t idesc_id[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) idesc_id[i] = idesc_with_sf_ids(p.idesc, i, i);
      const bool self_cp = !FP4 || p.mma_cp;
      uint32_t s = 0, phase = 0, tcount = 0;
      for (unsigned t; (t = tile_of_iter(p, tcount)) < total && !*abort_flag; ++tcount) {
        const Tile tile = decode_tile(p, t);
        TapWalk<MODE> tw;
        tw.init(p, tile);
        const int Q = tw.chunks(p);
        const int acc = acc_index(p, tcount);
        if (!mbar_wait(&tempty[acc], acc_phase(p, tcount) ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem + acc * p.BN;
        uint32_t accumulate = 0;
        for (int q0 = 0; q0 < Q; q0 += G) {
          // the scale copier signals sffull[s] once the stage's operands are in smem and its scale vectors in TMEM
          // E2M1: the scale copier signals sffull[s] once the stage's scale vectors are in TMEM.  8-bit operands: this
          // warp waits for the stage itself and its lane issues the (three) scale copies right before the MMAs that
          // read them - same thread, so the tensor pipe keeps the order, and no copy queues behind MMAs issued earlier.
          if (!mbar_wait(self_cp ? &full[s] : &sffull[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          tc_fence_after_sync();
          const uint32_t so = s * stage16;
          const uint32_t sfa_t = sf_base + s * SFC, sfb_t = sfa_t + SFB_OFF;
          const int natoms = min(G, Q - q0) * APC;
          if (elect_one()) {
            if (DUO) {
#pragma unroll
              for (int g = 0; g < SPA; ++g) {
                tmem_cp_32x128b_warpx4_2(sfa_t + 4 * g, sfa_desc0 + so + g * 32);
                tmem_cp_32x128b_warpx4_2(sfb_t + 4 * g * atoms_b, sfb_desc0 + so + g * atoms_b * 32);
                tmem_cp_32x128b_warpx4_2(sfb_t + 4 * (g * atoms_b + 1), sfb_desc0 + so + (g * atoms_b + 1) * 32);
              }
            } else if (self_cp) {
#pragma unroll
              for (int g = 0; g < SPA; ++g) {
                tmem_cp_32x128b_warpx4(sfa_t + 4 * g, sfa_desc0 + so + g * 32);
                tmem_cp_32x128b_warpx4(sfb_t + 4 * g * atoms_b, sfb_desc0 + so + g * atoms_b * 32);
                if (atoms_b > 1) tmem_cp_32x128b_warpx4(sfb_t + 4 * (g * atoms_b + 1), sfb_desc0 + so + (g * atoms_b + 1) * 32);
              }
            }
            uint32_t accu = accumulate;
#pragma unroll
            for (int a = 0; a < 4; ++a) {
              if (a < natoms) {
                const int c = a / APC, ja = a % APC;
                const uint64_t ad = a_desc0 + so + c * ((128 * KB) >> 4) + ja * 2;
                const uint64_t bd = b_desc0 + so + c * b_chunk16 + ja * 2;
                const int g = (a * SPA) >> 2, id = (a * SPA) & 3;
                if (DUO && KIND == 2) mma_nvf4_2(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                else if (DUO && KIND == 1) mma_mxf4_2(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                else if (DUO) mma_mxf8f6f4_2(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                else if (KIND == 2) mma_nvf4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                else if (KIND == 1) mma_mxf4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                else mma_mxf8f6f4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accu);
                accu = 1;
              }
            }
            if (DUO) tc_commit_2_multicast(&empty[s], 3); else tc_commit(&empty[s]);   // (a pair: frees the stage in both blocks)
          }
          __syncwarp();
          accumulate = 1;
          if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
        }
        if (elect_one()) {
          if (DUO) { if (Q > 0) tc_commit_2_multicast(&tfull[acc], 3); else { mbar_arrive(&tfull[acc]); mbar_arrive_remote(&tfull[acc], 1); } }
          else if (Q > 0) tc_commit(&tfull[acc]); else mbar_arrive(&tfull[acc]);
        }
        __syncwarp();
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ scale copier
    // Copies the stage's scale chunks smem -> TMEM (one TMEM scale buffer per pipeline stage) from its own
    // thread, so these copies overlap the MMA issuer's work on earlier stages.  The buffer of stage s is free
    // whenever full[s] completes: the producers refilled the stage only after the MMAs that read it committed.
    // E2M1 only (twice the scale bytes, up to six copies per stage); for 8-bit operands the MMA lane issues them.
    if (FP4 && !p.mma_cp) {
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint32_t sf_base = tmem + p.n_acc * p.BN;
      const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
      const uint64_t sfa_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes));
      const uint64_t sfb_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes + SFA_B));
      uint32_t s = 0, phase = 0;
      bool alive = true;
      for (unsigned i = 0, t; (t = tile_of_iter(p, i)) < total && alive && !*abort_flag; ++i) {
        const Tile tile = decode_tile(p, t);
        TapWalk<MODE> tw;
        tw.init(p, tile);
        const int Q = tw.chunks(p);
        for (int q0 = 0; q0 < Q; q0 += G) {
          if (!mbar_wait(&full[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; alive = false; break; }
          tc_fence_after_sync();
          const uint32_t so = s * stage16;
          const uint32_t sfa_t = sf_base + s * SFC, sfb_t = sfa_t + SFB_OFF;
          if (elect_one()) {
#pragma unroll
            for (int g = 0; g < SPA; ++g) {
              tmem_cp_32x128b_warpx4(sfa_t + 4 * g, sfa_desc0 + so + g * 32);
              for (int a = 0; a < atoms_b; ++a) tmem_cp_32x128b_warpx4(sfb_t + 4 * (g * atoms_b + a), sfb_desc0 + so + (g * atoms_b + a) * 32);
            }
            tc_commit(&sffull[s]);
          }
          __syncwarp();
          if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
        }
      }
    }
  }
  }
  // teardown: everyone meets here (all loops are bounded), then the allocating warp frees TMEM
  tc_fence_before_sync();
  __syncthreads();
  if (DUO) cluster_sync_all();   // nothing of the peer block is touched after this point
  if (warp == 1) { if (DUO) tmem_dealloc_2(tmem, 512); else tmem_dealloc(tmem, 512); }
}

template <int BPC>
__device__ __forceinline__ unsigned long long load_scale_bytes(const uint8_t* ptr) {
  if (BPC == 1) return __ldg(ptr);
  if (BPC == 2) return __ldg(reinterpret_cast<const unsigned short*>(ptr));
  if (BPC == 4) return __ldg(reinterpret_cast<const unsigned int*>(ptr));
  return __ldg(reinterpret_cast<const unsigned long long*>(ptr));
}

// Builds, in shared memory, the scale-vector chunks ([chunk][group][atom][512]) of the resident weight tile of
// the whole-tile kernel (channel tile 0).  Called by all threads of the block before the roles start (stride 1:
// tap q of the walk is weight tap q).
template <int KB, bool FP4>
__device__ __forceinline__ void halo_build_sfb(const ConvTcParams& p, uint8_t* s_sfb) {
  constexpr int G = 128 / KB, APC = KB / 32, SPA = FP4 ? 2 : 1, BPC = APC * SPA;
  const int taps = p.Kh * p.Kw;
  const int atoms_b = (p.BN + 127) / 128;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
#pragma unroll 1
  for (int st = warp; st < p.max_stages; st += nwarps) {
    unsigned long long acc[8] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
#pragma unroll 1
    for (int c = 0; c < G; ++c) {
      const int q = st * G + c;
      if (q < taps) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j < 4 * atoms_b && 32 * j < p.BN && 32 * j < p.Cd)
            acc[j] |= load_scale_bytes<BPC>(p.b_scales + ((long long)j * taps + q) * p.Kblocks) << (8 * c * BPC);
        }
      }
    }
    uint8_t* dst = s_sfb + (size_t)st * (512 * SPA * atoms_b) + lane * 16;
#pragma unroll
    for (int g = 0; g < SPA; ++g)
#pragma unroll 1
      for (int a = 0; a < atoms_b; ++a)
        *reinterpret_cast<uint4*>(dst + (g * atoms_b + a) * 512) =
            make_uint4((uint32_t)(acc[4 * a] >> (32 * g)), (uint32_t)(acc[4 * a + 1] >> (32 * g)), (uint32_t)(acc[4 * a + 2] >> (32 * g)),
                       (uint32_t)(acc[4 * a + 3] >> (32 * g)));
  }
  fence_proxy_async_smem();   // the scale copies read these through the async proxy
}

// ---- whole-tile-per-stage variant -------------------------------------------------------------------
// For stride-1 layers whose tap has at most 64 bytes of channels (one chunk per tap), the per-tap TMA boxes
// of the kernel above are tiny and their issue rate is the limit.  Here
//  * the weight tile (all taps, a pre-swizzled image written by the expansion kernel) and its scale chunks are
//    RESIDENT: one bulk copy when the channel tile changes (never, when the layer has a single channel tile),
//    its scale vectors copied to TMEM once;
//  * a pipeline stage holds the whole K range of a tile's activations, every stored pixel once (the data reuse
//    of Sec. IV-A): ONE TMA box [Kh rows][TN samples][TW + Kw - 1 columns][KB], and each tap's A operand is a
//    view into it: tap (kh, kw) starts at (kh * TN * WH + kw) * KB with 8-row groups WH * KB bytes apart (TW = 8:
//    one 8-row swizzle group per sample).
// Roles and barriers are those of conv_tc_kernel, plus bfull / bempty for the resident weight tile.
// With a single channel tile (p.fused) no preparation kernel runs at all: every block builds the weight image and
// its scale chunks in shared memory itself at start-up, and warp 3 expands each tile's activation scales (a
// Kh x (TW + Kw - 1) patch of tile scales: all rows of a tile lie in one 32-sample block) into the scale-vector
// chunks of the tile's stage, a few tiles ahead of the MMAs.
// TAPS > 0 fixes the tap count at compile time (the MMA issue loop is then fully unrolled with the tap offsets in
// registers: the single issuing thread is latency-bound, every instruction between two MMAs counts); 0 = any.
template <int MODE, int KB, bool FP4, int TAPS>
__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_halo_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_w,
                    const ConvTcParams p) {
  constexpr int G = 128 / KB, APC = KB / 32, SPA = FP4 ? 2 : 1;
  constexpr int LAYOUT = KB == 128 ? 2 : (KB == 64 ? 4 : 6);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int taps = TAPS > 0 ? TAPS : p.Kh * p.Kw;
  const int nsf = p.max_stages;                        // scale chunks (groups of 4 MMAs) per tile
  const int atoms_b = (p.BN + 127) / 128;
  const int b_bytes = taps * p.BN * KB;
  const int sfa_bytes = nsf * 512 * SPA, sfb_bytes = nsf * 512 * SPA * atoms_b;
  const int stage_bytes = p.halo_stage_bytes;
  uint8_t* stage0 = smem + p.halo_b_bytes;             // [weight image | its scale chunks] then the stages
  float* staging = reinterpret_cast<float*>(stage0 + (size_t)p.stages * stage_bytes);   // TMA-store epilogue only
  uint64_t* full = reinterpret_cast<uint64_t*>(stage0 + (size_t)p.stages * stage_bytes + (p.tma_store ? EPI_STAGING_BYTES : 0));
  uint64_t* empty = full + p.stages;
  uint64_t* sffull = empty + p.stages;
  uint64_t* tfull = sffull + p.stages;
  uint64_t* tempty = tfull + 2;
  uint64_t* bfull = tempty + 2;
  uint64_t* bempty = bfull + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bempty + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* tap_a = tmem_slot + 4;                     // per tap: offset of its A view / B rows, in 16-byte units
  uint32_t* tap_b = tap_a + 64;
  uint32_t* tap_p = tap_b + 64;                        // per tap: first pixel of its view in the tile's scale patch
  uint8_t* sc_tbl = reinterpret_cast<uint8_t*>(tap_p + 64);   // the tile's patch of raw scale bytes (<= 512)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;   // warp-uniform, see conv_tc_kernel
  const unsigned total = (unsigned)p.total_tiles;
  const unsigned tiles_per_c = (unsigned)(p.classes * p.tiles_w * p.tiles_h);   // tile order: (class, w, h) below the channel tile

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], p.fused ? 2 : 1); mbar_init(&empty[s], 1); mbar_init(&sffull[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 8); }
    mbar_init(bfull, 1); mbar_init(bempty, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tensormap(&map_a);
    if (p.tma_store) prefetch_tensormap(&map_out);
    pdl_wait();      // everything above touches only this block's shared memory and the kernel parameters
    if (p.fused) {   // the weight tile, all taps: one box, swizzled by the copy engine, while the block finishes setting up
      mbar_arrive_expect_tx(bfull, (uint32_t)b_bytes);
      tma_load_3d(smem, &map_w, bfull, 0, 0, 0);
    }
  }
  if ((int)threadIdx.x < taps) {
    const int kh = threadIdx.x / p.Kw, kw = threadIdx.x - kh * p.Kw;
    // forward reads halo row kh, column shift kw; the input gradient walks the taps in the same order but its
    // source pixel moves the other way
    const int hrow = MODE == MQ_OP_FWD ? kh : p.Kh - 1 - kh, wsh = MODE == MQ_OP_FWD ? kw : p.Kw - 1 - kw;
    const int aoff = (hrow * p.TN * p.WH + wsh) * KB;
    tap_a[threadIdx.x] = (uint32_t)aoff >> 4;
    tap_b[threadIdx.x] = (uint32_t)(threadIdx.x * p.BN * KB) >> 4;
    tap_p[threadIdx.x] = (uint32_t)(hrow * (p.TW + p.Kw - 1) + wsh);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  pdl_wait();
  if (p.fused) halo_build_sfb<KB, FP4>(p, smem + b_bytes);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  // TMEM columns: accumulators, the resident weight scale vectors (16 per chunk), then 8 per chunk per stage
  const uint32_t sfb_base = tmem + p.n_acc * p.BN;
  const uint32_t sfa_base = sfb_base + (uint32_t)nsf * 16;
  const uint32_t sfa_cols_stage = (uint32_t)nsf * 8;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    {
      uint32_t s = 0, phase = 0, bcount = 0;
      int cur_ct = -1;
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x) {
        const Tile tile = decode_tile(p, t);
        const int ct = tile.ct;
        if (!p.fused && ct != cur_ct) {
          // new weight tile: wait until the MMAs of the previous one have retired, then one copy of image + scales
          if (bcount > 0 && !mbar_wait(bempty, (bcount - 1) & 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          if (elect_one()) {
            mbar_arrive_expect_tx(bfull, (uint32_t)(b_bytes + sfb_bytes));
            bulk_load(smem, p.b_img + (size_t)ct * b_bytes, b_bytes, bfull);
            bulk_load(smem + b_bytes, p.sfb_img + ((size_t)tile.cls * p.tiles_c + ct) * sfb_bytes, sfb_bytes, bfull);
          }
          __syncwarp();
          cur_ct = ct; ++bcount;
        }
        if (!mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        uint8_t* sa = stage0 + (size_t)s * stage_bytes;
        // first source pixel of the halo: forward (h - ph, w0 - pw); input gradient (h + ph - (Kh-1), w0 + pw - (Kw-1))
        const int hs = MODE == MQ_OP_FWD ? tile.h - p.ph : tile.h + p.ph - (p.Kh - 1);
        const int ws = MODE == MQ_OP_FWD ? tile.w0 - p.pw : tile.w0 + p.pw - (p.Kw - 1);
        if (elect_one()) {
          mbar_arrive_expect_tx(&full[s], (uint32_t)(p.halo_box_bytes + (p.fused ? 0 : sfa_bytes)));
          tma_load_4d(sa, &map_a, &full[s], 0, ws, tile.n0, hs);
          if (!p.fused) bulk_load(sa + p.halo_a_bytes, p.sfa_img + (size_t)tile_m_index(p, tile) * sfa_bytes, sfa_bytes, &full[s]);
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: all taps of a tile per stage
    {
      const uint64_t a_desc_base = smem_desc_base(16, (uint32_t)(p.WH * KB), LAYOUT);   // 8-row groups one halo row apart
      const uint64_t b_desc_base = smem_desc_base(16, 8 * KB, LAYOUT);
      const uint32_t sb16 = smem_u32(smem) >> 4;
      uint32_t idesc_id[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) idesc_id[i] = idesc_with_sf_ids(p.idesc, i, i);
      uint32_t s = 0, phase = 0, tcount = 0, bcount = 0;
      int cur_ct = -1;
      constexpr int TU = TAPS > 0 ? TAPS : 1;
      uint32_t ta[TU], tb[TU];
#pragma unroll
      for (int q = 0; q < TU; ++q) { ta[q] = tap_a[q]; tb[q] = tap_b[q]; }
      const uint32_t acc_mask = (uint32_t)p.n_acc - 1, acc_shift = (uint32_t)p.n_acc - 1;   // n_acc is 1 or 2
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
        const int ct = p.tiles_c == 1 ? 0 : (int)((t / tiles_per_c) % (unsigned)p.tiles_c);
        const bool new_b = ct != cur_ct;
        if (new_b) {
          if (!mbar_wait(bfull, bcount & 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          cur_ct = ct; ++bcount;
        }
        const int acc = (int)(tcount & acc_mask);
        if (!mbar_wait(&tempty[acc], ((tcount >> acc_shift) & 1) ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        if (!mbar_wait(p.mma_cp ? &full[s] : &sffull[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem + acc * p.BN;
        const uint32_t sa16 = smem_u32(stage0 + (size_t)s * stage_bytes) >> 4;
        const uint32_t sfa_s = sfa_base + s * sfa_cols_stage;
        if (elect_one()) {
        if (p.mma_cp) {   // this lane issues the scale copies itself, right before the MMAs that read them
          const uint64_t sf_desc = smem_desc_base(0, 128, 0);
          if (new_b) {
            const uint32_t sfb_s = smem_u32(smem + b_bytes);
#pragma unroll 1
            for (int st = 0; st < nsf; ++st)
#pragma unroll
              for (int g = 0; g < SPA; ++g)
#pragma unroll 1
                for (int a2 = 0; a2 < atoms_b; ++a2)
                  tmem_cp_32x128b_warpx4(sfb_base + st * 16 + 4 * (g * atoms_b + a2), smem_desc(sf_desc, sfb_s + ((st * SPA + g) * atoms_b + a2) * 512));
          }
          const uint32_t sfa_sm = smem_u32(stage0 + (size_t)s * stage_bytes + p.halo_a_bytes);
#pragma unroll 1
          for (int st = 0; st < nsf; ++st) {
#pragma unroll
            for (int g = 0; g < SPA; ++g) tmem_cp_32x128b_warpx4(sfa_s + st * 8 + 4 * g, smem_desc(sf_desc, sfa_sm + (st * SPA + g) * 512));
          }
        }
        uint32_t accumulate = 0;
        auto issue_tap = [&](int q, uint32_t a16, uint32_t b16) {
          const int sfst = q / G;
          const uint32_t sfa_t = sfa_s + sfst * 8, sfb_t = sfb_base + sfst * 16;
#pragma unroll
          for (int ja = 0; ja < APC; ++ja) {
            const int atom = (q % G) * APC + ja;
            const int g = (atom * SPA) >> 2, id = (atom * SPA) & 3;
            const uint64_t ad = a_desc_base | (uint64_t)((a16 + 2 * ja) & 0x3FFF);
            const uint64_t bd = b_desc_base | (uint64_t)((b16 + 2 * ja) & 0x3FFF);
            if (FP4) mma_mxf4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accumulate);
            else mma_mxf8f6f4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accumulate);
            accumulate = 1;
          }
        };
        if (TAPS > 0) {
#pragma unroll
          for (int q = 0; q < TU; ++q) issue_tap(q, sa16 + ta[q], sb16 + tb[q]);
        } else {
#pragma unroll 1
          for (int q = 0; q < taps; ++q) issue_tap(q, sa16 + tap_a[q], sb16 + tap_b[q]);
        }
        tc_commit(&empty[s]);
        tc_commit(&tfull[acc]);
        if (p.tiles_c > 1) {
          const unsigned tn_ = t + gridDim.x;   // the block's next tile: release the weight tile if it needs another
          if (tn_ < total && (int)((tn_ / tiles_per_c) % (unsigned)p.tiles_c) != ct) tc_commit(bempty);
        }
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ scale copier: chunks smem -> TMEM
    if (!p.mma_cp) {
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      uint32_t s = 0, phase = 0, bcount = 0;
      int cur_ct = -1;
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x) {
        const int ct = p.tiles_c == 1 ? 0 : (int)((t / tiles_per_c) % (unsigned)p.tiles_c);
        const bool new_b = ct != cur_ct;
        if (new_b) {
          if (!p.fused && !mbar_wait(bfull, bcount & 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          cur_ct = ct; ++bcount;
        }
        if (!mbar_wait(&full[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        if (elect_one()) {
        if (new_b) {
          const uint32_t sfb_s = smem_u32(smem + b_bytes);
#pragma unroll 1
          for (int st = 0; st < nsf; ++st)
#pragma unroll
            for (int g = 0; g < SPA; ++g)
#pragma unroll 1
              for (int a = 0; a < atoms_b; ++a)
                tmem_cp_32x128b_warpx4(sfb_base + st * 16 + 4 * (g * atoms_b + a), smem_desc(sf_desc, sfb_s + ((st * SPA + g) * atoms_b + a) * 512));
        }
        const uint32_t sfa_sm = smem_u32(stage0 + (size_t)s * stage_bytes + p.halo_a_bytes);
        const uint32_t sfa_s = sfa_base + s * sfa_cols_stage;
#pragma unroll 1
        for (int st = 0; st < nsf; ++st) {
#pragma unroll
          for (int g = 0; g < SPA; ++g) tmem_cp_32x128b_warpx4(sfa_s + st * 8 + 4 * g, smem_desc(sf_desc, sfa_sm + (st * SPA + g) * 512));
        }
        tc_commit(&sffull[s]);
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp == 3) {
    // ------------------------------------------------------------------ activation-scale expander (fused mode)
    if (p.fused) {
      constexpr int BPC = APC * SPA;                       // scale bytes per tap per row = K-blocks of a tap
      const int WT = p.TW + p.Kw - 1, npix = p.Kh * WT;
      // this lane's patch entries e = lane + 32 i: (halo row, column, K-block), fixed for the whole kernel
      int e_h[4], e_w[4], e_k[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int e = lane + 32 * i, pe = e / BPC;
        e_k[i] = e - pe * BPC; e_h[i] = pe / WT; e_w[i] = pe - e_h[i] * WT;
        if (pe >= npix) e_h[i] = -1;
      }
      int twj[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) twj[j] = (32 * j + lane) & (p.TW - 1);
      uint32_t s = 0, phase = 0;
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x) {
        const Tile tile = decode_tile(p, t);
        const int hs = MODE == MQ_OP_FWD ? tile.h - p.ph : tile.h + p.ph - (p.Kh - 1);
        const int ws = MODE == MQ_OP_FWD ? tile.w0 - p.pw : tile.w0 + p.pw - (p.Kw - 1);
        const int nblk = tile.n0 >> 5;
        // raw tile scales of the patch (zero outside the image: those codes are zero-filled anyway)
        uint8_t raw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int hh = hs + e_h[i], ww = ws + e_w[i];
          raw[i] = 0;
          if (e_h[i] >= 0 && hh >= 0 && hh < p.Hs && ww >= 0 && ww < p.Ws)
            raw[i] = __ldg(p.a_scales + (((long long)hh * p.Ws + ww) * p.Nt + nblk) * p.Kblocks + e_k[i]);
        }
        bool ok = true;
        if (lane == 0) ok = mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { *abort_flag = 1; break; }
#pragma unroll
        for (int i = 0; i < 4; ++i) sc_tbl[lane + 32 * i] = raw[i];
        __syncwarp();
        uint8_t* dst = stage0 + (size_t)s * stage_bytes + p.halo_a_bytes + lane * 16;
#pragma unroll 1
        for (int st = 0; st < nsf; ++st) {
          unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
          for (int c = 0; c < G; ++c) {
            const int q = st * G + c;
            if (q < taps) {
              const uint32_t pb = tap_p[q];
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const uint8_t* src = sc_tbl + (pb + twj[j]) * BPC;
                unsigned long long v;
                if (BPC == 1) v = *src;
                else if (BPC == 2) v = *reinterpret_cast<const unsigned short*>(src);
                else v = *reinterpret_cast<const unsigned int*>(src);
                acc[j] |= v << (8 * c * BPC);
              }
            }
          }
#pragma unroll
          for (int g = 0; g < SPA; ++g)
            *reinterpret_cast<uint4*>(dst + (st * SPA + g) * 512) =
                make_uint4((uint32_t)(acc[0] >> (32 * g)), (uint32_t)(acc[1] >> (32 * g)), (uint32_t)(acc[2] >> (32 * g)), (uint32_t)(acc[3] >> (32 * g)));
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp >= 4 && warp < 12) {
    if (p.tma_store) epilogue_tma_role<MODE>(p, &map_out, staging, tmem, tfull, tempty, abort_flag, warp, lane, total);
    else epilogue_role<MODE>(p, tmem, tfull, tempty, abort_flag, warp, lane, total);
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---- scale expansion --------------------------------------------------------------------------------
// One warp per (tile, stage): writes the 512-byte scale-vector chunk(s) the MMA of that stage reads --
// row r of the tile at byte (r % 32) * 16 + (r / 32) * 4, four consecutive K-blocks per 32-bit word --
// from the compact tile scales.  A-side chunks exist per tile (without its channel index), B-side
// chunks per (stride class, channel tile).
template <int MODE, int KB, int KIND>
__global__ void __launch_bounds__(256) expand_conv_scales_kernel(const ConvTcParams p, unsigned n_tile_m) {
  constexpr bool FP4 = KIND != 0;
  pdl_wait();
  if (p.wt_fused && blockIdx.x >= p.expand_blocks) {
    // W -> W^T codes, one 32 x 32 (c_in, c_out) block of one tap per thread block (the work of weight_transpose_kernel)
    __shared__ uint8_t tile[32][33];  // [ci][co]
    unsigned b = blockIdx.x - p.expand_blocks;
    const int bx = (int)(b % (unsigned)p.wt_bx); b /= (unsigned)p.wt_bx;
    const int by = (int)(b % (unsigned)p.wt_by);
    const int tap = (int)(b / (unsigned)p.wt_by);
    const int taps = p.Kh * p.Kw, fp4 = FP4 ? 1 : 0;
    const int co0 = by * 32, ci0 = bx * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
    for (int r = ty; r < 32; r += 8) {
      const int co = co0 + r, ci = ci0 + tx;
      uint8_t v = 0;
      if (co < p.wt_Cout) {
        const long long e = ((long long)co * taps + tap) * p.wt_Cp + ci;
        v = fp4 ? (uint8_t)((p.wt_in[e >> 1] >> ((e & 1) * 4)) & 0xF) : p.wt_in[e];
      }
      tile[tx][r] = v;
    }
    __syncthreads();
    if (!fp4) {
      for (int r = ty; r < 32; r += 8) {
        const int ci = ci0 + r, co = co0 + tx;
        p.wt_out[((long long)ci * taps + tap) * p.wt_Cop + co] = tile[r][tx];
      }
    } else {
      for (int idx = ty * 32 + tx; idx < 32 * 16; idx += 256) {
        const int rr = idx >> 4, bb = idx & 15;
        const int ci = ci0 + rr, co = co0 + 2 * bb;
        p.wt_out[(((long long)ci * taps + tap) * p.wt_Cop + co) >> 1] = (uint8_t)(tile[rr][2 * bb] | (tile[rr][2 * bb + 1] << 4));
      }
    }
    return;
  }
  constexpr int G = 128 / KB, APC = KB / 32, SPA = KIND == 1 ? 2 : 1, BPC = APC * SPA;
  const int lane = threadIdx.x & 31;
  const unsigned wid = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const unsigned nA = conv_tc_sfa_chunks(p);
  const unsigned nB = (unsigned)(p.classes * p.tiles_c * p.max_stages);
  const int atoms_b = (p.BN + 127) / 128;
  if (KIND == 2) {
    // One E4M3 scale per 16 x 16 block (Eq. 5): a row's four scale bytes of an MMA (64 elements of K) are four consecutive
    // bytes of its 16-row block's scale line, and each MMA of a stage (group ga = chunk * APC + atom) gets a 512-byte
    // chunk of its own ([32 rows][row quarter][4 bytes]).  A: [Hs][Ws][ceil(N/16)][K/16]; B: [ceil(rows/16)][taps][K/16],
    // or, for the input gradient, gathered from the stored W scales [ceil(C_out/16)][taps][C_in_p/16] with K = C_out.
    const int Kb16 = p.Kblocks * 2, Nt16 = (p.N + 15) >> 4;
    if (G == 1 && p.sfa_dedup && wid < nA) {
      // shared chunks (unit strides, one chunk per stage), keyed as in the branch for the E8M0 kinds below:
      // wid = (((sample tile * row keys + row key) * column tiles + column tile) * Kw + kw) * cpt + chunk
      unsigned u = wid;
      ChunkPos pos;
      pos.ia = 0;
      pos.cc = (int)(u % (unsigned)p.cpt); u /= (unsigned)p.cpt;
      pos.ib = (int)(u % (unsigned)p.Kw); u /= (unsigned)p.Kw;
      Tile tile;
      tile.w0 = (int)(u % (unsigned)p.tiles_w) * p.TW; u /= (unsigned)p.tiles_w;
      const int hk = (int)(u % (unsigned)p.sfa_hk);
      tile.n0 = (int)(u / (unsigned)p.sfa_hk) * p.TN;
      tile.h = 0; tile.cls = 0; tile.c0 = 0; tile.ct = 0;
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int hs = hk + tw.hs0 - (MODE == MQ_OP_FWD ? 0 : p.Kh - 1);
      const int ws0 = src_w0(tw, pos);
      uint32_t val[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int r = 32 * j + lane;
        const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
        const int n = tile.n0 + tn, ws = ws0 + tw_;
        const bool ok = n < p.N && hs >= 0 && hs < p.Hs && ws >= 0 && ws < p.Ws;
        const uint8_t* rowp = p.a_scales + (((long long)hs * p.Ws + ws) * Nt16 + (n >> 4)) * Kb16 + pos.cc * (4 * APC);
#pragma unroll
        for (int ja = 0; ja < 4; ++ja) val[ja][j] = (ok && ja < APC) ? __ldg(reinterpret_cast<const unsigned int*>(rowp + 4 * ja)) : 0u;
      }
      uint8_t* dst = p.sfa_img + (size_t)wid * (512 * 4) + lane * 16;
#pragma unroll
      for (int ga = 0; ga < 4; ++ga) *reinterpret_cast<uint4*>(dst + ga * 512) = make_uint4(val[ga][0], val[ga][1], val[ga][2], val[ga][3]);
    } else if (wid < nA) {
      const unsigned tm = wid / (unsigned)p.max_stages;
      const int st = (int)(wid - tm * p.max_stages);
      const Tile tile = tile_of_m_index(p, tm);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      if (st * G >= Q) return;
      const int wstep = MODE == MQ_OP_FWD ? p.sw : 1;
      uint32_t val[4][4];
#pragma unroll
      for (int ga = 0; ga < 4; ++ga)
#pragma unroll
        for (int j = 0; j < 4; ++j) val[ga][j] = 0u;
#pragma unroll
      for (int c = 0; c < G; ++c) {
        const int q = st * G + c;
        if (q < Q) {
          ChunkPos pos;
          const int per_row = tw.nkw * p.cpt;
          pos.ia = q / per_row;
          const int rem = q - pos.ia * per_row;
          pos.ib = rem / p.cpt;
          pos.cc = rem - pos.ib * p.cpt;
          const int hs = src_h(tw, pos), ws0 = src_w0(tw, pos);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int r = 32 * j + lane;
            const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
            const int n = tile.n0 + tn, ws = ws0 + tw_ * wstep;
            if (n < p.N && hs >= 0 && hs < p.Hs && ws >= 0 && ws < p.Ws) {
              const uint8_t* rowp = p.a_scales + (((long long)hs * p.Ws + ws) * Nt16 + (n >> 4)) * Kb16 + pos.cc * (4 * APC);
#pragma unroll
              for (int ja = 0; ja < APC; ++ja) val[c * APC + ja][j] = __ldg(reinterpret_cast<const unsigned int*>(rowp + 4 * ja));
            }
          }
        }
      }
      uint8_t* dst = p.sfa_img + (size_t)wid * (512 * 4) + lane * 16;
#pragma unroll
      for (int ga = 0; ga < 4; ++ga) *reinterpret_cast<uint4*>(dst + ga * 512) = make_uint4(val[ga][0], val[ga][1], val[ga][2], val[ga][3]);
    } else if (wid < nA + nB) {
      unsigned idx = wid - nA;
      const int st = (int)(idx % (unsigned)p.max_stages); idx /= (unsigned)p.max_stages;
      const int ct = (int)(idx % (unsigned)p.tiles_c);
      Tile tile;
      tile.cls = (int)(idx / (unsigned)p.tiles_c); tile.ct = ct; tile.c0 = ct * p.BN; tile.w0 = 0; tile.n0 = 0; tile.h = 0;
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      if (st * G >= Q) return;
      const int taps_all = p.Kh * p.Kw;
      uint32_t val[4][8];
#pragma unroll
      for (int ga = 0; ga < 4; ++ga)
#pragma unroll
        for (int j = 0; j < 8; ++j) val[ga][j] = 0u;
#pragma unroll
      for (int c = 0; c < G; ++c) {
        const int q = st * G + c;
        if (q < Q) {
          ChunkPos pos;
          const int per_row = tw.nkw * p.cpt;
          pos.ia = q / per_row;
          const int rem = q - pos.ia * per_row;
          pos.ib = rem / p.cpt;
          pos.cc = rem - pos.ib * p.cpt;
          const int tap = tap_index(tw, pos);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int row = tile.c0 + 32 * j + lane;
            if (j < 4 * atoms_b && 32 * j < p.BN) {
              if (p.wt_fused) {
                if (row < p.wt_Cp) {
                  const int Cb_w = p.wt_Cp >> 4;
#pragma unroll
                  for (int ja = 0; ja < APC; ++ja) {
                    unsigned w = 0;
#pragma unroll
                    for (int kb = 0; kb < 4; ++kb)
                      w |= (unsigned)__ldg(p.wt_sc_in + ((long long)(pos.cc * (4 * APC) + 4 * ja + kb) * taps_all + tap) * Cb_w + (row >> 4)) << (8 * kb);
                    val[c * APC + ja][j] = w;
                  }
                }
              } else if (row < p.b_rows_total) {
                const uint8_t* rowp = p.b_scales + ((long long)(row >> 4) * taps_all + tap) * Kb16 + pos.cc * (4 * APC);
#pragma unroll
                for (int ja = 0; ja < APC; ++ja) val[c * APC + ja][j] = __ldg(reinterpret_cast<const unsigned int*>(rowp + 4 * ja));
              }
            }
          }
        }
      }
      uint8_t* dst = p.sfb_img + (size_t)(wid - nA) * (512 * 4 * atoms_b) + lane * 16;
#pragma unroll
      for (int ga = 0; ga < 4; ++ga)
        for (int a = 0; a < atoms_b; ++a)
          *reinterpret_cast<uint4*>(dst + (ga * atoms_b + a) * 512) = make_uint4(val[ga][4 * a], val[ga][4 * a + 1], val[ga][4 * a + 2], val[ga][4 * a + 3]);
    }
    return;
  }
  if (p.halo && wid >= nA + nB) {
    // weight tile images for the whole-tile variant: one 16-byte chunk per thread
    const int taps_all = p.Kh * p.Kw;
    constexpr int CPR = KB / 16;                       // chunks per row
    const unsigned chunks = (unsigned)(p.tiles_c * taps_all * p.BN) * CPR;
    const unsigned i = (wid - nA - nB) * 32u + (unsigned)lane;
    if (i < chunks) {
      const unsigned row_id = i / CPR; const int ch = (int)(i - row_id * CPR);
      const unsigned tt = row_id / (unsigned)p.BN; const int r = (int)(row_id - tt * p.BN);
      const int ct = (int)(tt / (unsigned)taps_all), tap = (int)(tt - (unsigned)ct * taps_all);
      const int row = ct * p.BN + r;
      uint4 v = make_uint4(0, 0, 0, 0);
      if (row < p.b_rows_total) v = __ldg(reinterpret_cast<const uint4*>(p.b_codes + ((size_t)row * taps_all + tap) * p.b_rowbytes) + ch);
      const int sw = KB == 128 ? (r & 7) : (KB == 64 ? ((r >> 1) & 3) : ((r >> 2) & 1));
      *reinterpret_cast<uint4*>(p.b_img + (size_t)row_id * KB + ((ch ^ sw) << 4)) = v;
    }
    return;
  }
  if (G == 1 && p.sfa_dedup && wid < nA) {
    // shared chunks: wid = (((sample tile * row keys + row key) * column tiles + column tile) * Kw + kw) * cpt + chunk
    unsigned u = wid;
    ChunkPos pos;
    pos.ia = 0;
    pos.cc = (int)(u % (unsigned)p.cpt); u /= (unsigned)p.cpt;
    pos.ib = (int)(u % (unsigned)p.Kw); u /= (unsigned)p.Kw;
    Tile tile;
    tile.w0 = (int)(u % (unsigned)p.tiles_w) * p.TW; u /= (unsigned)p.tiles_w;
    const int hk = (int)(u % (unsigned)p.sfa_hk);
    tile.n0 = (int)(u / (unsigned)p.sfa_hk) * p.TN;
    tile.h = 0; tile.cls = 0; tile.c0 = 0; tile.ct = 0;
    TapWalk<MODE> tw;
    tw.init(p, tile);
    const int hs = hk + tw.hs0 - (MODE == MQ_OP_FWD ? 0 : p.Kh - 1);   // hs0 of output row 0: -ph, or +ph for the input gradient
    const int ws0 = src_w0(tw, pos);
    unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = 32 * j + lane;
      const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
      const int n = tile.n0 + tn, ws = ws0 + tw_;
      if (n < p.N && hs >= 0 && hs < p.Hs && ws >= 0 && ws < p.Ws)
        acc[j] = load_scale_bytes<BPC>(p.a_scales + (((long long)hs * p.Ws + ws) * (p.line ? p.N : p.Nt) + (p.line ? n : (n >> 5))) * p.Kblocks + pos.cc * BPC);
    }
    uint8_t* dst = p.sfa_img + (size_t)wid * (512 * SPA) + lane * 16;
#pragma unroll
    for (int g = 0; g < SPA; ++g)
      *reinterpret_cast<uint4*>(dst + g * 512) = make_uint4((uint32_t)(acc[0] >> (32 * g)), (uint32_t)(acc[1] >> (32 * g)), (uint32_t)(acc[2] >> (32 * g)),
                                                          (uint32_t)(acc[3] >> (32 * g)));
  } else if (wid < nA) {
    const unsigned tm = wid / (unsigned)p.max_stages;
    const int st = (int)(wid - tm * p.max_stages);
    const Tile tile = tile_of_m_index(p, tm);
    TapWalk<MODE> tw;
    tw.init(p, tile);
    const int Q = tw.chunks(p);
    if (st * G >= Q) return;
    const int wstep = MODE == MQ_OP_FWD ? p.sw : 1;
    unsigned long long acc[4] = {0ull, 0ull, 0ull, 0ull};
#pragma unroll
    for (int c = 0; c < G; ++c) {
      const int q = st * G + c;
      if (q < Q) {
        ChunkPos pos;
        const int per_row = tw.nkw * p.cpt;
        pos.ia = q / per_row;
        const int rem = q - pos.ia * per_row;
        pos.ib = rem / p.cpt;
        pos.cc = rem - pos.ib * p.cpt;
        const int hs = src_h(tw, pos), ws0 = src_w0(tw, pos);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int r = 32 * j + lane;
          const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
          const int n = tile.n0 + tn, ws = ws0 + tw_ * wstep;
          if (n < p.N && hs >= 0 && hs < p.Hs && ws >= 0 && ws < p.Ws)
            acc[j] |= load_scale_bytes<BPC>(p.a_scales + (((long long)hs * p.Ws + ws) * (p.line ? p.N : p.Nt) + (p.line ? n : (n >> 5))) * p.Kblocks + pos.cc * BPC) << (8 * c * BPC);
        }
      }
    }
    uint8_t* dst = p.sfa_img + (size_t)wid * (512 * SPA) + lane * 16;
#pragma unroll
    for (int g = 0; g < SPA; ++g)
      *reinterpret_cast<uint4*>(dst + g * 512) = make_uint4((uint32_t)(acc[0] >> (32 * g)), (uint32_t)(acc[1] >> (32 * g)), (uint32_t)(acc[2] >> (32 * g)),
                                                          (uint32_t)(acc[3] >> (32 * g)));
  } else if (wid < nA + nB) {
    unsigned idx = wid - nA;
    const int st = (int)(idx % (unsigned)p.max_stages); idx /= (unsigned)p.max_stages;
    const int ct = (int)(idx % (unsigned)p.tiles_c);
    Tile tile;
    tile.cls = (int)(idx / (unsigned)p.tiles_c); tile.ct = ct; tile.c0 = ct * p.BN; tile.w0 = 0; tile.n0 = 0; tile.h = 0;
    TapWalk<MODE> tw;
    tw.init(p, tile);
    const int Q = tw.chunks(p);
    if (st * G >= Q) return;
    const int taps_all = p.Kh * p.Kw;
    unsigned long long acc[8] = {0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull, 0ull};
#pragma unroll
    for (int c = 0; c < G; ++c) {
      const int q = st * G + c;
      if (q < Q) {
        ChunkPos pos;
        const int per_row = tw.nkw * p.cpt;
        pos.ia = q / per_row;
        const int rem = q - pos.ia * per_row;
        pos.ib = rem / p.cpt;
        pos.cc = rem - pos.ib * p.cpt;
        const int tap = tap_index(tw, pos);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (j < 4 * atoms_b && 32 * j < p.BN && tile.c0 + 32 * j < p.Cd) {
            if (p.wt_fused) {
              // from the stored (not re-laid) weight scales: K-block kb is output-channel block kb of [C_out/32][taps][C_in_p/32]
              const int cib = (tile.c0 >> 5) + j, Ct_w = p.wt_Cp >> 5;
              unsigned long long bytes = 0;
#pragma unroll
              for (int kb = 0; kb < BPC; ++kb)
                bytes |= (unsigned long long)__ldg(p.wt_sc_in + ((long long)(pos.cc * BPC + kb) * taps_all + tap) * Ct_w + cib) << (8 * kb);
              acc[j] |= bytes << (8 * c * BPC);
            } else if (p.line) {
              // line blocks: every weight row has its own scale per K-block
              const int row = tile.c0 + 32 * j + lane;
              if (row < p.b_rows_total) acc[j] |= load_scale_bytes<BPC>(p.b_scales + ((long long)row * taps_all + tap) * p.Kblocks + pos.cc * BPC) << (8 * c * BPC);
            } else {
              acc[j] |= load_scale_bytes<BPC>(p.b_scales + ((long long)((tile.c0 >> 5) + j) * taps_all + tap) * p.Kblocks + pos.cc * BPC) << (8 * c * BPC);
            }
          }
        }
      }
    }
    uint8_t* dst = p.sfb_img + (size_t)(wid - nA) * (512 * SPA * atoms_b) + lane * 16;
#pragma unroll
    for (int g = 0; g < SPA; ++g)
      for (int a = 0; a < atoms_b; ++a)
        *reinterpret_cast<uint4*>(dst + (g * atoms_b + a) * 512) =
            make_uint4((uint32_t)(acc[4 * a] >> (32 * g)), (uint32_t)(acc[4 * a + 1] >> (32 * g)), (uint32_t)(acc[4 * a + 2] >> (32 * g)),
                       (uint32_t)(acc[4 * a + 3] >> (32 * g)));
  }
}

// ---- W -> W^T re-layout (codes only; scales are indexed in place) ------------------------------
// in:  [C_out][taps][C_in_p] codes;  out: [C_in_p][taps][C_out_p] codes (zero for c_out >= C_out)
__global__ void weight_transpose_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, const uint8_t* __restrict__ sc_in,
                                        uint8_t* __restrict__ sc_out, int Cout, int Cop, int Cp, int taps, int fp4) {
  pdl_wait();
  __shared__ uint8_t tile[32][33];  // [ci][co]
  const int tap = blockIdx.z;
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    // tile scales [C_out/32][taps][C_in_p/32] -> [C_in_p/32][taps][C_out_p/32]
    const int Ct = Cp / 32, Cot = Cop / 32;
    for (int i = threadIdx.y * 32 + threadIdx.x; i < Ct * Cot; i += 256) {
      const int cib = i / Cot, cob = i - cib * Cot;
      sc_out[((long long)cib * taps + tap) * Cot + cob] = sc_in[((long long)cob * taps + tap) * Ct + cib];
    }
  }
  const int co0 = blockIdx.y * 32, ci0 = blockIdx.x * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;  // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    const int co = co0 + r, ci = ci0 + tx;
    uint8_t v = 0;
    if (co < Cout) {
      const long long e = ((long long)co * taps + tap) * Cp + ci;
      v = fp4 ? (uint8_t)((in[e >> 1] >> ((e & 1) * 4)) & 0xF) : in[e];
    }
    tile[tx][r] = v;
  }
  __syncthreads();
  if (!fp4) {
    for (int r = ty; r < 32; r += 8) {
      const int ci = ci0 + r, co = co0 + tx;
      out[((long long)ci * taps + tap) * Cop + co] = tile[r][tx];
    }
  } else {
    // 32 ci rows x 16 bytes (two c_out codes per byte)
    for (int idx = ty * 32 + tx; idx < 32 * 16; idx += 256) {
      const int rr = idx >> 4, b = idx & 15;
      const int ci = ci0 + rr, co = co0 + 2 * b;
      out[(((long long)ci * taps + tap) * Cop + co) >> 1] = (uint8_t)(tile[rr][2 * b] | (tile[rr][2 * b + 1] << 4));
    }
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encoder() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess && qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

}  // namespace


static CUtensorMapL2promotion l2promo() { return CU_TENSOR_MAP_L2_PROMOTION_L2_256B; }
bool encode_tensor_map_u8(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                          const uint32_t* elem_strides, int swizzle_bytes, bool f32, int l2_promotion_bytes) {
  EncodeTiledFn fn = get_encoder();
  if (!fn) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = elem_strides ? elem_strides[i] : 1; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
  CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                        : swizzle_bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                        : swizzle_bytes == 32  ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = fn(map, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                  l2_promotion_bytes < 0 ? l2promo() : l2_promotion_bytes == 128 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : l2_promotion_bytes == 256 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B
                  : l2_promotion_bytes == 64 ? CU_TENSOR_MAP_L2_PROMOTION_L2_64B : CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

// A tiled map over packed 6-bit codes (16 in 12 bytes in global memory; in shared memory each group lands as the 12 bytes +
// 4 bytes of padding the MMA's 6-bit operand types want): dims, box and coordinates count codes, strides bytes.  The
// innermost extent must be a multiple of 128 codes, the box 128 codes wide, base 32-byte aligned, strides multiples of 32.
bool encode_tensor_map_p6(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                          const uint32_t* elem_strides) {
  EncodeTiledFn fn = get_encoder();
  if (!fn || (reinterpret_cast<uintptr_t>(base) & 31u) || dims[0] % 128 != 0 || box[0] != 128) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = elem_strides ? elem_strides[i] : 1; }
  for (int i = 0; i + 1 < rank; ++i) { st[i] = strides_bytes[i]; if (st[i] % 32 != 0) return false; }
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_16U6_ALIGN16B, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, l2promo(), CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

size_t conv_tc_smem_bytes(const ConvTcParams& p) {
  const size_t stage = A_STAGE_BYTES + (size_t)(p.duo ? p.BN / 2 : p.BN) * 128 + (p.kind_fp4 == 2 ? SFA_BYTES_NV + SFB_BYTES_NV : SFA_BYTES + SFB_BYTES);
  return 1024 + (size_t)p.stages * stage + (p.tma_store ? EPI_STAGING_BYTES : 0) + (3 * (size_t)p.stages + 4) * 8 + 64 + (p.mx_out ? 544 : 0);
}

template <int MODE, int KB, int FP4, int EPI = -1, bool DUO = false>
cudaError_t launch_conv_tc_inst(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_out, cudaStream_t s,
                                const CUtensorMap* map_sfa = nullptr, const CUtensorMap* map_sfb = nullptr) {
  static bool attr_set = false;
  const size_t smem = conv_tc_smem_bytes(p);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel<MODE, KB, FP4, EPI, DUO>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int sms = sm_count();
  const long long units = p.pair ? p.total_tiles / 2 : p.total_tiles;
  unsigned grid = (unsigned)(units < sms ? units : sms);
  count_launches(1);
  if (DUO) {   // clusters of two blocks; the tile count is even (the plan's condition), so is the grid
    if (!map_sfa || !map_sfb) return cudaErrorInvalidValue;
    grid &= ~1u;
    return launch_pdl_cluster(conv_tc_kernel<MODE, KB, FP4, EPI, DUO>, dim3(grid), dim3(tc_threads_of(EPI)), smem, s, 2u, map_a, map_b, map_out, *map_sfa, *map_sfb, p);
  }
  return launch_pdl(conv_tc_kernel<MODE, KB, FP4, EPI, DUO>, dim3(grid), dim3(tc_threads_of(EPI)), smem, s, map_a, map_b, map_out, map_a, map_a, p);
}

size_t conv_tc_sfa_bytes(const ConvTcParams& p) {
  return (size_t)conv_tc_sfa_chunks(p) * 512 * spa_of_kind(p.kind_fp4);
}
size_t conv_tc_sfb_bytes(const ConvTcParams& p) {
  return (size_t)p.classes * p.tiles_c * p.max_stages * 512 * spa_of_kind(p.kind_fp4) * ((p.BN + 127) / 128);
}

template <int MODE, int KB, int FP4>
cudaError_t launch_expand_inst(const ConvTcParams& p, cudaStream_t s) {
  const unsigned n_tile_m = (unsigned)(p.total_tiles / p.tiles_c);
  unsigned long long warps = (unsigned long long)conv_tc_sfa_chunks(p) + (unsigned long long)p.classes * p.tiles_c * p.max_stages;
  if (p.halo) warps += ((unsigned long long)p.tiles_c * p.Kh * p.Kw * p.BN * (KB / 16) + 31) / 32;
  const unsigned blocks = (unsigned)((warps + 7) / 8);
  count_launches(1);
  if (p.wt_fused) {
    ConvTcParams q = p;
    q.expand_blocks = blocks;
    const unsigned extra = (unsigned)(p.wt_bx * p.wt_by * p.Kh * p.Kw);
    return launch_pdl(expand_conv_scales_kernel<MODE, KB, FP4>, dim3(blocks + extra), dim3(256), 0, s, q, n_tile_m);
  }
  return launch_pdl(expand_conv_scales_kernel<MODE, KB, FP4>, dim3(blocks), dim3(256), 0, s, p, n_tile_m);
}

cudaError_t launch_expand_conv_scales(const ConvTcParams& p, cudaStream_t s) {
#define MQ_TC_CASE(M, K, F) if (p.mode == M && p.KB == K && p.kind_fp4 == F) return launch_expand_inst<M, K, F>(p, s)
  MQ_TC_CASE(MQ_OP_FWD, 128, 0); MQ_TC_CASE(MQ_OP_FWD, 64, 0); MQ_TC_CASE(MQ_OP_FWD, 32, 0);
  MQ_TC_CASE(MQ_OP_FWD, 128, 1); MQ_TC_CASE(MQ_OP_FWD, 64, 1); MQ_TC_CASE(MQ_OP_FWD, 32, 1);
  MQ_TC_CASE(MQ_OP_FWD, 128, 2); MQ_TC_CASE(MQ_OP_FWD, 64, 2); MQ_TC_CASE(MQ_OP_FWD, 32, 2);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 0); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 0); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 0);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 1); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 1); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 1);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 2); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 2); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 2);
#undef MQ_TC_CASE
  return cudaErrorInvalidValue;
}

template <int MODE, int KB, bool FP4, int TAPS>
cudaError_t launch_conv_tc_halo_taps(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_w, cudaStream_t s) {
  static bool attr_set = false;
  const size_t smem = 1024 + (size_t)p.halo_b_bytes + (size_t)p.stages * p.halo_stage_bytes + (p.tma_store ? EPI_STAGING_BYTES : 0) +
                      (3 * (size_t)p.stages + 6) * 8 + 16 + 3 * 64 * 4 + 512;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(conv_tc_halo_kernel<MODE, KB, FP4, TAPS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int sms = sm_count();
  const unsigned grid = (unsigned)(p.total_tiles < sms ? p.total_tiles : sms);
  count_launches(1);
  return launch_pdl(conv_tc_halo_kernel<MODE, KB, FP4, TAPS>, dim3(grid), dim3(TC_THREADS), smem, s, map_a, map_b, map_w, p);
}
template <int MODE, int KB, bool FP4>
cudaError_t launch_conv_tc_halo_inst(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_w, cudaStream_t s) {
  if (p.Kh * p.Kw == 9) return launch_conv_tc_halo_taps<MODE, KB, FP4, 9>(p, map_a, map_b, map_w, s);
  return launch_conv_tc_halo_taps<MODE, KB, FP4, 0>(p, map_a, map_b, map_w, s);
}

__global__ void __launch_bounds__(256) pack6_kernel(const uint4* __restrict__ in, uint4* __restrict__ out, size_t nchunks) {
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < nchunks; i += (size_t)gridDim.x * 256) {
    const uint4 v = __ldg(in + i);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    unsigned long long lo = 0ull, hi = 0ull;   // bits 0..63 and 64..95 of the 96-bit field
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const unsigned long long c = (w[e >> 2] >> (8 * (e & 3))) & 0x3Fu;
      const int bit = 6 * e;
      if (bit < 64) { lo |= c << bit; if (bit > 58) hi |= c >> (64 - bit); }
      else hi |= c << (bit - 64);
    }
    out[i] = make_uint4((uint32_t)lo, (uint32_t)(lo >> 32), (uint32_t)hi, 0u);
  }
}
cudaError_t launch_pack6(const uint8_t* in, uint8_t* out, size_t nbytes, cudaStream_t s) {
  const size_t nchunks = nbytes / 16;
  if (nchunks == 0) return cudaSuccess;
  size_t blocks = (nchunks + 255) / 256;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  count_launches(1);
  return launch_pdl(pack6_kernel, dim3((unsigned)blocks), dim3(256), 0, s, reinterpret_cast<const uint4*>(in), reinterpret_cast<uint4*>(out), nchunks);
}

// Packed 6-bit storage (16 codes in 12 bytes) -> what a kernel reads.  MODE 0: the MMA's container (the 12 bytes + 4 bytes of
// padding); 1: one code per byte; 2: E4M3 bytes of the same values (the weight gradient's 8-bit path).
template <int MODE, bool IS_E3M2>
__global__ void __launch_bounds__(256) unpack6_kernel(const uint32_t* __restrict__ in, uint4* __restrict__ out, size_t ngroups) {
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < ngroups; i += (size_t)gridDim.x * 256) {
    const uint32_t f[3] = {__ldg(in + 3 * i), __ldg(in + 3 * i + 1), __ldg(in + 3 * i + 2)};
    if (MODE == 0) { out[i] = make_uint4(f[0], f[1], f[2], 0u); continue; }
    uint32_t w[4];
    unpack6x16(f, w);
    if (MODE == 2) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t r = 0;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const unsigned short pair = (unsigned short)((w[q] >> (16 * h)) & 0xFFFF);
          const __half2_raw hr = __nv_cvt_fp6x2_to_halfraw2((__nv_fp6x2_storage_t)pair, IS_E3M2 ? __NV_E3M2 : __NV_E2M3);
          r |= (uint32_t)__nv_cvt_halfraw2_to_fp8x2(hr, __NV_SATFINITE, __NV_E4M3) << (16 * h);   // exact: the value is representable
        }
        w[q] = r;
      }
    }
    out[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
cudaError_t launch_unpack6(const uint8_t* in, uint8_t* out, size_t n_codes, int mode, int fmt6, cudaStream_t s) {
  const size_t ngroups = n_codes / 16;
  if (ngroups == 0) return cudaSuccess;
  size_t blocks = (ngroups + 255) / 256;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  count_launches(1);
  const uint32_t* src = reinterpret_cast<const uint32_t*>(in);
  uint4* dst = reinterpret_cast<uint4*>(out);
  if (mode == 0) return launch_pdl(unpack6_kernel<0, false>, dim3((unsigned)blocks), dim3(256), 0, s, src, dst, ngroups);
  if (mode == 1) return launch_pdl(unpack6_kernel<1, false>, dim3((unsigned)blocks), dim3(256), 0, s, src, dst, ngroups);
  if (fmt_base(fmt6) == MQ_E3M2) return launch_pdl(unpack6_kernel<2, true>, dim3((unsigned)blocks), dim3(256), 0, s, src, dst, ngroups);
  return launch_pdl(unpack6_kernel<2, false>, dim3((unsigned)blocks), dim3(256), 0, s, src, dst, ngroups);
}

template <bool IS_E3M2>
__global__ void __launch_bounds__(256) recode6_kernel(const uint4* __restrict__ in, uint4* __restrict__ out, size_t nchunks) {
  pdl_wait();
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < nchunks; i += (size_t)gridDim.x * 256) {
    const uint4 v = __ldg(in + i);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r = 0;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const unsigned short pair = (unsigned short)((w[q] >> (16 * h)) & 0xFFFF);
        const __half2_raw hr = __nv_cvt_fp6x2_to_halfraw2((__nv_fp6x2_storage_t)pair, IS_E3M2 ? __NV_E3M2 : __NV_E2M3);
        r |= (uint32_t)__nv_cvt_halfraw2_to_fp8x2(hr, __NV_SATFINITE, __NV_E4M3) << (16 * h);   // exact: the value is representable
      }
      w[q] = r;
    }
    out[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
cudaError_t launch_recode6_e4m3(const uint8_t* in, uint8_t* out, size_t nbytes, int fmt6, cudaStream_t s) {
  const size_t nchunks = nbytes / 16;
  if (nchunks == 0) return cudaSuccess;
  size_t blocks = (nchunks + 255) / 256;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  count_launches(1);
  if (fmt6 == MQ_E3M2) return launch_pdl(recode6_kernel<true>, dim3((unsigned)blocks), dim3(256), 0, s, reinterpret_cast<const uint4*>(in), reinterpret_cast<uint4*>(out), nchunks);
  return launch_pdl(recode6_kernel<false>, dim3((unsigned)blocks), dim3(256), 0, s, reinterpret_cast<const uint4*>(in), reinterpret_cast<uint4*>(out), nchunks);
}

__global__ void __launch_bounds__(256) recode4_kernel(const uint2* __restrict__ in, uint4* __restrict__ out, size_t nchunks) {
  pdl_wait();
  // E2M1 magnitudes 0, .5, 1, 1.5, 2, 3, 4, 6 as E4M3 bytes; the sign moves from bit 3 of the nibble to bit 7 of the byte
  const uint32_t lut_lo = 0x3C383000u, lut_hi = 0x4C484440u;
  for (size_t i = (size_t)blockIdx.x * 256 + threadIdx.x; i < nchunks; i += (size_t)gridDim.x * 256) {
    const uint2 v = __ldg(in + i);
    const uint32_t src[2] = {v.x, v.y};
    uint32_t w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint32_t r = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const uint32_t nib = (src[q >> 1] >> (16 * (q & 1) + 4 * b)) & 0xFu;
        r |= (__byte_perm(lut_lo, lut_hi, nib & 7u) & 0xFFu | ((nib & 8u) << 4)) << (8 * b);
      }
      w[q] = r;
    }
    out[i] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}
cudaError_t launch_recode4_e4m3(const uint8_t* in, uint8_t* out, size_t n_out, cudaStream_t s) {
  const size_t nchunks = n_out / 16;
  if (nchunks == 0) return cudaSuccess;
  size_t blocks = (nchunks + 255) / 256;
  if (blocks > sm_count() * 16) blocks = sm_count() * 16;
  count_launches(1);
  return launch_pdl(recode4_kernel, dim3((unsigned)blocks), dim3(256), 0, s, reinterpret_cast<const uint2*>(in), reinterpret_cast<uint4*>(out), nchunks);
}

cudaError_t launch_conv_tc(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_w, const CUtensorMap& map_out, cudaStream_t s,
                           const CUtensorMap* map_sfa, const CUtensorMap* map_sfb) {
  if (p.total_tiles <= 0 || p.total_tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
  if (p.duo) {   // pairs of blocks on 256 x 256 tiles: fp32 output, 128-byte K chunks, 8-bit or MX E2M1 operands
    if (p.halo || p.mx_out || p.KB != 128) return cudaErrorInvalidValue;
#define MQ_TC_DUO_CASE(M, F) if (p.mode == M && p.kind_fp4 == F) return launch_conv_tc_inst<M, 128, F, -1, true>(p, map_a, map_w, map_out, s, map_sfa, map_sfb)
    MQ_TC_DUO_CASE(MQ_OP_FWD, 0); MQ_TC_DUO_CASE(MQ_OP_FWD, 1); MQ_TC_DUO_CASE(MQ_OP_FWD, 2);
    MQ_TC_DUO_CASE(MQ_OP_BWD_DATA, 0); MQ_TC_DUO_CASE(MQ_OP_BWD_DATA, 1); MQ_TC_DUO_CASE(MQ_OP_BWD_DATA, 2);
#undef MQ_TC_DUO_CASE
    return cudaErrorInvalidValue;
  }
  if (p.halo) {
#define MQ_TC_HCASE(M, K, F) if (p.mode == M && p.KB == K && p.kind_fp4 == (F ? 1 : 0)) return launch_conv_tc_halo_inst<M, K, F>(p, map_a, map_out, map_w, s)
    MQ_TC_HCASE(MQ_OP_FWD, 64, false); MQ_TC_HCASE(MQ_OP_FWD, 32, false); MQ_TC_HCASE(MQ_OP_FWD, 64, true); MQ_TC_HCASE(MQ_OP_FWD, 32, true);
    MQ_TC_HCASE(MQ_OP_BWD_DATA, 64, false); MQ_TC_HCASE(MQ_OP_BWD_DATA, 32, false); MQ_TC_HCASE(MQ_OP_BWD_DATA, 64, true); MQ_TC_HCASE(MQ_OP_BWD_DATA, 32, true);
#undef MQ_TC_HCASE
    return cudaErrorInvalidValue;
  }
  if (p.mx_out) {   // the quantizing epilogue: one kernel instance per emitted format
#define MQ_TC_MX(M, K, F, E) if (p.mode == M && p.KB == K && p.kind_fp4 == (F ? 1 : 0) && p.mx_fmt == E) return launch_conv_tc_inst<M, K, F, E>(p, map_a, map_w, map_out, s)
#define MQ_TC_MX5(M, K, F) MQ_TC_MX(M, K, F, MQ_E4M3); MQ_TC_MX(M, K, F, MQ_E5M2); MQ_TC_MX(M, K, F, MQ_E2M1); MQ_TC_MX(M, K, F, MQ_E3M2); MQ_TC_MX(M, K, F, MQ_E2M3)
    MQ_TC_MX5(MQ_OP_FWD, 128, false); MQ_TC_MX5(MQ_OP_FWD, 64, false); MQ_TC_MX5(MQ_OP_FWD, 32, false);
    MQ_TC_MX5(MQ_OP_FWD, 128, true);  MQ_TC_MX5(MQ_OP_FWD, 64, true);  MQ_TC_MX5(MQ_OP_FWD, 32, true);
    MQ_TC_MX5(MQ_OP_BWD_DATA, 128, false); MQ_TC_MX5(MQ_OP_BWD_DATA, 64, false); MQ_TC_MX5(MQ_OP_BWD_DATA, 32, false);
    MQ_TC_MX5(MQ_OP_BWD_DATA, 128, true);  MQ_TC_MX5(MQ_OP_BWD_DATA, 64, true);  MQ_TC_MX5(MQ_OP_BWD_DATA, 32, true);
#undef MQ_TC_MX5
#undef MQ_TC_MX
    // the paper's own format in and out: kind 2 operands, emitted format 5
#define MQ_TC_TS(M, K) if (p.mode == M && p.KB == K && p.kind_fp4 == 2 && p.mx_fmt == 5) return launch_conv_tc_inst<M, K, 2, 5>(p, map_a, map_w, map_out, s)
    MQ_TC_TS(MQ_OP_FWD, 128); MQ_TC_TS(MQ_OP_FWD, 64); MQ_TC_TS(MQ_OP_FWD, 32);
    MQ_TC_TS(MQ_OP_BWD_DATA, 128); MQ_TC_TS(MQ_OP_BWD_DATA, 64); MQ_TC_TS(MQ_OP_BWD_DATA, 32);
#undef MQ_TC_TS
    return cudaErrorInvalidValue;
  }
#define MQ_TC_CASE(M, K, F) if (p.mode == M && p.KB == K && p.kind_fp4 == F) return launch_conv_tc_inst<M, K, F>(p, map_a, map_w, map_out, s)
  MQ_TC_CASE(MQ_OP_FWD, 128, 0); MQ_TC_CASE(MQ_OP_FWD, 64, 0); MQ_TC_CASE(MQ_OP_FWD, 32, 0);
  MQ_TC_CASE(MQ_OP_FWD, 128, 1); MQ_TC_CASE(MQ_OP_FWD, 64, 1); MQ_TC_CASE(MQ_OP_FWD, 32, 1);
  MQ_TC_CASE(MQ_OP_FWD, 128, 2); MQ_TC_CASE(MQ_OP_FWD, 64, 2); MQ_TC_CASE(MQ_OP_FWD, 32, 2);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 0); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 0); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 0);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 1); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 1); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 1);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, 2); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, 2); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, 2);
#undef MQ_TC_CASE
  return cudaErrorInvalidValue;
}

cudaError_t launch_weight_transpose(const uint8_t* w_codes, const uint8_t* w_scales, uint8_t* wt_codes, uint8_t* wt_scales, const Geom& g, int fmt,
                                    cudaStream_t s) {
  dim3 grid(g.Cp / 32, g.Cop / 32, g.Kh * g.Kw), block(32, 8);
  count_launches(1);
  return launch_pdl(weight_transpose_kernel, grid, block, 0, s, w_codes, wt_codes, w_scales, wt_scales, g.Cout, g.Cop, g.Cp, g.Kh * g.Kw, fmt == MQ_E2M1 ? 1 : 0);
}

}  // namespace mq
