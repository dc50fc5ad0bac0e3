// Tensor-core weight-gradient GEMM (G_Wf = G_Yf . X'^T, Sec. II-C / IV-B, Eq. 3), block-scaled as
// Eq. 7 with K-blocks of 32 samples at one output pixel: the stored X and G_Y are consumed along N,
// the second direction of their square quantization tiles.
//
//   D[co][(tap, ci)] = sum over (ho, wo, n) of G[ho, wo, n, co] * X[ho*s + kh - p, wo*s + kw - p, n, ci]
//
// 8-bit formats (MQ_WG_FP8): both operands are read exactly as stored ([pixel][n][c], c fastest) and handed
// to the MMA as MN-major tiles (K = n runs across rows of 128 channel bytes); no re-layout.
// E2M1: tcgen05 accepts 4-bit operands only K-major, so mq_conv_bwd_weight first permutes the nibbles of X
// and G_Y in scratch (scales untouched, nothing requantized):
//   MQ_WG_FP4_PIXEL  [pixel][c][n]; per pixel a [128 channels][n bytes] TMA box whose row length equals its
//                    swizzle span (16 bytes: unswizzled core matrices, two boxes side by side per MMA);
//   MQ_WG_FP4_FLAT   (stride 1) channel-blocked pieces over the zero-padded, flattened pixel axis q = h*Wp + w:
//                    the input pixel of output pixel q at tap (kh, kw) is q + kh*Wp + kw, so a stage of
//                    consecutive pixels is ONE contiguous, already swizzled run for each operand (bulk copy).
//
// A small kernel first expands the compact tile scales into the per-stage scale-vector chunks in scratch.
// One thread block per work item (128 output channels x one tap's block of input channels x a slice of
// the K range); partial sums go to scratch and are added in a fixed order by bwd_weight_reduce.
// Warps: 0 producer (TMA / bulk copies), 1 MMA issuer, 2 scale copier (smem -> TMEM), 4-7 epilogue.
#include <cstdlib>
#include "mq_conv_tc.cuh"
#include "mq_tcgen05.cuh"

namespace mq {
namespace {
using namespace tc;

constexpr int WG_THREADS = 320;   // MMA warp, scale copier / loader, eight more loader warps (four of them the epilogue)

// K-block b of stage st: output pixel and 32-sample block
__device__ __forceinline__ void stage_block(const WgradTcParams& p, int st, int b, int& ho, int& wo, int& nb) {
  const int px = b / p.BPP, sub = b - px * p.BPP;
  if (p.mode == MQ_WG_FP4_FLAT) {
    const int a = st * p.KPX + px;
    ho = a / p.Wp; wo = a - ho * p.Wp; nb = sub;
  } else {
    const int nc = st % p.nchunks; const int t = st / p.nchunks;
    const int wg = t % p.groups_w; ho = t / p.groups_w;
    wo = wg * p.KPX + px; nb = nc * p.BPP + sub;
  }
}

// ---- scale expansion, E4M3 scales per 16 x 16 block (kind 2): one warp per 2048-byte chunk of 128 rows --------------
// A stage is 16 K-blocks of 16 samples; MMA ga of the stage reads K-blocks 4 ga .. 4 ga + 3, four bytes per row, from
// its own 512-byte group [32 rows][row quarter][4 bytes].  Row r of quarter jj is channel 128 tile + 32 jj + r, whose
// scale line is that of its 16-channel block.  G_Y scales [Ho][Wo][ceil(N/16)][C_out_p/16], X scales [H][W][ceil(N/16)][C_in_p/16].
__device__ __forceinline__ void expand_wgrad_scales_nv_body(const WgradTcParams& p, unsigned block) {
  const int lane = threadIdx.x & 31;
  const long long wid = (long long)block * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int taps = p.Kh * p.Kw;
  const long long nA = (long long)p.m_tiles128 * p.stages_total;
  const int groups = taps / p.TG;
  const long long nB = p.sfb_S > 0 ? (long long)p.cb_tiles * p.sfb_S : (long long)p.cb_tiles * groups * p.stages_total * p.NB;
  if (wid >= nA + nB) return;
  const int Nt16 = (p.N + 15) >> 4, Cot16 = p.Cot * 2, Ct16 = p.Ct * 2;
  // A chunk holds 16 K-blocks x 8 row blocks (16 rows each) = 128 distinct scale bytes: lane (b16, jh) = (lane >> 1, lane & 1)
  // loads the four of K-block b16 and row blocks 4 jh .. 4 jh + 3; the words of the chunk are then assembled by shuffles
  // (a lane loading its own 64 bytes, two distinct addresses per warp-wide load, took 2.5 times as long).
  const int b16 = lane >> 1, jh = lane & 1;
  uint32_t mine = 0;
  uint8_t* dst = nullptr;
  const int st = wid < nA ? (int)(wid % p.stages_total) : (int)(((wid - nA) / p.NB) % p.stages_total);
  int ho, wo, nb;
  stage_block(p, st, b16 >> 1, ho, wo, nb);
  const int nb16 = 2 * nb + (b16 & 1);
  const bool kok = ho < p.Ho && wo < p.Wo && nb16 < Nt16;
  if (wid >= nA && p.sfb_S > 0) {
    // chunk of (channel block, padded start pixel s): K-block b is padded pixel s + b / BPP (row-major over the padded image,
    // running on into the next row: there the G_Y side is zero), sample block b % BPP; 128 channels of one tap panel
    const long long idx = wid - nA;
    const int s = (int)(idx % p.sfb_S), cb = (int)(idx / p.sfb_S);
    const int b = b16 >> 1, px = b / p.BPP;
    const int lin = s + px, hp = lin / p.Wp, wp = lin - hp * p.Wp;
    const int h = hp - p.ph, w = wp - p.pw;
    const int n16 = 2 * (b - px * p.BPP) + (b16 & 1);
    if (h >= 0 && h < p.H && w >= 0 && w < p.W && n16 < Nt16) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int cib16 = (cb * p.b_rows + 16 * (4 * jh + k)) >> 4;
        if (cib16 < Ct16) mine |= (uint32_t)__ldg(p.x_scales + (((long long)h * p.W + w) * Nt16 + n16) * Ct16 + cib16) << (8 * k);
      }
    }
    dst = p.sfb_img + idx * 2048;
  } else if (wid < nA) {
    const int mt = (int)(wid / p.stages_total);
    if (kok) {
      const uint8_t* line = p.g_scales + (((long long)ho * p.Wo + wo) * Nt16 + nb16) * Cot16;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int cob16 = mt * 8 + 4 * jh + k;
        if (cob16 < Cot16) mine |= (uint32_t)__ldg(line + cob16) << (8 * k);
      }
    }
    dst = p.sfa_img + wid * 2048;
  } else {
    long long idx = wid - nA;
    const int c = (int)(idx % p.NB); idx /= p.NB;
    idx /= p.stages_total;
    const int tg = (int)(idx % groups); const int cb = (int)(idx / groups);
    if (kok) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        // B rows of a tap group: tap-in-group major, input channel minor; chunk c holds rows [128c, 128c + 128); a 16-row
        // block lies inside one tap (b_rows is a multiple of 32)
        const int row = c * 128 + 16 * (4 * jh + k);
        const int tj = row / p.b_rows, rj = row - tj * p.b_rows;
        const int tap = tg * p.TG + tj;
        const int kh = tap / p.Kw, kw = tap - kh * p.Kw;
        const int cib16 = (cb * p.b_rows + rj) >> 4;
        const int h = ho * p.sh + kh - p.ph, w = wo * p.sw + kw - p.pw;
        if (tj < p.TG && cib16 < Ct16 && h >= 0 && h < p.H && w >= 0 && w < p.W)
          mine |= (uint32_t)__ldg(p.x_scales + (((long long)h * p.W + w) * Nt16 + nb16) * Ct16 + cib16) << (8 * k);
      }
    }
    dst = p.sfb_img + (wid - nA) * 2048;
  }
  // word (MMA ga, row quarter jj) of row `lane`: K-blocks 4 ga .. 4 ga + 3 of row block 2 jj + (lane >> 4)
  const int sh8 = 8 * (lane >> 4);
#pragma unroll
  for (int ga = 0; ga < 4; ++ga) {
    uint32_t w4[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      uint32_t word = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint32_t src = __shfl_sync(0xffffffffu, mine, ((4 * ga + k) << 1) | (jj >> 1));
        word |= ((src >> (16 * (jj & 1) + sh8)) & 0xffu) << (8 * k);
      }
      w4[jj] = word;
    }
    *reinterpret_cast<uint4*>(dst + ga * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
  }
}

// ---- scale expansion: one warp per 512*SPA-byte chunk ----------------------------------------------------
template <bool FP4>
__device__ __forceinline__ void expand_wgrad_scales_body(const WgradTcParams& p, unsigned block) {
  constexpr int SPA = FP4 ? 2 : 1, NBS = 4 * SPA;
  const int lane = threadIdx.x & 31;
  const long long wid = (long long)block * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int taps = p.Kh * p.Kw;
  const long long nA = (long long)p.m_tiles128 * p.stages_total;
  const int groups = taps / p.TG;
  // B-side chunks: E2M1 modes one per (channel block, tap group, stage); 8-bit mode one per (channel block, padded X
  // pixel, sample chunk) - a stage's chunk depends only on where its taps' pixels start, so the taps share them
  const long long nB = (FP4 && p.sfb_S > 0) ? (long long)p.cb_tiles * p.sfb_S
                     : FP4 ? (long long)p.cb_tiles * groups * p.stages_total * p.NB : (long long)p.cb_tiles * p.Hp * p.Wp * p.nchunks * p.NB;
  if (wid >= nA + nB) return;
  // this lane's byte: 32-row group j of the 128-row chunk, K-block b of the stage
  const int j = lane >> 3, b = lane & 7;
  uint32_t v = 0;
  uint8_t* dst;
  if (wid < nA) {
    const int mt = (int)(wid / p.stages_total), st = (int)(wid - (long long)mt * p.stages_total);
    const int cob = mt * 4 + j;
    if (b < NBS && cob < p.Cot) {
      int ho, wo, nb;
      stage_block(p, st, b, ho, wo, nb);
      if (ho < p.Ho && wo < p.Wo && nb < p.Nt) v = __ldg(p.g_scales + (((long long)ho * p.Wo + wo) * p.Nt + nb) * p.Cot + cob);
    }
    dst = p.sfa_img + wid * (512 * SPA);
  } else {
    long long idx = wid - nA;
    const int c = (int)(idx % p.NB); idx /= p.NB;
    if (!FP4) {
      // chunk (cb, hp, wp, nc): K-block b is pixel (hp - ph, wp - pw + (b / BPP) sw), sample block nc BPP + b % BPP
      const int nc = (int)(idx % p.nchunks); idx /= p.nchunks;
      const int wp = (int)(idx % p.Wp); idx /= p.Wp;
      const int hp = (int)(idx % p.Hp); const int cb = (int)(idx / p.Hp);
      // rows of the chunk: input channels of one tap, or (grouped thin mode) tap-in-row major, input channel minor - tap tj
      // reads the pixel tj further along the row
      const int row0 = c * 128 + 32 * j;
      const int tj = p.grp8 ? row0 / p.b_rows : 0;
      const int cib = p.grp8 ? (row0 - tj * p.b_rows) / 32 : (cb * p.b_rows + row0) / 32;
      if (b < NBS && cib < p.Ct && tj < p.TG) {
        const int px = b / p.BPP, nb = nc * p.BPP + (b - px * p.BPP);
        const int h = hp - p.ph, w = wp - p.pw + px * p.sw + tj;
        if (nb < p.Nt && h >= 0 && h < p.H && w >= 0 && w < p.W) v = __ldg(p.x_scales + (((long long)h * p.W + w) * p.Nt + nb) * p.Ct + cib);
      }
    } else if (p.sfb_S > 0) {
      // chunk of (channel block, padded start pixel s): K-block b is padded pixel s + b / BPP (row-major over the padded
      // image, running on into the next row: there the G_Y side is zero), sample block b % BPP; 128 channels of one tap panel
      idx = wid - nA;
      const int s = (int)(idx % p.sfb_S), cb = (int)(idx / p.sfb_S);
      const int cib = (cb * p.b_rows + 32 * j) / 32;
      if (b < NBS && cib < p.Ct) {
        const int px = b / p.BPP, nb = b - px * p.BPP;
        const int lin = s + px, hp = lin / p.Wp, wp = lin - hp * p.Wp;
        const int h = hp - p.ph, w = wp - p.pw;
        if (nb < p.Nt && h >= 0 && h < p.H && w >= 0 && w < p.W) v = __ldg(p.x_scales + (((long long)h * p.W + w) * p.Nt + nb) * p.Ct + cib);
      }
    } else {
    // B rows of a tap group: tap-in-group major, input channel minor; chunk c holds rows [128c, 128c + 128)
    const int st = (int)(idx % p.stages_total); idx /= p.stages_total;
    const int tg = (int)(idx % groups); const int cb = (int)(idx / groups);
    const int row0 = c * 128 + 32 * j;
    const int tj = row0 / p.b_rows, rj = row0 - tj * p.b_rows;
    const int tap = tg * p.TG + tj;
    const int kh = tap / p.Kw, kw = tap - kh * p.Kw;
    const int cib = (cb * p.b_rows + rj) / 32;
    if (b < NBS && tj < p.TG && cib < p.Ct) {
      int ho, wo, nb;
      stage_block(p, st, b, ho, wo, nb);
      const int h = ho * p.sh + kh - p.ph, w = wo * p.sw + kw - p.pw;
      if (ho < p.Ho && wo < p.Wo && nb < p.Nt && h >= 0 && h < p.H && w >= 0 && w < p.W)
        v = __ldg(p.x_scales + (((long long)h * p.W + w) * p.Nt + nb) * p.Ct + cib);
    }
    }
    dst = p.sfb_img + (wid - nA) * (512 * SPA);
  }
#pragma unroll
  for (int g = 0; g < SPA; ++g) {
    uint32_t w4[4];
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
      uint32_t word = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) word |= __shfl_sync(0xffffffffu, v, jj * 8 + 4 * g + k) << (8 * k);
      w4[jj] = word;
    }
    *reinterpret_cast<uint4*>(dst + g * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
  }
}

// A block's work item is (output-channel tile, tap group, input-channel block, K slice).  In the flat mode a tap
// group is the Kw taps of one kernel row: their B operands are views of the same run of consecutive pixels,
// shifted by one pixel (one piece) per tap, so a stage loads KPX + Kw - 1 pieces of X once and the stage's G_Y
// tile feeds Kw accumulators (Kw times less shared-memory traffic per FLOP than one tap per block).
template <bool FP4>
__global__ void __launch_bounds__(256) expand_wgrad_scales_kernel(const WgradTcParams p) { pdl_wait(); expand_wgrad_scales_body<FP4>(p, blockIdx.x); }
__global__ void __launch_bounds__(256) expand_wgrad_scales_nv_kernel(const WgradTcParams p) { pdl_wait(); expand_wgrad_scales_nv_body(p, blockIdx.x); }

//
// CTA2 (8-bit operands, C_out and C_in >= 256): the two blocks of a cluster compute a 256 x 256 tile with
// cta_group::2 MMAs.  Each block loads its own 128 output channels of G_Y and its own 128 of the tile's 256 input
// channels of X, so a block's shared memory receives and supplies two thirds of the bytes per FLOP of the one-block
// 128 x 256 tile -- and the shared-memory operand path is what bounds these kernels.  The leader block's threads issue
// the scale copies, MMAs and commits for the pair; the other block only loads, relays "my stage has landed" to the
// leader's barrier, and stores its half of the result.
template <int KIND, bool CTA2>
__global__ void __launch_bounds__(WG_THREADS, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const __grid_constant__ CUtensorMap map_p,
                const __grid_constant__ CUtensorMap map_sfa, const __grid_constant__ CUtensorMap map_sfb, const WgradTcParams p) {
  constexpr bool FP4 = KIND != 0;
  constexpr int SPA = KIND == 2 ? 4 : (KIND == 1 ? 2 : 1);     // scale bytes per MMA per row
  constexpr int SFC_BYTES = KIND == 2 ? 2048 : 1024;           // shared-memory bytes of a 128-row scale chunk
  constexpr uint32_t SFA_COLS = KIND == 2 ? 16u : 8u;          // TMEM columns of a 128-row scale chunk
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int TG = p.TG;
  const int stage_bytes = p.stage_bytes;               // A tile | B tile | A scale chunk (1024) | NB B scale chunks
  const int b_off = 128 * 128, sf_off = b_off + p.b_tile_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  uint64_t* empty = full + p.stages;
  uint64_t* sffull = empty + p.stages;
  uint64_t* tfull = sffull + p.stages;
  uint64_t* pfull = tfull + 1;                         // (spare)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pfull + p.stages);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  // Warp index and cluster rank go through a shuffle so that the compiler knows them to be warp-uniform: the role
  // loops below are run by whole warps, their arithmetic stays in the uniform datapath, and only the bulk-copy / MMA /
  // commit instructions themselves are issued by one elected lane.  (With `if (lane == 0)` around a role, every
  // operand of those instructions is first moved from a per-thread register, which more than doubles the cycles a
  // thread spends per MMA or copy.)
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

  // work item
  const uint32_t rank = CTA2 ? __shfl_sync(0xffffffffu, cluster_ctarank(), 0) : 0u;  // 0: leader
  int item = CTA2 ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int mu = item % p.m_tiles; item /= p.m_tiles;
  const int mt = CTA2 ? 2 * mu + (int)rank : mu;        // 128-row tile of output channels
  const int jt = item % p.j_tiles;
  const int split = item / p.j_tiles;
  const int tgi = jt / p.cb_tiles, cb = jt - tgi * p.cb_tiles;
  const int tap0 = tgi * TG;                            // first tap of the group (TG divides Kw)
  const int kh = tap0 / p.Kw, kw = tap0 - kh * p.Kw;
  const int co0 = mt * 128, ci0 = cb * p.b_rows;         // the tile's first output / input channel
  const int ci_ld = ci0 + (CTA2 ? 128 * (int)rank : 0);  // first input channel this block loads (its half, in a pair)
  const int st_begin = (int)((long long)p.stages_total * split / p.splits);
  const int st_end = (int)((long long)p.stages_total * (split + 1) / p.splits);
  const int nst = st_end - st_begin;
  const uint32_t acc_cols = (uint32_t)(TG * p.b_rows);  // accumulators first, then the per-stage scale buffers
  const uint32_t sf_cols = SFA_COLS * (1u + (uint32_t)p.NB);
  const bool has_b1 = p.mode == MQ_WG_FP8 && !CTA2 && p.b_rows > 128;   // a fifth loader: second X panel

  if (threadIdx.x == 0) {
#pragma unroll 1
    // full: one arrival per kind of copy
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], has_b1 ? 4 : 3); mbar_init(&empty[s], 1); mbar_init(&sffull[s], 1); mbar_init(&pfull[s], 1); }
    mbar_init(tfull, 1);
    *abort_flag = 0;
    mbar_fence_init();
    if (p.mode != MQ_WG_FP4_FLAT) { prefetch_tensormap(&map_a); prefetch_tensormap(&map_b); }
    prefetch_tensormap(&map_p);
  }
  if (warp == 1) {
    if (CTA2) { tmem_alloc_2(tmem_slot, p.tmem_cols); tmem_relinquish_2(); }
    else { tmem_alloc(tmem_slot, p.tmem_cols); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CTA2) cluster_sync_all();   // both blocks' barriers and tensor memory exist before anything crosses over
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();   // set-up above touched only shared memory, tensor memory and the kernel parameters

  // ------------------------------------------------------------------ loaders
  // A warp gets one bulk copy accepted per ~170 cycles whatever its size, and its loop around that copy (barrier
  // wait, addresses, coordinates) is a chain of dependent instructions, so the copies of a stage are spread over
  // warps: one KIND of copy per pair of warps (G_Y tile; X tile, one or two 128-channel panels; the two scale
  // chunks), the two warps of a kind taking even and odd stages.  Each kind arrives once per stage on the stage's
  // barrier with its own byte count.  The loaders include the epilogue warps, idle until the accumulators are final.
  // In a pair of blocks every copy of either block is counted on the LEADER's barrier: its loaders announce both
  // blocks' bytes, the peer's loaders only issue (no relay thread, no remote arrive in the loop).
  const int nkinds = has_b1 ? 4 : 3;
  const int lslot = FP4 ? (warp == 0 ? 0 : (warp >= 3 ? warp - 2 : -1))          // E2M1: warp 2 is the scale copier
                        : (warp == 0 ? 0 : (warp == 2 ? 1 : (warp >= 3 ? warp - 1 : -1)));
  if (lslot >= 0 && lslot < 2 * nkinds) {
    const int kidx = lslot >> 1, half = lslot & 1;
    const int kind = kidx == 0 ? 0 : (kidx == 1 ? 1 : ((kidx == 2 && has_b1) ? 2 : 3));   // 0 G_Y, 1 X, 2 second X panel, 3 scales
    const int taps = p.Kh * p.Kw;
    const uint8_t* sfa_src = p.sfa_img + ((size_t)mt * p.stages_total + st_begin) * (512 * SPA);
    const uint32_t sfb_bytes = (uint32_t)p.NB * 512 * SPA;
    // X-side scale chunks: per (tap group, stage), NB chunks each; or (sfb_S) per padded start pixel - the NB taps of the
    // stage are NB consecutive start pixels, the next stage starts KPX pixels on
    const uint32_t sfb_step = p.sfb_S > 0 ? (uint32_t)p.KPX * 512 * SPA : sfb_bytes;
    const uint8_t* sfb_src = p.sfb_S > 0 ? p.sfb_img + ((size_t)cb * p.sfb_S + (size_t)st_begin * p.KPX + (size_t)kh * p.Wp + kw) * (512 * SPA)
                                         : p.sfb_img + (((size_t)cb * (taps / TG) + tgi) * p.stages_total + st_begin) * sfb_bytes;
    const uint32_t a_bytes = 128 * 128, b_step = (uint32_t)p.b_rows * 128;
    const uint32_t b_bytes = (p.mode == MQ_WG_FP8 && !p.grp8) ? 128u * 128u : (uint32_t)p.b_tile_bytes;   // per loader
    const uint8_t* ga = nullptr; const uint8_t* gb = nullptr;
    if (p.mode == MQ_WG_FP4_FLAT) {
      ga = p.gt + (size_t)mt * p.gt_block_bytes + (size_t)st_begin * a_bytes;
      gb = p.xt + (size_t)cb * p.xt_block_bytes + ((size_t)st_begin * p.KPX + (size_t)kh * p.Wp + kw) * ((size_t)p.b_rows * p.KBn);
    }
    const uint32_t my_bytes = (kind == 0 ? a_bytes : (kind <= 2 ? b_bytes : 512u * SPA + sfb_bytes)) * (CTA2 ? 2u : 1u);
    const int sfa_row0 = (int)(((size_t)mt * p.stages_total + st_begin) * (2 * SPA));          // rows of 256 bytes (pair mode maps)
    int nc, wg, ho;                                            // of the first stage this warp handles
    {
      const int st = st_begin + half;
      nc = st % p.nchunks; const int t = st / p.nchunks;
      wg = t % p.groups_w; ho = t / p.groups_w;
    }
    uint32_t s = (uint32_t)half % (uint32_t)p.stages, phase = 0;   // stages >= 2
#pragma unroll 1
    for (int i = half; i < nst; i += 2) {
      // everything that does not depend on the stage being free comes before the wait
      uint8_t* sa = smem + (size_t)s * stage_bytes;
      uint8_t* sb = sa + b_off;
      uint8_t* ssf = sa + sf_off;
      uint64_t* bar = &full[s];
      const uint32_t lbar = CTA2 ? cluster_addr_of(bar, 0) : 0u;
      const int wo0 = wg * p.KPX;
      const int xw = wo0 * p.sw + kw - p.pw, xh = ho * p.sh + kh - p.ph;
      const int nrow = nc * p.BPP * 32;
      if (*abort_flag) break;
      if (!mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
      if (elect_one()) {
        if (rank == 0) mbar_arrive_expect_tx(bar, my_bytes);
        // 8-bit mode: the X-side chunk of (padded pixel, sample chunk); E2M1: of (tap group, stage)
        const long long xchunk = !FP4 ? ((((long long)cb * p.Hp + (xh + p.ph)) * p.Wp + (xw + p.pw)) * p.nchunks + nc) : 0;
        if (CTA2) {
          if (kind == 0) tma_load_4d_pair(sa, &map_a, lbar, co0, nrow, wo0, ho);
          else if (kind == 1) tma_load_4d_pair(sb, &map_b, lbar, ci_ld, nrow, xw, xh);
          else {
            tma_load_2d_pair(ssf, &map_sfa, lbar, 0, sfa_row0 + i * (2 * SPA));
            tma_load_2d_pair(ssf + SFC_BYTES, &map_sfb, lbar, 0, (int)(xchunk * (2 * SPA * p.NB)));
          }
        } else if (kind == 3) {
          bulk_load(ssf, sfa_src + (size_t)i * (512 * SPA), 512 * SPA, bar);
          bulk_load(ssf + SFC_BYTES, FP4 ? sfb_src + (size_t)i * sfb_step : p.sfb_img + (size_t)xchunk * sfb_bytes, sfb_bytes, bar);
        } else if (p.mode == MQ_WG_FP4_FLAT) {
          if (kind == 0) bulk_load(sa, ga + (size_t)i * a_bytes, a_bytes, bar);
          else bulk_load(sb, gb + (size_t)i * b_step, b_bytes, bar);          // KPX + TG - 1 consecutive pixels
        } else if (p.mode == MQ_WG_FP4_PIXEL) {
          // [pixel][c][n] re-laid codes: one box (n bytes, 128 channels) per pixel of the stage
#pragma unroll 1
          for (int px = 0; px < p.KPX; ++px) {
            if (kind == 0) tma_load_4d(sa + px * 128 * p.KBn, &map_a, bar, nc * p.KBn, co0, wo0 + px, ho);
            else tma_load_4d(sb + px * 128 * p.KBn, &map_b, bar, nc * p.KBn, ci0, (wo0 + px) * p.sw + kw - p.pw, xh);
          }
        } else {
          // stored [ho][wo][n][c] codes: box (128 channel bytes, n rows, pixels, 1)
          if (kind == 0) tma_load_4d(sa, &map_a, bar, co0, nrow, wo0, ho);
          else tma_load_4d(sb + (kind == 2 ? 128 * 128 : 0), &map_b, bar, ci_ld + (kind == 2 ? 128 : 0), nrow, xw, xh);
        }
      }
      __syncwarp();
      // two stages on: slot, then (sample chunk, pixel group, row) by counters, not divisions
      s += 2; if (s >= (uint32_t)p.stages) { s -= (uint32_t)p.stages; phase ^= 1; }
#pragma unroll
      for (int r = 0; r < 2; ++r)
        if (++nc == p.nchunks) { nc = 0; if (++wg == p.groups_w) { wg = 0; ++ho; } }
    }
  }
  __syncwarp();
  if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (the leader's, in a pair)
    if (rank == 0) {
      // 8-bit: MN-major tiles [K row][128 bytes], 128-byte swizzle, 8-row groups 1024 bytes apart; an MMA
      // takes 32 K rows (4096 bytes).  E2M1: K-major pieces [rows][KBn bytes], swizzle span = KBn (none for
      // 16: 8x16-byte core matrices, the next 16 bytes of K one piece further); an MMA takes 32 bytes of K.
      const uint32_t fp4_layout = p.KBn == 128 ? 2u : (p.KBn == 64 ? 4u : (p.KBn == 32 ? 6u : 0u));
      const uint32_t a_piece = 128 * p.KBn, b_piece = (uint32_t)p.b_rows * p.KBn;
      const uint64_t a_desc0 = smem_desc(FP4 ? smem_desc_base(a_piece, 8 * p.KBn, fp4_layout) : smem_desc_base(128 * 128, 1024, 2), smem_u32(smem));
      // grouped thin mode: MN-major panels of Cp bytes (swizzle span Cp), a tap's panel one pixel (32 BPP rows) after the
      // previous tap's, 8-row groups 8 Cp bytes apart
      const uint64_t b_desc0 = smem_desc(FP4 ? smem_desc_base(b_piece, 8 * p.KBn, fp4_layout)
                                             : (p.grp8 ? smem_desc_base(32 * p.BPP * p.Cp, 8 * p.Cp, p.Cp == 64 ? 4u : 6u) : smem_desc_base(128 * 128, 1024, 2)),
                                         smem_u32(smem + b_off));
      const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
      // The taps of a group are ONE wide B operand: tap j's view starts j pieces (= b_rows / 8 row groups) further,
      // which is exactly where rows [j * b_rows, (j + 1) * b_rows) of a (TG * b_rows)-row operand lie.  At most two
      // MMAs per K slice: N = n0 (<= 256) and the remaining n1 rows.
      const uint32_t idesc_n[2] = {p.idesc | ((uint32_t)(p.n0 >> 3) << 17), p.idesc | ((uint32_t)(p.n1 >> 3) << 17)};
      const uint32_t row16_1 = ((uint32_t)p.n0 * p.KBn) >> 4;   // second MMA: B rows from n0 on (flat mode only)
      const int nm = p.n1 > 0 ? 2 : 1;
      uint32_t ka16[4], kb16[4];   // offset of MMA a's K slice inside the stage's A / B tile, in 16-byte units
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        if (FP4) {
          const int piece = (32 * a) / p.KBn, off = (32 * a) % p.KBn;
          ka16[a] = (piece * a_piece + off) >> 4; kb16[a] = (piece * b_piece + off) >> 4;
        } else {
          ka16[a] = 256u * a;      // 32 K rows of 128 bytes per MMA
          // grouped thin mode: K slice a = (output pixel a / BPP, sample block a % BPP); its first tap's pixel lies sw strip pixels per output pixel on
          kb16[a] = p.grp8 ? (uint32_t)(((a / p.BPP) * p.sw * p.BPP + (a % p.BPP)) * 32 * p.Cp) >> 4 : 256u * a;
        }
      }
      const uint32_t sf_base = tmem + acc_cols;
      const uint64_t sf_desc0 = smem_desc(smem_desc_base(0, 128, 0), smem_u32(smem + sf_off));
      // Everything that does not depend on the stage is hoisted: this thread must hand the tensor core one MMA per
      // 128 cycles, and its own instructions are one dependent chain.
      uint32_t idesc_a[2][4], sfa_off[4], sfb_off[2][4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const uint32_t g = (uint32_t)(a * SPA) >> 2, id = (uint32_t)(a * SPA) & 3;
        sfa_off[a] = 4 * g;
#pragma unroll
        for (int m = 0; m < 2; ++m) {
          idesc_a[m][a] = idesc_with_sf_ids(idesc_n[m], id, id);
          sfb_off[m][a] = SFA_COLS + 4 * (g * (uint32_t)p.NB + (m ? (uint32_t)(p.n0 >> 7) : 0u));
        }
      }
      const uint32_t d1 = tmem + (uint32_t)p.n0;
      uint32_t s = 0, phase = 0, accumulate = 0;
      // Scale buffers in tensor memory: one per pipeline stage, or (sf_slots < stages: the wide scale vectors of kind 2 next to
      // a tap group's accumulators) fewer, taken in turn - a buffer is rewritten only after the MMAs that read it have
      // completed, which is what the stage's `empty` barrier reports.
      uint32_t ss = 0, es = 0, ephase = 0;   // scale slot of this stage; stage (and its parity) whose MMAs used that slot last
#pragma unroll 1
      for (int i = 0; i < nst; ++i) {   // another role's abort shows here as this thread's own bounded wait running out
        if (!mbar_wait((FP4 && !p.mma_cp) ? &sffull[s] : &full[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        if (FP4 && p.mma_cp && p.sf_slots < p.stages && i >= p.sf_slots) {
          if (!mbar_wait(&empty[es], ephase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          if (++es == (uint32_t)p.stages) { es = 0; ephase ^= 1; }
        }
        tc_fence_after_sync();
        const uint32_t so = s * stage16;
        const uint32_t sf_t = sf_base + ss * sf_cols;
        if (++ss == (uint32_t)p.sf_slots) ss = 0;
        const uint64_t ad = a_desc0 + so, bd = b_desc0 + so;
        if (!FP4 && nm == 1) {
          // 8-bit operands: this lane also issues the stage's three scale copies, right before the MMAs that read
          // them (same thread, so the tensor pipe keeps them in order).  A separate copier's copies would queue behind
          // the MMAs already issued and its completion signal would arrive only when those retire - one pipeline
          // bubble per stage.
          if (elect_one()) {
            const uint64_t sfd = sf_desc0 + so;
            if (CTA2) {
              tmem_cp_32x128b_warpx4_2(sf_t, sfd);
              tmem_cp_32x128b_warpx4_2(sf_t + 8, sfd + 64);
              tmem_cp_32x128b_warpx4_2(sf_t + 12, sfd + 96);
            } else {
              tmem_cp_32x128b_warpx4(sf_t, sfd);
              tmem_cp_32x128b_warpx4(sf_t + 8, sfd + 64);
              if (p.NB > 1) tmem_cp_32x128b_warpx4(sf_t + 12, sfd + 96);
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
              const uint32_t accu = a > 0 ? 1u : accumulate;
              const uint32_t id = idesc_n[0] | ((uint32_t)a << 4) | ((uint32_t)a << 29);
              if (CTA2) mma_mxf8f6f4_2(tmem, ad + 256u * a, bd + 256u * a, id, sf_t, sf_t + 8, accu);
              else mma_mxf8f6f4(tmem, ad + 256u * a, bd + kb16[a], id, sf_t, sf_t + 8, accu);
            }
            if (CTA2) tc_commit_2_multicast(&empty[s], 3); else tc_commit(&empty[s]);
          }
        } else
        if (elect_one()) {
        if (FP4 && p.mma_cp) {
          const uint64_t sfd = sf_desc0 + so;
#pragma unroll
          for (int g = 0; g < SPA; ++g) tmem_cp_32x128b_warpx4(sf_t + 4 * g, sfd + g * 32);
#pragma unroll 1
          for (int c = 0; c < p.NB; ++c)
#pragma unroll
            for (int g = 0; g < SPA; ++g) tmem_cp_32x128b_warpx4(sf_t + SFA_COLS + 4 * (g * p.NB + c), sfd + (SFC_BYTES >> 4) + (c * SPA + g) * 32);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const uint32_t accu = a > 0 ? 1u : accumulate;
          if (KIND == 2) mma_nvf4(tmem, ad + ka16[a], bd + kb16[a], idesc_a[0][a], sf_t + sfa_off[a], sf_t + sfb_off[0][a], accu);
          else if (FP4) mma_mxf4(tmem, ad + ka16[a], bd + kb16[a], idesc_a[0][a], sf_t + sfa_off[a], sf_t + sfb_off[0][a], accu);
          else if (CTA2) mma_mxf8f6f4_2(tmem, ad + ka16[a], bd + kb16[a], idesc_a[0][a], sf_t + sfa_off[a], sf_t + sfb_off[0][a], accu);
          else mma_mxf8f6f4(tmem, ad + ka16[a], bd + kb16[a], idesc_a[0][a], sf_t + sfa_off[a], sf_t + sfb_off[0][a], accu);
          if (nm == 2) {   // the remaining n1 rows of a tap group's operand (flat mode only)
            if (KIND == 2) mma_nvf4(d1, ad + ka16[a], bd + row16_1 + kb16[a], idesc_a[1][a], sf_t + sfa_off[a], sf_t + sfb_off[1][a], accu);
            else if (FP4) mma_mxf4(d1, ad + ka16[a], bd + row16_1 + kb16[a], idesc_a[1][a], sf_t + sfa_off[a], sf_t + sfb_off[1][a], accu);
            else mma_mxf8f6f4(d1, ad + ka16[a], bd + row16_1 + kb16[a], idesc_a[1][a], sf_t + sfa_off[a], sf_t + sfb_off[1][a], accu);
          }
        }
        if (CTA2) tc_commit_2_multicast(&empty[s], 3); else tc_commit(&empty[s]);   // frees the stage in both blocks
        }
        __syncwarp();
        accumulate = 1;
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
      if (elect_one()) {
        if (CTA2) {
          if (nst > 0) tc_commit_2_multicast(tfull, 3); else { mbar_arrive(tfull); mbar_arrive_remote(tfull, 1); }
        } else {
          if (nst > 0) tc_commit(tfull); else mbar_arrive(tfull);
        }
      }
      __syncwarp();
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ scale copier (smem -> per-stage TMEM buffers)
    // E2M1 only (twice the scale bytes, up to eight copies per stage); for 8-bit operands the MMA lane issues them.
    if (FP4 && !p.mma_cp) {
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint64_t sf_desc0 = smem_desc(sf_desc, smem_u32(smem + sf_off));
      const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
      const uint32_t sf_base = tmem + acc_cols;
      uint32_t s = 0, phase = 0;
      uint32_t ss = 0, es = 0, ephase = 0;   // see the MMA issuer
#pragma unroll 1
      for (int i = 0; i < nst && !*abort_flag; ++i) {
        if (!mbar_wait(&full[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        if (p.sf_slots < p.stages && i >= p.sf_slots) {
          if (!mbar_wait(&empty[es], ephase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          if (++es == (uint32_t)p.stages) { es = 0; ephase ^= 1; }
        }
        tc_fence_after_sync();
        const uint32_t so = s * stage16;
        const uint32_t sf_t = sf_base + ss * sf_cols;
        if (++ss == (uint32_t)p.sf_slots) ss = 0;
        if (elect_one()) {
#ifdef MQ_WG_SKIPCP
          if (i < p.stages)
#endif
          {
#pragma unroll
          for (int g = 0; g < SPA; ++g) {
            if (CTA2) tmem_cp_32x128b_warpx4_2(sf_t + 4 * g, sf_desc0 + so + g * 32);
            else tmem_cp_32x128b_warpx4(sf_t + 4 * g, sf_desc0 + so + g * 32);
          }
#pragma unroll 1
          for (int c = 0; c < p.NB; ++c) {     // B-side chunk c: rows [128c, 128c + 128) of the group's operand
#pragma unroll
            for (int g = 0; g < SPA; ++g) {
              if (CTA2) tmem_cp_32x128b_warpx4_2(sf_t + SFA_COLS + 4 * (g * p.NB + c), sf_desc0 + so + (SFC_BYTES >> 4) + (c * SPA + g) * 32);
              else tmem_cp_32x128b_warpx4(sf_t + SFA_COLS + 4 * (g * p.NB + c), sf_desc0 + so + (SFC_BYTES >> 4) + (c * SPA + g) * 32);
            }
          }
          }
          if (CTA2) tc_commit_2(&sffull[s]); else tc_commit(&sffull[s]);
        }
        __syncwarp();
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ------------------------------------------------------------------ epilogue: partial sums to scratch
    // Each warp moves its 32 rows, 32 columns at a time: TMEM -> registers -> a [32 rows][128 bytes] staging tile
    // (128-byte swizzle, so the 16-byte writes of a row do not collide) -> one TMA store into the partial-sum
    // tensor (columns, rows, split): coalesced lines, clipped at C_out.  The pipeline's shared memory is free by
    // now (tfull fires after the last MMA) and serves as staging, two tiles per warp.
    const int quad = warp & 3;
    bool ok = true;
    if (lane == 0) ok = mbar_wait(tfull, 0, p.status, MQ_ERR_TIMEOUT);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) {
      tc_fence_after_sync();
      const int ncols = min(p.b_rows, p.Cp - ci0);
      uint8_t* stg = smem + quad * (2 * 4096);
      uint32_t nbuf = 0;
#pragma unroll 1
      for (int j = 0; j < TG; ++j) {
        const int col0 = (tap0 + j) * p.Cp + ci0;
        const uint32_t taddr = tmem + (uint32_t)(j * p.b_rows) + ((uint32_t)(32 * quad) << 16);
#pragma unroll 1
        for (int c = 0; c < ncols; c += 32, ++nbuf) {
          uint32_t v[2][16];
          if (nst > 0) {
            tmem_ld_32x32b_x16(taddr + c, v[0]);
            tmem_ld_32x32b_x16(taddr + c + 16, v[1]);
            tmem_ld_wait();
          } else {
#pragma unroll
            for (int q = 0; q < 16; ++q) { v[0][q] = 0u; v[1][q] = 0u; }
          }
          uint8_t* buf = stg + (nbuf & 1) * 4096;
          if (lane == 0) bulk_wait_group_read<1>();      // the store that used this buffer two tiles ago has read it
          __syncwarp();
#pragma unroll
          for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int q = 0; q < 4; ++q)                  // 16-byte unit 4h + q of row `lane`
              *reinterpret_cast<uint4*>(buf + lane * 128 + (((4 * h + q) ^ (lane & 7)) << 4)) = make_uint4(v[h][4 * q], v[h][4 * q + 1], v[h][4 * q + 2], v[h][4 * q + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_3d(&map_p, buf, col0 + c, co0 + 32 * quad, split);
            bulk_commit_group();
          }
        }
      }
      if (lane == 0) bulk_wait_group_all();
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CTA2) cluster_sync_all();   // nothing of the peer block is touched after this point
  if (warp == 1) { if (CTA2) tmem_dealloc_2(tmem, p.tmem_cols); else tmem_dealloc(tmem, p.tmem_cols); }
}

// ---- E2M1 re-layout: stored [pixel][n][Cp] nibbles -> [pixel][Cp][Npad] nibbles (n fastest, zero for n >= N) ----
// One block: 8 pixels x 32 samples x 64 channels.  Reads rows of 32 bytes, writes 16 bytes per (pixel, channel).
__global__ void __launch_bounds__(256) fp4_to_n_major_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, int P, int N, int Cp, int Npad) {
  __shared__ uint8_t t[8][32][65];  // [pixel][n][c] one code per byte
  const int p0 = blockIdx.x * 8, n0 = blockIdx.y * 32, c0 = blockIdx.z * 64;
  const int tid = threadIdx.x;
  for (int i = tid; i < 512; i += 256) {
    const int px = i >> 6, n = (i >> 1) & 31, half = i & 1;
    uint4 v = make_uint4(0, 0, 0, 0);
    if (p0 + px < P && n0 + n < N && c0 + 32 * half < Cp)
      v = *reinterpret_cast<const uint4*>(in + (((long long)(p0 + px) * N + n0 + n) * Cp + c0 + 32 * half) / 2);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
      for (int b = 0; b < 8; ++b) t[px][n][32 * half + 8 * q + b] = (uint8_t)((w[q] >> (4 * b)) & 0xF);
  }
  __syncthreads();
  for (int i = tid; i < 512; i += 256) {
    const int px = i >> 6, c = i & 63;
    if (c0 + c < Cp && p0 + px < P) {
      uint32_t w[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t acc = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) acc |= (uint32_t)t[px][8 * q + b][c] << (4 * b);
        w[q] = acc;
      }
      *reinterpret_cast<uint4*>(out + (((long long)(p0 + px) * Cp + c0 + c) * Npad + n0) / 2) = make_uint4(w[0], w[1], w[2], w[3]);
    }
  }
}

// ---- E2M1 re-layout for the flat mode (see launch_fp4_to_flat) -------------------------------------------------
// One warp per (output pixel, 32-sample block, 64 channels): 1 KB in, 1 KB out, transposed in registers.  Lane
// (k, ng) = (lane & 7, lane >> 3) reads the 32-bit word of channels 8k..8k+7 for samples 8ng..8ng+7, swaps the
// 8 x 8 nibble block in three butterfly steps, and writes word ng of the 16-byte sample run of channels 8k..8k+7.
__device__ __forceinline__ void nibble_transpose_8x8(uint32_t (&w)[8]) {
#pragma unroll
  for (int a = 0; a < 8; a += 2) { const uint32_t x = ((w[a] >> 4) ^ w[a + 1]) & 0x0F0F0F0Fu; w[a + 1] ^= x; w[a] ^= x << 4; }
#pragma unroll
  for (int a = 0; a < 8; ++a)
    if ((a & 2) == 0) { const uint32_t x = ((w[a] >> 8) ^ w[a + 2]) & 0x00FF00FFu; w[a + 2] ^= x; w[a] ^= x << 8; }
#pragma unroll
  for (int a = 0; a < 4; ++a) { const uint32_t x = ((w[a] >> 16) ^ w[a + 4]) & 0x0000FFFFu; w[a + 4] ^= x; w[a] ^= x << 16; }
}

struct FlatArgs {
  const uint8_t* in; uint8_t* out;
  int Hs, Ws, N, Cs_p, P_out, Wp, off_h, off_w, rows, nblocks, KBn, ncg;
  unsigned units, blocks;
  int wide;   // 1: 256 samples x 256 channels per block through shared memory (whole lines in and out)
};
constexpr int FLAT_WIDE_PITCH = 33;                                   // words per staged row (132 bytes: conflict-free columns)
constexpr int FLAT_WIDE_SMEM = 2 * 256 * FLAT_WIDE_PITCH * 4;         // input tile + output tile
__device__ __forceinline__ void fp4_to_flat_body(const FlatArgs& fa, unsigned block, unsigned nblocks_grid) {
  const uint8_t* __restrict__ in = fa.in; uint8_t* __restrict__ out = fa.out;
  const int Hs = fa.Hs, Ws = fa.Ws, N = fa.N, Cs_p = fa.Cs_p, P_out = fa.P_out, Wp = fa.Wp, off_h = fa.off_h, off_w = fa.off_w;
  const int rows = fa.rows, nblocks = fa.nblocks, KBn = fa.KBn, ncg = fa.ncg;
  const unsigned units = fa.units;
  const int lane = threadIdx.x & 31;
  const int k = lane & 7, ng = lane >> 3;
  const int nbk = KBn >> 4;                        // 32-sample blocks per pixel
  const int cmax = nblocks * rows;
  const unsigned per_q = (unsigned)(ncg * nbk);
  for (unsigned u = block * 8u + (threadIdx.x >> 5); u < units; u += nblocks_grid * 8u) {
    const unsigned q = u / per_q, rem = u - q * per_q;
    const int nb = (int)(rem / (unsigned)ncg), cg = (int)(rem - (unsigned)nb * ncg);
    const int hq = (int)(q / (unsigned)Wp), wq = (int)q - hq * Wp;
    const int h = hq - off_h, w = wq - off_w;
    const int c0 = cg * 64 + 8 * k;                // this lane's 8 channels
    uint32_t wd[8];
    const bool pix_ok = h >= 0 && h < Hs && w >= 0 && w < Ws && c0 < Cs_p;
    const uint8_t* src = in + ((((long long)h * Ws + w) * N + nb * 32 + 8 * ng) * Cs_p + c0) / 2;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      wd[j] = 0u;
      if (pix_ok && nb * 32 + 8 * ng + j < N) wd[j] = __ldg(reinterpret_cast<const uint32_t*>(src + (long long)j * (Cs_p / 2)));
    }
    nibble_transpose_8x8(wd);                       // wd[i]: channel c0 + i, samples 8ng .. 8ng + 7
    if (c0 < cmax) {                                // rows is a multiple of 32: the lane's 8 channels share a block
      const int blk = c0 / rows, r0 = c0 - blk * rows;
      uint8_t* dst = out + (((long long)blk * P_out + q) * rows + r0) * KBn + 4 * ng;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int r = r0 + i;
        const int sw = KBn == 128 ? (r & 7) : (KBn == 64 ? ((r >> 1) & 3) : (KBn == 32 ? ((r >> 2) & 1) : 0));
        *reinterpret_cast<uint32_t*>(dst + (long long)i * KBn + ((nb ^ sw) << 4)) = wd[i];
      }
    }
  }
}

// Wide variant (256 samples per pixel, i.e. 128-byte pieces): a block takes (padded pixel, 256 channels), reads its
// 256 sample rows x 128 bytes as whole lines into shared memory, the warps transpose 32 x 64 sub-blocks in registers as
// above, and the 256 channel rows x 128 bytes leave as whole lines (the narrow variant reads 32-byte and writes
// 16-byte runs, which costs a memory request each).
__device__ __forceinline__ void fp4_to_flat_wide_body(const FlatArgs& fa, unsigned block, unsigned nblocks_grid, uint32_t* sm) {
  const uint8_t* __restrict__ in = fa.in; uint8_t* __restrict__ out = fa.out;
  uint32_t* sin = sm;
  uint32_t* sout = sm + 256 * FLAT_WIDE_PITCH;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const int k = lane & 7, ng = lane >> 3;
  const int ncgw = fa.ncg;                        // 256-channel groups
  const int cmax = fa.nblocks * fa.rows;
  const int row_t = t >> 3, ch_t = t & 7;          // this thread's row (+ 32 m) and 16-byte chunk of a 128-byte line
#pragma unroll 1
  for (unsigned u = block; u < fa.units; u += nblocks_grid) {
    const unsigned q = u / (unsigned)ncgw;
    const int cgw = (int)(u - q * (unsigned)ncgw);
    const int hq = (int)(q / (unsigned)fa.Wp), wq = (int)q - hq * fa.Wp;
    const int h = hq - fa.off_h, w = wq - fa.off_w;
    const bool pix_ok = h >= 0 && h < fa.Hs && w >= 0 && w < fa.Ws;
    const int cbase = cgw * 256;
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int row = row_t + 32 * m;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (pix_ok && row < fa.N && cbase + 32 * ch_t < fa.Cs_p)
        v = __ldg(reinterpret_cast<const uint4*>(in + ((((long long)h * fa.Ws + w) * fa.N + row) * fa.Cs_p + cbase + 32 * ch_t) / 2));
      uint32_t* d = sin + row * FLAT_WIDE_PITCH + 4 * ch_t;
      d[0] = v.x; d[1] = v.y; d[2] = v.z; d[3] = v.w;
    }
    __syncthreads();
#pragma unroll 1
    for (int sb = warp; sb < 32; sb += 8) {
      const int nb = sb >> 2, cg = sb & 3;
      uint32_t wd[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) wd[j] = sin[(nb * 32 + 8 * ng + j) * FLAT_WIDE_PITCH + cg * 8 + k];
      nibble_transpose_8x8(wd);                     // wd[i]: channel cg * 64 + 8k + i, samples nb * 32 + 8ng .. + 7
#pragma unroll
      for (int i = 0; i < 8; ++i) sout[(cg * 64 + 8 * k + i) * FLAT_WIDE_PITCH + ((nb ^ i) << 2) + ng] = wd[i];   // 128-byte swizzle: chunk nb ^ (row & 7)
    }
    __syncthreads();
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int row = row_t + 32 * m;
      const int c = cbase + row;
      if (c < cmax) {
        const int blk = c / fa.rows, r = c - blk * fa.rows;
        const uint32_t* sp = sout + row * FLAT_WIDE_PITCH + 4 * ch_t;
        *reinterpret_cast<uint4*>(out + (((long long)blk * fa.P_out + q) * fa.rows + r) * 128 + 16 * ch_t) = make_uint4(sp[0], sp[1], sp[2], sp[3]);
      }
    }
    // the next unit's fill of `sin` is ordered after this unit's reads of it by the second barrier above; its writes
    // to `sout` come after its own first barrier, which every thread reaches only after these reads
  }
}

// Preparation of the flat mode in one launch: blocks [0, x.blocks) re-lay X, the next g.blocks re-lay G_Y, the rest
// expand the scale chunks.
__global__ void __launch_bounds__(256) wgrad_flat_prep_kernel(const FlatArgs x, const FlatArgs gy, const WgradTcParams p) {
  extern __shared__ __align__(16) uint32_t flat_sm[];
  pdl_wait();
  if (blockIdx.x < x.blocks) { if (x.wide) fp4_to_flat_wide_body(x, blockIdx.x, x.blocks, flat_sm); else fp4_to_flat_body(x, blockIdx.x, x.blocks); }
  else if (blockIdx.x < x.blocks + gy.blocks) {
    if (gy.wide) fp4_to_flat_wide_body(gy, blockIdx.x - x.blocks, gy.blocks, flat_sm); else fp4_to_flat_body(gy, blockIdx.x - x.blocks, gy.blocks);
  } else if (p.kind == 2) expand_wgrad_scales_nv_body(p, blockIdx.x - x.blocks - gy.blocks);
  else expand_wgrad_scales_body<true>(p, blockIdx.x - x.blocks - gy.blocks);
}

}  // namespace

size_t wgrad_tc_smem_bytes(const WgradTcParams& p) { return 1024 + (size_t)p.stages * p.stage_bytes + (4 * (size_t)p.stages + 2) * 8 + 64; }

cudaError_t launch_wgrad_tc(const WgradTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_p, const CUtensorMap& map_sfa,
                            const CUtensorMap& map_sfb, cudaStream_t s) {
  static bool attr_set[4] = {false, false, false, false};
  const size_t smem = wgrad_tc_smem_bytes(p);
  const int f = p.cta2 ? 2 : (p.mode == MQ_WG_FP8 ? 0 : (p.kind == 2 ? 3 : 1));
  if (!attr_set[f]) {
    cudaError_t e = f == 2 ? cudaFuncSetAttribute(wgrad_tc_kernel<0, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)
                  : f == 1 ? cudaFuncSetAttribute(wgrad_tc_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)
                  : f == 3 ? cudaFuncSetAttribute(wgrad_tc_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)
                           : cudaFuncSetAttribute(wgrad_tc_kernel<0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[f] = true;
  }
  const unsigned grid = (unsigned)(p.m_tiles * p.j_tiles * p.splits) * (p.cta2 ? 2u : 1u);
  count_launches(1);
  if (f == 2) return launch_pdl_cluster(wgrad_tc_kernel<0, true>, dim3(grid), dim3(WG_THREADS), smem, s, 2u, map_a, map_b, map_p, map_sfa, map_sfb, p);
  if (f == 1) return launch_pdl(wgrad_tc_kernel<1, false>, dim3(grid), dim3(WG_THREADS), smem, s, map_a, map_b, map_p, map_sfa, map_sfb, p);
  if (f == 3) return launch_pdl(wgrad_tc_kernel<2, false>, dim3(grid), dim3(WG_THREADS), smem, s, map_a, map_b, map_p, map_sfa, map_sfb, p);
  return launch_pdl(wgrad_tc_kernel<0, false>, dim3(grid), dim3(WG_THREADS), smem, s, map_a, map_b, map_p, map_sfa, map_sfb, p);
}

cudaError_t launch_expand_wgrad_scales(const WgradTcParams& p, cudaStream_t s) {
  const long long nb = p.mode == MQ_WG_FP8 ? (long long)p.cb_tiles * p.Hp * p.Wp * p.nchunks * p.NB : (long long)p.cb_tiles * (p.Kh * p.Kw / p.TG) * p.stages_total * p.NB;
  const long long warps = (long long)p.m_tiles128 * p.stages_total + nb;
  const unsigned blocks = (unsigned)((warps + 7) / 8);
  count_launches(1);
  if (p.mode == MQ_WG_FP8) return launch_pdl(expand_wgrad_scales_kernel<false>, dim3(blocks), dim3(256), 0, s, p);
  if (p.kind == 2) return launch_pdl(expand_wgrad_scales_nv_kernel, dim3(blocks), dim3(256), 0, s, p);
  return launch_pdl(expand_wgrad_scales_kernel<true>, dim3(blocks), dim3(256), 0, s, p);
}

cudaError_t launch_fp4_to_n_major(const uint8_t* in, uint8_t* out, int P, int N, int Cp, int Npad, cudaStream_t s) {
  dim3 grid((P + 7) / 8, Npad / 32, (Cp + 63) / 64);
  fp4_to_n_major_kernel<<<grid, 256, 0, s>>>(in, out, P, N, Cp, Npad);
  count_launches(1);
  return cudaGetLastError();
}

static bool make_flat_args(FlatArgs* fa, const uint8_t* in, uint8_t* out, int Hs, int Ws, int N, int Cs_p, int P_out, int Wp, int off_h, int off_w, int rows,
                           int nblocks, int KBn) {
  fa->in = in; fa->out = out; fa->Hs = Hs; fa->Ws = Ws; fa->N = N; fa->Cs_p = Cs_p; fa->P_out = P_out; fa->Wp = Wp; fa->off_h = off_h; fa->off_w = off_w;
  fa->rows = rows; fa->nblocks = nblocks; fa->KBn = KBn;
  fa->wide = (KBn == 128 && nblocks * rows >= 256 && N <= 256 && !env_int("MQ_WGRAD_NO_WIDE_PREP", 0)) ? 1 : 0;
  if (fa->wide) {
    fa->ncg = (nblocks * rows + 255) / 256;
    const long long units = (long long)P_out * fa->ncg;
    if (units >= 0xffffffffLL) return false;
    fa->units = (unsigned)units;
    fa->blocks = (unsigned)(units < (long long)sm_count() * 3 ? (units < 1 ? 1 : units) : (long long)sm_count() * 3);
    return true;
  }
  fa->ncg = (nblocks * rows + 63) / 64;
  const long long units = (long long)P_out * (KBn / 16) * fa->ncg;
  if (units >= 0xffffffffLL) return false;
  fa->units = (unsigned)units;
  long long blocks = (units + 7) / 8;
  if (blocks > (long long)sm_count() * 32) blocks = (long long)sm_count() * 32;
  if (blocks < 1) blocks = 1;
  fa->blocks = (unsigned)blocks;
  return true;
}

cudaError_t launch_wgrad_flat_prep(const WgradTcParams& p, const uint8_t* x_codes, uint8_t* xt, int P_b, const uint8_t* g_codes, uint8_t* gt, int P_a,
                                   cudaStream_t s) {
  FlatArgs fx, fg;
  if (!make_flat_args(&fx, x_codes, xt, p.H, p.W, p.N, p.Cp, P_b, p.Wp, p.ph, p.pw, p.b_rows, p.cb_tiles, p.KBn)) return cudaErrorInvalidValue;
  if (!make_flat_args(&fg, g_codes, gt, p.Ho, p.Wo, p.N, p.Cot * 32, P_a, p.Wp, 0, 0, 128, p.m_tiles, p.KBn)) return cudaErrorInvalidValue;
  const long long warps = (long long)p.m_tiles128 * p.stages_total +
                          (p.sfb_S > 0 ? (long long)p.cb_tiles * p.sfb_S : (long long)p.cb_tiles * (p.Kh * p.Kw / p.TG) * p.stages_total * p.NB);
  const unsigned sc_blocks = (unsigned)((warps + 7) / 8);
  count_launches(1);
  const size_t smem = (fx.wide || fg.wide) ? (size_t)FLAT_WIDE_SMEM : 0;
  static bool attr_set = false;
  if (smem && !attr_set) {
    if (cudaFuncSetAttribute(wgrad_flat_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FLAT_WIDE_SMEM) != cudaSuccess) return cudaErrorInvalidValue;
    attr_set = true;
  }
  return launch_pdl(wgrad_flat_prep_kernel, dim3(fx.blocks + fg.blocks + sc_blocks), dim3(256), smem, s, fx, fg, p);
}

}  // namespace mq
