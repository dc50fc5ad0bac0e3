// Tensor-core implicit-GEMM kernel for mq_conv_fwd and mq_conv_bwd_data (Sec. II-C / IV-B GEMMs,
// block-scaled as Eq. 7) on sm_100a: tcgen05 block-scaled MMA with accumulators and scale vectors
// in tensor memory, operands brought by TMA straight from the stored channel-batch-first tensors
// (the im2col of Sec. IV-A is implicit: every tap is a shifted TMA box, out-of-image taps are the
// TMA zero fill).
//
// One persistent thread block per SM, 12 warps:
//   warp 0   TMA producer        one lane issues the A (gathered activation) and B (weight) boxes
//   warp 1   MMA issuer          one lane copies the stage's scale vectors smem -> TMEM and issues the MMAs
//   warps 2-3 scale expanders    (alternating stages) turn the compact tile scales (one E8M0 byte per 32x32 tile) into the
//                                per-row scale vectors the MMA reads, for the tap / K-block of each stage
//   warps 4-11 epilogue          TMEM -> registers -> global (fp32), overlapped with the next tile's main loop;
//                                two warps per TMEM lane quadrant, each taking half of the tile's columns
// A pipeline stage holds 128 bytes of K per row (four MMAs): one 128-byte box, or 128/KB boxes of KB
// bytes when a tap has fewer than 128 bytes of channels (then several taps share a stage).
// Every wait is bounded; on expiry the kernel records MQ_ERR_TIMEOUT in the status word and drains.
#include "mq_conv_tc.cuh"
#include "mq_tcgen05.cuh"

namespace mq {
namespace {
using namespace tc;

constexpr int TC_THREADS = 384;   // 12 warps: TMA, MMA, 2 scale expanders, 8 epilogue
constexpr int A_STAGE_BYTES = 128 * 128;
constexpr int SFA_BYTES = 1024;   // up to 2 groups of 4 scale bytes per row
constexpr int SFB_BYTES = 2048;   // up to 2 groups x 2 atoms of 128 rows
constexpr int SF_COLS = 24;       // TMEM columns of one scale buffer: 8 (A) + 16 (B)

// Cycle counters of block 0's roles (debug aid): [role][0] = cycles in the role's loop, [role][1] = cycles waiting.
__device__ unsigned long long g_prof[8][2];
#ifdef MQ_TC_PROFILE
#define PROF_BEGIN() const long long prof_t0 = clock64(); long long prof_wait = 0
#define PROF_WAIT(expr) ([&]() { const long long w0_ = clock64(); const bool r_ = (expr); prof_wait += clock64() - w0_; return r_; }())
#define PROF_END(role) do { if (blockIdx.x == 0) { g_prof[role][0] = clock64() - prof_t0; g_prof[role][1] = prof_wait; } } while (0)
#else
#define PROF_BEGIN() do { } while (0)
#define PROF_WAIT(expr) (expr)
#define PROF_END(role) do { } while (0)
#endif

struct Tile { int c0, w0, n0, h, cls; };

__device__ __forceinline__ Tile decode_tile(const ConvTcParams& p, unsigned t) {
  Tile q;
  unsigned u = t / (unsigned)p.tiles_c;
  q.c0 = (int)(t - u * p.tiles_c) * p.BN; t = u;
  u = t / (unsigned)p.tiles_w; q.w0 = (int)(t - u * p.tiles_w) * p.TW; t = u;
  u = t / (unsigned)p.tiles_n; q.n0 = (int)(t - u * p.tiles_n) * p.TN; t = u;
  u = t / (unsigned)p.tiles_h; q.h = (int)(t - u * p.tiles_h);
  q.cls = (int)u;
  return q;
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
      const int ch = t.cls / p.sw, cw = t.cls - ch * p.sw;
      const int kh0 = (ch + p.ph) % p.sh, kw0 = (cw + p.pw) % p.sw;
      nkh = kh0 < p.Kh ? (p.Kh - kh0 + p.sh - 1) / p.sh : 0;
      nkw = kw0 < p.Kw ? (p.Kw - kw0 + p.sw - 1) / p.sw : 0;
      hs0 = t.h + (ch + p.ph - kh0) / p.sh; ws0 = t.w0 + (cw + p.pw - kw0) / p.sw;
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

template <int MODE, int KB, bool FP4>
__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const ConvTcParams p) {
  constexpr int G = 128 / KB;          // chunks per stage
  constexpr int APC = KB / 32;         // MMA K-atoms (32 bytes) per chunk
  constexpr int SPA = FP4 ? 2 : 1;     // scale bytes per atom
  constexpr int BPC = APC * SPA;       // scale bytes per chunk: 1, 2, 4 or 8
  constexpr int LAYOUT = KB == 128 ? 2 : (KB == 64 ? 4 : 6);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  const int b_stage_bytes = p.BN * 128;
  const int stage_bytes = A_STAGE_BYTES + b_stage_bytes + SFA_BYTES + SFB_BYTES;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * stage_bytes);
  uint64_t* empty = full + p.stages;
  uint64_t* tfull = empty + p.stages;
  uint64_t* tempty = tfull + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int atoms_b = (p.BN + 127) / 128;
  const unsigned total = (unsigned)p.total_tiles;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 8); }
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      PROF_BEGIN();
      uint32_t s = 0, phase = 0;
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x) {
        const Tile tile = decode_tile(p, t);
        TapWalk<MODE> tw;
        tw.init(p, tile);
        const int Q = tw.chunks(p);
        ChunkPos pos;
        pos.reset();
        for (int q0 = 0; q0 < Q; q0 += G) {
          if (!PROF_WAIT(mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT))) { *abort_flag = 1; break; }
          const int nch = min(G, Q - q0);
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          uint8_t* sb = sa + A_STAGE_BYTES;
          mbar_arrive_expect_tx(&full[s], (uint32_t)nch * (128 + p.BN) * KB);
#pragma unroll
          for (int c = 0; c < G; ++c) {
            if (c < nch) {
              tma_load_4d(sa + c * 128 * KB, &map_a, &full[s], pos.cc * KB, src_w0(tw, pos), tile.n0, src_h(tw, pos));
              tma_load_3d(sb + c * p.BN * KB, &map_b, &full[s], pos.cc * KB, tap_index(tw, pos), tile.c0);
              pos.advance(tw, p.cpt);
            }
          }
          if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
        }
      }
      PROF_END(0);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint64_t op_desc = smem_desc_base(16, 8 * KB, LAYOUT);
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint32_t sf_base = tmem + p.n_acc * p.BN;
      const uint32_t stage16 = (uint32_t)stage_bytes >> 4;
      const uint64_t a_desc0 = smem_desc(op_desc, smem_u32(smem));
      const uint64_t b_desc0 = smem_desc(op_desc, smem_u32(smem + A_STAGE_BYTES));
      const uint64_t sfa_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes));
      const uint64_t sfb_desc0 = smem_desc(sf_desc, smem_u32(smem + A_STAGE_BYTES + b_stage_bytes + SFA_BYTES));
      const uint32_t b_chunk16 = (uint32_t)(p.BN * KB) >> 4;
      uint32_t idesc_id[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) idesc_id[i] = idesc_with_sf_ids(p.idesc, i, i);
      uint32_t s = 0, phase = 0, sfbuf = 0, tcount = 0;
      PROF_BEGIN();
      for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
        const Tile tile = decode_tile(p, t);
        TapWalk<MODE> tw;
        tw.init(p, tile);
        const int Q = tw.chunks(p);
        const int acc = tcount % p.n_acc;
        if (!PROF_WAIT(mbar_wait(&tempty[acc], ((tcount / p.n_acc) & 1) ^ 1, p.status, MQ_ERR_TIMEOUT))) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem + acc * p.BN;
        uint32_t accumulate = 0;
        for (int q0 = 0; q0 < Q; q0 += G) {
          if (!PROF_WAIT(mbar_wait(&full[s], phase, p.status, MQ_ERR_TIMEOUT))) { *abort_flag = 1; break; }
          tc_fence_after_sync();
          const uint32_t so = s * stage16;
          const uint32_t sfa_t = sf_base + sfbuf * SF_COLS, sfb_t = sfa_t + 8;
#pragma unroll
          for (int g = 0; g < SPA; ++g) {
            tmem_cp_32x128b_warpx4(sfa_t + 4 * g, sfa_desc0 + so + g * 32);
            for (int a = 0; a < atoms_b; ++a) tmem_cp_32x128b_warpx4(sfb_t + 4 * (g * atoms_b + a), sfb_desc0 + so + (g * atoms_b + a) * 32);
          }
          const int natoms = min(G, Q - q0) * APC;
#pragma unroll
          for (int a = 0; a < 4; ++a) {
            if (a < natoms) {
              constexpr int dummy = 0; (void)dummy;
              const int c = a / APC, ja = a % APC;
              const uint64_t ad = a_desc0 + so + c * ((128 * KB) >> 4) + ja * 2;
              const uint64_t bd = b_desc0 + so + c * b_chunk16 + ja * 2;
              const int g = (a * SPA) >> 2, id = (a * SPA) & 3;
              if (FP4) mma_mxf4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accumulate);
              else mma_mxf8f6f4(d_tmem, ad, bd, idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, accumulate);
              accumulate = 1;
            }
          }
          tc_commit(&empty[s]);
          sfbuf ^= 1;
          if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
        }
        if (Q > 0) tc_commit(&tfull[acc]); else mbar_arrive(&tfull[acc]);
      }
      PROF_END(1);
    }
  } else if (warp == 2 || warp == 3) {
    // ------------------------------------------------------------------ scale expanders (two warps, alternate stages)
    // The scale bytes of a chunk (one tap, KB bytes of channels) are contiguous in the stored scale
    // tensor, so a lane fetches them with one naturally aligned load.  Loads are issued RING stages
    // ahead of the stage being assembled and stay untouched in registers until then, which hides
    // their latency behind the pipeline.
    constexpr int RING = 4;
    const int NTL = p.TN >= 32 ? p.TN / 32 : 1;
    const int ncombos = p.TW * NTL;
    const int wstep = MODE == MQ_OP_FWD ? p.sw : 1;
    const int taps_all = p.Kh * p.Kw;
    const int ctw = lane / NTL, cnl = lane - ctw * NTL;   // this lane's A combo: column offset, 32-sample block
    // source lanes of the four rows 32j + lane this lane writes (row = tn * TW + tw)
    int src_lane[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = 32 * j + lane;
      src_lane[j] = (r & (p.TW - 1)) * NTL + ((r >> p.lgTW) >> 5);
    }
    struct Walk {
      unsigned t; Tile tile; TapWalk<MODE> tw; ChunkPos pos; int Q, q0; bool done;
      bool a_ok, b_ok; int a_nt; long long b_row;
    };
    auto load_tile = [&](Walk& w) {
      while (w.t < total) {
        w.tile = decode_tile(p, w.t);
        w.tw.init(p, w.tile);
        w.Q = w.tw.chunks(p);
        if (w.Q > 0) {
          w.q0 = 0; w.pos.reset();
          w.a_ok = lane < ncombos && (w.tile.n0 + cnl * 32) < p.N;
          w.a_nt = (w.tile.n0 + cnl * 32) >> 5;
          w.b_ok = lane < (p.BN + 31) / 32 && (w.tile.c0 + lane * 32) < p.Cd;
          w.b_row = (long long)((w.tile.c0 >> 5) + lane) * taps_all;
          return;
        }
        w.t += gridDim.x;
      }
      w.done = true;
    };
    // raw loads of one stage: up to G chunks x (A, B), 32 bits each (two words when a chunk has 8 bytes)
    struct Raw { uint32_t a[G == 1 ? 2 : G]; uint32_t b[G == 1 ? 2 : G]; };
    auto ld = [&](const uint8_t* ptr, uint32_t* dst) {
      if (BPC == 1) dst[0] = __ldg(ptr);
      else if (BPC == 2) dst[0] = __ldg(reinterpret_cast<const unsigned short*>(ptr));
      else if (BPC == 4) dst[0] = __ldg(reinterpret_cast<const unsigned int*>(ptr));
      else { const uint2 v = __ldg(reinterpret_cast<const uint2*>(ptr)); dst[0] = v.x; dst[1] = v.y; }
    };
    auto sf_load = [&](Walk& w, Raw& r) {
#pragma unroll
      for (int i = 0; i < (G == 1 ? 2 : G); ++i) { r.a[i] = 0u; r.b[i] = 0u; }
#pragma unroll
      for (int c = 0; c < G; ++c) {
        if (w.q0 + c < w.Q) {
          const int hs = src_h(w.tw, w.pos), ws = src_w0(w.tw, w.pos) + ctw * wstep;
          if (w.a_ok && hs >= 0 && hs < p.Hs && ws >= 0 && ws < p.Ws)
            ld(p.a_scales + (((long long)hs * p.Ws + ws) * p.Nt + w.a_nt) * p.Kblocks + w.pos.cc * BPC, &r.a[c]);
          if (w.b_ok) ld(p.b_scales + (w.b_row + tap_index(w.tw, w.pos)) * p.Kblocks + w.pos.cc * BPC, &r.b[c]);
          w.pos.advance(w.tw, p.cpt);
        }
      }
      w.q0 += G;
      if (w.q0 >= w.Q) { w.t += gridDim.x; load_tile(w); }
    };
    // stage scale words (4 bytes per group) from the raw chunk loads
    auto word = [&](const uint32_t* raw, int g) -> uint32_t {
      if (BPC == 8) return raw[g];                                   // G == 1: word g of the 8 bytes
      if (BPC == 4) return raw[g];                                   // FP8 KB=128 (G=1, g=0) or FP4 KB=64 (G=2: chunk g)
      if (BPC == 2) return G == 2 ? (raw[0] | (raw[1] << 16))        // FP8 KB=64: two chunks of 2 bytes, one group
                                  : (raw[2 * g] | (raw[2 * g + 1] << 16));  // FP4 KB=32: four chunks of 2 bytes, two groups
      return raw[0] | (raw[1] << 8) | (raw[2] << 16) | (raw[3] << 24);      // FP8 KB=32: four chunks of 1 byte
    };
    // advance a walk by one stage without loading (the other scale warp's stage)
    auto sf_skip = [&](Walk& w) {
#pragma unroll
      for (int c = 0; c < G; ++c)
        if (w.q0 + c < w.Q) w.pos.advance(w.tw, p.cpt);
      w.q0 += G;
      if (w.q0 >= w.Q) { w.t += gridDim.x; load_tile(w); }
    };
    Walk pre;
    pre.t = blockIdx.x; pre.done = false; load_tile(pre);
    if (warp == 3 && !pre.done) sf_skip(pre);
    unsigned n_stages_left = 0;   // stages this block will run: count by walking the tiles once
    for (unsigned t = blockIdx.x; t < total; t += gridDim.x) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      n_stages_left += (tw.chunks(p) + G - 1) / G;
    }
    Raw ring[RING];
#pragma unroll
    for (int d = 0; d < RING; ++d) {
#pragma unroll
      for (int i = 0; i < (G == 1 ? 2 : G); ++i) { ring[d].a[i] = 0u; ring[d].b[i] = 0u; }
      if (!pre.done) sf_load(pre, ring[d]);
      if (!pre.done) sf_skip(pre);
    }
    uint32_t s = 0, phase = 0;
    auto advance_stage = [&]() { if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; } };
    if (warp == 3 && n_stages_left > 0) { advance_stage(); --n_stages_left; }
    bool alive = true;
    PROF_BEGIN();
    while (alive && n_stages_left > 0) {
#pragma unroll
      for (int d = 0; d < RING; ++d) {
        if (n_stages_left == 0 || !alive) break;
        bool ok = true;
        if (lane == 0) ok = !*abort_flag && PROF_WAIT(mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT));
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { *abort_flag = 1; alive = false; break; }
        uint8_t* sfa = smem + (size_t)s * stage_bytes + A_STAGE_BYTES + b_stage_bytes;
        uint8_t* sfb = sfa + SFA_BYTES;
#pragma unroll
        for (int g = 0; g < SPA; ++g) {
          const uint32_t aw = word(ring[d].a, g), bw = word(ring[d].b, g);
          uint32_t w4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) w4[j] = __shfl_sync(0xffffffffu, aw, src_lane[j]);
          *reinterpret_cast<uint4*>(sfa + g * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          for (int a = 0; a < atoms_b; ++a) {
#pragma unroll
            for (int j = 0; j < 4; ++j) w4[j] = __shfl_sync(0xffffffffu, bw, 4 * a + j);
            *reinterpret_cast<uint4*>(sfb + (g * atoms_b + a) * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        advance_stage();
        --n_stages_left;
        if (n_stages_left > 0) { advance_stage(); --n_stages_left; }   // the other scale warp's stage
        if (!pre.done) sf_load(pre, ring[d]);
        if (!pre.done) sf_skip(pre);
      }
    }
    if (lane == 0 && warp == 2) PROF_END(2);
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;           // TMEM lane quadrant this warp may read
    const int half = (warp - 4) >> 2;    // warps 4-7 take the first half of the tile's columns, 8-11 the second
    const int r = 32 * quad + lane;
    const int tw_ = r & (p.TW - 1), tn = r >> p.lgTW;
    const int cbeg = half == 0 ? 0 : ((p.BN / 2 + 15) & ~15);
    const int cend = half == 0 ? ((p.BN / 2 + 15) & ~15) : p.BN;
    const long long cs = (long long)p.Hd * p.Wd;
    uint32_t tcount = 0;
    PROF_BEGIN();
    for (unsigned t = blockIdx.x; t < total && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      TapWalk<MODE> tw;
      tw.init(p, tile);
      const int Q = tw.chunks(p);
      const int acc = tcount % p.n_acc;
      bool ok = true;
      if (lane == 0) ok = PROF_WAIT(mbar_wait(&tfull[acc], (tcount / p.n_acc) & 1, p.status, MQ_ERR_TIMEOUT));
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      int yo, xo;
      if (MODE == MQ_OP_FWD) { yo = tile.h; xo = tile.w0 + tw_; }
      else { yo = tile.cls / p.sw + p.sh * tile.h; xo = tile.cls % p.sw + p.sw * (tile.w0 + tw_); }
      const int n = tile.n0 + tn;
      const bool row_ok = yo < p.Hd && xo < p.Wd && n < p.N;
      const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16);
      const bool full_cols = tile.c0 + p.BN <= p.Cd;
      float* o_nchw = p.out + (((long long)n * p.Cd + tile.c0 + cbeg) * p.Hd + yo) * p.Wd + xo;
      float* o_hwnc = p.out + (((long long)yo * p.Wd + xo) * p.N + n) * p.Cd + tile.c0 + cbeg;
      for (int c = cbeg; c < cend; c += 16) {
        uint32_t v[16];
        if (Q > 0) {
          tmem_ld_32x32b_x16(taddr + c, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
        if (row_ok) {
          if (p.out_layout == MQ_NCHW) {
            if (full_cols) {
#pragma unroll
              for (int j = 0; j < 16; ++j) { *o_nchw = __uint_as_float(v[j]); o_nchw += cs; }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j) { if (tile.c0 + c + j < p.Cd) *o_nchw = __uint_as_float(v[j]); o_nchw += cs; }
            }
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
      if (lane == 0) mbar_arrive(&tempty[acc]);
    }
    if (lane == 0 && warp == 4) PROF_END(3);
  }
  // teardown: everyone meets here (all loops are bounded), then the allocating warp frees TMEM
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---- W -> W^T re-layout (codes only; scales are indexed in place) ------------------------------
// in:  [C_out][taps][C_in_p] codes;  out: [C_in_p][taps][C_out_p] codes (zero for c_out >= C_out)
__global__ void weight_transpose_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, const uint8_t* __restrict__ sc_in,
                                        uint8_t* __restrict__ sc_out, int Cout, int Cop, int Cp, int taps, int fp4) {
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

extern "C" int mqdbg_read_prof(unsigned long long* out16) {
  return cudaMemcpyFromSymbol(out16, g_prof, sizeof(unsigned long long) * 16) == cudaSuccess ? 0 : 1;
}

bool encode_tensor_map_u8(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                          const uint32_t* elem_strides, int swizzle_bytes) {
  EncodeTiledFn fn = get_encoder();
  if (!fn) return false;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = elem_strides ? elem_strides[i] : 1; }
  for (int i = 0; i + 1 < rank; ++i) st[i] = strides_bytes[i];
  CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                        : swizzle_bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                        : swizzle_bytes == 32  ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

size_t conv_tc_smem_bytes(const ConvTcParams& p) {
  const size_t stage = A_STAGE_BYTES + (size_t)p.BN * 128 + SFA_BYTES + SFB_BYTES;
  return 1024 + (size_t)p.stages * stage + (2 * (size_t)p.stages + 4) * 8 + 64;
}

template <int MODE, int KB, bool FP4>
cudaError_t launch_conv_tc_inst(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, cudaStream_t s) {
  static bool attr_set = false;
  const size_t smem = conv_tc_smem_bytes(p);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel<MODE, KB, FP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned grid = (unsigned)(p.total_tiles < sms ? p.total_tiles : sms);
  conv_tc_kernel<MODE, KB, FP4><<<grid, TC_THREADS, smem, s>>>(map_a, map_b, p);
  return cudaGetLastError();
}

cudaError_t launch_conv_tc(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, cudaStream_t s) {
  if (p.total_tiles <= 0 || p.total_tiles > 0x7fffffffLL) return cudaErrorInvalidValue;
#define MQ_TC_CASE(M, K, F) if (p.mode == M && p.KB == K && (p.kind_fp4 != 0) == F) return launch_conv_tc_inst<M, K, F>(p, map_a, map_b, s)
  MQ_TC_CASE(MQ_OP_FWD, 128, false); MQ_TC_CASE(MQ_OP_FWD, 64, false); MQ_TC_CASE(MQ_OP_FWD, 32, false);
  MQ_TC_CASE(MQ_OP_FWD, 128, true);  MQ_TC_CASE(MQ_OP_FWD, 64, true);  MQ_TC_CASE(MQ_OP_FWD, 32, true);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, false); MQ_TC_CASE(MQ_OP_BWD_DATA, 64, false); MQ_TC_CASE(MQ_OP_BWD_DATA, 32, false);
  MQ_TC_CASE(MQ_OP_BWD_DATA, 128, true);  MQ_TC_CASE(MQ_OP_BWD_DATA, 64, true);  MQ_TC_CASE(MQ_OP_BWD_DATA, 32, true);
#undef MQ_TC_CASE
  return cudaErrorInvalidValue;
}

cudaError_t launch_weight_transpose(const uint8_t* w_codes, const uint8_t* w_scales, uint8_t* wt_codes, uint8_t* wt_scales, const Geom& g, int fmt,
                                    cudaStream_t s) {
  dim3 grid(g.Cp / 32, g.Cop / 32, g.Kh * g.Kw), block(32, 8);
  weight_transpose_kernel<<<grid, block, 0, s>>>(w_codes, wt_codes, w_scales, wt_scales, g.Cout, g.Cop, g.Cp, g.Kh * g.Kw, fmt == MQ_E2M1 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace mq
