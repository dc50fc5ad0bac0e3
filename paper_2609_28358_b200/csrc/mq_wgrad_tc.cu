// Tensor-core weight-gradient GEMM (G_Wf = G_Yf . X'^T, Sec. II-C / IV-B, Eq. 3), block-scaled as
// Eq. 7 with K-blocks of 32 samples at one output pixel: the stored X and G_Y are consumed along N,
// the second direction of their square quantization tiles.
//
//   D[co][(tap, ci)] = sum over (ho, wo, n) of G[ho, wo, n, co] * X[ho*s + kh - p, wo*s + kw - p, n, ci]
//
// 8-bit formats: both operands are read exactly as stored ([pixel][n][c], c fastest) and handed to the
// MMA as MN-major tiles (K = n runs across rows of 128 channel bytes); no re-layout, no requantization.
// E2M1: tcgen05 accepts 4-bit operands only K-major, so mq_conv_bwd_weight first transposes the codes of X
// and G_Y inside every pixel in scratch ([pixel][c][n], a pure permutation of nibbles, scales untouched);
// this kernel then loads, per pixel, a [128 channels][n bytes] K-major box whose row length equals its
// swizzle span (16 bytes: unswizzled core matrices, two boxes side by side per MMA).
//
// One thread block per work item (128 output channels x 128 (tap, ci) columns x a slice of the
// pixel range); partial sums go to scratch and are added in a fixed order by bwd_weight_reduce.
// Warps: 0 TMA producer, 1 MMA issuer, 2-3 scale expanders (alternating stages), 4-7 epilogue.
#include "mq_conv_tc.cuh"
#include "mq_tcgen05.cuh"

namespace mq {
namespace {
using namespace tc;

constexpr int WG_THREADS = 256;
constexpr int WG_STAGE_BYTES = 2 * 128 * 128 + 4 * 512;  // A 16 KB + B 16 KB + scale chunks (2 groups each)

// stage index -> (ho, wo group, n chunk), walked incrementally
struct KPos {
  int ho, wg, nc;
  __device__ __forceinline__ void set(const WgradTcParams& p, int st) {
    nc = st % p.nchunks; st /= p.nchunks;
    wg = st % p.groups_w; ho = st / p.groups_w;
  }
  __device__ __forceinline__ void next(const WgradTcParams& p) {
    if (++nc == p.nchunks) { nc = 0; if (++wg == p.groups_w) { wg = 0; ++ho; } }
  }
};

template <bool FP4>
__global__ void __launch_bounds__(WG_THREADS, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const WgradTcParams p) {
  constexpr int SPA = FP4 ? 2 : 1;     // scale bytes per MMA per row
  constexpr int NBS = 4 * SPA;         // K-blocks (scale bytes) per stage
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)p.stages * WG_STAGE_BYTES);
  uint64_t* empty = full + p.stages;
  uint64_t* tfull = empty + p.stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfull + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  // work item
  int item = blockIdx.x;
  const int mt = item % p.m_tiles; item /= p.m_tiles;
  const int jt = item % p.j_tiles;
  const int split = item / p.j_tiles;
  const int tap = jt / p.cb_tiles, cb = jt - tap * p.cb_tiles;
  const int kh = tap / p.Kw, kw = tap - kh * p.Kw;
  const int co0 = mt * 128, ci0 = cb * 128;
  const int st_begin = (int)((long long)p.stages_total * split / p.splits);
  const int st_end = (int)((long long)p.stages_total * (split + 1) / p.splits);
  const int nst = st_end - st_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
    mbar_init(tfull, 1);
    *abort_flag = 0;
    mbar_fence_init();
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 256); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      KPos k;
      k.set(p, st_begin);
      uint32_t s = 0, phase = 0;
      for (int i = 0; i < nst && !*abort_flag; ++i) {
        if (!mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        uint8_t* sa = smem + (size_t)s * WG_STAGE_BYTES;
        uint8_t* sb = sa + 128 * 128;
        mbar_arrive_expect_tx(&full[s], 2 * 128 * 128);
        const int wo0 = k.wg * p.KPX;
        if (FP4) {
          // [pixel][c][n] re-laid codes: one box (n bytes, 128 channels) per pixel of the stage
          for (int px = 0; px < p.KPX; ++px) {
            tma_load_4d(sa + px * 128 * p.KBn, &map_a, &full[s], k.nc * p.KBn, co0, wo0 + px, k.ho);
            tma_load_4d(sb + px * 128 * p.KBn, &map_b, &full[s], k.nc * p.KBn, ci0, (wo0 + px) * p.sw + kw - p.pw, k.ho * p.sh + kh - p.ph);
          }
        } else {
          // stored [ho][wo][n][c] codes: box (128 channel bytes, n rows, pixels, 1)
          tma_load_4d(sa, &map_a, &full[s], co0, k.nc * p.BPP * 32, wo0, k.ho);
          tma_load_4d(sb, &map_b, &full[s], ci0, k.nc * p.BPP * 32, wo0 * p.sw + kw - p.pw, k.ho * p.sh + kh - p.ph);
        }
        k.next(p);
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      // 8-bit: MN-major tiles [K row][128 bytes], 128-byte swizzle, 8-row groups 1024 bytes apart; an MMA
      // takes 32 K rows (4096 bytes).  E2M1: per-pixel K-major boxes [128 rows][KBn bytes], swizzle span
      // = KBn (none for 16: 8x16-byte core matrices, the next 16 bytes of K one box further); an MMA takes
      // 32 bytes of K.
      const uint32_t fp4_layout = p.KBn == 128 ? 2u : (p.KBn == 64 ? 4u : (p.KBn == 32 ? 6u : 0u));
      const uint64_t op_desc = FP4 ? smem_desc_base(128 * 16, 8 * p.KBn, fp4_layout) : smem_desc_base(128 * 128, 1024, 2);
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint32_t stage16 = WG_STAGE_BYTES >> 4;
      const uint64_t a_desc0 = smem_desc(op_desc, smem_u32(smem));
      const uint64_t b_desc0 = smem_desc(op_desc, smem_u32(smem + 128 * 128));
      const uint64_t sfa_desc0 = smem_desc(sf_desc, smem_u32(smem + 2 * 128 * 128));
      const uint64_t sfb_desc0 = smem_desc(sf_desc, smem_u32(smem + 2 * 128 * 128 + 1024));
      uint32_t koff16[4];   // offset of MMA a's K slice inside the stage's operand tile, in 16-byte units
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        if (FP4) { const int piece = (32 * a) / p.KBn, off = (32 * a) % p.KBn; koff16[a] = (uint32_t)(piece * 128 * p.KBn + off) >> 4; }
        else koff16[a] = 256u * a;
      }
      uint32_t idesc_id[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) idesc_id[i] = idesc_with_sf_ids(p.idesc, i, i);
      const uint32_t sf_base = tmem + 128;
      uint32_t s = 0, phase = 0, sfbuf = 0, accumulate = 0;
      for (int i = 0; i < nst && !*abort_flag; ++i) {
        if (!mbar_wait(&full[s], phase, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        const uint32_t so = s * stage16;
        const uint32_t sfa_t = sf_base + sfbuf * 16, sfb_t = sfa_t + 8;
#pragma unroll
        for (int g = 0; g < SPA; ++g) {
          tmem_cp_32x128b_warpx4(sfa_t + 4 * g, sfa_desc0 + so + g * 32);
          tmem_cp_32x128b_warpx4(sfb_t + 4 * g, sfb_desc0 + so + g * 32);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          const int g = (a * SPA) >> 2, id = (a * SPA) & 3;
          if (FP4) mma_mxf4(tmem, a_desc0 + so + koff16[a], b_desc0 + so + koff16[a], idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g, accumulate);
          else mma_mxf8f6f4(tmem, a_desc0 + so + koff16[a], b_desc0 + so + koff16[a], idesc_id[id], sfa_t + 4 * g, sfb_t + 4 * g, accumulate);
          accumulate = 1;
        }
        tc_commit(&empty[s]);
        sfbuf ^= 1;
        if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; }
      }
      if (nst > 0) tc_commit(tfull); else mbar_arrive(tfull);
    }
  } else if (warp == 2 || warp == 3) {
    // ------------------------------------------------------------------ scale expanders
    // Lane l < 4*SPA computes the A word (row group j = l / SPA, byte group g = l % SPA); lanes
    // 8..8+4*SPA the B words.  A word is the 4 scale bytes of 4 consecutive K-blocks (pixel, n block)
    // for one block of 32 channels.  Loads are issued RING stages ahead and left raw until used.
    constexpr int RING = 4;
    const int wid = warp - 2;
    const bool is_a = lane < 4 * SPA, is_b = lane >= 8 && lane < 8 + 4 * SPA;
    const int wl = is_b ? lane - 8 : lane;
    const int j = wl / SPA, g = wl - j * SPA;
    const int cblk = is_b ? (ci0 >> 5) + j : (co0 >> 5) + j;
    const bool lane_ok = (is_a && cblk < p.Cot) || (is_b && cblk < p.Ct);
    const uint8_t* base = is_b ? p.x_scales : p.g_scales;
    const int cstride = is_b ? p.Ct : p.Cot;
    auto sf_load = [&](const KPos& k, uint32_t* raw) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        raw[i] = 0u;
        const int b = 4 * g + i;                  // K-block of the stage
        const int px = b / p.BPP, nb = k.nc * p.BPP + (b - px * p.BPP);
        const int wo = k.wg * p.KPX + px;
        if (lane_ok && nb < p.Nt && wo < p.Wo) {
          int hh = k.ho, ww = wo, Wd = p.Wo;
          bool ok = true;
          if (is_b) {
            hh = k.ho * p.sh + kh - p.ph; ww = wo * p.sw + kw - p.pw; Wd = p.W;
            ok = hh >= 0 && hh < p.H && ww >= 0 && ww < p.W;
          }
          if (ok) raw[i] = __ldg(base + (((long long)hh * Wd + ww) * p.Nt + nb) * cstride + cblk);
        }
      }
    };
    KPos kpre;
    kpre.set(p, st_begin);
    int pre_left = nst;                       // stages not yet loaded (counting both warps' stages)
    auto pre_advance = [&]() { kpre.next(p); --pre_left; };
    if (wid == 1 && pre_left > 0) pre_advance();
    uint32_t ring[RING][4];
#pragma unroll
    for (int d = 0; d < RING; ++d) {
#pragma unroll
      for (int i = 0; i < 4; ++i) ring[d][i] = 0u;
      if (pre_left > 0) { sf_load(kpre, ring[d]); pre_advance(); if (pre_left > 0) pre_advance(); }
    }
    uint32_t s = 0, phase = 0;
    auto advance_stage = [&]() { if (++s == (uint32_t)p.stages) { s = 0; phase ^= 1; } };
    int left = nst;
    if (wid == 1 && left > 0) { advance_stage(); --left; }
    bool alive = true;
    while (alive && left > 0) {
#pragma unroll
      for (int d = 0; d < RING; ++d) {
        if (left == 0 || !alive) break;
        bool ok = true;
        if (lane == 0) ok = !*abort_flag && mbar_wait(&empty[s], phase ^ 1, p.status, MQ_ERR_TIMEOUT);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { *abort_flag = 1; alive = false; break; }
        uint8_t* sfa = smem + (size_t)s * WG_STAGE_BYTES + 2 * 128 * 128;
        uint8_t* sfb = sfa + 1024;
        const uint32_t word = ring[d][0] | (ring[d][1] << 8) | (ring[d][2] << 16) | (ring[d][3] << 24);
#pragma unroll
        for (int gg = 0; gg < SPA; ++gg) {
          uint32_t w4[4];
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) w4[jj] = __shfl_sync(0xffffffffu, word, jj * SPA + gg);
          *reinterpret_cast<uint4*>(sfa + gg * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
#pragma unroll
          for (int jj = 0; jj < 4; ++jj) w4[jj] = __shfl_sync(0xffffffffu, word, 8 + jj * SPA + gg);
          *reinterpret_cast<uint4*>(sfb + gg * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
        advance_stage(); --left;
        if (left > 0) { advance_stage(); --left; }
        if (pre_left > 0) { sf_load(kpre, ring[d]); pre_advance(); if (pre_left > 0) pre_advance(); }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: partial sums to scratch
    const int quad = warp & 3;
    const int r = 32 * quad + lane;
    bool ok = true;
    if (lane == 0) ok = mbar_wait(tfull, 0, p.status, MQ_ERR_TIMEOUT);
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    if (ok) {
      tc_fence_after_sync();
      const int co = co0 + r;
      const long long J = (long long)p.Kh * p.Kw * p.Cp;
      float* out = p.partial + ((long long)split * p.Cout + co) * J + (long long)tap * p.Cp + ci0;
      const int ncols = min(128, p.Cp - ci0);
      const uint32_t taddr = tmem + ((uint32_t)(32 * quad) << 16);
      for (int c = 0; c < ncols; c += 16) {
        uint32_t v[16];
        if (nst > 0) {
          tmem_ld_32x32b_x16(taddr + c, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int q = 0; q < 16; ++q) v[q] = 0u;
        }
        if (co < p.Cout) {
#pragma unroll
          for (int q = 0; q < 16; q += 4)   // Cp is a multiple of 32: whole float4s
            *reinterpret_cast<float4*>(out + c + q) = make_float4(__uint_as_float(v[q]), __uint_as_float(v[q + 1]), __uint_as_float(v[q + 2]), __uint_as_float(v[q + 3]));
        }
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 256);
}

// ---- E2M1 re-layout: stored [pixel][n][Cp] nibbles -> [pixel][Cp][Npad] nibbles (n fastest, zero for n >= N) ----
// One block: 8 pixels x 32 samples x 64 channels.  Reads rows of 32 bytes, writes 16 bytes per (pixel, channel).
__global__ void __launch_bounds__(256) fp4_to_n_major_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, int P, int N, int Cp, int Npad) {
  __shared__ uint8_t t[8][32][65];  // [pixel][n][c] one code per byte
  const int p0 = blockIdx.x * 8, n0 = blockIdx.y * 32, c0 = blockIdx.z * 64;
  const int tid = threadIdx.x;
  // load: 8 pixels x 32 rows x 32 bytes = 512 chunks of 16 bytes
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
  // store: 64 channels x 8 pixels x 16 bytes (32 samples)
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

}  // namespace

size_t wgrad_tc_smem_bytes(const WgradTcParams& p) { return 1024 + (size_t)p.stages * WG_STAGE_BYTES + (2 * (size_t)p.stages + 2) * 8 + 64; }

cudaError_t launch_wgrad_tc(const WgradTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, cudaStream_t s) {
  static bool attr_set[2] = {false, false};
  const size_t smem = wgrad_tc_smem_bytes(p);
  const int f = p.fp4 ? 1 : 0;
  if (!attr_set[f]) {
    cudaError_t e = f ? cudaFuncSetAttribute(wgrad_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024)
                      : cudaFuncSetAttribute(wgrad_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[f] = true;
  }
  const unsigned grid = (unsigned)(p.m_tiles * p.j_tiles * p.splits);
  if (f) wgrad_tc_kernel<true><<<grid, WG_THREADS, smem, s>>>(map_a, map_b, p);
  else wgrad_tc_kernel<false><<<grid, WG_THREADS, smem, s>>>(map_a, map_b, p);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_fp4_to_n_major(const uint8_t* in, uint8_t* out, int P, int N, int Cp, int Npad, cudaStream_t s) {
  dim3 grid((P + 7) / 8, Npad / 32, (Cp + 63) / 64);
  fp4_to_n_major_kernel<<<grid, 256, 0, s>>>(in, out, P, N, Cp, Npad);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace mq
