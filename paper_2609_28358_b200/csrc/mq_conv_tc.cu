// Tensor-core implicit-GEMM kernel for mq_conv_fwd and mq_conv_bwd_data (Sec. II-C / IV-B GEMMs,
// block-scaled as Eq. 7) on sm_100a: tcgen05 block-scaled MMA with accumulators and scale vectors
// in tensor memory, operands brought by TMA straight from the stored channel-batch-first tensors
// (the im2col of Sec. IV-A is implicit: every tap is a shifted TMA box, out-of-image taps are the
// TMA zero fill).
//
// One persistent thread block per SM, 8 warps:
//   warp 0   TMA producer        one lane issues the A (gathered activation) and B (weight) boxes
//   warp 1   MMA issuer          one lane copies the stage's scale vectors smem -> TMEM and issues the MMAs
//   warp 2   scale expander      turns the compact tile scales (one E8M0 byte per 32x32 tile) into the
//                                per-row scale vectors the MMA reads, for the tap / K-block of each stage
//   warps 4-7 epilogue           TMEM -> registers -> global (fp32), overlapped with the next tile's main loop
// A pipeline stage holds 128 bytes of K per row (four MMAs): one 128-byte box, or 128/KB boxes of KB
// bytes when a tap has fewer than 128 bytes of channels (then several taps share a stage).
// Every wait is bounded; on expiry the kernel records MQ_ERR_TIMEOUT in the status word and drains.
#include "mq_conv_tc.cuh"
#include "mq_tcgen05.cuh"

namespace mq {
namespace {
using namespace tc;

constexpr int TC_THREADS = 256;
constexpr int A_STAGE_BYTES = 128 * 128;
constexpr int SFA_BYTES = 1024;   // up to 2 groups of 4 scale bytes per row
constexpr int SFB_BYTES = 2048;   // up to 2 groups x 2 atoms of 128 rows
constexpr int SF_COLS = 24;       // TMEM columns of one scale buffer: 8 (A) + 16 (B)

struct Tile { int c0, w0, n0, h, cls; };
struct Tap { int kh, kw, hs, ws0; };

__device__ __forceinline__ Tile decode_tile(const ConvTcParams& p, long long t) {
  Tile q;
  q.c0 = (int)(t % p.tiles_c) * p.BN; t /= p.tiles_c;
  q.w0 = (int)(t % p.tiles_w) * p.TW; t /= p.tiles_w;
  q.n0 = (int)(t % p.tiles_n) * p.TN; t /= p.tiles_n;
  q.h = (int)(t % p.tiles_h); t /= p.tiles_h;
  q.cls = (int)t;
  return q;
}

// Taps that contribute to a tile.  Forward: all Kh*Kw.  Input gradient: the taps whose offset has the
// parity of the tile's class (h + pad - kh and w + pad - kw divisible by the stride).
__device__ __forceinline__ int tile_taps(const ConvTcParams& p, const Tile& t, int& nkw, int& kh0, int& kw0) {
  if (p.mode == MQ_OP_FWD) { nkw = p.Kw; kh0 = 0; kw0 = 0; return p.Kh * p.Kw; }
  const int ch = t.cls / p.sw, cw = t.cls % p.sw;
  kh0 = (ch + p.ph) % p.sh; kw0 = (cw + p.pw) % p.sw;
  const int nkh = kh0 < p.Kh ? (p.Kh - kh0 + p.sh - 1) / p.sh : 0;
  nkw = kw0 < p.Kw ? (p.Kw - kw0 + p.sw - 1) / p.sw : 0;
  return nkh * nkw;
}
__device__ __forceinline__ Tap tap_of(const ConvTcParams& p, const Tile& t, int i, int nkw, int kh0, int kw0) {
  Tap a;
  if (p.mode == MQ_OP_FWD) {
    a.kh = i / p.Kw; a.kw = i - a.kh * p.Kw;
    a.hs = t.h * p.sh + a.kh - p.ph;
    a.ws0 = t.w0 * p.sw + a.kw - p.pw;
  } else {
    const int ch = t.cls / p.sw, cw = t.cls % p.sw;
    const int ia = i / nkw, ib = i - ia * nkw;
    a.kh = kh0 + p.sh * ia; a.kw = kw0 + p.sw * ib;
    a.hs = t.h + (ch + p.ph - a.kh) / p.sh;    // exact division
    a.ws0 = t.w0 + (cw + p.pw - a.kw) / p.sw;
  }
  return a;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
conv_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const ConvTcParams p) {
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
  const int apc = p.KB / 32;                 // MMA K-atoms (32 bytes) per chunk
  const int spa = p.kind_fp4 ? 2 : 1;        // scale bytes per atom
  const int atoms_b = (p.BN + 127) / 128;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], 2); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 4); }
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
      uint32_t it = 0;
      for (long long t = blockIdx.x; t < p.total_tiles && !*abort_flag; t += gridDim.x) {
        const Tile tile = decode_tile(p, t);
        int nkw, kh0, kw0;
        const int ntaps = tile_taps(p, tile, nkw, kh0, kw0);
        const int Q = ntaps * p.cpt;
        for (int q0 = 0; q0 < Q; q0 += p.G, ++it) {
          const int s = it % p.stages;
          if (!mbar_wait(&empty[s], ((it / p.stages) & 1) ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          const int nch = min(p.G, Q - q0);
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          uint8_t* sb = sa + A_STAGE_BYTES;
          mbar_arrive_expect_tx(&full[s], (uint32_t)nch * (128 + p.BN) * p.KB);
          for (int c = 0; c < nch; ++c) {
            const int q = q0 + c;
            const int ti = q / p.cpt, cc = q - ti * p.cpt;
            const Tap tp = tap_of(p, tile, ti, nkw, kh0, kw0);
            tma_load_4d(sa + c * 128 * p.KB, &map_a, &full[s], cc * p.KB, tp.ws0, tile.n0, tp.hs);
            tma_load_3d(sb + c * p.BN * p.KB, &map_b, &full[s], cc * p.KB, tp.kh * p.Kw + tp.kw, tile.c0);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const int layout = p.KB == 128 ? 2 : (p.KB == 64 ? 4 : 6);
      const uint64_t op_desc = smem_desc_base(16, 8 * p.KB, layout);
      const uint64_t sf_desc = smem_desc_base(0, 128, 0);
      const uint32_t sf_base = tmem + p.n_acc * p.BN;
      uint32_t it = 0, tcount = 0;
      for (long long t = blockIdx.x; t < p.total_tiles && !*abort_flag; t += gridDim.x, ++tcount) {
        const Tile tile = decode_tile(p, t);
        int nkw, kh0, kw0;
        const int Q = tile_taps(p, tile, nkw, kh0, kw0) * p.cpt;
        const int acc = tcount % p.n_acc;
        if (!mbar_wait(&tempty[acc], ((tcount / p.n_acc) & 1) ^ 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
        tc_fence_after_sync();
        const uint32_t d_tmem = tmem + acc * p.BN;
        bool first = true;
        for (int q0 = 0; q0 < Q; q0 += p.G, ++it) {
          const int s = it % p.stages;
          if (!mbar_wait(&full[s], (it / p.stages) & 1, p.status, MQ_ERR_TIMEOUT)) { *abort_flag = 1; break; }
          tc_fence_after_sync();
          uint8_t* sa = smem + (size_t)s * stage_bytes;
          uint8_t* sb = sa + A_STAGE_BYTES;
          uint8_t* sfa = sb + b_stage_bytes;
          uint8_t* sfb = sfa + SFA_BYTES;
          const uint32_t sfa_t = sf_base + (it & 1) * SF_COLS, sfb_t = sfa_t + 8;
          for (int g = 0; g < spa; ++g) {
            tmem_cp_32x128b_warpx4(sfa_t + 4 * g, smem_desc(sf_desc, smem_u32(sfa + g * 512)));
            for (int a = 0; a < atoms_b; ++a)
              tmem_cp_32x128b_warpx4(sfb_t + 4 * (g * atoms_b + a), smem_desc(sf_desc, smem_u32(sfb + (g * atoms_b + a) * 512)));
          }
          const int natoms = min(p.G, Q - q0) * apc;
          for (int a = 0; a < natoms; ++a) {
            const int c = a / apc, ja = a - c * apc;
            const uint64_t ad = smem_desc(op_desc, smem_u32(sa + c * 128 * p.KB + ja * 32));
            const uint64_t bd = smem_desc(op_desc, smem_u32(sb + c * p.BN * p.KB + ja * 32));
            const int g = (a * spa) >> 2, id = (a * spa) & 3;
            const uint32_t idesc = idesc_with_sf_ids(p.idesc, id, id);
            if (p.kind_fp4) mma_mxf4(d_tmem, ad, bd, idesc, sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, first ? 0u : 1u);
            else mma_mxf8f6f4(d_tmem, ad, bd, idesc, sfa_t + 4 * g, sfb_t + 4 * g * atoms_b, first ? 0u : 1u);
            first = false;
          }
          tc_commit(&empty[s]);
        }
        if (Q > 0) tc_commit(&tfull[acc]); else mbar_arrive(&tfull[acc]);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ scale expander
    const int NTL = p.TN >= 32 ? p.TN / 32 : 1;
    const int ncombos = p.TW * NTL;
    const int wstep = p.mode == MQ_OP_FWD ? p.sw : 1;
    uint32_t it = 0;
    for (long long t = blockIdx.x; t < p.total_tiles && !*abort_flag; t += gridDim.x) {
      const Tile tile = decode_tile(p, t);
      int nkw, kh0, kw0;
      const int ntaps = tile_taps(p, tile, nkw, kh0, kw0);
      const int Q = ntaps * p.cpt;
      // this lane's A combo (column offset in the tile, 32-sample block) and B word (row block j, group g)
      const int ctw = lane / NTL, cnl = lane - ctw * NTL;
      const int a_nt = (tile.n0 + cnl * 32) >> 5;
      const bool a_lane_ok = lane < ncombos && (tile.n0 + cnl * 32) < p.N;
      const int bj = lane / spa, bg = lane - bj * spa;
      const int b_rowblock = (tile.c0 >> 5) + bj;
      const bool b_lane_ok = bj < (p.BN + 31) / 32 && (tile.c0 + bj * 32) < p.Cd;
      for (int q0 = 0; q0 < Q; q0 += p.G, ++it) {
        const int s = it % p.stages;
        bool ok = true;
        if (lane == 0) ok = mbar_wait(&empty[s], ((it / p.stages) & 1) ^ 1, p.status, MQ_ERR_TIMEOUT);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) { *abort_flag = 1; break; }
        uint8_t* sfa = smem + (size_t)s * stage_bytes + A_STAGE_BYTES + b_stage_bytes;
        uint8_t* sfb = sfa + SFA_BYTES;
        // scale bytes of the stage: byte b belongs to atom b / spa of the stage
        uint32_t aw[2] = {0u, 0u}, bw = 0u;
        for (int b = 0; b < 4 * spa; ++b) {
          const int atom = b / spa, sub = b - atom * spa;
          const int c = atom / apc, ja = atom - c * apc;
          const int q = q0 + c;
          if (q >= Q) break;
          const int ti = q / p.cpt, cc = q - ti * p.cpt;
          const Tap tp = tap_of(p, tile, ti, nkw, kh0, kw0);
          const int kblk = cc * (apc * spa) + ja * spa + sub;
          if (a_lane_ok) {
            const int ws = tp.ws0 + ctw * wstep;
            if (tp.hs >= 0 && tp.hs < p.Hs && ws >= 0 && ws < p.Ws) {
              const uint32_t v = __ldg(p.a_scales + (((long long)tp.hs * p.Ws + ws) * p.Nt + a_nt) * p.Kblocks + kblk);
              aw[b >> 2] |= v << (8 * (b & 3));
            }
          }
          if (b_lane_ok && (b >> 2) == bg) {
            const uint32_t v = __ldg(p.b_scales + (long long)b_rowblock * p.sb_row + (long long)(tp.kh * p.Kw + tp.kw) * p.sb_tap + (long long)kblk * p.sb_k);
            bw |= v << (8 * (b & 3));
          }
        }
        // rows 32j + lane of the tile: row = tn * TW + tw
        for (int g = 0; g < spa; ++g) {
          uint32_t w4[4];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int r = 32 * j + lane;
            const int tw = r & (p.TW - 1), tn = r >> p.lgTW;
            w4[j] = __shfl_sync(0xffffffffu, aw[g], tw * NTL + (tn >> 5));
          }
          *reinterpret_cast<uint4*>(sfa + g * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          for (int a = 0; a < atoms_b; ++a) {
#pragma unroll
            for (int j = 0; j < 4; ++j) w4[j] = __shfl_sync(0xffffffffu, bw, ((4 * a + j) * spa + g) & 31);
            *reinterpret_cast<uint4*>(sfb + (g * atoms_b + a) * 512 + lane * 16) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&full[s]);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp - 4;
    const int r = 32 * quad + lane;
    const int tw = r & (p.TW - 1), tn = r >> p.lgTW;
    uint32_t tcount = 0;
    for (long long t = blockIdx.x; t < p.total_tiles && !*abort_flag; t += gridDim.x, ++tcount) {
      const Tile tile = decode_tile(p, t);
      int nkw, kh0, kw0;
      const int Q = tile_taps(p, tile, nkw, kh0, kw0) * p.cpt;
      const int acc = tcount % p.n_acc;
      bool ok = true;
      if (lane == 0) ok = mbar_wait(&tfull[acc], (tcount / p.n_acc) & 1, p.status, MQ_ERR_TIMEOUT);
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      if (!ok) { *abort_flag = 1; break; }
      tc_fence_after_sync();
      int yo, xo;
      if (p.mode == MQ_OP_FWD) { yo = tile.h; xo = tile.w0 + tw; }
      else { yo = tile.cls / p.sw + p.sh * tile.h; xo = tile.cls % p.sw + p.sw * (tile.w0 + tw); }
      const int n = tile.n0 + tn;
      const bool row_ok = yo < p.Hd && xo < p.Wd && n < p.N;
      const uint32_t taddr = tmem + acc * p.BN + ((uint32_t)(32 * quad) << 16);
      for (int c = 0; c < p.BN; c += 16) {
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
            float* o = p.out + (((long long)n * p.Cd + tile.c0 + c) * p.Hd + yo) * p.Wd + xo;
            const long long cs = (long long)p.Hd * p.Wd;
#pragma unroll
            for (int j = 0; j < 16; ++j)
              if (tile.c0 + c + j < p.Cd) o[j * cs] = __uint_as_float(v[j]);
          } else {
            float* o = p.out + (((long long)yo * p.Wd + xo) * p.N + n) * p.Cd + tile.c0 + c;
            if (tile.c0 + c + 16 <= p.Cd && (p.Cd & 3) == 0) {
#pragma unroll
              for (int j = 0; j < 16; j += 4)
                *reinterpret_cast<float4*>(o + j) = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]), __uint_as_float(v[j + 3]));
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (tile.c0 + c + j < p.Cd) o[j] = __uint_as_float(v[j]);
            }
          }
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[acc]);
    }
  }
  // teardown: everyone meets here (all loops are bounded), then the allocating warp frees TMEM
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, 512);
}

// ---- W -> W^T re-layout (codes only; scales are indexed in place) ------------------------------
// in:  [C_out][taps][C_in_p] codes;  out: [C_in_p][taps][C_out_p] codes (zero for c_out >= C_out)
__global__ void weight_transpose_kernel(const uint8_t* __restrict__ in, uint8_t* __restrict__ out, int Cout, int Cop, int Cp, int taps, int fp4) {
  __shared__ uint8_t tile[32][33];  // [ci][co]
  const int tap = blockIdx.z;
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

cudaError_t launch_conv_tc(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, cudaStream_t s) {
  static bool attr_set = false;
  const size_t smem = conv_tc_smem_bytes(p);
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(conv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned grid = (unsigned)(p.total_tiles < sms ? p.total_tiles : sms);
  conv_tc_kernel<<<grid, TC_THREADS, smem, s>>>(map_a, map_b, p);
  return cudaGetLastError();
}

cudaError_t launch_weight_transpose(const uint8_t* w_codes, uint8_t* wt_codes, const Geom& g, int fmt, cudaStream_t s) {
  dim3 grid(g.Cp / 32, g.Cop / 32, g.Kh * g.Kw), block(32, 8);
  weight_transpose_kernel<<<grid, block, 0, s>>>(w_codes, wt_codes, g.Cout, g.Cop, g.Cp, g.Kh * g.Kw, fmt == MQ_E2M1 ? 1 : 0);
  return cudaGetLastError();
}

}  // namespace mq
