// Single-pass MX quantizer (Sec. III-A, Eq. 5-6 in the E8M0 form; square blocks of Sec. IV-B) that
// also re-lays the tensor into its channel-batch-first stored order (Sec. IV-A).
//
// The logical source (NCHW / OIHW fp32) is seen as R x C matrices at P positions with the position
// axis fastest in memory: element (p, r, c) lives at (r*C + c)*P + p.  A work item is one
// 32(r) x 32(c) tile at PS = 8 consecutive positions: 1024 source rows x 32 bytes, every 32-byte
// sector read exactly once.
//
// Main kernel (P % 4 == 0): persistent thread blocks loop over work items; the next item's 32 KB stream
// into shared memory with cp.async (16-byte copies, zero fill for out-of-range rows) while the current
// item is reduced and converted, so the block always has bytes in flight.  Per position: amax over the
// tile (per-thread max, one redux.sync per position, one shared-memory exchange), E8M0 code from the exponent field,
// hardware RNE+saturate conversion; a thread owns 4 adjacent channels so codes leave as 32-bit (FP8) or
// 16-bit (FP4) shared-memory stores, and each [n][c] slab is written with 16-byte global stores.
// Fallback kernel (any P, e.g. the 3x3 = 9 positions of a weight tensor): scalar loads, same arithmetic.
#include <cstdlib>

#include "mq_internal.cuh"
#include "mq_conv_tc.cuh"   // encode_tensor_map_u8
#include "mq_tcgen05.cuh"   // mbarrier and TMA wrappers

namespace mq {
namespace {

constexpr int PS = 8;           // positions per work item
constexpr int QT_THREADS = 256;
// input buffer: 1024 rows of 32 bytes, plus 16 bytes of padding after every 4 rows so that the 8 lanes of
// a quarter-warp (rows 4 apart) hit 8 different 16-byte bank groups
constexpr int QBUF_BYTES = 1024 * 32 + 256 * 16;

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
  const unsigned d = (unsigned)__cvta_generic_to_shared(dst);
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

struct Item { int p0, r0, c0, rt, ct; };
__device__ __forceinline__ Item item_of(unsigned it, int n_pstrips, int Ct, int psi = PS) {
  // channel tile fastest: the tiles that share an output line ([n][c] rows are c-contiguous) are produced
  // together, so full 128-byte lines reach L2 at about the same time; then position strip, then row tile
  Item q;
  const unsigned u = it / (unsigned)Ct;
  q.ct = (int)(it - u * (unsigned)Ct);
  q.rt = (int)(u / (unsigned)n_pstrips);
  const int ps = (int)(u - (unsigned)q.rt * (unsigned)n_pstrips);
  q.p0 = ps * psi; q.r0 = q.rt * 32; q.c0 = q.ct * 32;
  return q;
}

// R16 (tensors of at most 16 rows, e.g. a batch of 16 samples; NT = 256): the upper half of the 32-row tile would be
// padding, so an item takes 16 positions instead - buffer rows 16..31 hold rows 0..15 of the next eight positions - and
// every amax, scale and slab below is per (half, position).
// 16 consecutive one-byte codes at element index e (a multiple of 16): stored as they are, or - packed 6-bit storage - as
// the 12-byte field of their group
__device__ __forceinline__ void store_codes16(const QuantArgs& a, long long e, const uint4 val) {
  if (a.packed6) {
    const uint32_t w[4] = {val.x, val.y, val.z, val.w};
    uint32_t o[3];
    pack6x16(w, o);
    uint32_t* d = reinterpret_cast<uint32_t*>(a.codes + (e >> 4) * 12);
    d[0] = o[0]; d[1] = o[1]; d[2] = o[2];
  } else {
    *reinterpret_cast<uint4*>(a.codes + e) = val;
  }
}

template <int FMT, int NT, bool SR, bool R16 = false>   // NT threads per block: 256 (two tile rows per thread) or 512 (one); SR: stochastic rounding
__global__ void __launch_bounds__(NT) quantize_pipe_kernel(QuantArgs a, int n_pstrips, int Ct, unsigned n_items) {
  constexpr int RI = 512 / NT;      // tile rows per thread
  constexpr int NW = NT / 32;       // warps
  constexpr int CPT = 2048 / NT;    // 16-byte input chunks per thread
  extern __shared__ __align__(16) uint8_t qsmem[];
  uint8_t* buf0 = qsmem;
  uint8_t* buf1 = qsmem + QBUF_BYTES;
  uint8_t* stage = qsmem + 2 * QBUF_BYTES;                              // codes [p][r][32 B (FP8) | 16 B (FP4)]
  unsigned* red = reinterpret_cast<unsigned*>(stage + PS * 32 * 32);     // [warp][quad][4]

  pdl_wait();
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  // compute mapping: 4 adjacent channels x 2 rows x 4 positions per thread
  const int cq = t & 7, quad = (t >> 3) & 1, rs = t >> 4;
  constexpr int RB = FMT == MQ_E2M1 ? 16 : 32;   // bytes of a staged row

  // copy mapping: chunk (row, position quad) with row = (t >> 1) + (NT/2) m: channel (t >> 1) & 31, tile row
  // (t >> 6) + (NT/64) m
  constexpr int RSTEP = NT / 64;    // tile rows between a thread's consecutive chunks
  const int ld_cc = (t >> 1) & 31, ld_rr = t >> 6, ld_qd = t & 1;
  const int ld_row = t >> 1;
  const unsigned ld_dst = (unsigned)(ld_row * 32 + (ld_row >> 2) * 16 + ld_qd * 16);   // + m * RSTEP * (32 * 32 + 8 * 16)
  const long long row_step = (long long)RSTEP * a.C * a.P;   // floats between a thread's consecutive chunks
  auto issue = [&](unsigned it, uint8_t* buf) -> Item {
    const Item q = item_of(it, n_pstrips, Ct, R16 ? 2 * PS : PS);
    const int pq = q.p0 + 4 * ld_qd;
    const bool col_ok = (q.c0 + ld_cc) < a.C && pq < a.P;
    const float* src = a.src + ((long long)(q.r0 + ld_rr) * a.C + (q.c0 + ld_cc)) * a.P + pq;
    const int rows_left = a.R - q.r0 - ld_rr;     // tile row 4 m is valid while 4 m < rows_left
#pragma unroll
    for (int m = 0; m < CPT; ++m) {
      if (R16) {
        // buffer row ld_rr + 4 m: tensor row (ld_rr + 4 m) & 15 at the positions of half m >> 2
        const bool ok = (q.c0 + ld_cc) < a.C && pq + PS * (m >> 2) < a.P && RSTEP * (m & 3) < rows_left;
        cp_async16(buf + ld_dst + m * RSTEP * (32 * 32 + 8 * 16), ok ? src + (m & 3) * row_step + PS * (m >> 2) : a.src, ok);
      } else {
        const bool ok = col_ok && RSTEP * m < rows_left;
        cp_async16(buf + ld_dst + m * RSTEP * (32 * 32 + 8 * 16), ok ? src + m * row_step : a.src, ok);
      }
    }
    cp_async_commit();
    return q;
  };

  unsigned it = blockIdx.x;
  const unsigned n_it = (unsigned)n_items;
  Item q_next{};
  if (it < n_it) q_next = issue(it, buf0);
  int cur = 0;
  const unsigned quad_mask = quad ? 0xFF00FF00u : 0x00FF00FFu;   // the 16 lanes that share this thread's position quad
  for (; it < n_it; it += gridDim.x, cur ^= 1) {
    uint8_t* buf = cur ? buf1 : buf0;
    const unsigned nxt = it + gridDim.x;
    const Item q = q_next;
    if (nxt < n_it) { q_next = issue(nxt, cur ? buf0 : buf1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
    __syncthreads();   // the current item's bytes are visible to every thread

    float v[RI][4][4];   // [row i][channel k][position j]
#pragma unroll
    for (int i = 0; i < RI; ++i)
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int row = (rs + 16 * i) * 32 + 4 * cq + k;
        const float4 f = *reinterpret_cast<const float4*>(buf + row * 32 + (row >> 2) * 16 + quad * 16);
        v[i][k][0] = f.x; v[i][k][1] = f.y; v[i][k][2] = f.z; v[i][k][3] = f.w;
      }
    // amax per position on the bit patterns of |x| (order-preserving): thread, then the 16 lanes that share
    // this position quad (lane bits 0,1,2,4), then the 8 warps
    // HV = 1: one amax per position over both of the thread's rows; R16: one per (half, position)
    constexpr int HV = R16 ? RI : 1;
    unsigned m4[HV][4];
#pragma unroll
    for (int h = 0; h < HV; ++h)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float fm = 0.f;
#pragma unroll
        for (int i = 0; i < RI; ++i)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            if (!R16 || i == h) fm = fmaxf(fm, fabsf(v[i][k][j]));
        m4[h][j] = __reduce_max_sync(quad_mask, __float_as_uint(fm));
      }
    if ((lane & 23) == 0) {   // lanes 0 (quad 0) and 8 (quad 1)
#pragma unroll
      for (int h = 0; h < HV; ++h)
        *reinterpret_cast<uint4*>(&red[((warp * 2 + quad) * HV + h) * 4]) = make_uint4(m4[h][0], m4[h][1], m4[h][2], m4[h][3]);
    }
    __syncthreads();
    int code[HV][4];
#pragma unroll
    for (int h = 0; h < HV; ++h) {
      uint4 mx = make_uint4(0, 0, 0, 0);
#pragma unroll
      for (int w = 0; w < NW; ++w) {
        const uint4 r4 = *reinterpret_cast<const uint4*>(&red[((w * 2 + quad) * HV + h) * 4]);
        mx.x = max(mx.x, r4.x); mx.y = max(mx.y, r4.y); mx.z = max(mx.z, r4.z); mx.w = max(mx.w, r4.w);
      }
      code[h][0] = scale_code_of(mx.x, fmt_emax(FMT)); code[h][1] = scale_code_of(mx.y, fmt_emax(FMT));
      code[h][2] = scale_code_of(mx.z, fmt_emax(FMT)); code[h][3] = scale_code_of(mx.w, fmt_emax(FMT));
    }
    if (t < PS * HV) {       // position t of the item: half t >> 3 (R16), quad (t >> 2) & 1, j = t & 3
      const int h = t >> 3, qd = (t >> 2) & 1;
      unsigned mm = 0;
#pragma unroll
      for (int w = 0; w < NW; ++w) mm = max(mm, red[((w * 2 + qd) * HV + h) * 4 + (t & 3)]);
      if (q.p0 + t < a.P)
        a.scales[(long long)(q.p0 + t) * a.sc_stride_p + (long long)q.rt * a.sc_stride_r + q.ct] = (uint8_t)scale_code_of(mm, fmt_emax(FMT));
    }
    // index of element (row rs, channel 4 cq, position 4 quad) of this item in the logical tensor
    const long long e_base = ((long long)(q.r0 + rs) * a.C + q.c0 + 4 * cq) * a.P + q.p0 + 4 * quad;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int i = 0; i < RI; ++i) {
        const float f = scale_factor(code[R16 ? i : 0][j]);
        float x[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          x[k] = v[i][k][j] * f;
          if (SR) {
            // the thread's second row: 16 tensor rows on, or (R16) the same row eight positions on
            const long long e_off = R16 ? (long long)k * a.P + j + PS * i : ((long long)(16 * i) * a.C + k) * a.P + j;
            x[k] = sr_value<FMT>(x[k], (unsigned)e_base + (unsigned)e_off, sr_key(a, e_base + e_off));   // low word: modular arithmetic
          }
        }
        const unsigned lo = encode2<FMT>(x[0], x[1]);
        const unsigned hi = encode2<FMT>(x[2], x[3]);
        uint8_t* dst = R16 ? stage + ((PS * i + 4 * quad + j) * 16 + rs) * RB : stage + ((4 * quad + j) * 32 + rs + 16 * i) * RB;
        if (FMT == MQ_E2M1) *reinterpret_cast<unsigned short*>(dst + 2 * cq) = (unsigned short)(lo | (hi << 8));
        else *reinterpret_cast<unsigned*>(dst + 4 * cq) = lo | (hi << 16);
      }
    }
    __syncthreads();
    // copy out: per position a 32(r) x 32(c) slab; rows are contiguous runs of the stored tensor
    if (FMT == MQ_E2M1) {
      const int p = R16 ? t >> 4 : t >> 5, r = R16 ? t & 15 : t & 31;   // 256 rows of 16 bytes: [position][row]
      if (t < 256 && q.p0 + p < a.P && q.r0 + r < a.R) {
        const uint4 val = *reinterpret_cast<const uint4*>(stage + t * 16);
        const long long e = (long long)(q.p0 + p) * a.out_stride_p + (long long)(q.r0 + r) * a.out_stride_r + q.c0;
        *reinterpret_cast<uint4*>(a.codes + (e >> 1)) = val;
      }
    } else {
#pragma unroll
      for (int k = 0; k < 512 / NT; ++k) {
        const int id = t + NT * k;  // 512 chunks of 16 bytes: [position][row][half]
        const int p = R16 ? id >> 5 : id >> 6, r = R16 ? (id >> 1) & 15 : (id >> 1) & 31, half = id & 1;
        if (q.p0 + p < a.P && q.r0 + r < a.R) {
          const uint4 val = *reinterpret_cast<const uint4*>(stage + id * 16);
          const long long e = (long long)(q.p0 + p) * a.out_stride_p + (long long)(q.r0 + r) * a.out_stride_r + q.c0 + 16 * half;
          store_codes16(a, e, val);
        }
      }
    }
    // the next iteration's __syncthreads (after its wait) orders these reads of `stage` / `red` before their reuse
  }
}

// Fallback for sources whose position axis is not a multiple of 4 elements (no 16-byte rows): one block per item.
// LINE: line blocks - one scale per (position, row, 32 channels) instead of one per tile; the 32 channels of a line sit in
// 16 lanes of each of two neighbouring warps (shuffles, then one exchange through shared memory).
template <int FMT, bool SR, bool LINE = false>
__global__ void __launch_bounds__(QT_THREADS) quantize_simple_kernel(QuantArgs a, int n_pstrips, int Ct) {
  __shared__ __align__(16) unsigned red[8][2][4];
  __shared__ unsigned lred[LINE ? 8 : 1][2][8][4];
  __shared__ __align__(16) uint8_t stage[PS][32][32];   // one code per byte
  pdl_wait();
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  const Item q = item_of(blockIdx.x, n_pstrips, Ct);
  const int quad = t & 1, c = (t >> 1) & 31, rsub = t >> 6;
  const int pq = q.p0 + 4 * quad;
  float v[8][4];
  const bool c_ok = (q.c0 + c) < a.C;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int r = q.r0 + 4 * i + rsub;
    const bool ok = c_ok && r < a.R;
    const float* row = a.src + ((long long)r * a.C + (q.c0 + c)) * a.P;
#pragma unroll
    for (int j = 0; j < 4; ++j) v[i][j] = (ok && pq + j < a.P) ? __ldg(row + pq + j) : 0.f;
  }
  int code[LINE ? 8 : 1][4];
  if (LINE) {
    unsigned lm[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        unsigned mm = __float_as_uint(v[i][j]) & 0x7fffffffu;
#pragma unroll
        for (int off = 2; off < 32; off <<= 1) mm = max(mm, __shfl_xor_sync(0xffffffffu, mm, off));
        lm[i][j] = mm;
      }
    if (lane < 2) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) lred[warp][lane][i][j] = lm[i][j];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        code[i][j] = scale_code_of(max(lm[i][j], lred[warp ^ 1][quad][i][j]), fmt_emax(FMT));
        // the line's first channel sits in an even warp, lanes 0 (quad 0) and 1 (quad 1)
        if (c == 0 && q.p0 + 4 * quad + j < a.P && q.r0 + 4 * i + rsub < a.R)
          a.scales[(long long)(q.p0 + 4 * quad + j) * a.sc_stride_p + (long long)(q.r0 + 4 * i + rsub) * a.sc_stride_r + q.ct] = (uint8_t)code[i][j];
      }
  } else {
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
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      unsigned mm = 0;
#pragma unroll
      for (int w = 0; w < 8; ++w) mm = max(mm, red[w][quad][j]);
      code[0][j] = scale_code_of(mm, fmt_emax(FMT));
    }
    if (t < PS) {
      unsigned mm = 0;
#pragma unroll
      for (int w = 0; w < 8; ++w) mm = max(mm, red[w][t >> 2][t & 3]);
      if (q.p0 + t < a.P)
        a.scales[(long long)(q.p0 + t) * a.sc_stride_p + (long long)q.rt * a.sc_stride_r + q.ct] = (uint8_t)scale_code_of(mm, fmt_emax(FMT));
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j) {
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      float x0 = v[i][j] * scale_factor(code[LINE ? i : 0][j]), x1 = v[i + 1][j] * scale_factor(code[LINE ? i + 1 : 0][j]);
      if (SR) {
        const long long e0 = ((long long)(q.r0 + 4 * i + rsub) * a.C + (q.c0 + c)) * a.P + pq + j;
        const long long e1 = e0 + 4ll * a.C * a.P;
        x0 = sr_value<FMT>(x0, (unsigned)e0, sr_key(a, e0));
        x1 = sr_value<FMT>(x1, (unsigned)e1, sr_key(a, e1));
      }
      const unsigned two = encode2<FMT>(x0, x1);
      unsigned lo, hi;
      if (FMT == MQ_E2M1) { lo = two & 0xF; hi = (two >> 4) & 0xF; }
      else { lo = two & 0xFF; hi = (two >> 8) & 0xFF; }
      stage[4 * quad + j][4 * i + rsub][c] = (uint8_t)lo;
      stage[4 * quad + j][4 * (i + 1) + rsub][c] = (uint8_t)hi;
    }
  }
  __syncthreads();
  if (FMT == MQ_E2M1) {
    const int p = t >> 5, r = t & 31;
    if (q.p0 + p < a.P && q.r0 + r < a.R) {
      const uint4* srcw = reinterpret_cast<const uint4*>(&stage[p][r][0]);
      const uint4 lo = srcw[0], hi = srcw[1];
      const uint32_t in[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
      uint32_t outw[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        // 8 one-byte codes (two words) -> one word of 8 nibbles, lower index in the lower nibble
        const uint32_t w0 = in[2 * k], w1 = in[2 * k + 1];
        const uint32_t b0 = (w0 & 0xF) | ((w0 >> 4) & 0xF0) | ((w0 >> 8) & 0xF00) | ((w0 >> 12) & 0xF000);
        const uint32_t b1 = (w1 & 0xF) | ((w1 >> 4) & 0xF0) | ((w1 >> 8) & 0xF00) | ((w1 >> 12) & 0xF000);
        outw[k] = b0 | (b1 << 16);
      }
      const long long e = (long long)(q.p0 + p) * a.out_stride_p + (long long)(q.r0 + r) * a.out_stride_r + q.c0;
      *reinterpret_cast<uint4*>(a.codes + (e >> 1)) = make_uint4(outw[0], outw[1], outw[2], outw[3]);
    }
  } else {
#pragma unroll
    for (int k = 0; k < 2; ++k) {
      const int id = t + QT_THREADS * k;
      const int p = id >> 6, r = (id >> 1) & 31, half = id & 1;
      if (q.p0 + p < a.P && q.r0 + r < a.R) {
        const uint4 val = *reinterpret_cast<const uint4*>(&stage[p][r][16 * half]);
        const long long e = (long long)(q.p0 + p) * a.out_stride_p + (long long)(q.r0 + r) * a.out_stride_r + q.c0 + 16 * half;
        store_codes16(a, e, val);
      }
    }
  }
}


// ---- NCHW / OIHW source through TMA: whole 128-byte lines ---------------------------------------------------------
// A work item is one 32(r) x 32(c) tile at 32 consecutive positions: 1024 source rows of 128 bytes, so every global
// request is a full line.  The item arrives as up to four TMA boxes of 8 rows x 32 channels x 32 positions (32 KB,
// zero fill outside the tensor) in a ring of six slots fed by a loader warp.  Sixteen consumer warps take a box into
// REGISTERS as soon as it lands (lane = position, so the reads are conflict-free and a position's amax needs no
// shuffle: per-thread max, then one exchange across the 16 warps) and hand the slot back at once, so the ring keeps
// ~190 KB in flight per SM while the tile (64 values per thread) is scaled, converted with the hardware RNE + saturate
// conversions and laid out in a staging buffer [position][row][32 channels], which one TMA store (box = the tile's
// codes at 32 positions, clipped to the tensor) writes out.  Which (row, channel half) a thread takes is permuted by
// its lane, so that the 16-byte staging writes of a quarter-warp fall into different banks.
constexpr int TQ_CONSUMERS = 512;
constexpr int TQ_THREADS = TQ_CONSUMERS + 32;
constexpr int TQ_SLOTS = 6;
constexpr int TQ_BOX_FLOATS = 8 * 32 * 32;
constexpr int TQ_BOX_BYTES = TQ_BOX_FLOATS * 4;
constexpr int TQ_STAGE_BYTES = 32 * 32 * 32;
constexpr size_t TQ_SMEM = 128 + (size_t)TQ_SLOTS * TQ_BOX_BYTES + TQ_STAGE_BYTES + 16 * 32 * 4 + 2 * TQ_SLOTS * 8 + 16;

__device__ __forceinline__ bool mbar_wait_limit(uint64_t* bar, uint32_t parity, uint32_t limit, unsigned int* status, unsigned int tag) {
#pragma unroll 1
  for (uint32_t i = 0; i < limit; ++i) {
    if (tc::mbar_try_wait(bar, parity)) return true;
  }
  if (status) atomicMax(status, tag);
  return false;
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(TQ_CONSUMERS) : "memory"); }

// channel tile fastest (as item_of): the tiles that share an output line are produced together.  (Position strip fastest,
// so that neighbouring strips of the same source rows are read together, measured 0.69 against 0.77 of the copy rate on a
// 1.6 GB tensor and 0.78 against 0.72 on a 0.4 GB one: not kept.)
__device__ __forceinline__ Item tq_item_of(unsigned it, int n_pstrips, int Ct) { return item_of(it, n_pstrips, Ct, 32); }

// LINE: line blocks.  A line (32 channels of one row at one position) is held by two threads of neighbouring warps; they
// exchange their maxima through the (still unused) staging buffer and the one with the lower channels writes the scale.
// TS: the paper's own format (Eq. 4-6) - E2M1 elements, one E4M3 scale per 16 samples x 16 channels at a position, an
// fp32 scale per tensor.  A thread's 4 x 16 values are 2 x 16 of the block (samples 0-15, its channel half) and 2 x 16
// of the block 16 samples further; the 8 warps that hold the other samples of the same channel half are those of
// this warp's parity.  Every operation of Eq. 4-6 is one IEEE single-precision operation in the order written.
template <int FMT, bool SR, bool LINE, bool TS = false>
__global__ void __launch_bounds__(TQ_THREADS, 1)
quantize_tma_kernel(const __grid_constant__ CUtensorMap map_in, const __grid_constant__ CUtensorMap map_out, QuantArgs a, int n_pstrips, int Ct,
                    unsigned n_items) {
  extern __shared__ uint8_t tq_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tq_raw) + 127) & ~(uintptr_t)127);
  float* ring = reinterpret_cast<float*>(base);
  uint8_t* stage = base + (size_t)TQ_SLOTS * TQ_BOX_BYTES;
  unsigned* red = reinterpret_cast<unsigned*>(stage + TQ_STAGE_BYTES);
  uint64_t* full = reinterpret_cast<uint64_t*>(red + 16 * 32);
  uint64_t* empty = full + TQ_SLOTS;
  volatile unsigned* abort_flag = reinterpret_cast<volatile unsigned*>(empty + TQ_SLOTS);
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  const uint32_t limit = a.wait_limit ? a.wait_limit : tc::kWaitLimit;
  if (t == 0) {
    for (int s = 0; s < TQ_SLOTS; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 16); }
    *abort_flag = 0;
    tc::mbar_fence_init();
    tc::prefetch_tensormap(&map_in);
    tc::prefetch_tensormap(&map_out);
  }
  __syncthreads();
  pdl_wait();
  if (warp == 16) {
    // ---- loader: one lane arms a slot and issues its box as soon as the consumers have emptied it
    if (lane == 0) {
      int slot = 0;
      unsigned uses[TQ_SLOTS] = {0, 0, 0, 0, 0, 0};
      bool ok = true;
#pragma unroll 1
      for (unsigned it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
        const Item q = tq_item_of(it, n_pstrips, Ct);
        const int nb = min(4, (a.R - q.r0 + 7) >> 3);
#pragma unroll 1
        for (int b = 0; b < nb; ++b) {
          unsigned u = 0;
#pragma unroll
          for (int s = 0; s < TQ_SLOTS; ++s) u = s == slot ? uses[s] : u;
          if (*abort_flag) { ok = false; break; }
          if (u > 0 && !mbar_wait_limit(&empty[slot], (u - 1) & 1, limit, a.status, MQ_ERR_TIMEOUT)) { ok = false; break; }
          if (!a.debug_skip_loads) {
            tc::mbar_arrive_expect_tx(&full[slot], TQ_BOX_BYTES);
            tc::tma_load_3d(ring + (size_t)slot * TQ_BOX_FLOATS, &map_in, &full[slot], q.p0, q.c0, q.r0 + 8 * b);
#pragma unroll
            for (int s = 0; s < TQ_SLOTS; ++s) uses[s] += s == slot ? 1u : 0u;
          }
          slot = slot + 1 == TQ_SLOTS ? 0 : slot + 1;
        }
      }
      // on the way out (a wait gave up somewhere): let the copies still in flight land before the block's memory goes
      if (!ok || *abort_flag) {
#pragma unroll
        for (int s = 0; s < TQ_SLOTS; ++s)
          if (uses[s] > 0) mbar_wait_limit(&full[s], (uses[s] - 1) & 1, limit, a.status, MQ_ERR_TIMEOUT);
      }
    }
  } else {
    // ---- consumers
    const int n_sub = (warp >> 1) ^ ((lane >> 1) & 7);   // row within a box
    const int chalf = (warp & 1) ^ (lane & 1);           // which 16 of the tile's 32 channels
    const float* rd = ring + (n_sub * 32 + chalf * 16) * 32 + lane;
    constexpr int CB = FMT == MQ_E2M1 ? 8 : 16;          // bytes of 16 codes
    int slot = 0;
    unsigned phase = 0;
    bool dead = false;
    float tscale = 0.f, t6 = 0.f;
    unsigned own_max = 0;     // TS: bit pattern of the largest block maximum this thread has seen
    if (TS) {
      tscale = __fdiv_rn(*a.ts_amax, __fmul_rn(448.0f, 6.0f));                                  // Eq. 4
      t6 = __fmul_rn(tscale, 6.0f);
      if (blockIdx.x == 0 && t == 0) a.ts_stats[0] = tscale;
    }
#pragma unroll 1
    for (unsigned it = blockIdx.x; it < n_items; it += gridDim.x) {
      const Item q = tq_item_of(it, n_pstrips, Ct);
      const int nb = min(4, (a.R - q.r0 + 7) >> 3);
      float v[4][16];
      float fm = 0.f;
      float lm[(LINE || TS) ? 4 : 1];
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        if (LINE || TS) { lm[b] = 0.f; }
        if (b < nb) {
          if (!dead && !mbar_wait_limit(&full[slot], phase, limit, a.status, MQ_ERR_TIMEOUT)) { dead = true; *abort_flag = 1; }
          const float* src = rd + (size_t)slot * TQ_BOX_FLOATS;
#pragma unroll
          for (int k = 0; k < 16; ++k) {
            v[b][k] = src[k * 32];
            if (LINE || TS) lm[b] = fmaxf(lm[b], fabsf(v[b][k])); else fm = fmaxf(fm, fabsf(v[b][k]));
          }
          __syncwarp();
          if (lane == 0) tc::mbar_arrive(&empty[slot]);
          if (++slot == TQ_SLOTS) { slot = 0; phase ^= 1; }
        } else {
#pragma unroll
          for (int k = 0; k < 16; ++k) v[b][k] = 0.f;
        }
      }
      if (!LINE && !TS) red[warp * 32 + lane] = __float_as_uint(fm);
      if (t == 0) tc::bulk_wait_group_read<0>();    // the previous item's store has read the staging buffer
      consumer_sync();
      if (*abort_flag) break;    // uniform: written only between the previous item's last barrier and the one above
      int code[LINE ? 4 : 1];
      float den[2] = {0.f, 0.f};   // TS: Scale_b * T_scale of the thread's two blocks (0: the block encodes to signed zeros)
      if (TS) {
        unsigned* xch = reinterpret_cast<unsigned*>(stage);   // [sample half][warp][lane]
        xch[warp * 32 + lane] = __float_as_uint(fmaxf(lm[0], lm[1]));
        xch[(16 + warp) * 32 + lane] = __float_as_uint(fmaxf(lm[2], lm[3]));
        consumer_sync();
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          unsigned mx = 0;
#pragma unroll
          for (int k = 0; k < 8; ++k) mx = max(mx, xch[(16 * hf + (warp & 1) + 2 * k) * 32 + lane]);
          const float bmax = __uint_as_float(mx);
          own_max = max(own_max, mx);
          unsigned sc = 0;
          if (bmax > 0.f && tscale > 0.f) sc = (unsigned)__nv_cvt_float_to_fp8(__fdiv_rn(bmax, t6), __NV_SATFINITE, __NV_E4M3) & 0x7Fu;   // Eq. 5
          const __half_raw hr = __nv_cvt_fp8_to_halfraw((__nv_fp8_storage_t)sc, __NV_E4M3);
          const float bscale = __half2float(*reinterpret_cast<const __half*>(&hr));
          den[hf] = (bscale > 0.f && tscale > 0.f) ? __fmul_rn(bscale, tscale) : 0.f;
          // one thread per (position, sample half, channel half): warps 0 and 1 hold both channel halves of every position
          if ((warp >> 1) == 0 && q.p0 + lane < a.P && q.r0 + 16 * hf < a.R)
            a.scales[(long long)(q.p0 + lane) * a.sc_stride_p + (long long)(2 * q.rt + hf) * a.sc_stride_r + 2 * q.ct + chalf] = (uint8_t)sc;
        }
        consumer_sync();    // every exchange word has been read before the codes overwrite the buffer
      } else if (LINE) {
        unsigned* xch = reinterpret_cast<unsigned*>(stage);   // [box][warp][lane]
#pragma unroll
        for (int b = 0; b < 4; ++b) xch[(b * 16 + warp) * 32 + lane] = __float_as_uint(lm[b]);
        consumer_sync();
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          code[b] = scale_code_of(max(__float_as_uint(lm[b]), xch[(b * 16 + (warp ^ 1)) * 32 + lane]), fmt_emax(FMT));
          const int n = 8 * b + n_sub;
          if (b < nb && chalf == 0 && q.p0 + lane < a.P && q.r0 + n < a.R)
            a.scales[(long long)(q.p0 + lane) * a.sc_stride_p + (long long)(q.r0 + n) * a.sc_stride_r + q.ct] = (uint8_t)code[b];
        }
        consumer_sync();    // every exchange word has been read before the codes overwrite the buffer
      } else {
        unsigned mx = 0;
#pragma unroll
        for (int w = 0; w < 16; ++w) mx = max(mx, red[w * 32 + lane]);
        code[0] = scale_code_of(mx, fmt_emax(FMT));
        if (warp == 0 && q.p0 + lane < a.P)
          a.scales[(long long)(q.p0 + lane) * a.sc_stride_p + (long long)q.rt * a.sc_stride_r + q.ct] = (uint8_t)code[0];
      }
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        if (b < nb) {
          const float f = TS ? 0.f : scale_factor(code[LINE ? b : 0]);
          const float dn = den[b >> 1];
          const int n = 8 * b + n_sub;
          unsigned w4[4];
#pragma unroll
          for (int k = 0; k < 16; k += 4) {
            float x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (TS) x[j] = ts_div(v[b][k + j], dn);   // Eq. 6
              else x[j] = v[b][k + j] * f;
              if (SR && (!TS || dn > 0.f)) {
                const long long e = ((long long)(q.r0 + n) * a.C + q.c0 + chalf * 16 + k + j) * a.P + q.p0 + lane;
                x[j] = sr_value<FMT>(x[j], (unsigned)e, sr_key(a, e));
              }
            }
            const unsigned lo = encode2<FMT>(x[0], x[1]), hi = encode2<FMT>(x[2], x[3]);
            w4[k >> 2] = FMT == MQ_E2M1 ? (lo | (hi << 8)) : (lo | (hi << 16));
          }
          uint8_t* dst = stage + (lane * 32 + n) * (2 * CB) + chalf * CB;
          if (FMT == MQ_E2M1) *reinterpret_cast<uint2*>(dst) = make_uint2(w4[0] | (w4[1] << 16), w4[2] | (w4[3] << 16));
          else *reinterpret_cast<uint4*>(dst) = make_uint4(w4[0], w4[1], w4[2], w4[3]);
        }
      }
      tc::fence_proxy_async_smem();
      consumer_sync();
      if ((FMT == MQ_E3M2 || FMT == MQ_E2M3) && a.packed6) {
        // packed 6-bit storage: a row of the tile is 24 bytes - no TMA box.  Each thread packs two rows in place (32 -> 24
        // bytes of their slot), then the rows leave as 8-byte pieces, three neighbouring lanes per row, so that a row is one
        // request (the next item's first barrier orders these reads before the buffer is written again)
#pragma unroll
        for (int k = 0; k < 2; ++k) {
          uint4* sp = reinterpret_cast<uint4*>(stage + (t + TQ_CONSUMERS * k) * 32);
          const uint4 v0 = sp[0], v1 = sp[1];
          const uint32_t w0[4] = {v0.x, v0.y, v0.z, v0.w}, w1[4] = {v1.x, v1.y, v1.z, v1.w};
          uint32_t o0[3], o1[3];
          pack6x16(w0, o0);
          pack6x16(w1, o1);
          sp[0] = make_uint4(o0[0], o0[1], o0[2], o1[0]);
          *reinterpret_cast<uint2*>(sp + 1) = make_uint2(o1[1], o1[2]);
        }
        consumer_sync();
#pragma unroll
        for (int k = 0; k < 6; ++k) {
          const int id = t + TQ_CONSUMERS * k, row = id / 3, piece = id - 3 * row, p = row >> 5, n = row & 31;
          if (q.p0 + p < a.P && q.r0 + n < a.R) {
            const long long e = (long long)(q.p0 + p) * a.out_stride_p + (long long)(q.r0 + n) * a.out_stride_r + q.c0;
            *reinterpret_cast<uint2*>(a.codes + (e >> 4) * 12 + 8 * piece) = *reinterpret_cast<const uint2*>(stage + row * 32 + 8 * piece);
          }
        }
      } else if (t == 0) {
        // codes of the tile at 32 positions: box (32 channels, 32 rows, 32 positions), clipped to the tensor
        tc::tma_store_3d(&map_out, stage, q.c0 * (FMT == MQ_E2M1 ? 4 : 8) / 8, q.r0, q.p0);
        tc::bulk_commit_group();
      }
    }
    if (t == 0) tc::bulk_wait_group_all();
    if (TS && a.ts_track_max) {   // the tensor's own maximum for the next step (Sec. VII-B): one atomic per warp
      const unsigned wmax = __reduce_max_sync(0xffffffffu, own_max);
      if (lane == 0 && wmax != 0) atomicMax(reinterpret_cast<unsigned*>(a.ts_stats + 1), wmax);
    }
  }
  __syncthreads();
}

// ---- channel-fastest source ([H][W][N][C] activations / gradients, [Cout][Kh][Kw][Cin] weights) ------------------
// No re-layout is needed: a tile's 32 rows are runs of 32 consecutive floats.  One warp per (position, tile): lane
// (cq, rq) = (lane & 7, lane >> 3) loads 4 adjacent channels of rows rq, rq + 4, ... as one 128-bit load each (8 in
// flight), the amax is a per-lane max plus one redux.sync, and the codes leave as 32-bit words (FP8) or, pairing
// neighbouring lanes, 32-bit words of 8 E2M1 codes.  VEC = false takes any C and alignment with scalar loads.
template <int FMT, bool VEC, bool SR, bool LINE = false>   // LINE: one scale per row of the tile (line blocks), reduced over the 8 lanes of a row
__global__ void __launch_bounds__(256) quantize_cfast_kernel(QuantArgs a, unsigned Rt, unsigned Ct, unsigned n_items) {
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const int cq = lane & 7, rq = lane >> 3;
#pragma unroll 1
  for (unsigned it = blockIdx.x * 8u + (threadIdx.x >> 5); it < n_items; it += gridDim.x * 8u) {
    // channel tile fastest, then row tile, then position: consecutive warps read consecutive memory
    const unsigned ct = it % Ct; const unsigned u = it / Ct;
    const unsigned rt = u % Rt; const unsigned pos = u / Rt;
    const int r0 = (int)rt * 32 + rq, c0 = (int)ct * 32 + 4 * cq;
    const float* src = a.src + (long long)pos * a.src_stride_p + (long long)r0 * a.src_stride_r + c0;
    float4 v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      const float* q = src + (long long)(4 * i) * a.src_stride_r;
      if (r0 + 4 * i < a.R) {
        if (VEC) { if (c0 < a.C) v[i] = __ldg(reinterpret_cast<const float4*>(q)); }   // C % 4 == 0: whole quads
        else {
          if (c0 + 0 < a.C) v[i].x = __ldg(q + 0);
          if (c0 + 1 < a.C) v[i].y = __ldg(q + 1);
          if (c0 + 2 < a.C) v[i].z = __ldg(q + 2);
          if (c0 + 3 < a.C) v[i].w = __ldg(q + 3);
        }
      }
    }
    if (a.act) {
#pragma unroll
      for (int i = 0; i < 8; ++i)
        v[i] = make_float4(mx_activation(v[i].x, a.act), mx_activation(v[i].y, a.act), mx_activation(v[i].z, a.act), mx_activation(v[i].w, a.act));
    }
    int code[LINE ? 8 : 1];
    if (LINE) {
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        unsigned mm = __float_as_uint(fmaxf(fmaxf(fabsf(v[i].x), fabsf(v[i].y)), fmaxf(fabsf(v[i].z), fabsf(v[i].w))));
        mm = max(mm, __shfl_xor_sync(0xffffffffu, mm, 1));
        mm = max(mm, __shfl_xor_sync(0xffffffffu, mm, 2));
        mm = max(mm, __shfl_xor_sync(0xffffffffu, mm, 4));
        code[i] = scale_code_of(mm, fmt_emax(FMT));
        if (cq == 0 && r0 + 4 * i < a.R) a.scales[(long long)pos * a.sc_stride_p + (long long)(r0 + 4 * i) * a.sc_stride_r + ct] = (uint8_t)code[i];
      }
    } else {
      float m = 0.f;
#pragma unroll
      for (int i = 0; i < 8; ++i) m = fmaxf(fmaxf(m, fmaxf(fabsf(v[i].x), fabsf(v[i].y))), fmaxf(fabsf(v[i].z), fabsf(v[i].w)));
      code[0] = scale_code_of(__reduce_max_sync(0xffffffffu, __float_as_uint(m)), fmt_emax(FMT));
      if (lane == 0) a.scales[(long long)pos * a.sc_stride_p + (long long)rt * a.sc_stride_r + ct] = (uint8_t)code[0];
    }
    const long long pbase = (long long)pos * a.out_stride_p + c0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int r = r0 + 4 * i;
      const float f = scale_factor(code[LINE ? i : 0]);
      float x[4] = {v[i].x * f, v[i].y * f, v[i].z * f, v[i].w * f};
      if (SR) {
        const long long e0 = ((long long)r * a.C + c0) * a.P + pos;    // index in the logical tensor, whatever the source order
#pragma unroll
        for (int k = 0; k < 4; ++k) x[k] = sr_value<FMT>(x[k], (unsigned)e0 + (unsigned)k * (unsigned)a.P, sr_key(a, e0 + (long long)k * a.P));
      }
      const unsigned lo = encode2<FMT>(x[0], x[1]), hi = encode2<FMT>(x[2], x[3]);
      const long long e = pbase + (long long)r * a.out_stride_r;
      if (FMT == MQ_E2M1) {
        const unsigned mine = lo | (hi << 8);                       // 4 codes; the odd lane's go above the even lane's
        const unsigned other = __shfl_xor_sync(0xffffffffu, mine, 1);
        if ((lane & 1) == 0 && r < a.R) *reinterpret_cast<unsigned*>(a.codes + (e >> 1)) = mine | (other << 16);
      } else if ((FMT == MQ_E3M2 || FMT == MQ_E2M3) && a.packed6) {
        // packed 6-bit storage: a lane's four codes are 24 bits; lanes 4j .. 4j+3 hold a 12-byte group, its word k written by
        // lane 4j + k from its own bits and the next lane's
        const unsigned w = lo | (hi << 16);
        const unsigned t24 = (w & 0x3Fu) | ((w >> 2) & 0xFC0u) | ((w >> 4) & 0x3F000u) | ((w >> 6) & 0xFC0000u);
        const unsigned nxt = __shfl_down_sync(0xffffffffu, t24, 1);
        const int k = lane & 3;
        if (k < 3 && r < a.R) {
          const long long e16 = (e - 4 * k) >> 4;    // the group's index
          *reinterpret_cast<unsigned*>(a.codes + e16 * 12 + 4 * k) = (t24 >> (8 * k)) | (nxt << (24 - 8 * k));
        }
      } else {
        if (r < a.R) *reinterpret_cast<unsigned*>(a.codes + e) = lo | (hi << 16);
      }
    }
  }
}

template <int FMT>
cudaError_t launch_q_cfast(const QuantArgs& a, int Ct, cudaStream_t s) {
  const long long Rt = (a.R + 31) / 32;
  const long long items = (long long)a.P * Rt * Ct;
  if (items <= 0 || items > 0xffffffffLL) return cudaErrorInvalidValue;
  const bool vec = a.C % 4 == 0 && a.src_stride_p % 4 == 0 && a.src_stride_r % 4 == 0 && (reinterpret_cast<uintptr_t>(a.src) & 15) == 0;
  long long blocks = (items + 7) / 8;
  if (blocks > (long long)sm_count() * 64) blocks = (long long)sm_count() * 64;
  if (a.line) {
    if (a.sr) {
      if (vec) return launch_pdl(quantize_cfast_kernel<FMT, true, true, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
      return launch_pdl(quantize_cfast_kernel<FMT, false, true, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
    }
    if (vec) return launch_pdl(quantize_cfast_kernel<FMT, true, false, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
    return launch_pdl(quantize_cfast_kernel<FMT, false, false, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
  }
  if (a.sr) {
    if (vec) return launch_pdl(quantize_cfast_kernel<FMT, true, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
    return launch_pdl(quantize_cfast_kernel<FMT, false, true>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
  }
  if (vec) return launch_pdl(quantize_cfast_kernel<FMT, true, false>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
  return launch_pdl(quantize_cfast_kernel<FMT, false, false>, dim3((unsigned)blocks), dim3(256), 0, s, a, (unsigned)Rt, (unsigned)Ct, (unsigned)items);
}


template <int FMT>
cudaError_t launch_q_tma(const QuantArgs& a, cudaStream_t s) {
  const int bits = fmt_bits(FMT);
  CUtensorMap map_in, map_out;
  {
    const uint64_t dims[3] = {(uint64_t)a.P, (uint64_t)a.C, (uint64_t)a.R};
    const uint64_t strides[2] = {(uint64_t)a.P * 4, (uint64_t)a.C * a.P * 4};
    const uint32_t box[3] = {32u, 32u, 8u};
    // whole lines, each wanted once: no promotion to 256-byte fetches (measured: 0.72 -> 0.77 of the copy rate on 1.6 GB)
    if (!encode_tensor_map_u8(&map_in, a.src, 3, dims, strides, box, nullptr, 0, true, 128)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)a.Cp * bits / 8, (uint64_t)a.R, (uint64_t)a.P};
    const uint64_t strides[2] = {(uint64_t)a.out_stride_r * bits / 8, (uint64_t)a.out_stride_p * bits / 8};
    const uint32_t box[3] = {(uint32_t)(32 * bits / 8), 32u, 32u};
    if (!encode_tensor_map_u8(&map_out, a.codes, 3, dims, strides, box, nullptr, 0)) return cudaErrorInvalidValue;
  }
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(quantize_tma_kernel<FMT, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_tma_kernel<FMT, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_tma_kernel<FMT, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_tma_kernel<FMT, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int n_pstrips = (a.P + 31) / 32, Rt = (a.R + 31) / 32, Ct = a.Cp / 32;
  const long long n_items = (long long)n_pstrips * Rt * Ct;
  if (n_items <= 0 || n_items > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int sms = sm_count();
  const unsigned grid = (unsigned)(n_items < sms ? n_items : sms);
  if (a.line) {
    if (a.sr) return launch_pdl(quantize_tma_kernel<FMT, true, true>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
    return launch_pdl(quantize_tma_kernel<FMT, false, true>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
  }
  if (a.sr) return launch_pdl(quantize_tma_kernel<FMT, true, false>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
  return launch_pdl(quantize_tma_kernel<FMT, false, false>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
}

constexpr size_t QPIPE_SMEM = 2 * QBUF_BYTES + PS * 32 * 32 + 16 * 2 * 4 * sizeof(unsigned);

template <int FMT>
cudaError_t launch_q(const QuantArgs& a, int n_pstrips, int Ct, long long n_items, bool vec, bool r16, cudaStream_t s) {
  if (a.line) {   // line blocks without 16-byte rows (large aligned tensors take the whole-line kernel): the one-block-per-item kernel
    if (a.sr) return launch_pdl(quantize_simple_kernel<FMT, true, true>, dim3((unsigned)n_items), dim3(QT_THREADS), 0, s, a, n_pstrips, Ct);
    return launch_pdl(quantize_simple_kernel<FMT, false, true>, dim3((unsigned)n_items), dim3(QT_THREADS), 0, s, a, n_pstrips, Ct);
  }
  if (!vec) {
    if (a.sr) return launch_pdl(quantize_simple_kernel<FMT, true>, dim3((unsigned)n_items), dim3(QT_THREADS), 0, s, a, n_pstrips, Ct);
    return launch_pdl(quantize_simple_kernel<FMT, false>, dim3((unsigned)n_items), dim3(QT_THREADS), 0, s, a, n_pstrips, Ct);
  }
  static bool attr_set = false;
  const int ctas_per_sm = 2;   // 80 KB of shared memory per block; 256 threads (512-thread blocks measured slower: bound by instruction issue)
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(quantize_pipe_kernel<FMT, 256, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QPIPE_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_pipe_kernel<FMT, 256, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QPIPE_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_pipe_kernel<FMT, 256, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QPIPE_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_pipe_kernel<FMT, 256, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)QPIPE_SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int sms = sm_count();
  long long grid = (long long)sms * ctas_per_sm;
  if (grid > n_items) grid = n_items;
  if (r16 && a.sr) return launch_pdl(quantize_pipe_kernel<FMT, 256, true, true>, dim3((unsigned)grid), dim3(256), QPIPE_SMEM, s, a, n_pstrips, Ct, (unsigned)n_items);
  if (r16) return launch_pdl(quantize_pipe_kernel<FMT, 256, false, true>, dim3((unsigned)grid), dim3(256), QPIPE_SMEM, s, a, n_pstrips, Ct, (unsigned)n_items);
  if (a.sr) return launch_pdl(quantize_pipe_kernel<FMT, 256, true>, dim3((unsigned)grid), dim3(256), QPIPE_SMEM, s, a, n_pstrips, Ct, (unsigned)n_items);
  return launch_pdl(quantize_pipe_kernel<FMT, 256, false>, dim3((unsigned)grid), dim3(256), QPIPE_SMEM, s, a, n_pstrips, Ct, (unsigned)n_items);
}

}  // namespace

bool quantize_ts_tma_eligible(const QuantArgs& a) {
  const bool vec = (a.P % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.src) & 15) == 0);
  const long long elems = (long long)a.P * a.R * a.C;
  const int tv = env_int("MQ_QUANT_TMA", -1);   // 1 / 0 force the choice
  return vec && a.src_stride_r == 0 && a.fmt == MQ_E2M1 && (tv >= 0 ? tv != 0 : elems >= (1ll << 22));
}

cudaError_t launch_quantize_ts_tma(const QuantArgs& a0, const float* amax_src, float* stats, cudaStream_t s, bool track_max) {
  QuantArgs a = a0;
  a.ts_amax = amax_src; a.ts_stats = stats; a.ts_track_max = track_max ? 1 : 0;
  CUtensorMap map_in, map_out;
  {
    const uint64_t dims[3] = {(uint64_t)a.P, (uint64_t)a.C, (uint64_t)a.R};
    const uint64_t strides[2] = {(uint64_t)a.P * 4, (uint64_t)a.C * a.P * 4};
    const uint32_t box[3] = {32u, 32u, 8u};
    if (!encode_tensor_map_u8(&map_in, a.src, 3, dims, strides, box, nullptr, 0, true, 128)) return cudaErrorInvalidValue;
  }
  {
    const uint64_t dims[3] = {(uint64_t)a.Cp / 2, (uint64_t)a.R, (uint64_t)a.P};
    const uint64_t strides[2] = {(uint64_t)a.out_stride_r / 2, (uint64_t)a.out_stride_p / 2};
    const uint32_t box[3] = {16u, 32u, 32u};
    if (!encode_tensor_map_u8(&map_out, a.codes, 3, dims, strides, box, nullptr, 0)) return cudaErrorInvalidValue;
  }
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(quantize_tma_kernel<MQ_E2M1, false, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(quantize_tma_kernel<MQ_E2M1, true, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TQ_SMEM);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  const int n_pstrips = (a.P + 31) / 32, Rt = (a.R + 31) / 32, Ct = a.Cp / 32;
  const long long n_items = (long long)n_pstrips * Rt * Ct;
  if (n_items <= 0 || n_items > 0x7fffffffLL) return cudaErrorInvalidValue;
  const int sms = sm_count();
  const unsigned grid = (unsigned)(n_items < sms ? n_items : sms);
  if (a.sr) return launch_pdl(quantize_tma_kernel<MQ_E2M1, true, false, true>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
  return launch_pdl(quantize_tma_kernel<MQ_E2M1, false, false, true>, dim3(grid), dim3(TQ_THREADS), TQ_SMEM, s, map_in, map_out, a, n_pstrips, Ct, (unsigned)n_items);
}

cudaError_t launch_quantize(const QuantArgs& a, cudaStream_t s) {
  const bool vec = (a.P % 4 == 0) && ((reinterpret_cast<uintptr_t>(a.src) & 15) == 0);
  // at most 16 rows (e.g. a batch of 16 samples): items of 16 positions, see quantize_pipe_kernel
  const bool r16 = vec && !a.line && a.src_stride_r == 0 && a.R <= 16 && !env_int("MQ_QUANT_NO_R16", 0);
  const int psi = r16 ? 2 * PS : PS;
  const int n_pstrips = (a.P + psi - 1) / psi;
  const int Rt = (a.R + 31) / 32, Ct = a.Cp / 32;
  const long long n_items = (long long)n_pstrips * Rt * Ct;
  if (n_items <= 0 || n_items > 0x7fffffffLL) return cudaErrorInvalidValue;
  cudaError_t e;
  if (a.src_stride_r != 0) {   // channel-fastest source
    switch (a.fmt) {
      case MQ_E4M3: e = launch_q_cfast<MQ_E4M3>(a, Ct, s); break;
      case MQ_E5M2: e = launch_q_cfast<MQ_E5M2>(a, Ct, s); break;
      case MQ_E2M1: e = launch_q_cfast<MQ_E2M1>(a, Ct, s); break;
      case MQ_E3M2: e = launch_q_cfast<MQ_E3M2>(a, Ct, s); break;
      case MQ_E2M3: e = launch_q_cfast<MQ_E2M3>(a, Ct, s); break;
      default: return cudaErrorInvalidValue;
    }
    count_launches(1);
    return e;
  }
  // large tensors with 16-byte rows: whole-line TMA boxes (items of 32 positions); small ones keep the 8-position items,
  // which give a small tensor more blocks to spread over
  const long long elems = (long long)a.P * a.R * a.C;
  const int tv = env_int("MQ_QUANT_TMA", -1);   // 1 / 0 force the choice
  const bool tma = vec && (a.debug_skip_loads || (tv >= 0 ? tv != 0 : (elems >= (1ll << 22) || (a.line && elems >= (1ll << 18)))));
  if (a.debug_skip_loads && !tma) return cudaErrorInvalidValue;
  if (tma) {
    switch (a.fmt) {
      case MQ_E4M3: e = launch_q_tma<MQ_E4M3>(a, s); break;
      case MQ_E5M2: e = launch_q_tma<MQ_E5M2>(a, s); break;
      case MQ_E2M1: e = launch_q_tma<MQ_E2M1>(a, s); break;
      case MQ_E3M2: e = launch_q_tma<MQ_E3M2>(a, s); break;
      case MQ_E2M3: e = launch_q_tma<MQ_E2M3>(a, s); break;
      default: return cudaErrorInvalidValue;
    }
    count_launches(1);
    return e;
  }
  switch (a.fmt) {
    case MQ_E4M3: e = launch_q<MQ_E4M3>(a, n_pstrips, Ct, n_items, vec, r16, s); break;
    case MQ_E5M2: e = launch_q<MQ_E5M2>(a, n_pstrips, Ct, n_items, vec, r16, s); break;
    case MQ_E2M1: e = launch_q<MQ_E2M1>(a, n_pstrips, Ct, n_items, vec, r16, s); break;
    case MQ_E3M2: e = launch_q<MQ_E3M2>(a, n_pstrips, Ct, n_items, vec, r16, s); break;
    case MQ_E2M3: e = launch_q<MQ_E2M3>(a, n_pstrips, Ct, n_items, vec, r16, s); break;
    default: return cudaErrorInvalidValue;
  }
  count_launches(1);
  return e;
}

}  // namespace mq
