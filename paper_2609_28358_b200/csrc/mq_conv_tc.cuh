// Declarations shared by the tensor-core (tcgen05) convolution GEMM kernels and their host side.
#pragma once

#include <cuda.h>  // CUtensorMap (types only; the encoder is fetched through the runtime)

#include "mq_internal.cuh"

namespace mq {

// Parameters of the persistent implicit-GEMM kernel that serves mq_conv_fwd and mq_conv_bwd_data.
//
// GEMM view: D[(y, x, n)][c] = sum over taps and K-blocks of A[(y', x', n)][k] * B[c][tap][k], where
// A is a stored activation-like tensor ([Hs][Ws][N][Kp] codes, fwd: X, bwd_data: G_Y) gathered at a
// tap-dependent pixel, and B is a stored weight-like tensor ([rows][taps][Kp] codes, fwd: W,
// bwd_data: W re-laid as [C_in_p][taps][C_out_p]).
struct ConvTcParams {
  int mode;             // MQ_OP_FWD or MQ_OP_BWD_DATA
  int line;             // 1: line-block scales (forward only): a_scales [Hs][Ws][N][Kblocks], b_scales [rows][taps][Kblocks]
  int kind_fp4;         // 0: 8-bit formats (kind::mxf8f6f4, one E8M0 scale per 32 elements); 1: both operands E2M1 (kind::mxf4, E8M0 per 32);
                        // 2: both E2M1 with one E4M3 scale per 16 x 16 block and an fp32 scale per tensor (kind::mxf4nvf4, Eq. 4-6)
  const float* a_tscale;    // kind 2: the two tensors' fp32 scales (device); the epilogue multiplies the accumulator by their product
  const float* b_tscale;
  uint32_t idesc;       // instruction descriptor without scale ids
  int KB;               // bytes of K per row per TMA box: 128, 64 or 32 (= swizzle span)
  int G;                // boxes (chunks) per pipeline stage = 128 / KB
  int cpt;              // chunks per tap = row bytes / KB
  int BN;               // output channels per tile (multiple of 16, <= 256)
  int stages;
  int n_acc;            // accumulator buffers in TMEM (1 or 2)
  int TW, TN, lgTW, lgTN;  // tile = TW output columns x TN samples (TW * TN = 128), TW fastest among rows
  // geometry
  int N, Nt;
  int Hs, Ws;           // spatial extent of the gathered source (fwd: H, W; bwd_data: Ho, Wo)
  int Kblocks;          // 32-element K-blocks per tap (source channels / 32)
  int Hd, Wd;           // spatial extent of the output (fwd: Ho, Wo; bwd_data: H, W)
  int Cd;               // output channels (fwd: C_out; bwd_data: C_in)
  int Kh, Kw, sh, sw, ph, pw;
  // tiles
  int tiles_c, tiles_w, tiles_n, tiles_h, classes;  // classes = sh*sw parity classes (bwd_data), else 1
  long long total_tiles;
  uint32_t m_classes, m_tiles_w, m_tiles_h, m_tiles_c, m_sh, m_sw;   // ceil(2^32 / d) for the divisions by these (0: divide)
  // scales
  const uint8_t* a_scales;  // [Hs][Ws][Nt][Kblocks]
  const uint8_t* b_scales;  // [row blocks of 32][taps][Kblocks]
  // per-stage scale-vector chunks expanded by expand_conv_scales (scratch)
  uint8_t* sfa_img;         // [tile without the channel index][max_stages][512 * SPA]
  uint8_t* sfb_img;         // [class][channel tile][max_stages][512 * SPA * atoms_b]
  int max_stages;           // stages of the longest tile
  int sfa_dedup;            // 1: A-side chunks are stored once per (sample tile, source row, column tile, kw, chunk) - unit strides, one
                            // chunk per stage: tiles on neighbouring output rows read the same source row through different kh
  int sfa_hk;               // source-row keys per sample tile = output rows + Kh - 1
  // whole-tile-per-stage variant (small channel counts, stride 1): see conv_tc_halo_kernel
  int halo;                 // 1: use it
  int WH;                   // columns of the activation halo box = TW + Kw - 1
  int duo;                  // 1: clusters of two blocks on 256 x 256 tiles (cta_group::2), each loading half of the weight tile
  int snap;                 // 1: 256-column tiles, direct fp32 stores: the epilogue copies the accumulator into registers and frees it before storing
  int a_tx34;               // 1: the activation boxes come from packed 6-bit storage - a box counts 3/4 of its shared-memory bytes on the barrier
  int halo_box_bytes;       // bytes of one activation box = Kh * TN * WH * KB
  int halo_a_bytes;         // bytes of a tile's activation boxes (rounded up to 1024)
  int halo_stage_bytes;     // bytes of one pipeline stage (activation boxes + A-side scale chunks)
  int halo_b_bytes;         // bytes of the resident weight image + its scale chunks (rounded up to 1024)
  int fused;                // 1: single channel tile, stride 1: no preparation kernel (the blocks build the weight image, its
                            //    scale chunks and every tile's activation scale chunks themselves)
  int mma_cp;             // E2M1: 1 = the MMA lane issues the scale copies itself (no copier warp)
  int pair;                 // per-tap kernel, input gradient with column stride 2, NCHW output: see tile_of_iter
  int tma_store;            // 1: NCHW output written by TMA stores from per-warp staging slices
  const uint8_t* b_codes;   // weight-like codes [rows][taps][b_rowbytes] (source of the images below)
  int b_rows_total, b_rowbytes;
  uint8_t* b_img;           // [channel tile][tap][BN rows][KB], each row stored with the KB-byte swizzle applied
  // input gradient, per-tap kernel: the weight re-layout W -> W^T rides in the scale-expansion launch (extra blocks) and the
  // B-side chunks are gathered from the ORIGINAL tile scales, so the call needs one preparation launch instead of two
  int wt_fused;             // 1: on
  const uint8_t* wt_in;     // stored W codes [C_out][taps][C_in_p]
  uint8_t* wt_out;          // re-laid codes [C_in_p][taps][C_out_p]
  const uint8_t* wt_sc_in;  // stored W tile scales [C_out/32][taps][C_in_p/32]
  int wt_Cout, wt_Cop, wt_Cp, wt_bx, wt_by;   // channel counts; 32 x 32 blocks along C_in_p and C_out_p
  unsigned expand_blocks;   // blocks of the launch that expand scale chunks (the re-layout blocks follow)
  // output
  float* out;
  int out_layout;
  unsigned int* status;
  // quantizing epilogue (the producer emits the next tensor's MX tiles instead of fp32, see epilogue_mx_role)
  int mx_out;               // 1: on
  int mx_fmt, mx_act;       // element format of the emitted tensor (5: the paper's own format - E2M1, E4M3 scale per 16 x 16 block, fp32
                            // tensor scale from mx_ts_amax); activation applied first (mq_act)
  const float* mx_ts_amax;  // format 5: the maximum Eq. 4 takes (device; an earlier step's)
  float* mx_ts_stats;       // format 5: [0] receives T_scale, [1] (zero on entry) this tensor's own maximum
  uint8_t* mx_codes;        // [Hd][Wd][N][mx_Cp] codes
  uint8_t* mx_scales;       // [Hd][Wd][Nt][mx_Cp / 32] tile scales
  int mx_Cp;                // Cd rounded up to 32
};

// map_a: gathered activation codes.  map_w: weight codes, one tap per box (per-tap kernel) or all taps of a tile in one
// box (whole-tile kernel with fused preparation).  map_out: the fp32 NCHW output seen as (W, N, C, H), used when
// p.tma_store is set.
// 16-byte chunks of one-code-per-byte 6-bit codes -> 12 packed bytes (code i at bit 6 i) + 4 zero bytes
cudaError_t launch_pack6(const uint8_t* in, uint8_t* out, size_t nbytes, cudaStream_t s);
// packed 6-bit storage (16 codes in 12 bytes, n_codes a multiple of 16) -> mode 0: that container; 1: one code per byte;
// 2: E4M3 bytes of the same values (fmt6 says which 6-bit format)
cudaError_t launch_unpack6(const uint8_t* in, uint8_t* out, size_t n_codes, int mode, int fmt6, cudaStream_t s);
// one-code-per-byte E3M2 / E2M3 codes -> the E4M3 codes of the same values (every 6-bit value is an E4M3 value)
cudaError_t launch_recode6_e4m3(const uint8_t* in, uint8_t* out, size_t nbytes, int fmt6, cudaStream_t s);
// packed E2M1 codes (two per byte) -> the E4M3 codes of the same values, one per byte; n_out = elements = output bytes
cudaError_t launch_recode4_e4m3(const uint8_t* in, uint8_t* out, size_t n_out, cudaStream_t s);
// map_sfa, map_sfb: p.duo only - the two scale images as rows of 256 bytes (boxes of one stage's chunks)
cudaError_t launch_conv_tc(const ConvTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_w, const CUtensorMap& map_out, cudaStream_t s,
                           const CUtensorMap* map_sfa = nullptr, const CUtensorMap* map_sfb = nullptr);
// Expands the compact tile scales into the per-stage scale-vector chunks the MMA reads (p.sfa_img, p.sfb_img).
cudaError_t launch_expand_conv_scales(const ConvTcParams& p, cudaStream_t s);
size_t conv_tc_sfa_bytes(const ConvTcParams& p);
size_t conv_tc_sfb_bytes(const ConvTcParams& p);
size_t conv_tc_smem_bytes(const ConvTcParams& p);

// Re-lays the stored weight codes [C_out][taps][C_in_p] as [C_in_p][taps][C_out_p] and the tile scales
// [C_out/32][taps][C_in_p/32] as [C_in_p/32][taps][C_out_p/32] (bwd_data's B operand).  No requantization.
cudaError_t launch_weight_transpose(const uint8_t* w_codes, const uint8_t* w_scales, uint8_t* wt_codes, uint8_t* wt_scales, const Geom& g, int fmt,
                                    cudaStream_t s);

// Parameters of the tensor-core weight-gradient kernel (see mq_wgrad_tc.cu).
enum { MQ_WG_FP8 = 0, MQ_WG_FP4_PIXEL = 1, MQ_WG_FP4_FLAT = 2 };
struct WgradTcParams {
  int kind;             // 0: 8-bit operands (kind::mxf8f6f4); 1: E2M1 with E8M0 tile scales (kind::mxf4); 2: E2M1 with E4M3 scales per 16 x 16
                        // block (kind::mxf4nvf4; the tensors' fp32 scales are applied by bwd_weight_reduce) - modes FP4_PIXEL / FP4_FLAT
  int mode;             // MQ_WG_FP8: 8-bit operands as stored (MN-major TMA boxes); MQ_WG_FP4_PIXEL: E2M1 re-laid
                        // [pixel][c][n], one TMA box per pixel; MQ_WG_FP4_FLAT: stride 1, E2M1 re-laid as contiguous
                        // pre-swizzled pieces over the zero-padded, flattened pixel axis (bulk copies)
  uint32_t idesc;       // instruction descriptor without the N field
  int stages;
  int N, Nt, Ho, Wo, H, W, Cout, Cp, Ct, Cot, Kh, Kw, sh, sw, ph, pw;
  int BPP;              // K-blocks (32 samples) taken per pixel per stage
  int KPX;              // pixels per stage
  int KBn;              // E2M1: bytes of n per pixel per stage (= 16 * BPP)
  int nchunks;          // stages per pixel group
  int groups_w;         // ceil(Wo / KPX)
  int stages_total;     // pixel: Ho * groups_w * nchunks; flat: ceil(Ho * Wp / KPX)
  int Wp;               // padded width W + 2 * pw
  int Hp;               // padded height H + 2 * ph
  int b_rows;           // rows (input channels) of a B tile: 128, or min(128, Cp) in flat mode
  int m_tiles, j_tiles, cb_tiles, splits;   // j_tiles = (taps / TG) * cb_tiles; m_tiles counts work units along C_out
  int m_tiles128;       // 128-row tiles of output channels (= m_tiles, or 2 * m_tiles when cta2)
  int mma_cp;           // E2M1: 1 = the MMA lane issues the scale copies itself (no copier warp)
  int cta2;             // 1: pairs of blocks (clusters of 2) compute 256 x 256 tiles with cta_group::2 MMAs
  int TG;               // taps per block: 1, or Kw (flat mode: the taps of a kernel row share the stage's pixels)
  int sfb_S;            // flat E2M1 mode, 128 input channels per tap panel: > 0 = the X-side scale chunks are stored once per padded
                        // START pixel (sfb_S of them per channel block; tap (kh, kw) of stage st reads chunk st KPX + kh Wp + kw), not
                        // once per (tap group, stage, tap)
  int grp8;             // 8-bit operands, 32 or 64 bytes of input channels, unit strides: the Kw taps of a kernel row are one wide B operand
                        // (TG = Kw, b_rows = Cp) whose panels are views of one loaded strip of KPX + Kw - 1 pixels, one pixel apart
  int NB;               // 128-row chunks of the group's B rows = ceil(TG * b_rows / 128)
  int n0, n1;           // MMA widths per K slice: n0 = min(TG * b_rows, 256) and the rest (0: one MMA)
  int b_tile_bytes;     // bytes of X loaded per stage: b_rows * 128, flat mode (KPX + TG - 1) * b_rows * KBn
  int stage_bytes;      // A tile + B tile + (1 + NB) scale chunks of 1024 bytes, rounded up to 1024
  int sf_slots;         // scale buffers in tensor memory: = stages, or fewer (kind 2), used in turn
  int tmem_cols;        // TMEM allocation: accumulators (TG * b_rows) + stages * (8 + 8 * NB), a power of two
  const uint8_t* g_scales;  // [Ho][Wo][Nt][Cot]
  const uint8_t* x_scales;  // [H][W][Nt][Ct]
  const uint8_t* gt;        // flat: [co block][padded pixel][128][KBn]
  const uint8_t* xt;        // flat: [ci block][padded pixel][b_rows][KBn]
  long long gt_block_bytes, xt_block_bytes;
  uint8_t* sfa_img;         // [m tile][stage][512 * SPA]
  uint8_t* sfb_img;         // E2M1: [ci block][tap group][stage][NB][512 * SPA]; 8-bit: [ci block][Hp][Wp][sample chunk][NB][512]
  float* partial;           // [splits][Cout][taps * Cp]
  unsigned int* status;
};
// map_p: the partial sums as an fp32 tensor (taps * Cp columns, C_out rows, splits), box 32 x 32 x 1, 128-byte swizzle
cudaError_t launch_wgrad_tc(const WgradTcParams& p, const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_p, const CUtensorMap& map_sfa,
                            const CUtensorMap& map_sfb, cudaStream_t s);
cudaError_t launch_expand_wgrad_scales(const WgradTcParams& p, cudaStream_t s);
// E2M1 codes [P][N][Cp] -> [P][Cp][Npad] (n fastest, zero-padded): a permutation of nibbles, no requantization.
cudaError_t launch_fp4_to_n_major(const uint8_t* in, uint8_t* out, int P, int N, int Cp, int Npad, cudaStream_t s);
// Flat-mode preparation in one launch.  E2M1 codes [Hs][Ws][N][Cs_p] -> [channel block][q][rows][KBn] over the
// zero-padded, flattened pixel axis q = hq * Wp + wq in [0, P), source pixel (hq - off_h, wq - off_w), zero outside
// the image / beyond the channels, each [rows][KBn] piece stored with the shared-memory swizzle of span KBn already
// applied: X (P_b pixels, offsets = the padding, b_rows channels per block) and G_Y (P_a pixels, 128 channels per
// block); then the scale chunks of expand_wgrad_scales.
cudaError_t launch_wgrad_flat_prep(const WgradTcParams& p, const uint8_t* x_codes, uint8_t* xt, int P_b, const uint8_t* g_codes, uint8_t* gt, int P_a,
                                   cudaStream_t s);
// Adds the split partial sums in a fixed order and writes G_W in its final layout.
// ta, tb (device, may be null): fp32 tensor scales whose product the sums are multiplied by
cudaError_t launch_bwd_weight_reduce(const float* partial, float* out, const Geom& g, int splits, int layout, cudaStream_t s, const float* ta = nullptr,
                                     const float* tb = nullptr);

// Host: encode a tiled tensor map over bytes (or over fp32 elements when f32 is set: dims and box then count
// elements).  Strides in bytes (stride[0] implied contiguous), fastest dimension first.  l2_promotion_bytes: 0, 64, 128, 256,
// or -1 for the library's default.
bool encode_tensor_map_u8(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                          const uint32_t* box, const uint32_t* elem_strides, int swizzle_bytes, bool f32 = false, int l2_promotion_bytes = -1);

// The same over a tensor in packed 6-bit storage, 128-byte swizzle: dims, box and coordinates count codes (box[0] = 128).
bool encode_tensor_map_p6(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box,
                          const uint32_t* elem_strides);

}  // namespace mq
