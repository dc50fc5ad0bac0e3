/* mq.h -- C ABI of the MicroQonv hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, on one GPU, the three parts of a microscaling-quantized convolution
 * layer's training step as the paper lays them out:
 *   1. a single-pass MX quantizer applied once each to X, W and G_Y (Sec. III-A, Eq. 5-6; the
 *      square blocks and per-tensor directions of Sec. IV-B),
 *   2. the channel-batch-first im2col of the already-quantized activation (Sec. IV-A),
 *   3. the three block-scaled GEMMs Y, G_X, G_W (Sec. II-C, Sec. IV-B, Eq. 7).
 *
 * Conventions common to every call
 *   - All tensor pointers are DEVICE pointers unless a parameter says "host".  The caller owns
 *     every buffer, including workspace; the library allocates no device memory.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default stream) and
 *     return without synchronising.  Argument errors are detected on the host before anything is
 *     launched; on error nothing is enqueued and outputs are untouched.
 *   - Every device buffer must be 16-byte aligned.
 *   - Problem statement (Sec. II-A): X is N x C_in x H x W, W is C_out x C_in x Kh x Kw, G_Y and Y
 *     are N x C_out x Ho x Wo with Ho = floor((H + 2 pad_h - Kh) / stride_h) + 1 (likewise Wo).
 *     Cross-correlation, zero padding, dilation 1, groups 1, no bias.
 *
 * Stored MX tensors (the "channel-batch-first" layouts of Sec. IV-A / IV-B; Cp = C rounded up to 32)
 *   role X : codes [H][W][N][C_in_p],            scales [H][W][ceil(N/32)][C_in_p/32]
 *   role W : codes [C_out][Kh][Kw][C_in_p],      scales [ceil(C_out/32)][Kh][Kw][C_in_p/32]
 *   role DY: codes [Ho][Wo][N][C_out_p],         scales [Ho][Wo][ceil(N/32)][C_out_p/32]
 *   The channel axis is fastest.  E4M3 / E5M2 codes take one byte; E2M1 codes are packed two per
 *   byte, the lower channel index in bits 3:0.  Padded channels hold code 0.  A scale is one E8M0
 *   byte (value 2^(code-127)) shared by a 32 x 32 tile: 32 channels x 32 samples (X, DY) or
 *   32 input x 32 output channels (W) at one spatial / tap position, so that every 32-element
 *   line of a tile, in either contraction direction, is a standard MX block (Sec. IV-B).
 *
 * Packed 6-bit storage (MQ_E3M2_P6, MQ_E2M3_P6): the 6-bit element formats at the six bits per element Sec. VI counts
 *   for them.  Layouts as above; a group of 16 consecutive channels occupies 12 bytes, code k of the group in bits
 *   6k .. 6k+5 of that 96-bit little-endian field (so a row of Cp channels takes 3 Cp / 4 bytes, and the tensor 3/4 of
 *   the bytes of MQ_E3M2 / MQ_E2M3, which store one code per byte).  Scales are unchanged.  mq_qtensor_sizes,
 *   mq_im2col_sizes, mq_workspace_size, mq_quantize, mq_quantize_sr, mq_cbf_im2col, the three mq_conv_* GEMMs,
 *   mq_conv_bwd_data_static and mq_conv_layer_host accept them and give the results of the one-code-per-byte format bit
 *   for bit; the quantizing producer epilogues (mq_conv_*_mx) return MQ_ERR_UNSUPPORTED for them.  Activation and
 *   gradient tensors whose padded channel count is a multiple of 128 are read by the tensor-core GEMMs where they
 *   are stored; other operands pass through a copy in the call's scratch.
 *
 * Line blocks (MQ_BLOCK_LINE32): the one-directional block of Sec. III-A (Eq. 5-6) - 32 consecutive channels of ONE
 *   row (sample / output channel) share the scale, amax over those 32 elements.  Codes are laid out as above; scales
 *   have one entry per row instead of one per 32 rows:
 *   role X : scales [H][W][N][C_in_p/32]     role W : scales [C_out][Kh][Kw][C_in_p/32]     role DY: scales [Ho][Wo][N][C_out_p/32]
 *   Such a tensor can feed the GEMM that contracts over its channel axis (the forward GEMM for X and W) and no
 *   other: that is the limitation Sec. III-B / III-C derive the square blocks from.  mq_quantize, mq_cbf_im2col
 *   and mq_conv_fwd accept it; mq_conv_bwd_data and mq_conv_bwd_weight return MQ_ERR_UNSUPPORTED for it.
 *
 * The paper's own number format (MQ_BLOCK_TS16): Sec. III-A as written - an fp32 scale per TENSOR (Eq. 4:
 *   T_scale = max|X| / (448 * 6)), an E4M3 scale per block (Eq. 5: B_scale = CastE4M3(max|X_i| / (6 T_scale))) and E2M1
 *   elements (Eq. 6: Round(X_i / (B_scale T_scale))) - on the square blocks of Sec. IV-B with a side of 16, the finest
 *   scale granularity of the tensor cores' block-scaled E2M1 path (the paper's experiments use a side of 8).  Element
 *   format is MQ_E2M1; codes are laid out as above; scales hold one E4M3 byte per 16 x 16 block, in the order of the
 *   32 x 32 case with 16 in place of 32:
 *   role X : scales [H][W][ceil(N/16)][C_in_p/16]     role W : scales [ceil(C_out/16)][Kh][Kw][C_in_p/16]
 *   role DY: scales [Ho][Wo][ceil(N/16)][C_out_p/16]
 *   and mq_qtensor.tensor_scale points at two device floats: T_scale, and the tensor's own max|X| (kept so that a later
 *   step can use it as its estimate, Sec. VII-B).  Eq. 4-6 are evaluated in IEEE single precision, one rounding per
 *   written operation; both roundings go to nearest, ties to even, and saturate; a block of zeros has scale 0.
 *   All calls accept it (both operands of a GEMM must use it).  The three GEMMs run on the tensor cores (E4M3 scale per 16
 *   elements of the contraction axis, the tensors' fp32 scales applied to the accumulator) for the layers the MX E2M1
 *   path takes, on the CUDA-core kernels otherwise; the quantizing producer epilogue of this format is
 *   mq_conv_fwd_ts / mq_conv_bwd_data_ts (mq_conv_fwd_mx / mq_conv_bwd_data_mx do not take it).
 */
#ifndef MQ_H_
#define MQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MQ_OK = 0,
  MQ_ERR_INVALID_ARG = 1,      /* null pointer, non-positive dimension, unknown enum value        */
  MQ_ERR_UNSUPPORTED = 2,      /* a valid request this build does not implement                   */
  MQ_ERR_ALIGNMENT = 3,        /* a device pointer is not 16-byte aligned                         */
  MQ_ERR_BUFFER_TOO_SMALL = 4, /* a declared buffer size is smaller than the call needs           */
  MQ_ERR_CUDA = 5,             /* a CUDA runtime / driver call failed (launch, descriptor encode) */
  MQ_ERR_TIMEOUT = 6,          /* a bounded device-side wait gave up (see mq_last_device_status)  */
  MQ_ERR_STATIC_SCRATCH = 7    /* the layer needs more scratch than the built-in static array holds */
} mq_status;

typedef enum { MQ_E4M3 = 0, MQ_E5M2 = 1, MQ_E2M1 = 2,
               MQ_E3M2 = 3, MQ_E2M3 = 4,             /* element format, Sec. II-D; the 6-bit formats (Sec. V: the
                                                        activations of MicroQonv+, the "-6" variant) are stored one code
                                                        per byte, value in the low six bits, sign in bit 5 ...        */
               MQ_E3M2_P6 = 5, MQ_E2M3_P6 = 6 } mq_elem; /* ... or packed, 16 codes in 12 bytes (see above)            */
typedef enum { MQ_ROLE_X = 0, MQ_ROLE_W = 1, MQ_ROLE_DY = 2 } mq_role; /* which tensor, Sec. IV-B   */
typedef enum { MQ_NCHW = 0, MQ_HWNC = 1 } mq_layout;                   /* layout of an unquantized tensor */
typedef enum { MQ_BLOCK_TILE32 = 0,      /* 32 x 32 square block (Sec. IV-B), the default           */
               MQ_BLOCK_LINE32 = 1,      /* 1 x 32 line block along the channel axis (Sec. III-A)   */
               MQ_BLOCK_TS16 = 2 } mq_block; /* 16 x 16 square block, E4M3 block scale + fp32 tensor scale (Eq. 4-6) */
typedef enum { MQ_F32 = 0, MQ_BF16 = 1 } mq_dtype;                     /* element type of an unquantized tensor */
typedef enum { MQ_OP_FWD = 0, MQ_OP_BWD_DATA = 1, MQ_OP_BWD_WEIGHT = 2 } mq_op;
typedef enum { MQ_ACT_NONE = 0, MQ_ACT_RELU = 1, MQ_ACT_SILU = 2 } mq_act;   /* activation of the quantizing producer epilogue */

/* One convolution layer (Sec. II-A).  block_size must be 32 (the E8M0 block length). */
typedef struct {
  int N, C_in, H, W, C_out, Kh, Kw;
  int stride_h, stride_w, pad_h, pad_w;
  int block_size;
} mq_conv_desc;

/* A stored MX tensor: a view of caller-owned device memory, never freed by the library. */
typedef struct {
  void* codes;         /* element codes, layout above                 */
  uint8_t* scales;     /* E8M0 tile scales, layout above              */
  size_t codes_bytes;  /* size of the codes buffer                    */
  size_t scales_bytes; /* size of the scales buffer                   */
  int fmt;             /* mq_elem                                     */
  int role;            /* mq_role                                     */
  int block;           /* mq_block                                    */
  float* tensor_scale; /* MQ_BLOCK_TS16: two device floats (T_scale, max|X|), 8-byte aligned; else unused */
} mq_qtensor;

/* Size queries (host only, no GPU needed). */

/* Bytes of codes and scales of the stored MX tensor of `role` with blocks `block` (layouts above). */
mq_status mq_qtensor_sizes(const mq_conv_desc* desc, int role, int fmt, int block, size_t* codes_bytes, size_t* scales_bytes);

/* Bytes of X'_{Cin,N} (Sec. IV-A): codes [Ho][Wo][N][Kh][Kw][C_in_p], scales [Ho][Wo][ceil(N/32)][Kh][Kw][C_in_p/32]
 * (line blocks: [Ho][Wo][N][Kh][Kw][C_in_p/32]). */
mq_status mq_im2col_sizes(const mq_conv_desc* desc, int fmt, int block, size_t* codes_bytes, size_t* scales_bytes);

/* Bytes of scratch `op` (mq_op) needs for operand formats fmt_a, fmt_b (in the order of the call's
 * two mq_qtensor arguments) quantized in blocks `block`.  May be 0. */
mq_status mq_workspace_size(const mq_conv_desc* desc, int op, int fmt_a, int fmt_b, int block, size_t* bytes);

/* mq_quantize -- Sec. III-A (Eq. 5-6) in the E8M0 form of the original MX format (Sec. II-D), on the
 * square blocks and in the directions of Sec. IV-B; also re-lays the tensor into its stored order
 * (Sec. IV-A), so the tensor is read once and quantized once.
 *   per tile: amax = max |x| over the valid elements; scale code = clamp(floor(log2 amax) - emax
 *   + 127, 0, 254) (0 if amax = 0); element = round-to-nearest-even(x * 2^(127 - code)) on the
 *   element format's grid, saturating at its largest finite magnitude, sign kept.
 * src: device memory, 16-byte aligned, of element type `src_dtype` (MQ_F32; MQ_BF16 returns MQ_ERR_UNSUPPORTED in this
 * build); `src_layout` = MQ_NCHW (X: [N][C_in][H][W], W: [C_out][C_in][Kh][Kw],
 * G_Y: [N][C_out][Ho][Wo]) or MQ_HWNC, the channel-fastest order the convolution entry points can emit
 * (X: [H][W][N][C_in], W: [C_out][Kh][Kw][C_in], G_Y: [Ho][Wo][N][C_out]); both give the same stored
 * tensor bit for bit.  dst->codes / dst->scales receive the stored tensor; dst->fmt, dst->role and
 * dst->block select format, role and block shape; the *_bytes fields must be at least mq_qtensor_sizes().
 * Non-finite inputs are outside the contract (result unspecified, no fault). */
mq_status mq_quantize(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, void* stream);

/* mq_quantize_sr -- the same quantizer with the STOCHASTIC Round(.) of Eq. 6, which Sec. III-A assigns to the
 * gradient (activations and weights keep round-to-nearest); any role is accepted.  Tile scales are those of
 * mq_quantize.  Per element: with lo <= |x * 2^(127 - code)| < hi the neighbouring magnitudes of the element
 * format, the result is hi when u < (|x * 2^(127 - code)| - lo) / (hi - lo) and lo otherwise, sign kept; values on
 * the grid never move and magnitudes at or beyond the largest finite one saturate.  The paper names no generator;
 * here u = (top 23 bits of r + 1/2) / 2^23 with r = mix(low32(i) ^ key), key = mix(low32(seed) ^ mix(high32(seed) ^
 * mix(high32(i)))), i the element's index in the logical tensor ([N][C][H][W] / [C_out][C_in][Kh][Kw] order, for
 * either src_layout) and mix(x): x ^= x >> 16; x *= 0x7FEB352D; x ^= x >> 15; x *= 0x846CA68B; x ^= x >> 16 on
 * 32 bits.  The stored tensor is therefore a pure function of (src, seed): the same for both source layouts, on
 * every launch and on any number of GPUs.  Arguments, layouts and errors as for mq_quantize. */
mq_status mq_quantize_sr(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, unsigned long long seed,
                         void* stream);

/* mq_quantize_ts -- quantizer of the paper's own format (dst->block = MQ_BLOCK_TS16, dst->fmt = MQ_E2M1) with control over
 * where Eq. 4 takes the tensor's maximum from.  amax_in = NULL: from this tensor (two passes over `src`: a reduction,
 * then the quantizer); mq_quantize on such a dst does exactly this.  amax_in = a device fp32: from that value - e.g.
 * the max|X| an earlier step left in its tensor_scale[1] (statistics of previous batches, Sec. VII-B), so that the
 * quantizer needs no result of a reduction over this tensor (large NCHW / OIHW sources are then read ONCE, the quantizer
 * collecting this tensor's maximum as it goes); elements beyond the estimate saturate.  amax_in must not point into
 * dst->tensor_scale (the call rewrites both words).  Either way dst->tensor_scale[0] receives T_scale and
 * dst->tensor_scale[1] this tensor's own max|X|.
 * seed_or_null: NULL = round to nearest; else a host pointer to the 64-bit seed of the stochastic Round(.) of Eq. 6 (the
 * gradient's rounding; draws as in mq_quantize_sr). */
mq_status mq_quantize_ts(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, const float* amax_in,
                         const unsigned long long* seed_or_null, void* stream);

/* mq_cbf_im2col -- channel-batch-first im2col (Sec. IV-A) of the quantized activation `xq` (role X):
 * row (kh,kw,c), column (ho,wo,n) of X' is the stored code at pixel (ho*stride+kh-pad,
 * wo*stride+kw-pad); tile scales are gathered alongside; out-of-image taps are zero bytes (codes
 * and scale).  No arithmetic on values: an element keeps its single quantized value everywhere.
 * cols_codes / cols_scales: sizes from mq_im2col_sizes() for xq->fmt and xq->block. */
mq_status mq_cbf_im2col(const mq_conv_desc* desc, const mq_qtensor* xq, void* cols_codes, uint8_t* cols_scales, void* stream);

/* mq_conv_fwd -- Y_{f Cout,N} = W_{f Cout,Cin} . X'_{Cin,N} (Sec. II-C, IV-B; Eq. 1), block-scaled as
 * Eq. 7 with K-blocks of 32 input channels at one tap; X' is formed on the fly from `xq`.
 * y: `y_dtype` elements (MQ_F32; MQ_BF16 returns MQ_ERR_UNSUPPORTED in this build), `y_layout` MQ_NCHW
 * ([N][C_out][Ho][Wo]) or MQ_HWNC ([Ho][Wo][N][C_out]); fp32 accumulation.
 * xq and wq must have the same block shape; with line blocks the K-blocks carry one scale per row (Eq. 7 as written).
 * workspace: ws_bytes >= mq_workspace_size(desc, MQ_OP_FWD, xq->fmt, wq->fmt, xq->block) (may be NULL if 0). */
mq_status mq_conv_fwd(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, void* y, int y_dtype, int y_layout,
                      void* workspace, size_t ws_bytes, void* stream);

/* mq_conv_bwd_data -- G_X' = W_f^T . G_Yf followed by the col2im reordering (Sec. II-C, IV-B; Eq. 2):
 * the exact adjoint of mq_conv_fwd in X, K-blocks of 32 output channels at one tap.
 * dx: `dx_dtype` elements (MQ_F32), MQ_NCHW ([N][C_in][H][W]) or MQ_HWNC ([H][W][N][C_in]).
 * W is contracted along C_out, across its stored channel lines (the second direction of its blocks), which only
 * square blocks allow: line-block operands give MQ_ERR_UNSUPPORTED. */
mq_status mq_conv_bwd_data(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, void* dx, int dx_dtype, int dx_layout,
                           void* workspace, size_t ws_bytes, void* stream);

/* mq_conv_bwd_data_static -- the same computation as mq_conv_bwd_data for callers that cannot hand the
 * library a scratch buffer because they cannot allocate device memory at all.  (The paper has no
 * counterpart for this call; it exists for integration reasons only.)  Typical cases: a plug-in that runs
 * inside a host application which owns the allocator and forbids cudaMalloc on its streams, code running
 * while a memory pool is frozen, or a tiny embedding that links the library without any allocator.  Such
 * a caller still supplies the inputs (wq, dyq) and the output (dx); only the scratch is taken care of.
 *
 * The scratch that mq_conv_bwd_data takes as `workspace` (the weight codes and tile scales re-laid for the
 * input-gradient GEMM, and the per-stage scale-vector chunks expanded from the tile scales) lives here in a
 * static array inside the library's device image, MQ_STATIC_SCRATCH_BYTES (16 MiB) long; every GPU that
 * loads the library keeps that much memory reserved until the process exits.  A layer whose
 * mq_workspace_size(desc, MQ_OP_BWD_DATA, ...) exceeds it is rejected with MQ_ERR_STATIC_SCRATCH and nothing
 * is launched (for scale: N=32, 128->64 channels, 80x80, 3x3 needs about 6 MB).
 * The call performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *
 * Arguments are checked exactly as by mq_conv_bwd_data (same codes), then the size limit.
 * First use on a device: every call looks up the array's device address for the current device (nothing is
 * cached, so a cudaDeviceReset between calls is harmless); the first such lookup on a device may load the
 * library's device code, so make the first call outside of any stream capture.
 * Sharing: all calls on a device use the same array and it keeps whatever the previous call left in it;
 * each call overwrites every byte it later reads, so nothing needs clearing, but two calls whose kernels
 * overlap on the GPU (different streams, no ordering between them) race on the array -- order them. */
#define MQ_STATIC_SCRATCH_BYTES (16u << 20)
mq_status mq_conv_bwd_data_static(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, void* dx, int dx_dtype, int dx_layout,
                                  void* stream);

/* Producer epilogue that quantizes.  The paper's cost model quantizes a tensor on chip, when its producer has it, and only
 * then stores it (Sec. V, the DRAM model: activations leave the chip in their quantized form); these two calls are the
 * GEMMs above with that order: the epilogue applies the activation and writes the NEXT tensor's stored MX form instead
 * of fp32, so the fp32 tensor never exists in HBM and the separate mq_quantize pass over it disappears.
 *
 * mq_conv_fwd_mx:      Y = act(conv(X, W)), emitted as the stored activation of the next layer: yq has role MQ_ROLE_X
 *                      and the layouts of a role-X tensor of N x C_out x Ho x Wo (codes [Ho][Wo][N][C_out_p], scales
 *                      [Ho][Wo][ceil(N/32)][C_out_p/32]); yq->fmt selects its element format.
 *                      act (mq_act): none, ReLU max(y, 0), or SiLU y / (1 + exp(-y)), evaluated in fp32.
 * mq_conv_bwd_data_mx: G_X, emitted as the stored output gradient of the previous layer: dxq has role MQ_ROLE_DY and the
 *                      layouts of N x C_in x H x W (codes [H][W][N][C_in_p], scales [H][W][ceil(N/32)][C_in_p/32]).
 * Arithmetic of the emitted tensor: exactly mq_quantize's (tile amax over valid elements of the fp32 result, E8M0 floor
 * rule, round-to-nearest-even, saturating, padded channels code 0) applied to the fp32-accumulated GEMM result.
 * Square blocks only.  Layers the tensor-core kernels do not take (a tap's channel row not a multiple of 32 bytes, an
 * E2M1 operand mixed with a one-byte format) give the same result in two launches inside the call: the CUDA-core GEMM
 * writes fp32 into the workspace and the quantizer, applying the activation, reads it back.
 * workspace: ws_bytes >= mq_conv_mx_workspace_size(desc, op, fmt of the first operand, fmt of the second). */
mq_status mq_conv_mx_workspace_size(const mq_conv_desc* desc, int op, int fmt_a, int fmt_b, size_t* bytes);
mq_status mq_conv_fwd_mx(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, int act, mq_qtensor* yq, void* workspace,
                         size_t ws_bytes, void* stream);
mq_status mq_conv_bwd_data_mx(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, mq_qtensor* dxq, void* workspace,
                              size_t ws_bytes, void* stream);

/* The same producer epilogue in the paper's own number format (Sec. III-A, Eq. 4-6; MQ_BLOCK_TS16 operands AND emitted tensor).
 * Eq. 4 needs the emitted tensor's maximum before its first element can be scaled, which a single pass over the
 * accumulators cannot know: the maximum is SUPPLIED, from statistics of earlier batches (Sec. VII-B), as for mq_quantize_ts.
 *   amax_in: device pointer to one fp32, the maximum Eq. 4 uses (4-byte aligned; e.g. the previous step's
 *            tensor_scale[1] of the same tensor).  Values beyond it saturate (block scale at 448, elements at 6).
 *   yq / dxq: caller-allocated MQ_BLOCK_TS16 / MQ_E2M1 tensor with the sizes of mq_qtensor_sizes for the NEXT layer's
 *            role-X tensor (N x C_out x Ho x Wo), resp. the previous layer's role-DY tensor (N x C_in x H x W): codes
 *            [pixel][N][C_p / 2], scales [pixel][ceil(N/16)][C_p/16] E4M3 bytes; on return tensor_scale[0] =
 *            amax_in / (448 x 6) and tensor_scale[1] = the emitted tensor's own max|value| (for the next step).
 * Arithmetic: mq_quantize_ts's, one IEEE single-precision operation per written operation of Eq. 4-6, applied to the
 * fp32-accumulated GEMM result times the two operands' tensor scales, after the activation.  Round-to-nearest-even.
 * Layers the tensor-core kernels do not take run as two launches inside the call, as above.
 * workspace: ws_bytes >= mq_conv_ts_workspace_size(desc, op).  Errors as mq_conv_fwd_mx; operands or output that are not
 * MQ_BLOCK_TS16 give MQ_ERR_UNSUPPORTED, a null amax_in MQ_ERR_INVALID_ARG. */
mq_status mq_conv_ts_workspace_size(const mq_conv_desc* desc, int op, size_t* bytes);
mq_status mq_conv_fwd_ts(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, int act, const float* amax_in, mq_qtensor* yq,
                         void* workspace, size_t ws_bytes, void* stream);
mq_status mq_conv_bwd_data_ts(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, const float* amax_in, mq_qtensor* dxq,
                              void* workspace, size_t ws_bytes, void* stream);

/* mq_conv_bwd_weight -- G_Wf = G_Yf . X'^T (Sec. II-C, IV-B; Eq. 3), K-blocks of 32 samples at one
 * output pixel: the stored X and G_Y are read along N, the other direction of their square blocks.
 * dw: fp32 OIHW ([C_out][C_in][Kh][Kw]) for MQ_NCHW, or [C_out][Kh][Kw][C_in] for MQ_HWNC.
 * The reduction over (ho,wo,n) is split across thread blocks through `workspace` and summed in a
 * fixed order (deterministic).  dw: `dw_dtype` elements (MQ_F32).  Line-block operands give MQ_ERR_UNSUPPORTED
 * (the contraction runs along N, across the lines). */
mq_status mq_conv_bwd_weight(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* dyq, void* dw, int dw_dtype, int dw_layout,
                             void* workspace, size_t ws_bytes, void* stream);

/* mq_conv_layer_host -- one whole pass of the path for a layer whose tensors live in HOST memory:
 * copies X, W, G_Y (fp32; NCHW / OIHW / N.C_out.Ho.Wo; pinned memory makes the copies asynchronous)
 * into `arena`, runs mq_quantize on each once, mq_cbf_im2col, mq_conv_fwd, mq_conv_bwd_data and
 * mq_conv_bwd_weight, and copies Y, G_X, G_W (fp32, MQ_NCHW layouts) back to the host buffers.
 * The kernels are enqueued on `stream`; the copies run on two library-owned side streams (one per direction,
 * created on first use, no device memory involved) tied to `stream` by events, so uploads and downloads
 * overlap the kernels; `stream` waits for the last download, so the host results are valid after `stream`
 * is synchronised and successive calls on one stream stay ordered.
 * The step runs slab by slab along the batch (slabs of whole 32-sample tiles, at most 8): every call above needs only the
 * slab's own samples (and W), so slab k + 1 uploads and slab k's Y and G_X download while the kernels run.  Y and G_X
 * are exactly the device calls' results; G_W is the sum of the slabs' weight gradients, added in slab order.
 * arena: device memory, arena_bytes >= mq_conv_layer_host_arena_size(); contents are scratch. */
mq_status mq_conv_layer_host_arena_size(const mq_conv_desc* desc, int fmt_x, int fmt_w, int fmt_dy, size_t* bytes);
mq_status mq_conv_layer_host(const mq_conv_desc* desc, int fmt_x, int fmt_w, int fmt_dy, const float* x_host, const float* w_host,
                             const float* dy_host, float* y_host, float* dx_host, float* dw_host, void* arena, size_t arena_bytes,
                             void* stream);

/* Diagnostic: how many kernels this library has launched so far in this process (all entry points). */
unsigned long long mq_kernel_launch_count(void);

/* Diagnostic: the library's MQ_* environment knobs (alternate kernel paths, kept for testing and measurement) are read
 * once each, on first use, so that mq_workspace_size and the call it sizes always plan alike.  This call makes the next
 * use of every knob read the environment again.  Not for use while another thread is inside the library. */
void mq_reload_env(void);

/* Diagnostic self-test of the give-up path of the library's bounded device-side waits (the paper has no counterpart).
 * Launches the quantizer's TMA pipeline for role X or DY (dst->role; H*W resp. Ho*Wo a multiple of 4, else
 * MQ_ERR_UNSUPPORTED) on `src` (fp32 NCHW) with its loader issuing NO copies and every barrier wait limited to `polls`
 * polls (1 .. 2^20): nothing ever arrives, each wait runs out, the kernel records MQ_ERR_TIMEOUT in the device status
 * word, leaves its loops, and returns normally - nothing hangs, traps or faults, the context stays usable.  dst's buffers
 * (sizes as for mq_quantize) are left with unspecified contents.  Afterwards mq_last_device_status() reports
 * MQ_ERR_TIMEOUT once and clears the word. */
mq_status mq_selftest_wait_timeout(const mq_conv_desc* desc, const void* src, mq_qtensor* dst, unsigned polls, void* stream);

/* Human-readable name of a status code (static storage). */
const char* mq_status_string(int status);

/* Synchronises `stream`, then reads and clears the device-side status word that kernels set when a
 * bounded wait gives up.  Returns MQ_OK, MQ_ERR_TIMEOUT or MQ_ERR_CUDA. */
mq_status mq_last_device_status(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* MQ_H_ */
