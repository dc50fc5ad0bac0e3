// extern "C" entry points: argument validation, size arithmetic, kernel selection.
#include <atomic>
#include <cstdlib>
#include <map>
#include <mutex>
#include <string>

#include "mq_internal.cuh"
#include "mq_conv_tc.cuh"

namespace mq {

__device__ unsigned int g_device_status = 0;  // set by kernels when a bounded wait gives up

static std::atomic<unsigned long long> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// environment knobs, read once each (see mq_internal.cuh)
static std::mutex g_env_mutex;
static std::map<std::string, std::pair<bool, int>> g_env;   // name -> (set in the environment, value)
int env_int(const char* name, int dflt) {
  std::lock_guard<std::mutex> lock(g_env_mutex);
  auto it = g_env.find(name);
  if (it == g_env.end()) {
    const char* v = std::getenv(name);
    it = g_env.emplace(name, std::make_pair(v != nullptr, v ? std::atoi(v) : 0)).first;
  }
  return it->second.first ? it->second.second : dflt;
}
static void env_forget() {
  std::lock_guard<std::mutex> lock(g_env_mutex);
  g_env.clear();
}

namespace {

bool valid_fmt_unpacked(int f) { return f == MQ_E4M3 || f == MQ_E5M2 || f == MQ_E2M1 || f == MQ_E3M2 || f == MQ_E2M3; }
bool valid_fmt(int f) { return valid_fmt_unpacked(f) || fmt_is_packed6(f); }
bool valid_role(int r) { return r == MQ_ROLE_X || r == MQ_ROLE_W || r == MQ_ROLE_DY; }
bool valid_block(int b) { return b == MQ_BLOCK_TILE32 || b == MQ_BLOCK_LINE32 || b == MQ_BLOCK_TS16; }
bool valid_dtype(int t) { return t == MQ_F32 || t == MQ_BF16; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

mq_status check_desc(const mq_conv_desc* d) {
  if (!d) return MQ_ERR_INVALID_ARG;
  if (d->N <= 0 || d->C_in <= 0 || d->H <= 0 || d->W <= 0 || d->C_out <= 0 || d->Kh <= 0 || d->Kw <= 0) return MQ_ERR_INVALID_ARG;
  if (d->stride_h <= 0 || d->stride_w <= 0 || d->pad_h < 0 || d->pad_w < 0) return MQ_ERR_INVALID_ARG;
  if (d->H + 2 * d->pad_h < d->Kh || d->W + 2 * d->pad_w < d->Kw) return MQ_ERR_INVALID_ARG;
  if (d->block_size != 32) return MQ_ERR_UNSUPPORTED;
  return MQ_OK;
}

struct View { long long P, R, C, Cp; };
View view_of(const Geom& g, int role) {
  View v;
  if (role == MQ_ROLE_X) { v.P = (long long)g.H * g.W; v.R = g.N; v.C = g.Cin; v.Cp = g.Cp; }
  else if (role == MQ_ROLE_W) { v.P = (long long)g.Kh * g.Kw; v.R = g.Cout; v.C = g.Cin; v.Cp = g.Cp; }
  else { v.P = (long long)g.Ho * g.Wo; v.R = g.N; v.C = g.Cout; v.Cp = g.Cop; }
  return v;
}

void sizes_of(const Geom& g, int role, int fmt, int block, size_t* cb, size_t* sb) {
  View v = view_of(g, role);
  *cb = (size_t)(v.P * v.R * v.Cp) * fmt_store_bits(fmt) / 8;
  if (block == MQ_BLOCK_TS16) *sb = (size_t)(v.P * ((v.R + 15) / 16) * (v.Cp / 16));
  else *sb = (size_t)(v.P * (block == MQ_BLOCK_LINE32 ? v.R : (v.R + 31) / 32) * (v.Cp / 32));
}

mq_status check_qtensor(const Geom& g, const mq_qtensor* q, int role) {
  if (!q || !q->codes || !q->scales) return MQ_ERR_INVALID_ARG;
  if (!valid_fmt(q->fmt) || q->role != role || !valid_block(q->block)) return MQ_ERR_INVALID_ARG;
  if (q->block == MQ_BLOCK_TS16) {   // the paper's own format: E2M1 elements and a tensor-scale buffer
    if (q->fmt != MQ_E2M1 || !q->tensor_scale) return MQ_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(q->tensor_scale) & 7u) return MQ_ERR_ALIGNMENT;
  }
  if (!aligned16(q->codes) || !aligned16(q->scales)) return MQ_ERR_ALIGNMENT;
  size_t cb, sb;
  sizes_of(g, role, q->fmt, q->block, &cb, &sb);
  if (q->codes_bytes < cb || q->scales_bytes < sb) return MQ_ERR_BUFFER_TOO_SMALL;
  return MQ_OK;
}


// ---- tensor-core path: eligibility, tile shape, tensor maps ------------------------------------

// fwd / bwd_data run on the tcgen05 kernel when both operands are 8-bit formats or both are E2M1 and a
// tap's channel row is a whole number of 32-byte MMA K-atoms.
bool conv_tc_eligible(int op, const Geom& g, int fmt_x_like, int fmt_w) {
  if (op != MQ_OP_FWD && op != MQ_OP_BWD_DATA) return false;
  if (env_int("MQ_DISABLE_TC", 0)) return false;
  const bool fp4 = fmt_x_like == MQ_E2M1 && fmt_w == MQ_E2M1;
  const bool fp8 = fmt_x_like != MQ_E2M1 && fmt_w != MQ_E2M1;
  if (!fp4 && !fp8) return false;
  // 6-bit operands: the tensor core reads them as 16 codes packed into 12 bytes + 4 bytes of padding (along K), not one
  // code per byte as they are stored; run_conv_tc packs them into scratch first (MQ_TC_NO_FP6=1: CUDA-core kernels)
  if ((fmt_is_6bit(fmt_x_like) || fmt_is_6bit(fmt_w)) && env_int("MQ_TC_NO_FP6", 0)) return false;
  const int Kp = op == MQ_OP_FWD ? g.Cp : g.Cop;
  const int rowbytes = Kp * (fp4 ? 4 : 8) / 8;
  return rowbytes % 32 == 0;
}

size_t wt_codes_bytes(const Geom& g, int fmt_w) {
  return ((size_t)g.Cp * g.Kh * g.Kw * g.Cop * fmt_bits(fmt_w) / 8 + 255) / 256 * 256;
}
size_t up256(size_t v) { return (v + 255) / 256 * 256; }

// Output columns per tile.  Rows of a tile are TW consecutive output columns x TN = 128/TW samples with the
// column index fastest.  An NCHW store writes runs of TW floats and the store path is bound by the NUMBER of
// runs (about 2.2 cycles each per SM, measured), so the choice weighs the tile's MMA time against its store time
// and both against the padding the tile shape wastes at the edges.
//   k_bytes: bytes of K per tile row (taps x channel bytes); bn: output channels per tile.
//   serial: the tile's store is not overlapped with the next tile's MMAs (a single 256-column accumulator).
//   pair: the tiles of the even and the odd output columns are stored together (stride-2 input gradient): runs of
//   2 tw floats, and the two accumulators belong to one pair, so the store is not overlapped either.
int choose_tw(int w_eff, int N, int layout, double k_bytes, int bn, bool thin, bool serial, bool pair) {
  const int forced = env_int("MQ_TC_TW", 0);
  if (forced > 0) return forced;
  if (thin) return 8;   // the whole-tile kernel (8-column tiles): its per-tile loads beat any per-tap shape on thin layers
  const double t_mma = k_bytes / 32.0 * 107.0 * (bn / 128.0 < 0.5 ? 0.5 : bn / 128.0);
  int best = 1;
  double best_cost = 1e30;
  for (int tw = 1; tw <= 32; tw *= 2) {
    const int tn = 128 / tw;
    const double waste = (double)((w_eff + tw - 1) / tw * tw) / w_eff * (double)((N + tn - 1) / tn * tn) / N;
    double t_store = 128.0 * (bn * 4.0 / 128.0) * 2.2;          // [H][W][N][C] output: whole lines
    const int run = pair ? 2 * tw : tw;
    if (layout == MQ_NCHW) t_store = 128.0 * bn / run * 2.2 * (run < 8 ? 8.0 / run : 1.0);   // runs below a 32-byte sector cost a sector each
    double cost = waste * ((serial || pair) ? t_mma + t_store : (t_mma > t_store ? t_mma : t_store));
    if (cost < best_cost * (1.0 - 1e-9)) { best_cost = cost; best = tw; }
  }
  return best;
}

// Geometry of a tensor-core fwd / bwd_data call and the layout of its scratch:
//   [W re-laid codes | W re-laid scales]  (bwd_data only)  [A-side scale chunks][B-side scale chunks]
struct ConvTcPlan {
  ConvTcParams p;
  int rowbytes, rows_b;
  size_t off_wt_scales, off_sfa, off_sfb, off_bimg, off_pack_a, off_pack_b, total;   // off_pack_*: packed copies of 6-bit operands
};

// line: line-block operands (forward only).  mx: the quantizing epilogue (tiles of at most 4 output columns, channel tiles
// of whole 32-channel blocks, per-tap kernel).
// ts16: the paper's own format (E2M1 elements, one E4M3 scale per 16 x 16 block, an fp32 scale per tensor): kind::mxf4nvf4, per-tap kernel.
bool conv_tc_plan(int op, const Geom& g, int fmt_x_like, int fmt_w, int layout, ConvTcPlan* out, bool line = false, bool mx = false, bool ts16 = false) {
  const bool fp4 = fmt_w == MQ_E2M1;
  if (ts16 && (!fp4 || fmt_x_like != MQ_E2M1 || line)) return false;
  const int bits = fp4 ? 4 : 8;
  const int taps = g.Kh * g.Kw;
  ConvTcParams p{};
  p.mode = op;
  p.kind_fp4 = ts16 ? 2 : (fp4 ? 1 : 0);
  p.N = g.N; p.Nt = g.Nt;
  p.Kh = g.Kh; p.Kw = g.Kw; p.sh = g.sh; p.sw = g.sw; p.ph = g.ph; p.pw = g.pw;
  int Kp;
  if (op == MQ_OP_FWD) {
    Kp = g.Cp; p.Hs = g.H; p.Ws = g.W; p.Hd = g.Ho; p.Wd = g.Wo; p.Cd = g.Cout; out->rows_b = g.Cout;
    p.tiles_h = g.Ho; p.classes = 1;
  } else {
    Kp = g.Cop; p.Hs = g.Ho; p.Ws = g.Wo; p.Hd = g.H; p.Wd = g.W; p.Cd = g.Cin; out->rows_b = g.Cp;
    p.tiles_h = (g.H + g.sh - 1) / g.sh; p.classes = g.sh * g.sw;
  }
  p.Kblocks = Kp / 32;
  const int rowbytes = Kp * bits / 8;
  out->rowbytes = rowbytes;
  p.KB = rowbytes % 128 == 0 ? 128 : (rowbytes % 64 == 0 ? 64 : 32);
  p.G = 128 / p.KB;
  p.cpt = rowbytes / p.KB;
  const int w_eff = op == MQ_OP_FWD ? g.Wo : (g.W + g.sw - 1) / g.sw;
  // line blocks (one scale per row): the per-tap kernel, whose preparation launch lays out the scale vectors row by row
  const bool thin = !line && !mx && !ts16 && g.sh == 1 && g.sw == 1 && p.cpt == 1 && p.KB <= 64 && !env_int("MQ_TC_NO_HALO", 0);
  p.line = line ? 1 : 0;
  const int cd16 = mx ? (p.Cd + 31) / 32 * 32 : (p.Cd + 15) / 16 * 16;
  p.BN = cd16 <= 128 ? cd16 : 128;
  p.mx_out = mx ? 1 : 0;
  // 256-channel tiles halve the re-reads of the activation tile but leave tensor memory for one accumulator only, so
  // the epilogue no longer overlaps the next tile: worth it for 8-bit layers whose main loop is long (measured: +30 %
  // at 2304+ bytes of K per row)
  if (!fp4 && p.Cd >= 256 && (double)taps * rowbytes >= 2048.0 && (op == MQ_OP_FWD || (g.sh == 1 && g.sw == 1))) p.BN = 256;
  // 1x1 layers: the activation tile is the whole of a tile's loads, so halving its re-reads pays although the main loop is short
  // (measured, N = 256, 8-bit, fp32 / quantized output: 256 channels 56x56 324 -> 207 us / 217 -> 196 us; 512 channels 56x56
  // 531 -> 528 / 464 -> 410 us; 512 channels 28x28 181 -> 175 / 133 -> 127 us)
  // E2M1 likewise: 512 channels 56x56 550 -> 364 us, 256 channels 56x56 290 -> 173 us
  if (p.Cd >= 256 && taps == 1 && g.sh == 1 && g.sw == 1 && !env_int("MQ_TC_1X1_BN128", 0)) p.BN = 256;
  // E2M1: the same trade (measured with the tile widths chosen below: 256 channels 28x28 -13 %, 512 channels 14x14 -6 %,
  // 56x56 -10 %)
  const double act_bytes = (double)p.Hs * p.Ws * g.N * rowbytes;
  if (fp4 && p.Cd >= 256 && (double)taps * rowbytes >= 1024.0 && (op == MQ_OP_FWD || (g.sh == 1 && g.sw == 1)) && !env_int("MQ_TC_FP4_BN128", 0)) p.BN = 256;
  {
    const int forced_bn_ = env_int("MQ_TC_BN", 0);
    const int bn_ = (forced_bn_ >= 32 && forced_bn_ <= 256 && forced_bn_ % 32 == 0) ? (forced_bn_ < cd16 ? forced_bn_ : cd16) : p.BN;
    const int nkh_ = op == MQ_OP_FWD ? g.Kh : (g.Kh + g.sh - 1) / g.sh, nkw_ = op == MQ_OP_FWD ? g.Kw : (g.Kw + g.sw - 1) / g.sw;
    // with a single accumulator the store time adds to the tile's time instead of hiding behind the next tile: wider
    // tiles (longer store runs) then win - as long as the activations stay in L2 (measured: 28x28 -11 %, 56x56 +11 %)
    const bool serial = bn_ > 128 && act_bytes <= 110e6;
    const bool pair_hint = !mx && op == MQ_OP_BWD_DATA && g.sw == 2 && layout == MQ_NCHW && p.Wd % 2 == 0 && bn_ <= 128 && !env_int("MQ_TC_NO_PAIR", 0);
    p.TW = choose_tw(w_eff, g.N, layout, (double)nkh_ * nkw_ * rowbytes, bn_ < 128 ? bn_ : (serial ? bn_ : 128), thin, serial, pair_hint);
    if (mx) {   // a sample tile (32 samples) must lie inside a GEMM tile: 1, 2 or 4 columns; the least edge padding wins, then the
                // narrowest: with one column a warp's 32 rows ARE a sample tile, and the epilogue needs no exchange between warps
                // (measured, N = 256, 4 -> 1 columns: 1x1 512 channels 56x56 417 -> 368 us, 3x3 stride 2 input gradient 267 -> 234 us)
      double best = 1e30;
      for (int tw = 1; tw <= (ts16 ? 2 : 4); tw <<= 1) {   // emitting 16-sample blocks: a warp's rows must hold whole blocks (1 or 2 columns)
        const int tn = 128 / tw;
        const double waste = (double)((w_eff + tw - 1) / tw * tw) / w_eff * (double)((g.N + tn - 1) / tn * tn) / g.N;
        if (waste < best * (1.0 - 1e-9)) { best = waste; p.TW = tw; }
      }
      const int ftw = env_int("MQ_TC_MX_TW", 0);
      if (ftw == 1 || ftw == 2 || (ftw == 4 && !ts16)) p.TW = ftw;
    }
  }
  if (p.TW < 1 || p.TW > 32 || (p.TW & (p.TW - 1))) return false;
  p.TN = 128 / p.TW;
  p.lgTW = 0;
  while ((1 << p.lgTW) < p.TW) ++p.lgTW;
  const int forced_bn = env_int("MQ_TC_BN", 0);
  if (forced_bn >= 32 && forced_bn <= 256 && forced_bn % 32 == 0) p.BN = forced_bn < cd16 ? forced_bn : cd16;
  if (mx && (p.BN % 32 != 0 || p.TW > (ts16 ? 2 : 4))) return false;
  p.tiles_c = (p.Cd + p.BN - 1) / p.BN;
  p.tiles_w = (w_eff + p.TW - 1) / p.TW;
  p.tiles_n = (g.N + p.TN - 1) / p.TN;
  p.total_tiles = (long long)p.tiles_c * p.tiles_w * p.tiles_n * p.tiles_h * p.classes;
  if (p.total_tiles > 0x7fffffffLL) return false;
  p.lgTN = 7 - p.lgTW;
  {
    // multiply-high reciprocals for the per-tile index arithmetic: exact while numerator * divisor < 2^32
    bool exact = true;
    auto magic = [&](int d) -> uint32_t {
      if (d <= 1) return 0u;
      if ((unsigned long long)p.total_tiles * (unsigned long long)d >= (1ull << 32)) { exact = false; return 0u; }
      return (uint32_t)(((1ull << 32) + (unsigned long long)d - 1) / (unsigned long long)d);
    };
    p.m_classes = magic(p.classes); p.m_tiles_w = magic(p.tiles_w); p.m_tiles_h = magic(p.tiles_h); p.m_tiles_c = magic(p.tiles_c);
    p.m_sh = magic(g.sh); p.m_sw = magic(g.sw);
    if (!exact) return false;
  }
  // NCHW output through TMA stores (unit-stride output columns, rows of 16-byte multiples): worth its 64 KB of
  // staging only in the whole-tile kernel, whose pipeline is short; the per-tap kernel keeps its stages
  // (NCHW: rows of TW floats, at least 16 bytes; [H][W][N][C]: rows of 32 channels whatever the tile's width, whole 32-channel
  // groups per column half)
  // Strided input gradient, channel-fastest output: the staged epilogue writes a parity class through a tensor map that steps sw
  // pixels along W.  Not for NCHW: there W is the innermost axis and a class's first column (x = 1 for the odd one) would be
  // a TMA coordinate that is not on a 16-byte boundary, which the hardware refuses; NCHW keeps the paired direct stores.
  const bool strided_out = op == MQ_OP_BWD_DATA && (g.sh != 1 || g.sw != 1);
  const bool s2_tma_ok = strided_out && layout == MQ_HWNC && g.sw <= 8 && !env_int("MQ_TC_NO_S2_TMA", 0);
  const bool tma_store_ok = (!strided_out || s2_tma_ok) && p.TW <= 32 &&
                            (layout == MQ_NCHW ? (p.TW >= 4 && p.Wd % 4 == 0) : (p.Cd % 4 == 0 && p.BN % 64 == 0));
  // ... and for 1x1 layers, whose main loop is a handful of stages: the tile's time is its store (measured 4-12 % faster, 28x28 and
  // 56x56 images, 256 and 512 channels)
  // ... and for the channel-fastest output order, where a direct store is one 16-byte request per row and instruction - the request
  // count, not the bytes, bounds the store path (measured, N = 256, 512 channels: 1x1 56x56 841 -> 443 us, 3x3 28x28 447 -> 396 us,
  // the latter 2.39 PFLOP/s against 2.15 for the NCHW order)
  p.tma_store = !mx && tma_store_ok && (env_int("MQ_TC_TMA_STORE", 0) || ((taps == 1 || layout == MQ_HWNC || strided_out) && !env_int("MQ_TC_NO_TMA_STORE", 0))) ? 1 : 0;
  const size_t stage_bytes = 128 * 128 + (size_t)p.BN * 128 + (ts16 ? 6144 : 3072);
  const int sf_cols = ts16 ? 48 : 24;
  int stages = (int)((227 * 1024 - 2048 - (p.tma_store ? 65536 : 0)) / stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) return false;
  p.stages = stages;
  // TMEM (512 columns): accumulators (BN columns each) + one 24-column (E4M3 scales per 16: 48-column) scale buffer per pipeline stage
  while (stages > 2 && p.BN + sf_cols * stages > 512) --stages;
  p.stages = stages;
  p.n_acc = (2 * p.BN + sf_cols * stages <= 512) ? 2 : 1;
  if (p.n_acc * p.BN + sf_cols * stages > 512) return false;
  p.mma_cp = env_int("MQ_TC_NO_MMA_CP", 0) ? 0 : 1;   // E2M1 too: the bubble behind a copier warp costs more than the lane's extra issues
  p.pair = !mx && !p.tma_store && op == MQ_OP_BWD_DATA && g.sw == 2 && layout == MQ_NCHW && p.Wd % 2 == 0 && p.n_acc == 2 && p.total_tiles % 2 == 0 &&
           !env_int("MQ_TC_NO_PAIR", 0);
  const int nkh = op == MQ_OP_FWD ? g.Kh : (g.Kh + g.sh - 1) / g.sh, nkw = op == MQ_OP_FWD ? g.Kw : (g.Kw + g.sw - 1) / g.sw;
  p.max_stages = (nkh * nkw * p.cpt + p.G - 1) / p.G;
  // one 256-column accumulator: the epilogue copies it into registers and frees it before storing (with the staged TMA
  // stores only when a tile has at least MQ_TC_SNAP_MIN_STAGES pipeline stages of MMAs to overlap: E2M1 1x1 512 channels, two
  // stages per tile, measured 384-407 us without and 517-601 us with it; E4M3, four stages, 562-567 against 521 us)
  p.snap = (!mx && ((p.BN == 256 && p.n_acc == 1 && !p.pair) || (p.pair && p.BN == 128)) && !env_int("MQ_TC_NO_SNAP", 0) &&
            (!p.tma_store || p.max_stages >= env_int("MQ_TC_SNAP_MIN_STAGES", 4))) ? 1 : 0;
  const uint32_t fa = fp4 ? 1u : fmt_mma_code(fmt_x_like);   // kind::mxf4: 1 = E2M1; kind::mxf8f6f4: E4M3 0, E5M2 1, E2M3 3, E3M2 4
  const uint32_t fb = fp4 ? 1u : fmt_mma_code(fmt_w);
  // pairs of blocks on 256 x 256 tiles (see conv_tc_kernel's DUO): tiles 2k and 2k + 1 must exist and share the channel tile
  // (and have at least eight pipeline stages of MMAs per tile: 1x1 layers, four stages, measured 538-548 us without, 609 us with it)
  p.duo = (p.snap && !p.halo && p.KB == 128 && p.classes == 1 && p.mma_cp && p.total_tiles % 2 == 0 &&
           (p.tiles_w * p.tiles_h) % 2 == 0 && !fmt_is_6bit(fmt_x_like) && !fmt_is_6bit(fmt_w) && p.max_stages >= 8 && !env_int("MQ_TC_NO_DUO", 0)) ? 1 : 0;
  if (p.duo) {   // half of the weight tile per block: a stage is 16 KB smaller, the ring two stages deeper
    int st = (int)((227 * 1024 - 2048 - (p.tma_store ? 65536 : 0)) / (stage_bytes - (size_t)p.BN * 64));
    if (st > 8) st = 8;
    while (st > 2 && p.BN + sf_cols * st > 512) --st;
    p.stages = st;
  }
  // bit 23: scale type, 1 = E8M0, 0 = E4M3 (kind::mxf4nvf4)
  p.idesc = (fa << 7) | (fb << 10) | ((uint32_t)(p.BN >> 3) << 17) | (ts16 ? 0u : (1u << 23)) | (((p.duo ? 256u : 128u) >> 4) << 24);
  // whole-tile-per-stage variant: stride 1, one chunk per tap (<= 64 bytes of channels).  One box with the column
  // halo needs 8-column tiles; one box per column shift takes 8, 16 or 32 columns (longer NCHW store runs).
  p.halo = 0;
  if (!line && !mx && !ts16 && g.sh == 1 && g.sw == 1 && p.cpt == 1 && p.KB <= 64 && taps <= 64 && !env_int("MQ_TC_NO_HALO", 0)) {
    const int spa = fp4 ? 2 : 1, atoms_b = (p.BN + 127) / 128;
    if (p.TW == 8) {
      p.WH = p.TW + g.Kw - 1;
      p.halo_box_bytes = g.Kh * p.WH * p.TN * p.KB;
      p.halo_a_bytes = (p.halo_box_bytes + 1023) / 1024 * 1024;
      p.halo_stage_bytes = (p.halo_a_bytes + p.max_stages * 512 * spa + 1023) / 1024 * 1024;
      p.halo_b_bytes = (taps * p.BN * p.KB + p.max_stages * 512 * spa * atoms_b + 1023) / 1024 * 1024;
      const int halo_tma = tma_store_ok && !env_int("MQ_TC_NO_TMA_STORE", 0) ? 1 : 0;
      int hst = (227 * 1024 - 4096 - p.halo_b_bytes - (halo_tma ? 65536 : 0)) / p.halo_stage_bytes;
      if (hst > 4) hst = 4;
      // TMEM: accumulator(s), 16 columns per chunk of resident weight scales, 8 per chunk per stage
      while (hst >= 2 && p.BN + 16 * p.max_stages + 8 * p.max_stages * hst > 512) --hst;
      if (hst >= 2 && p.WH <= 256) {
        p.halo = 1;
        p.tma_store = halo_tma;
        p.fused = p.tiles_c == 1 && p.TN <= 32 && g.Kh * (p.TW + g.Kw - 1) * (p.KB / 32) * spa <= 128 && !env_int("MQ_TC_NO_FUSED", 0);
        p.stages = hst;
        p.n_acc = (2 * p.BN + 16 * p.max_stages + 8 * p.max_stages * hst <= 512) ? 2 : 1;
      }
    }
  }
  // unit strides and one 128-byte chunk per stage: the activation-side scale chunk of (tile, kh) equals that of the tile one
  // output row further with kh - 1, so chunks are stored per source row - Kh times fewer to expand
  p.sfa_dedup = (!p.halo && p.KB == 128 && g.sh == 1 && g.sw == 1 && !env_int("MQ_TC_NO_SFA_DEDUP", 0)) ? 1 : 0;
  p.sfa_hk = p.tiles_h + g.Kh - 1;
  out->p = p;
  size_t o = 0;
  out->off_wt_scales = 0;
  if (op == MQ_OP_BWD_DATA) { o = wt_codes_bytes(g, fmt_w); out->off_wt_scales = o; o += up256((size_t)g.Ct * taps * g.Cot * (ts16 ? 4 : 1)); }
  out->off_sfa = o; o += up256(conv_tc_sfa_bytes(p));
  out->off_sfb = o; o += up256(conv_tc_sfb_bytes(p));
  out->off_bimg = o;
  if (p.halo) o += up256((size_t)p.tiles_c * taps * p.BN * p.KB);
  out->off_pack_a = o;
  if (fmt_is_6bit(fmt_x_like)) o += up256((size_t)p.Hs * p.Ws * g.N * rowbytes);
  out->off_pack_b = o;
  if (fmt_is_6bit(fmt_w)) o += up256((size_t)out->rows_b * taps * rowbytes);
  out->total = o;
  return true;
}

// Scratch of a forward / input-gradient call: the tensor-core plan's where one exists (it depends on the output layout: the
// larger of the two), never less than what the CUDA-core kernels need, which take the layers a plan refuses.
size_t conv_tc_workspace(int op, const Geom& g, int fmt_x_like, int fmt_w, bool line, bool ts16 = false) {
  size_t need = conv_generic_workspace(op, g);
  for (int layout = 0; layout < 2; ++layout) {   // the tile shape, hence the scratch, depends on the output layout
    ConvTcPlan pl;
    if (conv_tc_plan(op, g, fmt_x_like, fmt_w, layout, &pl, line, false, ts16) && pl.total > need) need = pl.total;
  }
  return need;
}

// Every tensor map of the call is encoded before its first launch, so a failing encode leaves nothing enqueued.
mq_status run_conv_tc(int op, const Geom& g, ConvTcPlan& pl, const mq_qtensor* qx_like, const mq_qtensor* qw, float* out, int layout, void* ws,
                      unsigned int* status, cudaStream_t stream) {
  ConvTcParams& p = pl.p;
  const int taps = g.Kh * g.Kw;
  uint8_t* base = static_cast<uint8_t*>(ws);
  // where the kernels will find their operands: as stored, or in scratch (W re-laid for the input gradient; 6-bit operands
  // repacked - 16 codes -> 12 packed bytes + 4 bytes of padding per 16-byte chunk, the container of the MMA's 6-bit types)
  const uint8_t* w_stored = static_cast<const uint8_t*>(qw->codes);
  const uint8_t* x_stored = static_cast<const uint8_t*>(qx_like->codes);
  // (operands in packed 6-bit storage - 16 codes in 12 bytes - reach that container by a copy that pads each group; the
  // weights of the input gradient arrive here one code per byte whatever their storage: their re-layout reads bytes)
  const int fx = fmt_base(qx_like->fmt), fw = fmt_base(qw->fmt);
  const bool pk_x = fmt_is_packed6(qx_like->fmt), pk_w = fmt_is_packed6(qw->fmt);
  if (pk_w && op != MQ_OP_FWD) return MQ_ERR_INVALID_ARG;
  const uint8_t* b_unpacked = op == MQ_OP_FWD ? w_stored : base;
  const uint8_t* b_codes = fmt_is_6bit(fw) ? base + pl.off_pack_b : b_unpacked;
  const uint8_t* a_codes = fmt_is_6bit(fx) ? base + pl.off_pack_a : x_stored;
  uint8_t* wt_scales = base + pl.off_wt_scales;
  bool separate_transpose = false;
  if (op == MQ_OP_FWD) {
    p.b_scales = qw->scales;
  } else {
    // per-tap kernel, operands that need no repacking: the re-layout rides in the scale-expansion launch
    p.wt_fused = (!p.halo && !fmt_is_6bit(fw) && (p.kind_fp4 == 2 || !env_int("MQ_TC_NO_WT_FUSED", 0))) ? 1 : 0;   // kind 2: this route only
    if (p.wt_fused) {
      p.wt_in = w_stored; p.wt_out = base; p.wt_sc_in = qw->scales;
      p.wt_Cout = g.Cout; p.wt_Cop = g.Cop; p.wt_Cp = g.Cp; p.wt_bx = g.Cp / 32; p.wt_by = g.Cop / 32;
    } else separate_transpose = true;
    p.b_scales = wt_scales;
  }
  p.a_scales = qx_like->scales;
  p.a_tscale = qx_like->tensor_scale; p.b_tscale = qw->tensor_scale;
  p.sfa_img = base + pl.off_sfa;
  p.sfb_img = base + pl.off_sfb;
  p.b_codes = b_codes; p.b_rows_total = pl.rows_b; p.b_rowbytes = pl.rowbytes; p.b_img = base + pl.off_bimg;
  p.out = out; p.out_layout = layout; p.status = status;

  CUtensorMap map_a, map_w;
  bool direct_x = false;
  {
    const uint64_t rb = (uint64_t)pl.rowbytes;
    const uint64_t dims[4] = {rb, (uint64_t)p.Ws, (uint64_t)g.N, (uint64_t)p.Hs};
    const uint64_t strides[3] = {(uint64_t)g.N * rb, rb, (uint64_t)p.Ws * g.N * rb};
    const uint32_t wst = op == MQ_OP_FWD ? (uint32_t)g.sw : 1u;
    uint32_t box[4] = {(uint32_t)p.KB, (uint32_t)((p.TW - 1) * wst + 1), (uint32_t)p.TN, 1u};
    if (p.halo) { box[1] = (uint32_t)p.WH; box[3] = (uint32_t)g.Kh; }   // the whole halo of a tile in one box
    const uint32_t es[4] = {1u, wst, 1u, 1u};
    // a packed activation / gradient tensor with rows of whole 128-code boxes is read where it is stored (the copy engine pads
    // each 12-byte group on its way into shared memory): no scratch copy, no pass over the tensor before the GEMM
    if (pk_x && p.KB == 128 && rb % 128 == 0 && !env_int("MQ_TC_NO_P6_DIRECT", 0)) {
      const uint64_t ps[3] = {strides[0] * 3 / 4, strides[1] * 3 / 4, strides[2] * 3 / 4};
      direct_x = encode_tensor_map_p6(&map_a, x_stored, 4, dims, ps, box, es);
    }
    if (!direct_x && !encode_tensor_map_u8(&map_a, a_codes, 4, dims, strides, box, es, p.KB)) return MQ_ERR_CUDA;
    p.a_tx34 = direct_x ? 1 : 0;
    if (direct_x && p.halo) p.halo_box_bytes = p.halo_box_bytes * 3 / 4;
  }
  map_w = map_a;
  if (p.halo) {
    if (p.fused) {
      // all taps of the weight tile in one box: dims ordered (channel bytes, rows, taps)
      const uint64_t rb = (uint64_t)pl.rowbytes;
      const uint64_t dims[3] = {rb, (uint64_t)pl.rows_b, (uint64_t)taps};
      const uint64_t strides[2] = {(uint64_t)taps * rb, rb};
      const uint32_t box[3] = {(uint32_t)p.KB, (uint32_t)p.BN, (uint32_t)taps};
      if (!encode_tensor_map_u8(&map_w, b_codes, 3, dims, strides, box, nullptr, p.KB)) return MQ_ERR_CUDA;
    }
  } else {
    const uint64_t rb = (uint64_t)pl.rowbytes;
    const uint64_t dims[3] = {rb, (uint64_t)taps, (uint64_t)pl.rows_b};
    const uint64_t strides[2] = {rb, (uint64_t)taps * rb};
    const uint32_t box[3] = {(uint32_t)p.KB, 1u, (uint32_t)(p.duo ? p.BN / 2 : p.BN)};   // (a pair of blocks: each loads half of the tile's rows)
    if (!encode_tensor_map_u8(&map_w, b_codes, 3, dims, strides, box, nullptr, p.KB)) return MQ_ERR_CUDA;
  }
  CUtensorMap map_sfa = map_a, map_sfb = map_a;
  if (p.duo) {   // the scale images as rows of 256 bytes: one box = the chunks of one stage
    const uint32_t spa = p.kind_fp4 == 2 ? 4u : (p.kind_fp4 == 1 ? 2u : 1u), atoms_b = (uint32_t)(p.BN + 127) / 128;
    const uint64_t da[2] = {256, (uint64_t)(conv_tc_sfa_bytes(p) / 256)}, db[2] = {256, (uint64_t)(conv_tc_sfb_bytes(p) / 256)}, st[1] = {256};
    const uint32_t ba[2] = {256u, 2u * spa}, bb[2] = {256u, 2u * spa * atoms_b};
    if (!encode_tensor_map_u8(&map_sfa, p.sfa_img, 2, da, st, ba, nullptr, 0)) return MQ_ERR_CUDA;
    if (!encode_tensor_map_u8(&map_sfb, p.sfb_img, 2, db, st, bb, nullptr, 0)) return MQ_ERR_CUDA;
  }
  CUtensorMap map_out = map_a;
  if (p.tma_store) {
    if (reinterpret_cast<uintptr_t>(out) % 16 != 0) p.tma_store = 0;
    else {
      if (layout == MQ_NCHW) {
        // the output seen as (W, N, C, H); one epilogue warp's 32 rows x the channels of a column half (at most 64)
        const uint64_t dims[4] = {(uint64_t)p.Wd, (uint64_t)g.N, (uint64_t)p.Cd, (uint64_t)p.Hd};
        const uint64_t strides[3] = {(uint64_t)p.Cd * p.Hd * p.Wd * 4, (uint64_t)p.Hd * p.Wd * 4, (uint64_t)p.Wd * 4};
        const int half_cols = (p.BN / 2 + 15) & ~15;
        const uint32_t box[4] = {(uint32_t)p.TW, (uint32_t)(32 / p.TW), (uint32_t)(half_cols < 64 ? half_cols : 64), 1u};
        if (!encode_tensor_map_u8(&map_out, out, 4, dims, strides, box, nullptr, 0, true)) return MQ_ERR_CUDA;
      } else {
        // [Ho][Wo][N][C] seen as (C, W, N, H) -- the order of a tile's rows: a warp's 32 rows x 32 channels, rows of 128
        // bytes with the 128-byte swizzle
        const uint64_t dims[4] = {(uint64_t)p.Cd, (uint64_t)p.Wd, (uint64_t)g.N, (uint64_t)p.Hd};
        const uint64_t strides[3] = {(uint64_t)g.N * p.Cd * 4, (uint64_t)p.Cd * 4, (uint64_t)p.Wd * g.N * p.Cd * 4};
        // strided input gradient: a parity class's columns are sw pixels apart - the box steps sw along W (TW of its pixels land)
        const uint32_t esw = op == MQ_OP_BWD_DATA ? (uint32_t)g.sw : 1u;
        const uint32_t box[4] = {32u, (uint32_t)p.TW * esw, (uint32_t)(32 / p.TW), 1u};
        const uint32_t es[4] = {1u, esw, 1u, 1u};
        if (!encode_tensor_map_u8(&map_out, out, 4, dims, strides, box, es, 128, true)) return MQ_ERR_CUDA;
      }
    }
  }
  // ---- launches
  if (separate_transpose && launch_weight_transpose(w_stored, qw->scales, base, wt_scales, g, fw, stream) != cudaSuccess) return MQ_ERR_CUDA;
  if (fmt_is_6bit(fx) && !direct_x) {
    const size_t n = (size_t)p.Hs * p.Ws * g.N * pl.rowbytes;
    if ((pk_x ? launch_unpack6(x_stored, base + pl.off_pack_a, n, 0, fx, stream) : launch_pack6(x_stored, base + pl.off_pack_a, n, stream)) != cudaSuccess) return MQ_ERR_CUDA;
  }
  if (fmt_is_6bit(fw)) {
    const size_t n = (size_t)pl.rows_b * taps * pl.rowbytes;
    if ((pk_w ? launch_unpack6(b_unpacked, base + pl.off_pack_b, n, 0, fw, stream) : launch_pack6(b_unpacked, base + pl.off_pack_b, n, stream)) != cudaSuccess) return MQ_ERR_CUDA;
  }
  if (!(p.halo && p.fused) && launch_expand_conv_scales(p, stream) != cudaSuccess) return MQ_ERR_CUDA;
  return launch_conv_tc(p, map_a, map_w, map_out, stream, &map_sfa, &map_sfb) == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

// ---- weight gradient on tensor cores ---------------------------------------------------------------
// Scratch: [split-K partials][A-side scale chunks][B-side scale chunks][E2M1: re-laid X][E2M1: re-laid G_Y]
struct WgradPlan {
  bool ok;
  WgradTcParams p;
  int Npad, P_a, P_b;
  size_t off_sfa, off_sfb, off_xt, off_gt, total;
  bool recode4;   // E2M1 operands re-encoded as E4M3 bytes for the 8-bit path
};

// ts16: the paper's own format (E4M3 scales per 16 x 16 block): the two E2M1 modes with kind::mxf4nvf4
WgradPlan wgrad_plan(const Geom& g, int fmt_x, int fmt_g, bool ts16 = false) {
  WgradPlan w{};
  if (ts16 && (fmt_x != MQ_E2M1 || fmt_g != MQ_E2M1 || env_int("MQ_TC_NO_TS16", 0))) return w;
  if (env_int("MQ_DISABLE_TC", 0) || env_int("MQ_DISABLE_TC_WGRAD", 0)) return w;
  const bool fp4_in = fmt_x == MQ_E2M1 && fmt_g == MQ_E2M1;
  const bool fp8_in = fmt_x != MQ_E2M1 && fmt_g != MQ_E2M1;
  if (!fp4_in && !fp8_in) return w;
  // E2M1 layers that the flat mode below does not take (stride 2, batches that are not 1, 2, 4 or 8 sample tiles): every
  // E2M1 value is an E4M3 value, so the codes are re-encoded exactly as E4M3 bytes in scratch and the 8-bit path (stored
  // order read MN-major, block pairs) runs - faster than the per-pixel E2M1 mode (MQ_WGRAD_FP4_PIXEL=1 keeps that mode)
  const bool flat_ok = fp4_in && g.sh == 1 && g.sw == 1 && (g.Nt == 1 || g.Nt == 2 || g.Nt == 4 || g.Nt == 8) && !env_int("MQ_WGRAD_NO_FLAT", 0);
  const bool recode4 = fp4_in && !flat_ok && !ts16 && !env_int("MQ_WGRAD_FP4_PIXEL", 0);   // (E4M3 block scales are no E8M0 scales: not for ts16)
  const bool fp4 = fp4_in && !recode4;
  const bool fp8 = fp8_in || recode4;
  w.recode4 = recode4;
  // 6-bit operands: this GEMM reads its operands MN-major (K = samples), where the MMA's packed 6-bit container (packed
  // along K) does not apply; every E3M2 / E2M3 value is also an E4M3 value, so the codes are re-encoded exactly as
  // E4M3 bytes in scratch and the 8-bit path runs unchanged (MQ_TC_NO_FP6=1: CUDA-core kernels)
  if ((fmt_is_6bit(fmt_x) || fmt_is_6bit(fmt_g)) && env_int("MQ_TC_NO_FP6", 0)) return w;
  WgradTcParams& p = w.p;
  p.N = g.N; p.Nt = g.Nt; p.Ho = g.Ho; p.Wo = g.Wo; p.H = g.H; p.W = g.W; p.Cout = g.Cout; p.Cp = g.Cp; p.Ct = g.Ct; p.Cot = g.Cot;
  p.Kh = g.Kh; p.Kw = g.Kw; p.sh = g.sh; p.sw = g.sw; p.ph = g.ph; p.pw = g.pw;
  const bool flat = fp4 && g.sh == 1 && g.sw == 1 && (g.Nt == 1 || g.Nt == 2 || g.Nt == 4 || g.Nt == 8) && !env_int("MQ_WGRAD_NO_FLAT", 0);
  p.mode = fp8 ? MQ_WG_FP8 : (flat ? MQ_WG_FP4_FLAT : MQ_WG_FP4_PIXEL);
  p.kind = ts16 ? 2 : (fp4 ? 1 : 0);
  const int sf_cols1 = ts16 ? 16 : 8;       // TMEM columns and shared-memory bytes of one 128-row scale chunk
  const int sf_bytes1 = ts16 ? 2048 : 1024;
  if (fp4) p.BPP = flat ? g.Nt : (g.Nt >= 5 ? 8 : (g.Nt >= 3 ? 4 : g.Nt));
  else p.BPP = g.Nt >= 3 ? 4 : g.Nt;
  p.KPX = (fp4 ? 8 : 4) / p.BPP;
  p.KBn = 16 * p.BPP;
  p.nchunks = (g.Nt + p.BPP - 1) / p.BPP;
  w.Npad = 32 * p.BPP * p.nchunks;
  p.groups_w = (g.Wo + p.KPX - 1) / p.KPX;
  p.Wp = g.W + 2 * g.pw;
  p.Hp = g.H + 2 * g.ph;
  p.mma_cp = env_int("MQ_WGRAD_MMA_CP", 0);
  p.stages_total = flat ? (g.Ho * p.Wp + p.KPX - 1) / p.KPX : g.Ho * p.groups_w * p.nchunks;
  p.b_rows = flat ? (g.Cp < 128 ? g.Cp : 128) : 128;
  // 8-bit operands: 256 input channels per MMA when the layer has them (the kernel is bound by the tensor core's
  // shared-memory operand reads, and a wider N reads the G_Y tile once for twice the work)
  if (fp8 && g.Cp >= 256 && !env_int("MQ_WGRAD_N128", 0)) p.b_rows = 256;
  p.m_tiles = (g.Cout + 127) / 128;
  p.m_tiles128 = p.m_tiles;
  // Pairs of blocks on 256 x 256 tiles (cta_group::2) when both channel counts allow it: half the X bytes per block
  // and stage, so six pipeline stages instead of four, and one MMA instruction per 256 x 256 x 32 for the issuing lane.
  p.cta2 = fp8 && p.b_rows == 256 && g.Cout >= 256 && !env_int("MQ_WGRAD_NO_CTA2", 0);
  if (p.cta2) { p.m_tiles = (g.Cout + 255) / 256; p.m_tiles128 = 2 * p.m_tiles; }
  // Thin 8-bit layers (32 or 64 input channels, unit strides): with one tap per block a 128-row B tile is mostly zero
  // fill.  Instead the Kw taps of a kernel row form one B operand of Kw * Cp rows: a stage loads a strip of
  // KPX + Kw - 1 pixels once ([pixel][sample][Cp bytes], swizzle span = Cp) and tap kw's panel is that strip one pixel
  // further - Kw times fewer stages, G_Y loads and MMA instructions.
  // (With a column stride the strip is the contiguous run of (KPX - 1) sw + Kw input pixels: output pixel a's tap kw is
  // input pixel a sw + kw of the strip, so panels stay one pixel apart and K slices sw pixels apart.)
  p.grp8 = (fp8 && !p.cta2 && g.Kw > 1 && (g.Cp == 32 || g.Cp == 64) && g.Kw * g.Cp <= 256 && !env_int("MQ_WGRAD_NO_GROUP8", 0)) ? 1 : 0;
  if (p.grp8) p.b_rows = g.Cp;
  p.cb_tiles = (g.Cp + p.b_rows - 1) / p.b_rows;
  // taps per block: a whole kernel row in the flat mode when its accumulators fit in tensor memory
  p.TG = p.grp8 ? g.Kw : 1;
  if (flat && g.Kw > 1 && g.Kw * p.b_rows + 2 * sf_cols1 * (1 + (g.Kw * p.b_rows + 127) / 128) <= 512 && !env_int("MQ_WGRAD_NO_GROUP", 0)) p.TG = g.Kw;
  p.NB = (p.TG * p.b_rows + 127) / 128;
  p.n0 = p.TG * p.b_rows < 256 ? p.TG * p.b_rows : 256;
  p.n1 = p.TG * p.b_rows - p.n0;
  p.j_tiles = (g.Kh * g.Kw / p.TG) * p.cb_tiles;
  const int items = p.m_tiles * p.j_tiles;
  int splits = env_int("MQ_WGRAD_SPLITS", 0);
  const int units = p.cta2 ? sm_count() / 2 : sm_count();   // blocks, or pairs of blocks, that run at once
  if (splits <= 0) splits = items >= units ? 1 : units / items;
  if (splits > p.stages_total) splits = p.stages_total;
  if (splits < 1) splits = 1;
  p.splits = splits;
  p.b_tile_bytes = flat ? (p.KPX + p.TG - 1) * p.b_rows * p.KBn : (p.cta2 ? 128 : p.b_rows) * 128;   // a pair's blocks load half of X each
  if (p.grp8) p.b_tile_bytes = ((p.KPX - 1) * g.sw + p.TG) * 32 * p.BPP * g.Cp;
  p.stage_bytes = (128 * 128 + p.b_tile_bytes + (1 + p.NB) * sf_bytes1 + 1023) / 1024 * 1024;
  {
    int st = (227 * 1024 - 2048) / p.stage_bytes;
    if (st > 6) st = 6;
    int slots = st;
    // kind 2: the scale buffers are twice as wide; rather than giving up pipeline stages, fewer buffers are used in turn
    if (ts16 && !env_int("MQ_WGRAD_TS_NO_SLOTS", 0)) { while (slots > 2 && p.TG * p.b_rows + slots * sf_cols1 * (1 + p.NB) > 512) --slots; }
    else { while (st > 2 && p.TG * p.b_rows + st * sf_cols1 * (1 + p.NB) > 512) --st; slots = st; }
    p.stages = st;
    p.sf_slots = slots;
    const int cols = p.TG * p.b_rows + slots * sf_cols1 * (1 + p.NB);
    p.tmem_cols = cols <= 256 ? 256 : 512;
    if (st < 2 || cols > 512) return w;
  }
  const int spa = ts16 ? 4 : (fp4 ? 2 : 1);
  w.P_a = p.stages_total * p.KPX;
  w.P_b = (w.P_a + (g.Kh - 1) * p.Wp + g.Kw - 1 + 7) / 8 * 8;
  size_t o = up256((size_t)splits * g.Cout * g.Kh * g.Kw * g.Cp * sizeof(float));
  w.off_sfa = o; o += up256((size_t)p.m_tiles128 * p.stages_total * 512 * spa);
  // flat mode with whole 128-channel tap panels: the X-side scale chunks once per padded start pixel (Kh Kw / KPX times fewer)
  p.sfb_S = (flat && p.b_rows == 128 && !env_int("MQ_WGRAD_NO_SFB_DEDUP", 0)) ? w.P_b : 0;
  w.off_sfb = o; o += up256(fp8 ? (size_t)p.cb_tiles * p.Hp * p.Wp * p.nchunks * p.NB * 512
                                : p.sfb_S > 0 ? ((size_t)p.cb_tiles * p.sfb_S + p.NB) * 512 * spa
                                              : (size_t)p.cb_tiles * (g.Kh * g.Kw / p.TG) * p.stages_total * p.NB * 512 * spa);
  w.off_xt = o;
  if (flat) { p.xt_block_bytes = (long long)w.P_b * p.b_rows * p.KBn; o += up256((size_t)p.cb_tiles * p.xt_block_bytes); }
  else if (fp4) o += up256((size_t)g.Cp * g.H * g.W * w.Npad / 2);
  else if (fmt_is_6bit(fmt_x) || recode4) o += up256((size_t)g.H * g.W * g.N * g.Cp);     // X re-encoded as E4M3
  w.off_gt = o;
  if (flat) { p.gt_block_bytes = (long long)w.P_a * 128 * p.KBn; o += up256((size_t)p.m_tiles * p.gt_block_bytes); }
  else if (fp4) o += up256((size_t)g.Cop * g.Ho * g.Wo * w.Npad / 2);
  else if (fmt_is_6bit(fmt_g) || recode4) o += up256((size_t)g.Ho * g.Wo * g.N * g.Cop);  // G_Y re-encoded as E4M3
  w.total = o;
  w.ok = true;
  return w;
}

mq_status run_wgrad_tc(const Geom& g, WgradPlan& w, const mq_qtensor* qx, const mq_qtensor* qg, float* out, int layout, void* ws,
                       unsigned int* status, cudaStream_t stream) {
  uint8_t* base = static_cast<uint8_t*>(ws);
  float* partial = reinterpret_cast<float*>(base);
  WgradTcParams& p = w.p;
  p.g_scales = qg->scales; p.x_scales = qx->scales; p.partial = partial; p.status = status;
  p.sfa_img = base + w.off_sfa; p.sfb_img = base + w.off_sfb;
  uint8_t* xt = base + w.off_xt;
  uint8_t* gt = base + w.off_gt;
  CUtensorMap map_a{}, map_b{};
  const uint32_t sf_type = p.kind == 2 ? 0u : (1u << 23);   // instruction descriptor bit 23: E8M0 scales (0: E4M3)
  if (p.mode == MQ_WG_FP4_FLAT) {
    p.xt = xt; p.gt = gt;
    p.idesc = (1u << 7) | (1u << 10) | sf_type | ((128u >> 4) << 24);
  } else if (p.mode == MQ_WG_FP4_PIXEL) {
    if (launch_fp4_to_n_major(static_cast<const uint8_t*>(qx->codes), xt, g.H * g.W, g.N, g.Cp, w.Npad, stream) != cudaSuccess) return MQ_ERR_CUDA;
    if (launch_fp4_to_n_major(static_cast<const uint8_t*>(qg->codes), gt, g.Ho * g.Wo, g.N, g.Cop, w.Npad, stream) != cudaSuccess) return MQ_ERR_CUDA;
    p.idesc = (1u << 7) | (1u << 10) | sf_type | ((128u >> 4) << 24);
    const uint64_t nb = (uint64_t)w.Npad / 2;
    const int swz = p.KBn >= 32 ? p.KBn : 0;
    {
      const uint64_t dims[4] = {nb, (uint64_t)g.Cop, (uint64_t)g.Wo, (uint64_t)g.Ho};
      const uint64_t strides[3] = {nb, (uint64_t)g.Cop * nb, (uint64_t)g.Wo * g.Cop * nb};
      const uint32_t box[4] = {(uint32_t)p.KBn, 128u, 1u, 1u};
      if (!encode_tensor_map_u8(&map_a, gt, 4, dims, strides, box, nullptr, swz)) return MQ_ERR_CUDA;
    }
    {
      const uint64_t dims[4] = {nb, (uint64_t)g.Cp, (uint64_t)g.W, (uint64_t)g.H};
      const uint64_t strides[3] = {nb, (uint64_t)g.Cp * nb, (uint64_t)g.W * g.Cp * nb};
      const uint32_t box[4] = {(uint32_t)p.KBn, 128u, 1u, 1u};
      if (!encode_tensor_map_u8(&map_b, xt, 4, dims, strides, box, nullptr, swz)) return MQ_ERR_CUDA;
    }
  } else {
    const uint8_t* g_codes = static_cast<const uint8_t*>(qg->codes);
    const uint8_t* x_codes = static_cast<const uint8_t*>(qx->codes);
    int fmt_g_eff = fmt_base(qg->fmt), fmt_x_eff = fmt_base(qx->fmt);
    if (fmt_is_6bit(fmt_x_eff)) {   // (from either storage of the 6-bit codes)
      const size_t n = (size_t)g.H * g.W * g.N * g.Cp;
      if ((fmt_is_packed6(qx->fmt) ? launch_unpack6(x_codes, xt, n, 2, fmt_x_eff, stream) : launch_recode6_e4m3(x_codes, xt, n, fmt_x_eff, stream)) != cudaSuccess) return MQ_ERR_CUDA;
      x_codes = xt; fmt_x_eff = MQ_E4M3;
    }
    if (fmt_is_6bit(fmt_g_eff)) {
      const size_t n = (size_t)g.Ho * g.Wo * g.N * g.Cop;
      if ((fmt_is_packed6(qg->fmt) ? launch_unpack6(g_codes, gt, n, 2, fmt_g_eff, stream) : launch_recode6_e4m3(g_codes, gt, n, fmt_g_eff, stream)) != cudaSuccess) return MQ_ERR_CUDA;
      g_codes = gt; fmt_g_eff = MQ_E4M3;
    }
    if (w.recode4) {
      if (launch_recode4_e4m3(x_codes, xt, (size_t)g.H * g.W * g.N * g.Cp, stream) != cudaSuccess) return MQ_ERR_CUDA;
      if (launch_recode4_e4m3(g_codes, gt, (size_t)g.Ho * g.Wo * g.N * g.Cop, stream) != cudaSuccess) return MQ_ERR_CUDA;
      x_codes = xt; g_codes = gt; fmt_x_eff = MQ_E4M3; fmt_g_eff = MQ_E4M3;
    }
    const uint32_t fa = fmt_mma_code(fmt_g_eff), fb = fmt_mma_code(fmt_x_eff);
    p.idesc = (fa << 7) | (fb << 10) | (1u << 15) | (1u << 16) | (1u << 23) | (((p.cta2 ? 256u : 128u) >> 4) << 24);
    {
      const uint64_t rb = (uint64_t)g.Cop;
      const uint64_t dims[4] = {rb, (uint64_t)g.N, (uint64_t)g.Wo, (uint64_t)g.Ho};
      const uint64_t strides[3] = {rb, (uint64_t)g.N * rb, (uint64_t)g.Wo * g.N * rb};
      const uint32_t box[4] = {128u, (uint32_t)(p.BPP * 32), (uint32_t)p.KPX, 1u};
      if (!encode_tensor_map_u8(&map_a, g_codes, 4, dims, strides, box, nullptr, 128)) return MQ_ERR_CUDA;
    }
    {
      const uint64_t rb = (uint64_t)g.Cp;
      const uint64_t dims[4] = {rb, (uint64_t)g.N, (uint64_t)g.W, (uint64_t)g.H};
      const uint64_t strides[3] = {rb, (uint64_t)g.N * rb, (uint64_t)g.W * g.N * rb};
      uint32_t box[4] = {128u, (uint32_t)(p.BPP * 32), (uint32_t)((p.KPX - 1) * g.sw + 1), 1u};
      uint32_t es[4] = {1u, 1u, (uint32_t)g.sw, 1u};
      if (p.grp8) { box[0] = (uint32_t)g.Cp; box[2] = (uint32_t)((p.KPX - 1) * g.sw + p.TG); es[2] = 1u; }   // the contiguous strip of a kernel row's taps, rows of Cp bytes
      if (!encode_tensor_map_u8(&map_b, x_codes, 4, dims, strides, box, es, p.grp8 ? g.Cp : 128)) return MQ_ERR_CUDA;
    }
  }
  if (p.mode == MQ_WG_FP4_FLAT) {
    if (launch_wgrad_flat_prep(p, static_cast<const uint8_t*>(qx->codes), xt, w.P_b, static_cast<const uint8_t*>(qg->codes), gt, w.P_a, stream) != cudaSuccess)
      return MQ_ERR_CUDA;
  } else if (launch_expand_wgrad_scales(p, stream) != cudaSuccess) return MQ_ERR_CUDA;
  CUtensorMap map_p{};
  {
    const uint64_t J = (uint64_t)g.Kh * g.Kw * g.Cp;
    const uint64_t dims[3] = {J, (uint64_t)g.Cout, (uint64_t)p.splits};
    const uint64_t strides[2] = {J * 4, (uint64_t)g.Cout * J * 4};
    const uint32_t box[3] = {32u, 32u, 1u};
    if (!encode_tensor_map_u8(&map_p, partial, 3, dims, strides, box, nullptr, 128, true)) return MQ_ERR_CUDA;
  }
  CUtensorMap map_sfa{}, map_sfb{};
  if (p.cta2) {   // a pair's scale chunks travel as tiled copies too (rows of 256 bytes), so that they can count on the leader's barrier
    const int spa = 1;   // 8-bit operands only
    const uint64_t rows_a = (uint64_t)p.m_tiles128 * p.stages_total * 2 * spa;
    const uint64_t rows_b = (uint64_t)p.cb_tiles * p.Hp * p.Wp * p.nchunks * p.NB * 2 * spa;
    const uint64_t da[2] = {256, rows_a}, db[2] = {256, rows_b}, st[1] = {256};
    const uint32_t ba[2] = {256u, (uint32_t)(2 * spa)}, bb[2] = {256u, (uint32_t)(2 * spa * p.NB)};
    if (!encode_tensor_map_u8(&map_sfa, p.sfa_img, 2, da, st, ba, nullptr, 0)) return MQ_ERR_CUDA;
    if (!encode_tensor_map_u8(&map_sfb, p.sfb_img, 2, db, st, bb, nullptr, 0)) return MQ_ERR_CUDA;
  }
  if (launch_wgrad_tc(p, map_a, map_b, map_p, map_sfa, map_sfb, stream) != cudaSuccess) return MQ_ERR_CUDA;
  const bool tsc = p.kind == 2;
  return launch_bwd_weight_reduce(partial, out, g, p.splits, layout, stream, tsc ? qx->tensor_scale : nullptr, tsc ? qg->tensor_scale : nullptr) == cudaSuccess
             ? MQ_OK : MQ_ERR_CUDA;
}

// address of the current device's status word (a __device__ variable has one instance per device and per context:
// looked up on every call, a host-side table lookup, so that no address outlives a cudaDeviceReset)
unsigned int* device_status_ptr() {
  void* q = nullptr;
  if (cudaGetSymbolAddress(&q, g_device_status) != cudaSuccess) return nullptr;
  return static_cast<unsigned int*>(q);
}

// argument checks common to the three convolution entry points (everything but the workspace)
mq_status check_conv_args(int op, const mq_conv_desc* desc, const mq_qtensor* qa, int role_a, const mq_qtensor* qb, int role_b, const void* out, int dtype,
                          int layout) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  const Geom g = make_geom(*desc);
  if ((st = check_qtensor(g, qa, role_a)) != MQ_OK) return st;
  if ((st = check_qtensor(g, qb, role_b)) != MQ_OK) return st;
  if (!out) return MQ_ERR_INVALID_ARG;
  if (layout != MQ_NCHW && layout != MQ_HWNC) return MQ_ERR_INVALID_ARG;
  if (!valid_dtype(dtype)) return MQ_ERR_INVALID_ARG;
  if (!aligned16(out)) return MQ_ERR_ALIGNMENT;
  if (qa->block != qb->block) return MQ_ERR_UNSUPPORTED;
  // a line-quantized tensor serves the GEMM that contracts along its lines and no other (Sec. III-B, III-C)
  if (qa->block == MQ_BLOCK_LINE32 && op != MQ_OP_FWD) return MQ_ERR_UNSUPPORTED;
  if (dtype != MQ_F32) return MQ_ERR_UNSUPPORTED;
  return MQ_OK;
}

// Does a forward / input-gradient call of this layer, formats and output layout run on the tensor cores?  (formats: one code per byte)
bool conv_takes_tc(int op, const Geom& g, int fmt_x_like, int fmt_w, int layout, bool line, bool ts16, ConvTcPlan* pl) {
  return (!ts16 || !env_int("MQ_TC_NO_TS16", 0)) && (op == MQ_OP_FWD || op == MQ_OP_BWD_DATA) && conv_tc_eligible(op, g, fmt_x_like, fmt_w) &&
         conv_tc_plan(op, g, fmt_x_like, fmt_w, layout, pl, line, false, ts16);
}

// Operands in packed 6-bit storage: scratch, behind the call's own, for the one-code-per-byte copies of the operands no
// kernel of the call's route reads packed - the weights of the input gradient (their re-layout reads bytes) and both
// operands of a layer the CUDA-core kernels take.  (The tensor-core routes read a packed activation / gradient tensor
// through the copy that builds the MMA's container, which a one-code-per-byte tensor needs as well.)
struct PackedExtra { bool keep_a, keep_b; size_t bytes_a, bytes_b; };
int operand_role(int op, int which) {
  if (op == MQ_OP_FWD) return which == 0 ? MQ_ROLE_X : MQ_ROLE_W;
  if (op == MQ_OP_BWD_DATA) return which == 0 ? MQ_ROLE_W : MQ_ROLE_DY;
  return which == 0 ? MQ_ROLE_X : MQ_ROLE_DY;
}
PackedExtra packed_extra(int op, const Geom& g, int fmt_a, int fmt_b, int block) {
  PackedExtra e{false, false, 0, 0};
  const bool pa = fmt_is_packed6(fmt_a), pb = fmt_is_packed6(fmt_b);
  if (!pa && !pb) return e;
  const int fa = fmt_base(fmt_a), fb = fmt_base(fmt_b);
  const bool line = block == MQ_BLOCK_LINE32, ts16 = block == MQ_BLOCK_TS16;
  bool tc = true;    // on the tensor cores whatever the output layout
  ConvTcPlan pl;
  if (op == MQ_OP_BWD_WEIGHT) tc = wgrad_plan(g, fa, fb, ts16).ok;
  else for (int layout = 0; layout < 2; ++layout) tc = tc && conv_takes_tc(op, g, op == MQ_OP_FWD ? fa : fb, op == MQ_OP_FWD ? fb : fa, layout, line, ts16, &pl);
  e.keep_a = pa && (!tc || op == MQ_OP_BWD_DATA);
  e.keep_b = pb && !tc;
  const View va = view_of(g, operand_role(op, 0)), vb = view_of(g, operand_role(op, 1));
  e.bytes_a = e.keep_a ? ((size_t)(va.P * va.R * va.Cp) + 255) / 256 * 256 : 0;
  e.bytes_b = e.keep_b ? ((size_t)(vb.P * vb.R * vb.Cp) + 255) / 256 * 256 : 0;
  return e;
}
size_t conv_workspace_unpacked(int op, const Geom& g, int fa, int fb, int block) {
  const bool line = block == MQ_BLOCK_LINE32, ts16 = block == MQ_BLOCK_TS16;
  size_t bytes = conv_generic_workspace(op, g);
  if (op == MQ_OP_FWD && conv_tc_eligible(op, g, fa, fb)) bytes = conv_tc_workspace(op, g, fa, fb, line, ts16);
  if (op == MQ_OP_BWD_DATA && conv_tc_eligible(op, g, fb, fa)) bytes = conv_tc_workspace(op, g, fb, fa, false, ts16);
  if (op == MQ_OP_BWD_WEIGHT) {
    const WgradPlan w = wgrad_plan(g, fa, fb, ts16);
    if (w.ok) bytes = w.total;
  }
  return bytes;
}

mq_status run_conv(int op, const mq_conv_desc* desc, const mq_qtensor* qa_in, int role_a, const mq_qtensor* qb_in, int role_b,
                   void* out, int dtype, int layout, void* ws, size_t ws_bytes, void* stream) {
  mq_status st = check_conv_args(op, desc, qa_in, role_a, qb_in, role_b, out, dtype, layout);
  if (st != MQ_OK) return st;
  Geom g = make_geom(*desc);
  if (ws && !aligned16(ws)) return MQ_ERR_ALIGNMENT;
  size_t need = 0;
  mq_workspace_size(desc, op, qa_in->fmt, qb_in->fmt, qa_in->block, &need);
  if (need > 0 && (!ws || ws_bytes < need)) return MQ_ERR_BUFFER_TOO_SMALL;
  const int fa = fmt_base(qa_in->fmt), fb = fmt_base(qb_in->fmt);
  const bool ts16 = qa_in->block == MQ_BLOCK_TS16, line = qa_in->block == MQ_BLOCK_LINE32;
  // which route: tensor cores when the layer is eligible AND a plan exists for it; everything else runs on the CUDA-core kernels
  ConvTcPlan pl;
  WgradPlan wp;
  wp.ok = false;
  const bool conv_tc = op != MQ_OP_BWD_WEIGHT && conv_takes_tc(op, g, op == MQ_OP_FWD ? fa : fb, op == MQ_OP_FWD ? fb : fa, layout, line, ts16, &pl);
  if (op == MQ_OP_BWD_WEIGHT) wp = wgrad_plan(g, fa, fb, ts16);
  const bool tc = conv_tc || wp.ok;
  // operands in packed 6-bit storage that this route reads one code per byte: copies behind the call's own scratch
  mq_qtensor qa_v = *qa_in, qb_v = *qb_in;
  if (fmt_is_packed6(qa_in->fmt) || fmt_is_packed6(qb_in->fmt)) {
    const PackedExtra pe = packed_extra(op, g, qa_in->fmt, qb_in->fmt, qa_in->block);
    uint8_t* extra = static_cast<uint8_t*>(ws) + (conv_workspace_unpacked(op, g, fa, fb, qa_in->block) + 255) / 256 * 256;
    if (fmt_is_packed6(qa_in->fmt) && (!tc || op == MQ_OP_BWD_DATA)) {
      const View v = view_of(g, role_a);
      if (launch_unpack6(static_cast<const uint8_t*>(qa_in->codes), extra, (size_t)(v.P * v.R * v.Cp), 1, fa, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MQ_ERR_CUDA;
      qa_v.codes = extra; qa_v.fmt = fa; qa_v.codes_bytes = pe.bytes_a;
    }
    if (fmt_is_packed6(qb_in->fmt) && !tc) {
      const View v = view_of(g, role_b);
      if (launch_unpack6(static_cast<const uint8_t*>(qb_in->codes), extra + pe.bytes_a, (size_t)(v.P * v.R * v.Cp), 1, fb, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MQ_ERR_CUDA;
      qb_v.codes = extra + pe.bytes_a; qb_v.fmt = fb; qb_v.codes_bytes = pe.bytes_b;
    }
  }
  const mq_qtensor* qa = &qa_v;
  const mq_qtensor* qb = &qb_v;
  if (conv_tc) {
    const mq_qtensor* qx_like = op == MQ_OP_FWD ? qa : qb;
    const mq_qtensor* qw = op == MQ_OP_FWD ? qb : qa;
    return run_conv_tc(op, g, pl, qx_like, qw, static_cast<float*>(out), layout, ws, device_status_ptr(), static_cast<cudaStream_t>(stream));
  }
  if (wp.ok) return run_wgrad_tc(g, wp, qa, qb, static_cast<float*>(out), layout, ws, device_status_ptr(), static_cast<cudaStream_t>(stream));
  ConvArgs a;
  a.g = g;
  a.a_codes = static_cast<const uint8_t*>(qa->codes); a.a_scales = qa->scales; a.fmt_a = qa->fmt;
  a.b_codes = static_cast<const uint8_t*>(qb->codes); a.b_scales = qb->scales; a.fmt_b = qb->fmt;
  a.out = static_cast<float*>(out); a.out_layout = layout; a.workspace = ws; a.ws_bytes = ws_bytes;
  a.line = qa->block == MQ_BLOCK_LINE32 ? 1 : 0;
  a.ts16 = qa->block == MQ_BLOCK_TS16 ? 1 : 0;
  a.a_tscale = qa->tensor_scale; a.b_tscale = qb->tensor_scale;
  cudaError_t e = launch_conv_generic(op, a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

}  // namespace

bool pdl_enabled() { return env_int("MQ_NO_PDL", 0) == 0; }

}  // namespace mq

using namespace mq;

extern "C" {

mq_status mq_qtensor_sizes(const mq_conv_desc* desc, int role, int fmt, int block, size_t* codes_bytes, size_t* scales_bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_role(role) || !valid_fmt(fmt) || !valid_block(block) || !codes_bytes || !scales_bytes) return MQ_ERR_INVALID_ARG;
  sizes_of(make_geom(*desc), role, fmt, block, codes_bytes, scales_bytes);
  return MQ_OK;
}

mq_status mq_im2col_sizes(const mq_conv_desc* desc, int fmt, int block, size_t* codes_bytes, size_t* scales_bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt) || !valid_block(block) || !codes_bytes || !scales_bytes) return MQ_ERR_INVALID_ARG;
  Geom g = make_geom(*desc);
  *codes_bytes = (size_t)g.Ho * g.Wo * g.N * g.Kh * g.Kw * g.Cp * fmt_store_bits(fmt) / 8;
  if (block == MQ_BLOCK_TS16) *scales_bytes = (size_t)g.Ho * g.Wo * ((g.N + 15) / 16) * g.Kh * g.Kw * (g.Cp / 16);
  else *scales_bytes = (size_t)g.Ho * g.Wo * (block == MQ_BLOCK_LINE32 ? g.N : g.Nt) * g.Kh * g.Kw * g.Ct;
  return MQ_OK;
}

mq_status mq_workspace_size(const mq_conv_desc* desc, int op, int fmt_a, int fmt_b, int block, size_t* bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt_a) || !valid_fmt(fmt_b) || !valid_block(block) || !bytes) return MQ_ERR_INVALID_ARG;
  if (op != MQ_OP_FWD && op != MQ_OP_BWD_DATA && op != MQ_OP_BWD_WEIGHT) return MQ_ERR_INVALID_ARG;
  if (block == MQ_BLOCK_LINE32 && op != MQ_OP_FWD) return MQ_ERR_UNSUPPORTED;
  const Geom g = make_geom(*desc);
  if (block == MQ_BLOCK_TS16 && (fmt_a != MQ_E2M1 || fmt_b != MQ_E2M1)) return MQ_ERR_INVALID_ARG;
  *bytes = conv_workspace_unpacked(op, g, fmt_base(fmt_a), fmt_base(fmt_b), block);
  if (fmt_is_packed6(fmt_a) || fmt_is_packed6(fmt_b)) {
    const PackedExtra pe = packed_extra(op, g, fmt_a, fmt_b, block);
    *bytes = (*bytes + 255) / 256 * 256 + pe.bytes_a + pe.bytes_b;
  }
  return MQ_OK;
}

static mq_status quantize_impl(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, int sr, unsigned long long seed,
                               void* stream, unsigned wait_limit = 0, int skip_loads = 0, const float* amax_in = nullptr) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!src || !dst || !valid_role(dst->role)) return MQ_ERR_INVALID_ARG;
  if (src_layout != MQ_NCHW && src_layout != MQ_HWNC) return MQ_ERR_INVALID_ARG;
  if (!valid_dtype(src_dtype)) return MQ_ERR_INVALID_ARG;
  Geom g = make_geom(*desc);
  if ((st = check_qtensor(g, dst, dst->role)) != MQ_OK) return st;
  if (!aligned16(src)) return MQ_ERR_ALIGNMENT;
  if (src_dtype != MQ_F32) return MQ_ERR_UNSUPPORTED;
  View v = view_of(g, dst->role);
  QuantArgs a{};
  a.src = static_cast<const float*>(src);
  a.codes = static_cast<uint8_t*>(dst->codes);
  a.scales = dst->scales;
  a.P = (int)v.P; a.R = (int)v.R; a.C = (int)v.C; a.Cp = (int)v.Cp;
  a.line = dst->block == MQ_BLOCK_LINE32 ? 1 : 0;
  const bool ts16 = dst->block == MQ_BLOCK_TS16;
  const long long Rt = ts16 ? (v.R + 15) / 16 : (a.line ? v.R : (v.R + 31) / 32), Ct = ts16 ? v.Cp / 16 : v.Cp / 32;   // scale blocks per position
  if (dst->role == MQ_ROLE_W) {  // [r][p][c]
    a.out_stride_p = v.Cp; a.out_stride_r = v.P * v.Cp;
    a.sc_stride_p = Ct; a.sc_stride_r = v.P * Ct;
  } else {                       // [p][r][c]
    a.out_stride_p = v.R * v.Cp; a.out_stride_r = v.Cp;
    a.sc_stride_p = Rt * Ct; a.sc_stride_r = Ct;
  }
  a.fmt = fmt_base(dst->fmt);
  a.packed6 = fmt_is_packed6(dst->fmt) ? 1 : 0;
  a.src_stride_p = 0; a.src_stride_r = 0;
  if (src_layout == MQ_HWNC) {   // channel-fastest source: activations / gradients [pixel][n][c], weights [cout][tap][cin]
    if (dst->role == MQ_ROLE_W) { a.src_stride_p = v.C; a.src_stride_r = v.P * v.C; }
    else { a.src_stride_p = v.R * v.C; a.src_stride_r = v.C; }
  }
  a.status = device_status_ptr();
  a.act = 0;
  a.wait_limit = wait_limit; a.debug_skip_loads = skip_loads;
  a.sr = sr;
  a.sr_seed_lo = (unsigned)seed; a.sr_seed_hi = (unsigned)(seed >> 32);
  a.sr_key0 = sr_mix32(a.sr_seed_lo ^ sr_mix32(a.sr_seed_hi ^ sr_mix32(0u)));
  a.sr_wide = ((unsigned long long)v.P * (unsigned long long)v.R * (unsigned long long)v.C >= (1ull << 32) || env_int("MQ_SR_WIDE", 0)) ? 1 : 0;
  cudaError_t e = ts16 ? launch_quantize_ts(a, amax_in, dst->tensor_scale, static_cast<cudaStream_t>(stream)) : launch_quantize(a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

mq_status mq_quantize_ts(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, const float* amax_in,
                         const unsigned long long* seed_or_null, void* stream) {
  if (dst && dst->block != MQ_BLOCK_TS16) return MQ_ERR_INVALID_ARG;
  if (amax_in && (reinterpret_cast<uintptr_t>(amax_in) & 3u)) return MQ_ERR_ALIGNMENT;
  if (amax_in && dst && dst->tensor_scale && amax_in >= static_cast<const float*>(dst->tensor_scale) &&
      amax_in < static_cast<const float*>(dst->tensor_scale) + 2) return MQ_ERR_INVALID_ARG;   // the call rewrites both words
  return quantize_impl(desc, src, src_dtype, src_layout, dst, seed_or_null ? 1 : 0, seed_or_null ? *seed_or_null : 0ull, stream, 0, 0, amax_in);
}

mq_status mq_quantize(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, void* stream) {
  return quantize_impl(desc, src, src_dtype, src_layout, dst, 0, 0ull, stream);
}

mq_status mq_quantize_sr(const mq_conv_desc* desc, const void* src, int src_dtype, int src_layout, mq_qtensor* dst, unsigned long long seed,
                         void* stream) {
  return quantize_impl(desc, src, src_dtype, src_layout, dst, 1, seed, stream);
}

mq_status mq_selftest_wait_timeout(const mq_conv_desc* desc, const void* src, mq_qtensor* dst, unsigned polls, void* stream) {
  if (polls == 0 || polls > (1u << 20)) return MQ_ERR_INVALID_ARG;
  if (dst && dst->role == MQ_ROLE_W) return MQ_ERR_UNSUPPORTED;
  if (desc && dst && (long long)(dst->role == MQ_ROLE_X ? desc->H * desc->W : 0) % 4 != 0) return MQ_ERR_UNSUPPORTED;
  if (dst && dst->block != MQ_BLOCK_TILE32) return MQ_ERR_UNSUPPORTED;
  return quantize_impl(desc, src, MQ_F32, MQ_NCHW, dst, 0, 0ull, stream, polls, 1);
}

mq_status mq_cbf_im2col(const mq_conv_desc* desc, const mq_qtensor* xq, void* cols_codes, uint8_t* cols_scales, void* stream) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  Geom g = make_geom(*desc);
  if ((st = check_qtensor(g, xq, MQ_ROLE_X)) != MQ_OK) return st;
  if (!cols_codes || !cols_scales) return MQ_ERR_INVALID_ARG;
  if (!aligned16(cols_codes) || !aligned16(cols_scales)) return MQ_ERR_ALIGNMENT;
  Im2colArgs a;
  a.codes = static_cast<const uint8_t*>(xq->codes);
  a.scales = xq->scales;
  a.out_codes = static_cast<uint8_t*>(cols_codes);
  a.out_scales = cols_scales;
  a.g = g;
  a.fmt = xq->fmt;
  a.line = xq->block == MQ_BLOCK_LINE32 ? 1 : 0;
  a.ts16 = xq->block == MQ_BLOCK_TS16 ? 1 : 0;
  cudaError_t e = launch_im2col(a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

mq_status mq_conv_fwd(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, void* y, int y_dtype, int y_layout,
                      void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_FWD, desc, xq, MQ_ROLE_X, wq, MQ_ROLE_W, y, y_dtype, y_layout, workspace, ws_bytes, stream);
}

mq_status mq_conv_bwd_data(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, void* dx, int dx_dtype, int dx_layout,
                           void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, dx, dx_dtype, dx_layout, workspace, ws_bytes, stream);
}

mq_status mq_conv_bwd_weight(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* dyq, void* dw, int dw_dtype, int dw_layout,
                             void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_BWD_WEIGHT, desc, xq, MQ_ROLE_X, dyq, MQ_ROLE_DY, dw, dw_dtype, dw_layout, workspace, ws_bytes, stream);
}

// ---- producer epilogue that quantizes: forward / input-gradient GEMM emitting the next tensor's MX form ----------------
namespace {
// sizes of the emitted tensor: [Hd][Wd][N][Cd rounded up to 32] codes, one scale per (pixel, 32 samples, 32 channels)
void mx_out_sizes(const Geom& g, int op, int fmt, size_t* cb, size_t* sb) {
  const long long P = op == MQ_OP_FWD ? (long long)g.Ho * g.Wo : (long long)g.H * g.W;
  const long long Cp = op == MQ_OP_FWD ? g.Cop : g.Cp;
  *cb = (size_t)(P * g.N * Cp) * fmt_bits(fmt) / 8;
  *sb = (size_t)(P * g.Nt * (Cp / 32));
}
// ts: the paper's own format in and out (MQ_BLOCK_TS16 everywhere); ts_amax: the maximum Eq. 4 takes for the emitted tensor
mq_status run_conv_mx(int op, const mq_conv_desc* desc, const mq_qtensor* qa, int role_a, const mq_qtensor* qb, int role_b, int act, mq_qtensor* out,
                      int role_out, void* ws, size_t ws_bytes, void* stream, size_t* size_query, bool ts = false, const float* ts_amax = nullptr) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  const Geom g = make_geom(*desc);
  int fmt_x_like, fmt_w;
  if (size_query) {   // formats only: qa / qb carry them in their fmt fields
    fmt_x_like = op == MQ_OP_FWD ? qa->fmt : qb->fmt; fmt_w = op == MQ_OP_FWD ? qb->fmt : qa->fmt;
  } else if (ts) {
    if ((st = check_qtensor(g, qa, role_a)) != MQ_OK) return st;
    if ((st = check_qtensor(g, qb, role_b)) != MQ_OK) return st;
    if (!out || !out->codes || !out->scales || !out->tensor_scale || out->fmt != MQ_E2M1 || out->role != role_out || !ts_amax) return MQ_ERR_INVALID_ARG;
    if (act != MQ_ACT_NONE && act != MQ_ACT_RELU && act != MQ_ACT_SILU) return MQ_ERR_INVALID_ARG;
    if (qa->block != MQ_BLOCK_TS16 || qb->block != MQ_BLOCK_TS16 || out->block != MQ_BLOCK_TS16) return MQ_ERR_UNSUPPORTED;
    if (!aligned16(out->codes) || !aligned16(out->scales) || (ws && !aligned16(ws)) || (reinterpret_cast<uintptr_t>(out->tensor_scale) & 7u) ||
        (reinterpret_cast<uintptr_t>(ts_amax) & 3u)) return MQ_ERR_ALIGNMENT;
    const long long P = op == MQ_OP_FWD ? (long long)g.Ho * g.Wo : (long long)g.H * g.W;
    const long long Cdp = op == MQ_OP_FWD ? g.Cop : g.Cp;
    if (out->codes_bytes < (size_t)(P * g.N * Cdp / 2) || out->scales_bytes < (size_t)(P * ((g.N + 15) / 16) * (Cdp / 16))) return MQ_ERR_BUFFER_TOO_SMALL;
    fmt_x_like = fmt_w = MQ_E2M1;
  } else {
    if ((st = check_qtensor(g, qa, role_a)) != MQ_OK) return st;
    if ((st = check_qtensor(g, qb, role_b)) != MQ_OK) return st;
    if (!out || !out->codes || !out->scales || !valid_fmt(out->fmt) || !valid_block(out->block) || out->role != role_out) return MQ_ERR_INVALID_ARG;
    if (act != MQ_ACT_NONE && act != MQ_ACT_RELU && act != MQ_ACT_SILU) return MQ_ERR_INVALID_ARG;
    if (!aligned16(out->codes) || !aligned16(out->scales) || (ws && !aligned16(ws))) return MQ_ERR_ALIGNMENT;
    size_t cb, sb;
    mx_out_sizes(g, op, out->fmt, &cb, &sb);
    if (out->codes_bytes < cb || out->scales_bytes < sb) return MQ_ERR_BUFFER_TOO_SMALL;
    if (qa->block != MQ_BLOCK_TILE32 || qb->block != MQ_BLOCK_TILE32 || out->block != MQ_BLOCK_TILE32) return MQ_ERR_UNSUPPORTED;
    if (fmt_is_packed6(qa->fmt) || fmt_is_packed6(qb->fmt) || fmt_is_packed6(out->fmt)) return MQ_ERR_UNSUPPORTED;   // packed 6-bit storage: not here
    fmt_x_like = op == MQ_OP_FWD ? qa->fmt : qb->fmt; fmt_w = op == MQ_OP_FWD ? qb->fmt : qa->fmt;
  }
  ConvTcPlan pl;
  if (!conv_tc_eligible(op, g, fmt_x_like, fmt_w) || !conv_tc_plan(op, g, fmt_x_like, fmt_w, MQ_HWNC, &pl, false, true, ts)) {
    // layers the tensor-core kernels do not take: the same result in two launches - the CUDA-core GEMM writes fp32
    // [pixel][sample][channel] into scratch and the channel-fastest quantizer, which applies the activation, reads it back
    const long long P = op == MQ_OP_FWD ? (long long)g.Ho * g.Wo : (long long)g.H * g.W;
    const int Cd = op == MQ_OP_FWD ? g.Cout : g.Cin, Cdp = op == MQ_OP_FWD ? g.Cop : g.Cp;
    const size_t y_bytes = up256((size_t)P * g.N * Cd * sizeof(float));
    const size_t total = y_bytes + up256(conv_generic_workspace(op, g));
    if (size_query) { *size_query = total; return MQ_OK; }
    if (!ws || ws_bytes < total) return MQ_ERR_BUFFER_TOO_SMALL;
    uint8_t* base = static_cast<uint8_t*>(ws);
    ConvArgs a;
    a.g = g;
    a.a_codes = static_cast<const uint8_t*>(qa->codes); a.a_scales = qa->scales; a.fmt_a = qa->fmt;
    a.b_codes = static_cast<const uint8_t*>(qb->codes); a.b_scales = qb->scales; a.fmt_b = qb->fmt;
    a.out = reinterpret_cast<float*>(base); a.out_layout = MQ_HWNC; a.workspace = base + y_bytes; a.ws_bytes = ws_bytes - y_bytes; a.line = 0;
    a.ts16 = ts ? 1 : 0; a.a_tscale = ts ? qa->tensor_scale : nullptr; a.b_tscale = ts ? qb->tensor_scale : nullptr;
    if (launch_conv_generic(op, a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return MQ_ERR_CUDA;
    QuantArgs q{};
    q.src = reinterpret_cast<const float*>(base); q.codes = static_cast<uint8_t*>(out->codes); q.scales = out->scales;
    q.P = (int)P; q.R = g.N; q.C = Cd; q.Cp = Cdp;
    q.out_stride_p = (long long)g.N * Cdp; q.out_stride_r = Cdp;
    q.sc_stride_p = ts ? (long long)((g.N + 15) / 16) * (Cdp / 16) : (long long)g.Nt * (Cdp / 32); q.sc_stride_r = ts ? Cdp / 16 : Cdp / 32;
    q.src_stride_p = (long long)g.N * Cd; q.src_stride_r = Cd;
    q.fmt = out->fmt; q.act = act; q.status = device_status_ptr();
    if (ts) return launch_quantize_ts(q, ts_amax, out->tensor_scale, static_cast<cudaStream_t>(stream)) == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
    return launch_quantize(q, static_cast<cudaStream_t>(stream)) == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
  }
  if (size_query) { *size_query = pl.total; return MQ_OK; }
  if (pl.total > 0 && (!ws || ws_bytes < pl.total)) return MQ_ERR_BUFFER_TOO_SMALL;
  pl.p.mx_fmt = ts ? 5 : out->fmt; pl.p.mx_act = act;   // 5: the emitted tensor is in the paper's own format
  pl.p.mx_codes = static_cast<uint8_t*>(out->codes); pl.p.mx_scales = out->scales;
  pl.p.mx_Cp = op == MQ_OP_FWD ? g.Cop : g.Cp;
  if (ts) {
    pl.p.mx_ts_amax = ts_amax; pl.p.mx_ts_stats = out->tensor_scale;
    // the tensor's own maximum is collected with atomicMax on its bit pattern: start from zero
    if (cudaMemsetAsync(out->tensor_scale + 1, 0, sizeof(float), static_cast<cudaStream_t>(stream)) != cudaSuccess) return MQ_ERR_CUDA;
  }
  const mq_qtensor* qx_like = op == MQ_OP_FWD ? qa : qb;
  const mq_qtensor* qw = op == MQ_OP_FWD ? qb : qa;
  return run_conv_tc(op, g, pl, qx_like, qw, nullptr, MQ_HWNC, ws, device_status_ptr(), static_cast<cudaStream_t>(stream));
}
}  // namespace

mq_status mq_conv_mx_workspace_size(const mq_conv_desc* desc, int op, int fmt_a, int fmt_b, size_t* bytes) {
  if (!bytes || !valid_fmt(fmt_a) || !valid_fmt(fmt_b) || (op != MQ_OP_FWD && op != MQ_OP_BWD_DATA)) return MQ_ERR_INVALID_ARG;
  if (fmt_is_packed6(fmt_a) || fmt_is_packed6(fmt_b)) return MQ_ERR_UNSUPPORTED;
  mq_qtensor a{}, b{};
  a.fmt = fmt_a; b.fmt = fmt_b;
  return run_conv_mx(op, desc, &a, 0, &b, 0, 0, nullptr, 0, nullptr, 0, nullptr, bytes);
}

mq_status mq_conv_fwd_mx(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, int act, mq_qtensor* yq, void* workspace, size_t ws_bytes,
                         void* stream) {
  return run_conv_mx(MQ_OP_FWD, desc, xq, MQ_ROLE_X, wq, MQ_ROLE_W, act, yq, MQ_ROLE_X, workspace, ws_bytes, stream, nullptr);
}

mq_status mq_conv_bwd_data_mx(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, mq_qtensor* dxq, void* workspace, size_t ws_bytes,
                              void* stream) {
  return run_conv_mx(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, MQ_ACT_NONE, dxq, MQ_ROLE_DY, workspace, ws_bytes, stream, nullptr);
}

mq_status mq_conv_ts_workspace_size(const mq_conv_desc* desc, int op, size_t* bytes) {
  if (!bytes || (op != MQ_OP_FWD && op != MQ_OP_BWD_DATA)) return MQ_ERR_INVALID_ARG;
  mq_qtensor a{}, b{};
  a.fmt = MQ_E2M1; b.fmt = MQ_E2M1;
  return run_conv_mx(op, desc, &a, 0, &b, 0, 0, nullptr, 0, nullptr, 0, nullptr, bytes, true, nullptr);
}

mq_status mq_conv_fwd_ts(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, int act, const float* amax_in, mq_qtensor* yq, void* workspace,
                         size_t ws_bytes, void* stream) {
  if (!xq || !wq) return MQ_ERR_INVALID_ARG;
  return run_conv_mx(MQ_OP_FWD, desc, xq, MQ_ROLE_X, wq, MQ_ROLE_W, act, yq, MQ_ROLE_X, workspace, ws_bytes, stream, nullptr, true, amax_in);
}

mq_status mq_conv_bwd_data_ts(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, const float* amax_in, mq_qtensor* dxq, void* workspace,
                              size_t ws_bytes, void* stream) {
  if (!wq || !dyq) return MQ_ERR_INVALID_ARG;
  return run_conv_mx(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, MQ_ACT_NONE, dxq, MQ_ROLE_DY, workspace, ws_bytes, stream, nullptr, true, amax_in);
}

// ---- allocation-free variant of mq_conv_bwd_data ---------------------------------------------------
// Scratch for callers that cannot allocate: a static array in the device image.  In host code the name
// below is only a handle for the runtime, not a device address; the address is looked up with
// cudaGetSymbolAddress (with the caller's device current) and that pointer is what the kernels receive.
// The lookup is repeated on every call - after the first one on a device, which may load the module, it is a
// host-side table lookup - so no cached address can outlive a cudaDeviceReset of its context.
static __device__ __align__(256) unsigned char g_static_scratch[MQ_STATIC_SCRATCH_BYTES];

mq_status mq_conv_bwd_data_static(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, void* dx, int dx_dtype, int dx_layout,
                                  void* stream) {
  // the ordinary call's argument checks first, so that a bad argument is reported as such whatever the layer's size
  mq_status st = check_conv_args(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, dx, dx_dtype, dx_layout);
  if (st != MQ_OK) return st;
  size_t need = 0;
  if ((st = mq_workspace_size(desc, MQ_OP_BWD_DATA, wq->fmt, dyq->fmt, wq->block, &need)) != MQ_OK) return st;
  if (need > MQ_STATIC_SCRATCH_BYTES) return MQ_ERR_STATIC_SCRATCH;
  void* addr = nullptr;
  if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return MQ_ERR_CUDA;
  return run_conv(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, dx, dx_dtype, dx_layout, addr, MQ_STATIC_SCRATCH_BYTES, stream);
}

namespace {
// The step runs slab by slab along the batch (slabs of whole 32-sample tiles, at most 8 of them): the quantized tensors, the
// im2col and the GEMMs of a slab need that slab's samples only (W in full), so the upload of slab k + 1 and the download of
// slab k's Y and G_X overlap the computation, and both copy engines stay busy for the whole step.  G_W is the sum of the
// slabs' weight gradients, added in slab order.
struct LayerArena {
  size_t off_x, off_w, off_g, off_y, off_dx, off_dw, off_dwp, off_ws, off_ic, off_is, total;
  size_t off_qc[3], off_qs[3];
  size_t nx, nw, ng, qc[3], qs[3], ic, is, ws;
  int slab_n, slabs;        // samples per slab (the last may hold fewer), number of slabs
};
size_t up256(size_t v) { return (v + 255) / 256 * 256; }
LayerArena layer_arena(const mq_conv_desc* desc, const int fmts[3]) {
  Geom g = make_geom(*desc);
  LayerArena L{};
  L.nx = (size_t)g.N * g.Cin * g.H * g.W * 4;
  L.nw = (size_t)g.Cout * g.Cin * g.Kh * g.Kw * 4;
  L.ng = (size_t)g.N * g.Cout * g.Ho * g.Wo * 4;
  size_t o = 0;
  auto take = [&](size_t n) { size_t r = o; o += up256(n); return r; };
  L.off_x = take(L.nx); L.off_w = take(L.nw); L.off_g = take(L.ng);
  L.off_y = take(L.ng); L.off_dx = take(L.nx); L.off_dw = take(L.nw);
  int max_slabs = env_int("MQ_HOST_SLABS", 8);
  max_slabs = max_slabs < 1 ? 1 : (max_slabs > 8 ? 8 : max_slabs);
  const int tiles_per_slab = (g.Nt + max_slabs - 1) / max_slabs;
  L.slab_n = 32 * tiles_per_slab;
  L.slabs = (g.N + L.slab_n - 1) / L.slab_n;
  L.off_dwp = L.slabs > 1 ? take((size_t)L.slabs * up256(L.nw)) : 0;
  mq_conv_desc ds = *desc;
  ds.N = L.slabs > 1 ? L.slab_n : g.N;     // the largest slab sizes the per-slab buffers
  const Geom gs = make_geom(ds);
  sizes_of(gs, 0, fmts[0], MQ_BLOCK_TILE32, &L.qc[0], &L.qs[0]);
  sizes_of(g, 1, fmts[1], MQ_BLOCK_TILE32, &L.qc[1], &L.qs[1]);
  sizes_of(gs, 2, fmts[2], MQ_BLOCK_TILE32, &L.qc[2], &L.qs[2]);
  for (int r = 0; r < 3; ++r) { L.off_qc[r] = take(L.qc[r]); L.off_qs[r] = take(L.qs[r]); }
  mq_im2col_sizes(&ds, fmts[0], MQ_BLOCK_TILE32, &L.ic, &L.is);
  L.off_ic = take(L.ic); L.off_is = take(L.is);
  L.ws = 0;
  const int ops[3] = {MQ_OP_FWD, MQ_OP_BWD_DATA, MQ_OP_BWD_WEIGHT};
  const int fa[3] = {fmts[0], fmts[1], fmts[0]}, fb[3] = {fmts[1], fmts[2], fmts[2]};
  for (int pass = 0; pass < 2; ++pass) {     // the full slab, and the ragged last one (its plans may need more scratch)
    mq_conv_desc dq = ds;
    if (pass == 1) { dq.N = g.N - (L.slabs - 1) * L.slab_n; if (L.slabs == 1 || dq.N == ds.N) break; }
    for (int i = 0; i < 3; ++i) { size_t b = 0; mq_workspace_size(&dq, ops[i], fa[i], fb[i], MQ_BLOCK_TILE32, &b); if (b > L.ws) L.ws = b; }
  }
  L.off_ws = take(L.ws);
  L.total = o;
  return L;
}
}  // namespace

// Side streams and events of mq_conv_layer_host, created once per device (no device memory is allocated).
// G_W = sum over the slabs of their weight gradients, in slab order (float4 body, scalar tail)
__global__ void __launch_bounds__(256) sum_slabs_kernel(const float4* __restrict__ part4, float4* __restrict__ out4, long long n4, long long stride4, int slabs,
                                                        const float* __restrict__ part, float* __restrict__ out, long long n) {
  const long long t0 = (long long)blockIdx.x * blockDim.x + threadIdx.x, step = (long long)gridDim.x * blockDim.x;
  for (long long i = t0; i < n4; i += step) {
    float4 a = __ldg(part4 + i);
    for (int k = 1; k < slabs; ++k) { const float4 b = __ldg(part4 + (long long)k * stride4 + i); a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; }
    out4[i] = a;
  }
  for (long long i = 4 * n4 + t0; i < n; i += step) {
    float a = __ldg(part + i);
    for (int k = 1; k < slabs; ++k) a += __ldg(part + (long long)k * stride4 * 4 + i);
    out[i] = a;
  }
}

constexpr int HOST_EVENTS = 48;   // start, W, final, and four per slab (at most 8 slabs)
struct HostPipe { cudaStream_t h2d, d2h; cudaEvent_t ev[HOST_EVENTS]; bool ready; };
static HostPipe* host_pipe() {
  static HostPipe pipes[32];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 32) return nullptr;
  HostPipe* hp = &pipes[dev];
  if (!hp->ready) {
    if (cudaStreamCreateWithFlags(&hp->h2d, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&hp->d2h, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    for (int i = 0; i < HOST_EVENTS; ++i)
      if (cudaEventCreateWithFlags(&hp->ev[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    hp->ready = true;
  }
  return hp;
}

mq_status mq_conv_layer_host_arena_size(const mq_conv_desc* desc, int fmt_x, int fmt_w, int fmt_dy, size_t* bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt_x) || !valid_fmt(fmt_w) || !valid_fmt(fmt_dy) || !bytes) return MQ_ERR_INVALID_ARG;
  const int fmts[3] = {fmt_x, fmt_w, fmt_dy};
  *bytes = layer_arena(desc, fmts).total;
  return MQ_OK;
}

mq_status mq_conv_layer_host(const mq_conv_desc* desc, int fmt_x, int fmt_w, int fmt_dy, const float* x_host, const float* w_host,
                             const float* dy_host, float* y_host, float* dx_host, float* dw_host, void* arena, size_t arena_bytes,
                             void* stream) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt_x) || !valid_fmt(fmt_w) || !valid_fmt(fmt_dy)) return MQ_ERR_INVALID_ARG;
  if (!x_host || !w_host || !dy_host || !y_host || !dx_host || !dw_host || !arena) return MQ_ERR_INVALID_ARG;
  if (!aligned16(arena)) return MQ_ERR_ALIGNMENT;
  const int fmts[3] = {fmt_x, fmt_w, fmt_dy};
  LayerArena L = layer_arena(desc, fmts);
  if (arena_bytes < L.total) return MQ_ERR_BUFFER_TOO_SMALL;
  uint8_t* base = static_cast<uint8_t*>(arena);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // Copies run on two side streams of their own (one per direction: the copy engines are full duplex) and are tied to
  // the caller's stream by events.  Slab by slab: upload X_k and G_Y_k; quantize, im2col, forward -> download Y_k;
  // input gradient -> download G_X_k; weight gradient of the slab into its own buffer.  The caller's stream waits for
  // the last download: synchronising it is enough.
  HostPipe* hp = host_pipe();
  if (!hp) return MQ_ERR_CUDA;
  auto ok = [](cudaError_t e) { return e == cudaSuccess; };
  const Geom g = make_geom(*desc);
  const int S = L.slabs;
  cudaEvent_t* ev = hp->ev;     // 0 start, 1 W uploaded, 2 G_W ready, 3 last download; 4 + 4k .. : X_k, G_Y_k uploaded, Y_k, G_X_k ready
  if (!ok(cudaEventRecord(ev[0], s)) || !ok(cudaStreamWaitEvent(hp->h2d, ev[0], 0)) || !ok(cudaStreamWaitEvent(hp->d2h, ev[0], 0))) return MQ_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(base + L.off_w, w_host, L.nw, cudaMemcpyHostToDevice, hp->h2d)) || !ok(cudaEventRecord(ev[1], hp->h2d))) return MQ_ERR_CUDA;
  const size_t x_per_n = (size_t)g.Cin * g.H * g.W * 4, g_per_n = (size_t)g.Cout * g.Ho * g.Wo * 4;
  for (int k = 0; k < S; ++k) {
    const size_t n0 = (size_t)k * L.slab_n, nk = (size_t)(k == S - 1 ? g.N - (int)n0 : L.slab_n);
    if (!ok(cudaMemcpyAsync(base + L.off_x + n0 * x_per_n, reinterpret_cast<const uint8_t*>(x_host) + n0 * x_per_n, nk * x_per_n, cudaMemcpyHostToDevice, hp->h2d)) ||
        !ok(cudaEventRecord(ev[4 + 4 * k], hp->h2d))) return MQ_ERR_CUDA;
    if (!ok(cudaMemcpyAsync(base + L.off_g + n0 * g_per_n, reinterpret_cast<const uint8_t*>(dy_host) + n0 * g_per_n, nk * g_per_n, cudaMemcpyHostToDevice, hp->h2d)) ||
        !ok(cudaEventRecord(ev[5 + 4 * k], hp->h2d))) return MQ_ERR_CUDA;
  }
  mq_qtensor q[3];
  for (int r = 0; r < 3; ++r) {
    q[r].codes = base + L.off_qc[r]; q[r].scales = base + L.off_qs[r];
    q[r].codes_bytes = L.qc[r]; q[r].scales_bytes = L.qs[r]; q[r].fmt = fmts[r]; q[r].role = r; q[r].block = MQ_BLOCK_TILE32; q[r].tensor_scale = nullptr;
  }
  void* ws = L.ws ? base + L.off_ws : nullptr;
  if (!ok(cudaStreamWaitEvent(s, ev[1], 0))) return MQ_ERR_CUDA;
  if ((st = mq_quantize(desc, base + L.off_w, MQ_F32, MQ_NCHW, &q[1], stream)) != MQ_OK) return st;
  for (int k = 0; k < S; ++k) {
    const size_t n0 = (size_t)k * L.slab_n, nk = (size_t)(k == S - 1 ? g.N - (int)n0 : L.slab_n);
    mq_conv_desc dk = *desc;
    dk.N = (int)nk;
    uint8_t* xk = base + L.off_x + n0 * x_per_n;
    uint8_t* gk = base + L.off_g + n0 * g_per_n;
    uint8_t* yk = base + L.off_y + n0 * g_per_n;
    uint8_t* dxk = base + L.off_dx + n0 * x_per_n;
    void* dwk = S > 1 ? static_cast<void*>(base + L.off_dwp + (size_t)k * ((L.nw + 255) / 256 * 256)) : static_cast<void*>(base + L.off_dw);
    if (!ok(cudaStreamWaitEvent(s, ev[4 + 4 * k], 0))) return MQ_ERR_CUDA;
    if ((st = mq_quantize(&dk, xk, MQ_F32, MQ_NCHW, &q[0], stream)) != MQ_OK) return st;
    if ((st = mq_cbf_im2col(&dk, &q[0], base + L.off_ic, base + L.off_is, stream)) != MQ_OK) return st;
    if ((st = mq_conv_fwd(&dk, &q[0], &q[1], yk, MQ_F32, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
    if (!ok(cudaEventRecord(ev[6 + 4 * k], s)) || !ok(cudaStreamWaitEvent(hp->d2h, ev[6 + 4 * k], 0))) return MQ_ERR_CUDA;
    if (!ok(cudaMemcpyAsync(reinterpret_cast<uint8_t*>(y_host) + n0 * g_per_n, yk, nk * g_per_n, cudaMemcpyDeviceToHost, hp->d2h))) return MQ_ERR_CUDA;
    if (!ok(cudaStreamWaitEvent(s, ev[5 + 4 * k], 0))) return MQ_ERR_CUDA;
    if ((st = mq_quantize(&dk, gk, MQ_F32, MQ_NCHW, &q[2], stream)) != MQ_OK) return st;
    if ((st = mq_conv_bwd_data(&dk, &q[1], &q[2], dxk, MQ_F32, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
    if (!ok(cudaEventRecord(ev[7 + 4 * k], s)) || !ok(cudaStreamWaitEvent(hp->d2h, ev[7 + 4 * k], 0))) return MQ_ERR_CUDA;
    if (!ok(cudaMemcpyAsync(reinterpret_cast<uint8_t*>(dx_host) + n0 * x_per_n, dxk, nk * x_per_n, cudaMemcpyDeviceToHost, hp->d2h))) return MQ_ERR_CUDA;
    if ((st = mq_conv_bwd_weight(&dk, &q[0], &q[2], dwk, MQ_F32, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
  }
  if (S > 1) {
    const long long n4 = (long long)(L.nw / 16), stride4 = (long long)((L.nw + 255) / 256 * 256 / 16);
    unsigned blocks = (unsigned)((n4 + 255) / 256);
    if (blocks > (unsigned)sm_count() * 8) blocks = (unsigned)sm_count() * 8;
    if (blocks < 1) blocks = 1;
    sum_slabs_kernel<<<blocks, 256, 0, s>>>(reinterpret_cast<const float4*>(base + L.off_dwp), reinterpret_cast<float4*>(base + L.off_dw), n4, stride4, S,
                                          reinterpret_cast<const float*>(base + L.off_dwp), reinterpret_cast<float*>(base + L.off_dw), (long long)(L.nw / 4));
    count_launches(1);
    if (cudaGetLastError() != cudaSuccess) return MQ_ERR_CUDA;
  }
  if (!ok(cudaEventRecord(ev[2], s)) || !ok(cudaStreamWaitEvent(hp->d2h, ev[2], 0))) return MQ_ERR_CUDA;
  if (!ok(cudaMemcpyAsync(dw_host, base + L.off_dw, L.nw, cudaMemcpyDeviceToHost, hp->d2h))) return MQ_ERR_CUDA;
  if (!ok(cudaEventRecord(ev[3], hp->d2h)) || !ok(cudaStreamWaitEvent(s, ev[3], 0))) return MQ_ERR_CUDA;
  return MQ_OK;
}

unsigned long long mq_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

void mq_reload_env(void) { env_forget(); }

const char* mq_status_string(int status) {
  switch (status) {
    case MQ_OK: return "MQ_OK";
    case MQ_ERR_INVALID_ARG: return "MQ_ERR_INVALID_ARG";
    case MQ_ERR_UNSUPPORTED: return "MQ_ERR_UNSUPPORTED";
    case MQ_ERR_ALIGNMENT: return "MQ_ERR_ALIGNMENT";
    case MQ_ERR_BUFFER_TOO_SMALL: return "MQ_ERR_BUFFER_TOO_SMALL";
    case MQ_ERR_CUDA: return "MQ_ERR_CUDA";
    case MQ_ERR_TIMEOUT: return "MQ_ERR_TIMEOUT";
    case MQ_ERR_STATIC_SCRATCH: return "MQ_ERR_STATIC_SCRATCH";
    default: return "MQ_ERR_UNKNOWN";
  }
}

mq_status mq_last_device_status(void* stream) {
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) return MQ_ERR_CUDA;
  unsigned int v = 0, zero = 0;
  if (cudaMemcpyFromSymbol(&v, g_device_status, sizeof(v)) != cudaSuccess) return MQ_ERR_CUDA;
  if (v != 0 && cudaMemcpyToSymbol(g_device_status, &zero, sizeof(zero)) != cudaSuccess) return MQ_ERR_CUDA;
  return v == 0 ? MQ_OK : MQ_ERR_TIMEOUT;
}

}  // extern "C"
