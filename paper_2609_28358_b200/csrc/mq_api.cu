// extern "C" entry points: argument validation, size arithmetic, kernel selection.
#include "mq_internal.cuh"

namespace mq {

__device__ unsigned int g_device_status = 0;  // set by kernels when a bounded wait gives up

namespace {

bool valid_fmt(int f) { return f == MQ_E4M3 || f == MQ_E5M2 || f == MQ_E2M1; }
bool valid_role(int r) { return r == MQ_ROLE_X || r == MQ_ROLE_W || r == MQ_ROLE_DY; }
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

void sizes_of(const Geom& g, int role, int fmt, size_t* cb, size_t* sb) {
  View v = view_of(g, role);
  *cb = (size_t)(v.P * v.R * v.Cp) * fmt_bits(fmt) / 8;
  *sb = (size_t)(v.P * ((v.R + 31) / 32) * (v.Cp / 32));
}

mq_status check_qtensor(const Geom& g, const mq_qtensor* q, int role) {
  if (!q || !q->codes || !q->scales) return MQ_ERR_INVALID_ARG;
  if (!valid_fmt(q->fmt) || q->role != role) return MQ_ERR_INVALID_ARG;
  if (!aligned16(q->codes) || !aligned16(q->scales)) return MQ_ERR_ALIGNMENT;
  size_t cb, sb;
  sizes_of(g, role, q->fmt, &cb, &sb);
  if (q->codes_bytes < cb || q->scales_bytes < sb) return MQ_ERR_BUFFER_TOO_SMALL;
  return MQ_OK;
}

mq_status run_conv(int op, const mq_conv_desc* desc, const mq_qtensor* qa, int role_a, const mq_qtensor* qb, int role_b,
                   void* out, int layout, void* ws, size_t ws_bytes, void* stream) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  Geom g = make_geom(*desc);
  if ((st = check_qtensor(g, qa, role_a)) != MQ_OK) return st;
  if ((st = check_qtensor(g, qb, role_b)) != MQ_OK) return st;
  if (!out) return MQ_ERR_INVALID_ARG;
  if (layout != MQ_NCHW && layout != MQ_HWNC) return MQ_ERR_INVALID_ARG;
  if (!aligned16(out) || (ws && !aligned16(ws))) return MQ_ERR_ALIGNMENT;
  size_t need = 0;
  mq_workspace_size(desc, op, qa->fmt, qb->fmt, &need);
  if (need > 0 && (!ws || ws_bytes < need)) return MQ_ERR_BUFFER_TOO_SMALL;
  ConvArgs a;
  a.g = g;
  a.a_codes = static_cast<const uint8_t*>(qa->codes); a.a_scales = qa->scales; a.fmt_a = qa->fmt;
  a.b_codes = static_cast<const uint8_t*>(qb->codes); a.b_scales = qb->scales; a.fmt_b = qb->fmt;
  a.out = static_cast<float*>(out); a.out_layout = layout; a.workspace = ws; a.ws_bytes = ws_bytes;
  cudaError_t e = launch_conv_generic(op, a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

}  // namespace
}  // namespace mq

using namespace mq;

extern "C" {

mq_status mq_qtensor_sizes(const mq_conv_desc* desc, int role, int fmt, size_t* codes_bytes, size_t* scales_bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_role(role) || !valid_fmt(fmt) || !codes_bytes || !scales_bytes) return MQ_ERR_INVALID_ARG;
  sizes_of(make_geom(*desc), role, fmt, codes_bytes, scales_bytes);
  return MQ_OK;
}

mq_status mq_im2col_sizes(const mq_conv_desc* desc, int fmt, size_t* codes_bytes, size_t* scales_bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt) || !codes_bytes || !scales_bytes) return MQ_ERR_INVALID_ARG;
  Geom g = make_geom(*desc);
  *codes_bytes = (size_t)g.Ho * g.Wo * g.N * g.Kh * g.Kw * g.Cp * fmt_bits(fmt) / 8;
  *scales_bytes = (size_t)g.Ho * g.Wo * g.Nt * g.Kh * g.Kw * g.Ct;
  return MQ_OK;
}

mq_status mq_workspace_size(const mq_conv_desc* desc, int op, int fmt_a, int fmt_b, size_t* bytes) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!valid_fmt(fmt_a) || !valid_fmt(fmt_b) || !bytes) return MQ_ERR_INVALID_ARG;
  if (op != MQ_OP_FWD && op != MQ_OP_BWD_DATA && op != MQ_OP_BWD_WEIGHT) return MQ_ERR_INVALID_ARG;
  *bytes = conv_generic_workspace(op, make_geom(*desc));
  return MQ_OK;
}

mq_status mq_quantize(const mq_conv_desc* desc, const void* src, int src_layout, mq_qtensor* dst, void* stream) {
  mq_status st = check_desc(desc);
  if (st != MQ_OK) return st;
  if (!src || !dst || !valid_role(dst->role)) return MQ_ERR_INVALID_ARG;
  if (src_layout != MQ_NCHW && src_layout != MQ_HWNC) return MQ_ERR_INVALID_ARG;
  if (src_layout != MQ_NCHW) return MQ_ERR_UNSUPPORTED;
  Geom g = make_geom(*desc);
  if ((st = check_qtensor(g, dst, dst->role)) != MQ_OK) return st;
  if (!aligned16(src)) return MQ_ERR_ALIGNMENT;
  View v = view_of(g, dst->role);
  QuantArgs a;
  a.src = static_cast<const float*>(src);
  a.codes = static_cast<uint8_t*>(dst->codes);
  a.scales = dst->scales;
  a.P = (int)v.P; a.R = (int)v.R; a.C = (int)v.C; a.Cp = (int)v.Cp;
  const long long Rt = (v.R + 31) / 32, Ct = v.Cp / 32;
  if (dst->role == MQ_ROLE_W) {  // [r][p][c]
    a.out_stride_p = v.Cp; a.out_stride_r = v.P * v.Cp;
    a.sc_stride_p = Ct; a.sc_stride_r = v.P * Ct;
  } else {                       // [p][r][c]
    a.out_stride_p = v.R * v.Cp; a.out_stride_r = v.Cp;
    a.sc_stride_p = Rt * Ct; a.sc_stride_r = Ct;
  }
  a.fmt = dst->fmt;
  cudaError_t e = launch_quantize(a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
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
  cudaError_t e = launch_im2col(a, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? MQ_OK : MQ_ERR_CUDA;
}

mq_status mq_conv_fwd(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* wq, void* y, int y_layout,
                      void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_FWD, desc, xq, MQ_ROLE_X, wq, MQ_ROLE_W, y, y_layout, workspace, ws_bytes, stream);
}

mq_status mq_conv_bwd_data(const mq_conv_desc* desc, const mq_qtensor* wq, const mq_qtensor* dyq, void* dx, int dx_layout,
                           void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_BWD_DATA, desc, wq, MQ_ROLE_W, dyq, MQ_ROLE_DY, dx, dx_layout, workspace, ws_bytes, stream);
}

mq_status mq_conv_bwd_weight(const mq_conv_desc* desc, const mq_qtensor* xq, const mq_qtensor* dyq, void* dw, int dw_layout,
                             void* workspace, size_t ws_bytes, void* stream) {
  return run_conv(MQ_OP_BWD_WEIGHT, desc, xq, MQ_ROLE_X, dyq, MQ_ROLE_DY, dw, dw_layout, workspace, ws_bytes, stream);
}

namespace {
struct LayerArena {
  size_t off_x, off_w, off_g, off_y, off_dx, off_dw, off_ws, off_ic, off_is, total;
  size_t off_qc[3], off_qs[3];
  size_t nx, nw, ng, qc[3], qs[3], ic, is, ws;
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
  for (int r = 0; r < 3; ++r) {
    sizes_of(g, r, fmts[r], &L.qc[r], &L.qs[r]);
    L.off_qc[r] = take(L.qc[r]); L.off_qs[r] = take(L.qs[r]);
  }
  mq_im2col_sizes(desc, fmts[0], &L.ic, &L.is);
  L.off_ic = take(L.ic); L.off_is = take(L.is);
  L.ws = 0;
  const int ops[3] = {MQ_OP_FWD, MQ_OP_BWD_DATA, MQ_OP_BWD_WEIGHT};
  const int fa[3] = {fmts[0], fmts[1], fmts[0]}, fb[3] = {fmts[1], fmts[2], fmts[2]};
  for (int i = 0; i < 3; ++i) { size_t b = 0; mq_workspace_size(desc, ops[i], fa[i], fb[i], &b); if (b > L.ws) L.ws = b; }
  L.off_ws = take(L.ws);
  L.total = o;
  return L;
}
}  // namespace

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
  if (cudaMemcpyAsync(base + L.off_x, x_host, L.nx, cudaMemcpyHostToDevice, s) != cudaSuccess) return MQ_ERR_CUDA;
  if (cudaMemcpyAsync(base + L.off_w, w_host, L.nw, cudaMemcpyHostToDevice, s) != cudaSuccess) return MQ_ERR_CUDA;
  if (cudaMemcpyAsync(base + L.off_g, dy_host, L.ng, cudaMemcpyHostToDevice, s) != cudaSuccess) return MQ_ERR_CUDA;
  mq_qtensor q[3];
  const size_t src_off[3] = {L.off_x, L.off_w, L.off_g};
  for (int r = 0; r < 3; ++r) {
    q[r].codes = base + L.off_qc[r]; q[r].scales = base + L.off_qs[r];
    q[r].codes_bytes = L.qc[r]; q[r].scales_bytes = L.qs[r]; q[r].fmt = fmts[r]; q[r].role = r;
    if ((st = mq_quantize(desc, base + src_off[r], MQ_NCHW, &q[r], stream)) != MQ_OK) return st;
  }
  if ((st = mq_cbf_im2col(desc, &q[0], base + L.off_ic, base + L.off_is, stream)) != MQ_OK) return st;
  void* ws = L.ws ? base + L.off_ws : nullptr;
  if ((st = mq_conv_fwd(desc, &q[0], &q[1], base + L.off_y, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
  if ((st = mq_conv_bwd_data(desc, &q[1], &q[2], base + L.off_dx, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
  if ((st = mq_conv_bwd_weight(desc, &q[0], &q[2], base + L.off_dw, MQ_NCHW, ws, L.ws, stream)) != MQ_OK) return st;
  if (cudaMemcpyAsync(y_host, base + L.off_y, L.ng, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MQ_ERR_CUDA;
  if (cudaMemcpyAsync(dx_host, base + L.off_dx, L.nx, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MQ_ERR_CUDA;
  if (cudaMemcpyAsync(dw_host, base + L.off_dw, L.nw, cudaMemcpyDeviceToHost, s) != cudaSuccess) return MQ_ERR_CUDA;
  return MQ_OK;
}

const char* mq_status_string(int status) {
  switch (status) {
    case MQ_OK: return "MQ_OK";
    case MQ_ERR_INVALID_ARG: return "MQ_ERR_INVALID_ARG";
    case MQ_ERR_UNSUPPORTED: return "MQ_ERR_UNSUPPORTED";
    case MQ_ERR_ALIGNMENT: return "MQ_ERR_ALIGNMENT";
    case MQ_ERR_BUFFER_TOO_SMALL: return "MQ_ERR_BUFFER_TOO_SMALL";
    case MQ_ERR_CUDA: return "MQ_ERR_CUDA";
    case MQ_ERR_TIMEOUT: return "MQ_ERR_TIMEOUT";
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
