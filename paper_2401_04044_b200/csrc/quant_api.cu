// C ABI of the quantised split (Section 5.2): layout of the packed blob, the quantising pack, the expansion for
// inspection and the few-token forward's plan.  Kernels: quant_pack.cu, decode_quant.cu.
#include <cstring>

#include "internal.h"
#include "quant.h"
#include "quant_plan.h"

namespace ffsp {

ffsplit_status launch_quant_pack(ffsplit_ctx* ctx, const __nv_bfloat16* W, long long ld, int utype, const int* idx,
                                 int n_out, int n_k, int groups, int bits, unsigned char* dst, cudaStream_t st);
ffsplit_status launch_quant_unpack(ffsplit_ctx* ctx, const unsigned char* src, int n_out, int n_k, int groups, int bits,
                                   unsigned char* codes, float* scale, float* lo, cudaStream_t st);

namespace {

using namespace qnt;

constexpr size_t kAlignQ = 256;
inline size_t align_q(size_t v) { return (v + kAlignQ - 1) / kAlignQ * kAlignQ; }

ffsplit_status check_quant_shape(ffsplit_ctx* ctx, const ffsplit_shape* s, int k) {
  if (!s) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "shape is NULL");
  if (s->d < 1 || s->m < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "d and m must be >= 1");
  if (s->act < 0 || s->act > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown activation");
  if (s->dtype != FFSPLIT_BF16) return fail(ctx, FFSPLIT_ERR_DTYPE, "the quantised split takes bf16 layers");
  if (s->d % 8 != 0) return fail(ctx, FFSPLIT_ERR_SHAPE, "bf16 layers need d to be a multiple of 8");
  if (k < 0 || k > s->m) return fail(ctx, FFSPLIT_ERR_SHAPE, "k must be in [0, m]");
  return FFSPLIT_OK;
}

void layout_quant(const ffsplit_shape& s, int k, QuantHeader* h) {
  std::memset(h, 0, sizeof(*h));
  h->magic = kQuantMagic; h->version = kQuantVersion;
  h->d = s.d; h->m = s.m; h->act = s.act; h->k = k; h->ml = s.m - k; h->n_in = s.act == FFSPLIT_SWIGLU ? 2 : 1;
  h->gd = even_groups(s.d); h->gk = k > 0 ? even_groups(k) : 0; h->gl = h->ml > 0 ? even_groups(h->ml) : 0;
  h->k8 = (k + 7) / 8 * 8; h->ml8 = (h->ml + 7) / 8 * 8;
  size_t off = sizeof(QuantHeader);
  auto take = [&](int sec, size_t bytes) { h->off[sec] = off; off = align_q(off + bytes); };
  take(QS_U1, static_cast<size_t>(k) * h->gd * kGroupBytes8);
  take(QS_U2, static_cast<size_t>(h->ml) * h->gd * kGroupBytes3);
  if (h->n_in == 2) {
    take(QS_U1U, static_cast<size_t>(k) * h->gd * kGroupBytes8);
    take(QS_U2U, static_cast<size_t>(h->ml) * h->gd * kGroupBytes3);
  }
  take(QS_V1, static_cast<size_t>(s.d) * h->gk * kGroupBytes8);
  take(QS_V2, static_cast<size_t>(s.d) * h->gl * kGroupBytes3);
  take(QS_B1H, static_cast<size_t>(h->k8 > 0 ? h->k8 : 8) * 4);
  take(QS_B1L, static_cast<size_t>(h->ml8 > 0 ? h->ml8 : 8) * 4);
  take(QS_B2, static_cast<size_t>(s.d) * 4);
  h->total_bytes = off;
  // codes at their width plus one (scale, lo) pair of float32 per real group, and the float32 biases
  const double gd = (s.d + kGroup - 1) / kGroup;
  auto part = [&](double n, double bits) {
    if (n <= 0) return 0.0;
    const double gv = static_cast<double>((static_cast<long long>(n) + kGroup - 1) / kGroup);
    return (h->n_in * n * s.d * bits + n * s.d * bits) / 8.0 + 8.0 * (h->n_in * n * gd + s.d * gv);
  };
  h->logical_bytes = static_cast<uint64_t>(part(k, 8) + part(h->ml, 3) + 4.0 * (s.m + s.d));
}

bool quant_header_valid(const QuantHeader& h, size_t blob_bytes) {
  if (h.magic != kQuantMagic || h.version != kQuantVersion) return false;
  if (h.d < 1 || h.m < 1 || h.act < 0 || h.act > 2 || h.k < 0 || h.k > h.m || h.d % 8 != 0) return false;
  ffsplit_shape s{h.d, h.m, h.act, FFSPLIT_BF16};
  QuantHeader ref;
  layout_quant(s, h.k, &ref);
  if (std::memcmp(&ref, &h, sizeof(h)) != 0) return false;
  return blob_bytes >= h.total_bytes;
}

struct QSplits { int s1, s2a, s2b; };
QSplits quant_splits(const QuantHeader& h, int T) {
  const int gmax = quant_groups_max(stream_x_rows(T));
  auto need = [&](int g) { return g <= 0 ? 0 : (g + gmax - 1) / gmax; };
  QSplits q;
  q.s1 = need(h.gd); q.s2a = need(h.gk); q.s2b = need(h.gl);
  return q;
}
size_t quant_scratch_bytes(const QuantHeader& h, int T) {
  const QSplits q = quant_splits(h, T);
  const size_t n1 = static_cast<size_t>(h.n_in) * (h.k8 + h.ml8);
  return align_q(static_cast<size_t>(q.s1) * 8 * n1 * 4) + align_q(static_cast<size_t>(q.s2a + q.s2b) * 8 * h.d * 4);
}

}  // namespace
}  // namespace ffsp

using namespace ffsp;
using namespace ffsp::qnt;

extern "C" {

ffsplit_status ffsplit_quant_pack_size(const ffsplit_shape* shape, int32_t k, size_t* padded_bytes, size_t* logical_bytes) {
  ffsplit_status s = check_quant_shape(nullptr, shape, k);
  if (s != FFSPLIT_OK) return s;
  QuantHeader h;
  layout_quant(*shape, k, &h);
  if (padded_bytes) *padded_bytes = h.total_bytes;
  if (logical_bytes) *logical_bytes = h.logical_bytes;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_quant_workspace_size(const ffsplit_shape* shape, int32_t k, size_t* bytes) {
  if (!bytes) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_quant_shape(nullptr, shape, k);
  if (s != FFSPLIT_OK) return s;
  QuantHeader h;
  layout_quant(*shape, k, &h);
  size_t need = 0;
  for (int T : {1, 2, 4, 8}) {
    const size_t n = quant_scratch_bytes(h, T);
    if (n > need) need = n;
  }
  *bytes = kCtrlBytes + need;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_quant_pack(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                  const int32_t* heavy_idx, int32_t k, const int32_t* light_idx, void* blob,
                                  size_t blob_bytes, void* stream) {
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  ctx->prep_active = false;
  ctx->prep.n = 0;
  int dev = -1;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaGetDevice");
  if (dev != ctx->device) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "the context's device is not the current device");
  if (!ctx->ws || ctx->ws_bytes < kCtrlBytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "no workspace set (ffsplit_set_workspace)");
  ffsplit_status s = check_quant_shape(ctx, shape, k);
  if (s != FFSPLIT_OK) return s;
  if (!wt || !wt->W1 || !wt->W2 || !blob) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  const int ml = shape->m - k;
  if ((k > 0 && !heavy_idx) || (ml > 0 && !light_idx)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "index list is NULL");
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  if (gated && (!wt->W1u || wt->b1)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "SwiGLU needs W1u and no b1");
  if (!aligned16(wt->W1) || !aligned16(wt->W2) || (gated && !aligned16(wt->W1u)))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(blob) % kAlignQ != 0) return fail(ctx, FFSPLIT_ERR_ALIGN, "blob must be 256-byte aligned");
  QuantHeader h;
  layout_quant(*shape, k, &h);
  if (blob_bytes < h.total_bytes) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "blob buffer too small (ffsplit_quant_pack_size)");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* b = static_cast<unsigned char*>(blob);
  const int d = shape->d, m = shape->m;
  const __nv_bfloat16* W1 = static_cast<const __nv_bfloat16*>(wt->W1);
  const __nv_bfloat16* W1u = static_cast<const __nv_bfloat16*>(wt->W1u);
  const __nv_bfloat16* W2 = static_cast<const __nv_bfloat16*>(wt->W2);
  // biases: b1[h2], b1[light] (zero padded to k8, ml8), b2, and the check that h2 is ascending and in range
  if ((s = launch_pack_bias(ctx, FFSPLIT_BF16, wt->b1, wt->b2, heavy_idx, m, k, d, reinterpret_cast<float*>(b + h.off[QS_B1H]),
                            h.k8, reinterpret_cast<float*>(b + h.off[QS_B1L]), h.ml8, reinterpret_cast<float*>(b + h.off[QS_B2]),
                            st)) != FFSPLIT_OK)
    return s;
  // U-type: one neuron's input weights per packed row, groups along d
  if ((s = launch_quant_pack(ctx, W1, m, 1, heavy_idx, k, d, h.gd, 8, b + h.off[QS_U1], st)) != FFSPLIT_OK) return s;
  if ((s = launch_quant_pack(ctx, W1, m, 1, light_idx, ml, d, h.gd, 3, b + h.off[QS_U2], st)) != FFSPLIT_OK) return s;
  if (gated) {
    if ((s = launch_quant_pack(ctx, W1u, m, 1, heavy_idx, k, d, h.gd, 8, b + h.off[QS_U1U], st)) != FFSPLIT_OK) return s;
    if ((s = launch_quant_pack(ctx, W1u, m, 1, light_idx, ml, d, h.gd, 3, b + h.off[QS_U2U], st)) != FFSPLIT_OK) return s;
  }
  // V-type: one output column per packed row, groups along the part's neurons
  if (k > 0 && (s = launch_quant_pack(ctx, W2, d, 0, heavy_idx, d, k, h.gk, 8, b + h.off[QS_V1], st)) != FFSPLIT_OK) return s;
  if (ml > 0 && (s = launch_quant_pack(ctx, W2, d, 0, light_idx, d, ml, h.gl, 3, b + h.off[QS_V2], st)) != FFSPLIT_OK) return s;
  ffsplit_ctx::QuantEntry& ent = ctx->qblobs[blob];
  std::memcpy(ent.header, &h, sizeof(h));
  ent.bytes = h.total_bytes;
  ent.hash = header_hash_host(&h);
  ce = cudaMemcpyAsync(blob, ent.header, sizeof(h), cudaMemcpyHostToDevice, st);
  return check_cuda(ctx, ce, "cudaMemcpyAsync(quantised blob header)");
}

ffsplit_status ffsplit_quant_blob_open(ffsplit_ctx* ctx, const void* blob, size_t blob_bytes, void* stream) {
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  if (!blob) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "blob is NULL");
  if (reinterpret_cast<uintptr_t>(blob) % kAlignQ != 0) return fail(ctx, FFSPLIT_ERR_ALIGN, "blob must be 256-byte aligned");
  if (blob_bytes < sizeof(QuantHeader)) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "blob_bytes is smaller than a header");
  ctx->qblobs.erase(blob);
  QuantHeader h;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&h, blob, sizeof(h), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(quantised blob header)");
  if (!quant_header_valid(h, blob_bytes)) return fail(ctx, FFSPLIT_ERR_BAD_BLOB, "not a quantised packed layer (bad header, or larger than blob_bytes)");
  ffsplit_ctx::QuantEntry& ent = ctx->qblobs[blob];
  std::memcpy(ent.header, &h, sizeof(h));
  ent.bytes = blob_bytes;
  ent.hash = header_hash_host(&h);
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_quant_unpack(ffsplit_ctx* ctx, const void* blob, int32_t which, uint8_t* codes, float* scale,
                                    float* lo, void* stream) {
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  auto it = ctx->qblobs.find(blob);
  if (it == ctx->qblobs.end()) return fail(ctx, FFSPLIT_ERR_BAD_BLOB, "quantised blob not known to this context");
  if (which < QS_U1 || which > QS_V2 || !codes || !scale || !lo) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "bad argument");
  QuantHeader h;
  std::memcpy(&h, it->second.header, sizeof(h));
  const bool heavy = which == QS_U1 || which == QS_U1U || which == QS_V1;
  const bool vtype = which == QS_V1 || which == QS_V2;
  if ((which == QS_U1U || which == QS_U2U) && h.n_in != 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "the layer has no up projection");
  const int part = heavy ? h.k : h.ml;
  const int n_out = vtype ? h.d : part, n_k = vtype ? part : h.d;
  const int groups = vtype ? (heavy ? h.gk : h.gl) : h.gd;
  return launch_quant_unpack(ctx, static_cast<const unsigned char*>(blob) + h.off[which], n_out, n_k, groups, heavy ? 8 : 3, codes,
                             scale, lo, static_cast<cudaStream_t>(stream));
}

ffsplit_status ffsplit_quant_forward(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T, void* Y, void* stream) {
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  int dev = -1;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaGetDevice");
  if (dev != ctx->device) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "the context's device is not the current device");
  if (!ctx->ws || ctx->ws_bytes < kCtrlBytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "no workspace set (ffsplit_set_workspace)");
  if (!blob || !X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  if (!aligned16(X) || !aligned16(Y)) return fail(ctx, FFSPLIT_ERR_ALIGN, "X and Y must be 16-byte aligned");
  auto it = ctx->qblobs.find(blob);
  if (it == ctx->qblobs.end())
    return fail(ctx, FFSPLIT_ERR_BAD_BLOB, "quantised blob not known to this context: pack it here or register it with ffsplit_quant_blob_open()");
  QuantHeader h;
  std::memcpy(&h, it->second.header, sizeof(h));
  const unsigned char* b = static_cast<const unsigned char*>(blob);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ctx->score_prep.valid = false;
  const bool gated = h.act == FFSPLIT_SWIGLU;
  const int d = h.d, G = ctx->num_sms;
  const long long n1 = static_cast<long long>(h.n_in) * (h.k8 + h.ml8);
  // the tokens go through the kernel eight at a time
  for (int64_t t0 = 0; t0 < T; t0 += 8) {
    const int Tc = static_cast<int>(T - t0 < 8 ? T - t0 : 8);
    const QSplits sp = quant_splits(h, Tc);
    if (kCtrlBytes + quant_scratch_bytes(h, Tc) > ctx->ws_bytes)
      return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for the quantised forward (ffsplit_quant_workspace_size)");
    // the kernel's unit arithmetic is 32-bit: 17 units per 8-bit row, 7 per 3-bit row, times the k ranges
    const double units1 = (17.0 * h.k + 7.0 * h.ml) * h.n_in * sp.s1, units2 = 17.0 * d * (sp.s2a > sp.s2b ? sp.s2a : sp.s2b);
    if ((units1 > units2 ? units1 : units2) * (G + 1) >= 2147483648.0)
      return fail(ctx, FFSPLIT_ERR_SHAPE, "quantised forward: layer too large for the unit arithmetic");
    float* z = reinterpret_cast<float*>(ctx->ws + kCtrlBytes);
    float* ys = reinterpret_cast<float*>(ctx->ws + kCtrlBytes + align_q(static_cast<size_t>(sp.s1) * 8 * n1 * 4));
    QParams p;
    std::memset(&p, 0, sizeof(p));
    p.T = Tc; p.act = h.act; p.ctrl = ctx->status();
    p.x_rows = stream_x_rows(Tc);
    p.x_pitch = 2 * stream_kx_max(p.x_rows) + 64;
    p.guard = t0 == 0 ? reinterpret_cast<const unsigned long long*>(blob) : nullptr;
    p.guard_hash = it->second.hash;
    auto add_seg = [](QPhase& ph, const unsigned char* W, int groups, int rows, int bits, int x_off, int out_col) {
      if (rows <= 0) return;
      QSegment& s = ph.seg[ph.nseg++];
      s.W = W; s.row_bytes = static_cast<long long>(groups) * (bits == 8 ? kGroupBytes8 : kGroupBytes3);
      s.rows = rows; s.bits = bits; s.x_off = x_off; s.out_col = out_col;
    };
    // ---- phase 1: z = X [U1~ | U2~] (SwiGLU: and the up projections behind them), raw
    {
      QPhase& ph = p.ph[p.nph++];
      ph.sync_before = 1; ph.G = h.gd; ph.S = sp.s1;
      add_seg(ph, b + h.off[QS_U1], h.gd, h.k, 8, 0, 0);
      add_seg(ph, b + h.off[QS_U2], h.gd, h.ml, 3, 0, h.k8);
      if (gated) {
        add_seg(ph, b + h.off[QS_U1U], h.gd, h.k, 8, 0, h.k8 + h.ml8);
        add_seg(ph, b + h.off[QS_U2U], h.gd, h.ml, 3, 0, 2 * h.k8 + h.ml8);
      }
      StreamInPart& in = ph.in[0];
      ph.nin = 1;
      in.col_begin = 0; in.col_end = d; in.kind = STREAM_IN_BF16;
      in.src = static_cast<const __nv_bfloat16*>(X) + t0 * d; in.ld = d;
      ph.out = z; ph.out_ld = n1;
    }
    // ---- phase 2: the heavy part sigma(z_H + b1[h2]) V1~ and the light part sigma(z_L + b1[light]) V2~
    auto part_phase = [&](int sec, int groups, int n_part, int bits, int src_col, int splits, int slice0, int sec_bias, bool sync) {
      if (n_part <= 0) return;
      QPhase& ph = p.ph[p.nph++];
      ph.sync_before = sync ? 1 : 0; ph.G = groups; ph.S = splits; ph.slice0 = slice0;
      add_seg(ph, b + h.off[sec], groups, d, bits, 0, 0);
      StreamInPart& in = ph.in[0];
      ph.nin = 1;
      in.col_begin = 0; in.col_end = n_part; in.kind = gated ? STREAM_IN_GATED : STREAM_IN_ACT;
      in.nslices = sp.s1; in.src = z; in.ld = n1; in.slice_stride = 8 * n1; in.src_col = src_col;
      in.gate_off = h.k8 + h.ml8;
      in.bias = gated ? nullptr : reinterpret_cast<const float*>(b + h.off[sec_bias]);
      ph.out = ys; ph.out_ld = d;
    };
    part_phase(QS_V1, h.gk, h.k, 8, 0, sp.s2a, 0, QS_B1H, true);
    part_phase(QS_V2, h.gl, h.ml, 3, h.k8, sp.s2b, sp.s2a, QS_B1L, h.k <= 0);
    // ---- closing reduction: Y = all slices + b2
    {
      QPhase& rd = p.ph[p.nph++];
      rd.kind = 1; rd.sync_before = 1;
      StreamInPart& in = rd.in[0];
      rd.nin = 1;
      in.col_begin = 0; in.col_end = d; in.kind = STREAM_IN_LINEAR; in.nslices = sp.s2a + sp.s2b; in.src = ys; in.ld = d;
      in.slice_stride = 8ll * d;
      rd.y = static_cast<__nv_bfloat16*>(Y) + t0 * d; rd.y_ld = d; rd.y_bias = reinterpret_cast<const float*>(b + h.off[QS_B2]);
      rd.y_cols = d;
    }
    const ffsplit_status s = decode_quant_launch(ctx, p, static_cast<double>(h.logical_bytes) + 4.0 * Tc * d, st);
    if (s != FFSPLIT_OK) return s;
  }
  return FFSPLIT_OK;
}

}  // extern "C"
