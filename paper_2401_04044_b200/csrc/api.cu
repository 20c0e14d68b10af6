// C ABI of libffsplit: argument validation, memory layouts (workspace, packed
// blob) and the sequencing of kernels for score / select / pack / forward.
#include <cstdlib>
#include <cstring>

#include "internal.h"

using namespace ffsp;

namespace ffsp {

ffsplit_status fail(ffsplit_ctx* ctx, ffsplit_status code, const std::string& msg) {
  if (ctx) ctx->err = msg;
  return code;
}

ffsplit_status check_cuda(ffsplit_ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return FFSPLIT_OK;
  if (ctx) ctx->err = std::string(what) + ": " + cudaGetErrorString(e);
  return FFSPLIT_ERR_CUDA;
}

int prof_open(ffsplit_ctx* ctx, int cls, double work, cudaStream_t st) {
  if (!ctx->profiling) return -1;
  ffsplit_ctx::ProfRec r;
  r.cls = cls;
  r.work = work;
  if (cudaEventCreate(&r.a) != cudaSuccess) return -1;
  if (cudaEventCreate(&r.b) != cudaSuccess) { cudaEventDestroy(r.a); return -1; }
  cudaEventRecord(r.a, st);
  ctx->prof.push_back(r);
  return static_cast<int>(ctx->prof.size()) - 1;
}

void prof_close(ffsplit_ctx* ctx, int handle, cudaStream_t st) {
  if (handle >= 0) cudaEventRecord(ctx->prof[handle].b, st);
}

ffsplit_status launch_decode_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                     long long T, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                     cudaStream_t st, unsigned long long guard_hash);
bool decode_path_applies(const ffsplit_ctx* ctx, const BlobHeader& h, long long T);
char* noalloc_control_block(int device);   // nullptr until ffsplit_forward_noalloc has run on that device
size_t decode_scratch_bytes(int dtype, long long T);

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct SplitDims {
  int k, r, ml, k_pad, r_pad, ml_pad, kp_rp, n_in;
};

SplitDims make_dims(const ffsplit_shape& s, int k, int r) {
  SplitDims o;
  o.k = k;
  o.r = r;
  o.ml = s.m - k;
  o.n_in = s.act == FFSPLIT_SWIGLU ? 2 : 1;
  o.k_pad = round_up(k, 16);
  o.r_pad = round_up(r, 16);
  o.ml_pad = r > 0 ? round_up(o.ml, 16) : 0;
  if (o.k_pad + o.r_pad == 0) o.k_pad = 16;  // keeps the last GEMM non-empty: Y = b2
  o.kp_rp = o.k_pad + o.r_pad;
  return o;
}

ffsplit_status check_shape(ffsplit_ctx* ctx, const ffsplit_shape* s) {
  if (!s) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "shape is NULL");
  if (s->d < 1 || s->m < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "d and m must be >= 1");
  if (s->act < 0 || s->act > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown activation");
  if (s->dtype != FFSPLIT_F32 && s->dtype != FFSPLIT_BF16) return fail(ctx, FFSPLIT_ERR_DTYPE, "unknown dtype");
  if (s->dtype == FFSPLIT_BF16 && s->d % 8 != 0)
    return fail(ctx, FFSPLIT_ERR_SHAPE, "bf16 layers need d to be a multiple of 8");
  return FFSPLIT_OK;
}

ffsplit_status check_split(ffsplit_ctx* ctx, const ffsplit_shape* s, int k, int r) {
  if (k < 0 || k > s->m) return fail(ctx, FFSPLIT_ERR_SHAPE, "k must be in [0, m]");
  const int ml = s->m - k;
  const int rmax = s->d < ml ? s->d : ml;
  if (r < 0 || r > rmax) return fail(ctx, FFSPLIT_ERR_SHAPE, "r must be in [0, min(d, m - k)]");
  return FFSPLIT_OK;
}

void layout_blob(const ffsplit_shape& s, const SplitDims& D, BlobHeader* h) {
  std::memset(h, 0, sizeof(*h));
  const size_t es = elem_size(s.dtype);
  h->magic = kBlobMagic;
  h->version = kBlobVersion;
  h->d = s.d; h->m = s.m; h->act = s.act; h->dtype = s.dtype;
  h->k = D.k; h->r = D.r; h->n_in = D.n_in;
  h->k_pad = D.k_pad; h->r_pad = D.r_pad; h->ml_pad = D.ml_pad; h->ml = D.ml;
  size_t off = sizeof(BlobHeader);
  // U1^T, A1^T (and the SwiGLU up factor) are adjacent with the same pitch d, so
  // that [U1 | A1]^T and [A1 | A1u]^T can each be read as one matrix.
  h->off[SEC_U1T] = off;  off += (size_t)D.k_pad * s.d * es;
  h->off[SEC_A1T] = off;  off += (size_t)D.r_pad * s.d * es;
  if (D.n_in == 2) { h->off[SEC_A1UT] = off; off += (size_t)D.r_pad * s.d * es; }
  off = align_up(off);
  if (D.n_in == 2) { h->off[SEC_U1UT] = off; off = align_up(off + (size_t)D.k_pad * s.d * es); }
  h->off[SEC_B1T] = off;  off = align_up(off + (size_t)D.ml_pad * D.r_pad * es);
  if (D.n_in == 2) { h->off[SEC_B1UT] = off; off = align_up(off + (size_t)D.ml_pad * D.r_pad * es); }
  h->off[SEC_A2T] = off;  off = align_up(off + (size_t)D.r_pad * D.ml_pad * es);
  h->off[SEC_V1B2T] = off; off = align_up(off + (size_t)s.d * D.kp_rp * es);
  h->off[SEC_B1H] = off;  off = align_up(off + (size_t)D.k_pad * 4);
  h->off[SEC_B1L] = off;  off = align_up(off + (size_t)D.ml_pad * 4);
  h->off[SEC_B2] = off;   off = align_up(off + (size_t)s.d * 4);
  h->total_bytes = off;
  const size_t params = (size_t)(D.n_in + 1) * ((size_t)s.d * D.k + (size_t)D.r * (s.d + D.ml));
  h->logical_bytes = es * (params + s.m + s.d);
}

SplitDims dims_of(const BlobHeader& h) {
  SplitDims D;
  D.k = h.k; D.r = h.r; D.ml = h.ml; D.k_pad = h.k_pad; D.r_pad = h.r_pad; D.ml_pad = h.ml_pad;
  D.kp_rp = h.k_pad + h.r_pad; D.n_in = h.n_in;
  return D;
}

bool header_valid(const BlobHeader& h, size_t blob_bytes) {
  if (h.magic != kBlobMagic || h.version != kBlobVersion) return false;
  ffsplit_shape s{h.d, h.m, h.act, h.dtype};
  if (s.d < 1 || s.m < 1 || s.act < 0 || s.act > 2 || (s.dtype != 0 && s.dtype != 1)) return false;
  if (h.k < 0 || h.k > h.m || h.r < 0) return false;
  BlobHeader ref;
  layout_blob(s, make_dims(s, h.k, h.r), &ref);
  if (std::memcmp(&ref, &h, sizeof(BlobHeader)) != 0) return false;
  return blob_bytes == 0 || blob_bytes >= h.total_bytes;
}

struct FwdLayout { size_t ap, q, hl, skp, skp_bytes, xs, ys, dscratch, end; };
// The T x mL buffer of the unfused light chain doubles as the fp32 partial buffer of
// the fused kernel (only one of the two paths runs in a call).
FwdLayout fwd_layout(const SplitDims& D, int d, int dtype, int act, long long T) {
  FwdLayout L;
  const size_t es = elem_size(dtype);
  size_t off = 0;
  L.ap = off; off = align_up(off + (size_t)T * D.kp_rp * es);
  L.q = off;  off = align_up(off + (size_t)T * D.n_in * D.r_pad * es);
  size_t hl = (size_t)T * D.ml_pad * es;
  if (fused_light_applies(dtype, act, D.r_pad, D.ml_pad)) {
    const size_t fs = fused_light_scratch_bytes(T, D.r_pad);
    if (fs > hl) hl = fs;
  }
  if (fused_layer_applies(dtype, act, d, D.k, D.k_pad, D.r_pad, D.ml_pad, T, 1 << 20)) {   // whatever the SM count
    const size_t fs = fused_layer_scratch_bytes(T, D.r_pad);
    if (fs > hl) hl = fs;
  }
  L.hl = off; off = align_up(off + hl);
  // fp32 partials of the light chain's second product when it is cut along K (up to four of [T, r_pad])
  L.skp_bytes = (dtype == FFSPLIT_BF16 && D.r_pad > 0 && T > 64) ? static_cast<size_t>(4) * T * D.r_pad * 4 : 0;
  L.skp = off; off = align_up(off + L.skp_bytes);
  L.xs = off; off = align_up(off + (size_t)T * d * es);
  L.ys = off; off = align_up(off + (size_t)T * d * es);
  L.dscratch = off; off = align_up(off + decode_scratch_bytes(dtype, T));   // few-token path: split-K partials
  L.end = off;
  return L;
}

struct ScoreLayout { size_t w1t, w1ut, b1f, w, partial, end; int groups; };
ScoreLayout score_layout(const ffsplit_shape& s, long long T) {
  ScoreLayout L;
  const size_t es = elem_size(s.dtype);
  size_t off = 0;
  L.w1t = off;  off = align_up(off + (size_t)s.m * s.d * es);
  L.w1ut = off; if (s.act == FFSPLIT_SWIGLU) off = align_up(off + (size_t)s.m * s.d * es);
  L.b1f = off;  off = align_up(off + (size_t)s.m * 4);
  L.w = off;    off = align_up(off + (size_t)s.m * 4);
  L.groups = s.dtype == FFSPLIT_BF16 ? 4 * (int)((T + 127) / 128) : (int)((T + 63) / 64);
  L.partial = off; off = align_up(off + (size_t)L.groups * s.m * 4);
  L.end = off;
  return L;
}

ffsplit_status check_ctx(ffsplit_ctx* ctx, bool need_ws) {
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  ctx->prep_active = false;   // a batch left open by a call that failed half-way is dropped
  ctx->prep.n = 0;
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaGetDevice");
  if (dev != ctx->device) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "the context's device is not the current device");
  if (need_ws && (!ctx->ws || ctx->ws_bytes < kCtrlBytes))
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "no workspace set (ffsplit_set_workspace)");
  return FFSPLIT_OK;
}

// A blob is known to a context once ffsplit_pack() wrote it or ffsplit_blob_open() registered it there;
// nothing is opened implicitly (a header read inside a forward would be a synchronous copy that is not
// ordered after whatever produced the blob).
const ffsplit_ctx::BlobEntry* find_blob(ffsplit_ctx* ctx, const void* blob, ffsplit_status* st) {
  auto it = ctx->blobs.find(blob);
  if (it != ctx->blobs.end()) return &it->second;
  *st = fail(ctx, FFSPLIT_ERR_BAD_BLOB,
             "blob not known to this context: pack it here or register it with ffsplit_blob_open()");
  return nullptr;
}

// The three-stage split forward (Eq. 2) as a sequence of GEMMs with fused epilogues.
// guard_hash != 0: the first kernel checks that the header in device memory still is the one registered.
ffsplit_status run_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X, long long T,
                           void* Y, cudaStream_t st, unsigned long long guard_hash) {
  const SplitDims D = dims_of(h);
  const size_t es = elem_size(h.dtype);
  const int d = h.d;
  char* base = ctx->ws + kCtrlBytes;
  ctx->score_prep.valid = false;   // the forward buffers share the workspace with the scoring buffers
  const FwdLayout L = fwd_layout(D, d, h.dtype, h.act, T);
  const bool few = decode_path_applies(ctx, h, T);
  if (kCtrlBytes + (T <= 64 ? L.end : L.xs) > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this forward (ffsplit_workspace_size)");
  char* AP = base + L.ap;
  char* Q = base + L.q;
  char* HL = base + L.hl;
  if (few) return launch_decode_forward(ctx, h, blob, X, T, Y, AP, Q, HL, base + L.dscratch, st, guard_hash);
  const unsigned long long* guard = guard_hash ? reinterpret_cast<const unsigned long long*>(blob) : nullptr;
  const float* b1h = reinterpret_cast<const float*>(blob + h.off[SEC_B1H]);
  const float* b1l = reinterpret_cast<const float*>(blob + h.off[SEC_B1L]);
  const float* b2 = reinterpret_cast<const float*>(blob + h.off[SEC_B2]);
  const bool gated = h.act == FFSPLIT_SWIGLU;
  const bool light = D.r_pad > 0 && D.ml > 0;
  ffsplit_status s;
  GemmArgs g;
  // 13..64 tokens of a bf16 layer: the stage GEMMs below with the operands exchanged (weights as accumulator rows)
  const bool few_tc = h.dtype == FFSPLIT_BF16 && T <= 64;
  void* few_ptr = few_tc ? base + L.dscratch : nullptr;
  int n_gemm = 0;       // products launched so far by this call
  const size_t few_bytes = few_tc ? decode_scratch_bytes(h.dtype, T) : 0;

  // ---- small hidden widths: the whole layer in one launch, a cluster of four CTAs per 128-token tile
  if (light && ctx->use_layer_kernel && fused_layer_applies(h.dtype, h.act, d, D.k, D.k_pad, D.r_pad, D.ml_pad, T, ctx->num_sms))
    return launch_fused_layer(ctx, h, blob, X, T, HL, AP, D.kp_rp, Y, guard_hash, st);

  // ---- stage 1: [A_H | Q] = X [U1 | A1], activation on the heavy columns only
  if (!gated) {
    std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
    g.A0 = X; g.lda0 = d;
    g.B0 = blob + h.off[SEC_U1T]; g.ldb0 = d;
    g.M = T; g.N = D.kp_rp; g.K = d;
    g.algo_flops = 2.0 * T * d * (D.k + D.r);
    g.epi.C0 = AP; g.epi.ld0 = D.kp_rp;
    g.epi.C1 = Q; g.epi.ld1 = D.r_pad;
    g.epi.n_split = D.k_pad; g.epi.n_act = D.k_pad; g.epi.n_bias = D.k_pad;
    g.epi.bias = b1h; g.epi.act = h.act;
    g.epi.guard = guard; g.epi.guard_hash = guard_hash;
    if ((s = launch_gemm(ctx, h.dtype, g, st)) != FFSPLIT_OK) return s;
  } else {
    std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
    g.A0 = X; g.lda0 = d; g.B0 = blob + h.off[SEC_U1T]; g.ldb0 = d;
    g.A1 = X; g.lda1 = d; g.B1 = blob + h.off[SEC_U1UT]; g.ldb1 = d;
    g.M = T; g.N = D.k_pad; g.K = d;
    g.algo_flops = 4.0 * T * d * D.k;
    g.epi.C0 = AP; g.epi.ld0 = D.kp_rp;
    g.epi.n_split = D.k_pad; g.epi.n_act = D.k_pad; g.epi.act = h.act;
    g.epi.guard = guard; g.epi.guard_hash = guard_hash;
    if ((s = launch_gemm(ctx, h.dtype, g, st)) != FFSPLIT_OK) return s;
    if (light) {
      std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
      g.A0 = X; g.lda0 = d; g.B0 = blob + h.off[SEC_A1T]; g.ldb0 = d;  // [A1 | A1u]^T
      g.M = T; g.N = 2 * D.r_pad; g.K = d;
      g.algo_flops = 4.0 * T * d * D.r;
      g.epi.C0 = Q; g.epi.ld0 = 2 * D.r_pad; g.epi.n_split = g.N; g.epi.act = h.act;
      if ((s = launch_gemm(ctx, h.dtype, g, st)) != FFSPLIT_OK) return s;
    }
  }
  // ---- stage 2: P = sigma(Q B1 + b1[light]) A2, written next to A_H
  if (ctx->use_fused < 0) {
    const char* env = std::getenv("FFSPLIT_NO_FUSED");
    ctx->use_fused = (env && env[0] == '1') ? 0 : 1;
  }
  const long long tiles_m = (T + 127) / 128;
  if (light && ctx->use_fused && !few_tc && fused_light_applies(h.dtype, h.act, D.r_pad, D.ml_pad) && tiles_m <= kMaxTicketTiles) {
    if ((s = launch_fused_light(ctx, Q, D.r_pad, T, blob + h.off[SEC_B1T], blob + h.off[SEC_A2T], b1l, D.r_pad,
                                D.ml_pad, h.act, AP + (size_t)D.k_pad * es, D.kp_rp, HL, ctx->tickets(),
                                4.0 * T * D.r * D.ml, st)) != FFSPLIT_OK)
      return s;
  } else if (light) {
    std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
    g.A0 = Q; g.lda0 = (long long)D.n_in * D.r_pad;
    g.B0 = blob + h.off[SEC_B1T]; g.ldb0 = D.r_pad;
    if (gated) {
      g.A1 = Q + (size_t)D.r_pad * es; g.lda1 = g.lda0;
      g.B1 = blob + h.off[SEC_B1UT]; g.ldb1 = D.r_pad;
    }
    g.M = T; g.N = D.ml_pad; g.K = D.r_pad;
    g.algo_flops = 2.0 * D.n_in * T * D.r * D.ml;
    g.epi.C0 = HL; g.epi.ld0 = D.ml_pad;
    g.epi.n_split = g.N; g.epi.n_act = g.N; g.epi.n_bias = gated ? 0 : g.N;
    g.epi.bias = b1l; g.epi.act = h.act;
    if ((s = launch_gemm(ctx, h.dtype, g, st)) != FFSPLIT_OK) return s;

    std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
    g.A0 = HL; g.lda0 = D.ml_pad;
    g.B0 = blob + h.off[SEC_A2T]; g.ldb0 = D.ml_pad;
    g.M = T; g.N = D.r_pad; g.K = D.ml_pad;
    g.algo_flops = 2.0 * T * D.r * D.ml;
    g.epi.C0 = AP + (size_t)D.k_pad * es; g.epi.ld0 = D.kp_rp;
    g.epi.n_split = g.N; g.epi.act = h.act;
    g.splitk = L.skp_bytes ? base + L.skp : nullptr; g.splitk_bytes = L.skp_bytes;
    if ((s = launch_gemm(ctx, h.dtype, g, st)) != FFSPLIT_OK) return s;
  }
  // ---- stage 3: Y = [A_H | P] [V1 ; B2] + b2 (heavy and light parts in one accumulator)
  std::memset(&g, 0, sizeof(g));
    g.few = few_ptr; g.few_bytes = few_bytes; g.weights_stable = n_gemm++ > 0;
  g.A0 = AP; g.lda0 = D.kp_rp;
  g.B0 = blob + h.off[SEC_V1B2T]; g.ldb0 = D.kp_rp;
  g.M = T; g.N = d; g.K = light ? D.kp_rp : D.k_pad;
  g.algo_flops = 2.0 * T * d * (D.k + (light ? D.r : 0));
  g.epi.C0 = Y; g.epi.ld0 = d;
  g.epi.n_split = d; g.epi.n_bias = d; g.epi.bias = b2; g.epi.act = h.act;
  return launch_gemm(ctx, h.dtype, g, st);
}


// ---- a stack of layers, layer l reading layer l-1's output ------------------------------------
// The intermediate outputs alternate between two buffers placed behind the largest per-layer forward layout.
struct StackLayout { size_t ping, pong, end; };
ffsplit_status stack_layout(ffsplit_ctx* ctx, const void* const* blobs, int n_layers, long long T, StackLayout* out) {
  size_t body = 0;
  int d = -1, dtype = -1;
  for (int l = 0; l < n_layers; ++l) {
    ffsplit_status s = FFSPLIT_OK;
    const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blobs[l], &s);
    if (!ent) return s;
    const BlobHeader& h = ent->h;
    if (l == 0) { d = h.d; dtype = h.dtype; }
    else if (h.d != d || h.dtype != dtype)
      return fail(ctx, FFSPLIT_ERR_SHAPE, "the layers of a stack must share the hidden width and the dtype");
    const size_t e = fwd_layout(dims_of(h), h.d, h.dtype, h.act, T).end;
    if (e > body) body = e;
  }
  const size_t act = align_up(static_cast<size_t>(T) * d * elem_size(dtype));
  out->ping = body;
  out->pong = body + act;
  out->end = body + 2 * act;
  return FFSPLIT_OK;
}

}  // namespace
}  // namespace ffsp

static ffsplit_status forward_stack_impl(ffsplit_ctx* ctx, const void* const* blobs, int n_layers, const void* X,
                                         long long T, void* Y, cudaStream_t st, bool host) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if (!blobs || n_layers < 1 || !X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor or empty stack");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  if (!host && (!aligned16(X) || !aligned16(Y))) return fail(ctx, FFSPLIT_ERR_ALIGN, "X and Y must be 16-byte aligned");
  StackLayout SL;
  if ((s = stack_layout(ctx, blobs, n_layers, T, &SL)) != FFSPLIT_OK) return s;
  if (kCtrlBytes + SL.end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this stack (ffsplit_stack_workspace_size)");
  char* base = ctx->ws + kCtrlBytes;
  char* buf[2] = {base + SL.ping, base + SL.pong};
  const BlobHeader& h0 = ctx->blobs.find(blobs[0])->second.h;
  const size_t bytes = static_cast<size_t>(T) * h0.d * elem_size(h0.dtype);
  const void* in = X;
  int which = 0;
  if (host) {
    cudaError_t e = cudaMemcpyAsync(buf[0], X, bytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(X)");
    in = buf[0];
    which = 1;
  }
  for (int l = 0; l < n_layers; ++l) {
    const ffsplit_ctx::BlobEntry& ent = ctx->blobs.find(blobs[l])->second;
    const bool last = l == n_layers - 1;
    void* out = (last && !host) ? Y : static_cast<void*>(buf[which]);
    if ((s = run_forward(ctx, ent.h, static_cast<const char*>(blobs[l]), in, T, out, st, ent.hash)) != FFSPLIT_OK) return s;
    in = out;
    which ^= 1;
  }
  if (host) {
    cudaError_t e = cudaMemcpyAsync(Y, in, bytes, cudaMemcpyDeviceToHost, st);
    return check_cuda(ctx, e, "cudaMemcpyAsync(Y)");
  }
  return FFSPLIT_OK;
}

namespace ffsp {
// One packed FFN layer inside another entry point (the encoder block): same checks and path as ffsplit_forward.
ffsplit_status run_ffn_forward(ffsplit_ctx* ctx, const void* blob, const void* X, long long T, void* Y, cudaStream_t st) {
  ffsplit_status s = FFSPLIT_OK;
  const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blob, &s);
  if (!ent) return s;
  return run_forward(ctx, ent->h, static_cast<const char*>(blob), X, T, Y, st, ent->hash);
}
// Bytes of the workspace (behind the control block) that forward of this blob at T tokens uses.
size_t ffn_forward_workspace_end(ffsplit_ctx* ctx, const void* blob, long long T, ffsplit_status* status, int* d, int* dtype) {
  const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blob, status);
  if (!ent) return 0;
  if (d) *d = ent->h.d;
  if (dtype) *dtype = ent->h.dtype;
  return fwd_layout(dims_of(ent->h), ent->h.d, ent->h.dtype, ent->h.act, T).end;
}
}  // namespace ffsp

// =====================================================================================
extern "C" {

int32_t ffsplit_version(void) { return 100; }

const char* ffsplit_last_error(const ffsplit_ctx* ctx) {
  return ctx ? ctx->err.c_str() : "no context";
}

ffsplit_status ffsplit_profile_begin(ffsplit_ctx* ctx) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  for (auto& r : ctx->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  ctx->prof.clear();
  ctx->profiling = true;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_profile_end(ffsplit_ctx* ctx, void* stream, int32_t kernel_class, int32_t* launches,
                                   double* total_ms, double* total_work) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  ctx->profiling = false;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaStreamSynchronize");
  int n = 0;
  double ms = 0.0, work = 0.0;
  for (auto& r : ctx->prof) {
    if (r.cls != kernel_class) continue;
    float t = 0.f;
    if (cudaEventSynchronize(r.b) == cudaSuccess && cudaEventElapsedTime(&t, r.a, r.b) == cudaSuccess) {
      ++n; ms += t; work += r.work;
    }
  }
  cudaGetLastError();
  if (launches) *launches = n;
  if (total_ms) *total_ms = ms;
  if (total_work) *total_work = work;
  return FFSPLIT_OK;
}

int64_t ffsplit_launch_count(const ffsplit_ctx* ctx) { return ctx ? ctx->launches : 0; }

ffsplit_status ffsplit_create(ffsplit_ctx** out, int device) {
  if (!out) return FFSPLIT_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) {
    cudaGetLastError();
    return FFSPLIT_ERR_CUDA;
  }
  int major = 0, minor = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, device) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return FFSPLIT_ERR_CUDA;
  if (major != 10) return FFSPLIT_ERR_ARCH;
  ffsplit_ctx* c = new ffsplit_ctx();
  c->device = device;
  c->cc_major = major;
  c->cc_minor = minor;
  c->num_sms = sms;
  if (const char* env = std::getenv("FFSPLIT_GEMM_TWO_M")) c->gemm_two_m = env[0] == '0' ? 0 : env[0] == '2' ? 2 : 1;
  if (const char* env = std::getenv("FFSPLIT_GEMM_ARES")) c->gemm_ares = env[0] == '0' ? 0 : 1;
  if (const char* env = std::getenv("FFSPLIT_GEMM_PANEL")) c->gemm_panel = std::atoi(env);
  if (const char* env = std::getenv("FFSPLIT_GEMM_SPLIT_K")) c->gemm_split_k = env[0] == '0' ? 0 : 1;
  if (const char* env = std::getenv("FFSPLIT_FEW_TENSOR_MIN")) c->few_tensor_min = std::atoi(env);
  if (const char* env = std::getenv("FFSPLIT_LAYER_KERNEL")) c->use_layer_kernel = env[0] == '0' ? 0 : 1;
  if (const char* env = std::getenv("FFSPLIT_DECODE_LAYER")) c->decode_one_launch = env[0] == '0' ? 0 : 1;
  if (const char* env = std::getenv("FFSPLIT_DECODE_STREAM")) c->decode_stream = env[0] == '0' ? 0 : env[0] == '2' ? 2 : 1;
  *out = c;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_destroy(ffsplit_ctx* ctx) {
  if (ctx) for (auto& r : ctx->prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
  delete ctx;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_workspace_size(const ffsplit_shape* shape, int64_t T_fwd, int64_t T_cal, int32_t k, int32_t r,
                                      size_t* bytes) {
  if (!bytes) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_shape(nullptr, shape);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_split(nullptr, shape, k, r)) != FFSPLIT_OK) return s;
  if (T_fwd < 0 || T_cal < 0) return FFSPLIT_ERR_INVALID_ARG;
  const SplitDims D = make_dims(*shape, k, r);
  size_t need = 0;
  if (T_fwd > 0) {
    need = fwd_layout(D, shape->d, shape->dtype, shape->act, T_fwd).end;
  }
  if (T_cal > 0) {
    const size_t sc = score_layout(*shape, T_cal).end;
    if (sc > need) need = sc;
  }
  *bytes = kCtrlBytes + need;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_set_workspace(ffsplit_ctx* ctx, void* dev_ptr, size_t bytes) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  if (!dev_ptr || bytes < kCtrlBytes) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace needs >= 65536 bytes");
  if (reinterpret_cast<uintptr_t>(dev_ptr) % kAlign != 0)
    return fail(ctx, FFSPLIT_ERR_ALIGN, "workspace must be 256-byte aligned");
  cudaError_t e = cudaMemset(dev_ptr, 0, kCtrlBytes);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemset(control block)");
  ctx->ws = static_cast<char*>(dev_ptr);
  ctx->ws_bytes = bytes;
  ctx->tmaps.clear();
  ctx->score_prep.valid = false;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_poll(ffsplit_ctx* ctx, void* stream) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaStreamSynchronize");
  // Two places can hold a device-side condition: the control block of the workspace (if one is set) and
  // the control block inside the built-in scratch of ffsplit_forward_noalloc (if that has run on this device).
  char* blocks[2] = {ctx->ws, noalloc_control_block(ctx->device)};
  const char* where[2] = {"workspace", "built-in scratch"};
  for (int b = 0; b < 2; ++b) {
    if (!blocks[b]) continue;
    int words[4] = {0, 0, 0, 0};
    e = cudaMemcpy(words, blocks[b], sizeof(words), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpy(status block)");
    if (words[0] == 0) continue;
    e = cudaMemset(blocks[b], 0, kCtrlBytes);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemset(control block)");
    ctx->err = "device status " + std::to_string(words[0]) + " (detail " + std::to_string(words[1]) + ", kernel " +
               std::to_string(words[2]) + ", " + where[b] + ")";
    return static_cast<ffsplit_status>(words[0]);
  }
  return FFSPLIT_OK;
}

// Arguments of a scoring call, checked.
static ffsplit_status check_score_args(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                       const void* X, int64_t T, int32_t mode, const float* energy) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_shape(ctx, shape)) != FFSPLIT_OK) return s;
  if (!wt || !wt->W1 || !wt->W2 || !X || !energy) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  if (mode < 0 || mode > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown score mode");
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  if (gated && (!wt->W1u || wt->b1)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "SwiGLU needs W1u and no b1");
  if (!aligned16(wt->W1) || !aligned16(wt->W2) || (gated && !aligned16(wt->W1u)))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  return FFSPLIT_OK;
}

// U^T (K-major for the contraction over d), the fp32 bias and ||V_j||^2 into the scoring region of the
// workspace, as one batched launch -- unless that region still holds them from an earlier batch of the same
// accumulation.
static ffsplit_status score_prepare(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                    const ScoreLayout& L, bool need_w, bool may_reuse, cudaStream_t st) {
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  const int d = shape->d, m = shape->m, dt = shape->dtype;
  ffsplit_ctx::ScorePrep& c = ctx->score_prep;
  const bool same = c.valid && c.W1 == wt->W1 && c.W1u == wt->W1u && c.b1 == wt->b1 && c.W2 == wt->W2 && c.d == d &&
                    c.m == m && c.act == shape->act && c.dtype == dt;
  if (may_reuse && same && (c.has_w || !need_w)) return FFSPLIT_OK;
  char* base = ctx->ws + kCtrlBytes;
  ffsplit_status s;
  c.valid = false;
  prep_begin(ctx);
  if ((s = launch_transpose(ctx, dt, wt->W1, m, d, m, base + L.w1t, d, d, m, nullptr, d, st)) != FFSPLIT_OK) return s;
  if (gated && (s = launch_transpose(ctx, dt, wt->W1u, m, d, m, base + L.w1ut, d, d, m, nullptr, d, st)) != FFSPLIT_OK)
    return s;
  if (!gated && (s = launch_to_f32(ctx, dt, wt->b1, m, reinterpret_cast<float*>(base + L.b1f), st)) != FFSPLIT_OK) return s;
  if (need_w && (s = launch_row_energy(ctx, dt, wt->W2, m, d, reinterpret_cast<float*>(base + L.w), st)) != FFSPLIT_OK)
    return s;
  if ((s = prep_flush(ctx, dt, st)) != FFSPLIT_OK) return s;
  c.valid = true; c.has_w = need_w;
  c.W1 = wt->W1; c.W1u = wt->W1u; c.b1 = wt->b1; c.W2 = wt->W2; c.d = d; c.m = m; c.act = shape->act; c.dtype = dt;
  return FFSPLIT_OK;
}

// One batch of calibration tokens (device memory) through the product with the column-energy epilogue.
static ffsplit_status score_batch(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ScoreLayout& L, const void* X,
                                  int64_t T, int32_t mode, int32_t accumulate, float* energy, float* scores,
                                  cudaStream_t st) {
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  const int d = shape->d, m = shape->m, dt = shape->dtype;
  char* base = ctx->ws + kCtrlBytes;
  float* b1f = reinterpret_cast<float*>(base + L.b1f);
  float* w = reinterpret_cast<float*>(base + L.w);
  float* partial = reinterpret_cast<float*>(base + L.partial);
  GemmArgs g;
  std::memset(&g, 0, sizeof(g));
  g.A0 = X; g.lda0 = d; g.B0 = base + L.w1t; g.ldb0 = d;
  if (gated) { g.A1 = X; g.lda1 = d; g.B1 = base + L.w1ut; g.ldb1 = d; }
  g.M = T; g.N = m; g.K = d;
  g.algo_flops = 2.0 * (gated ? 2 : 1) * T * (double)d * m;
  g.epi.col_partial = partial;
  g.epi.n_bias = gated ? 0 : m; g.epi.bias = b1f; g.epi.n_act = m; g.epi.n_split = m;
  g.epi.act = shape->act; g.epi.score_abs = mode == FFSPLIT_SCORE_SUM_NORM;
  ffsplit_status s;
  if ((s = launch_gemm(ctx, dt, g, st)) != FFSPLIT_OK) return s;
  // row groups this batch produced (a last, shorter chunk fills fewer than the layout has room for)
  const int groups = dt == FFSPLIT_BF16 ? 4 * static_cast<int>((T + 127) / 128) : static_cast<int>((T + 63) / 64);
  return launch_score_finalize(ctx, partial, groups, m, w, energy, scores, mode, accumulate, st);
}

ffsplit_status ffsplit_score(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt, const void* X,
                             int64_t T, int32_t mode, int32_t accumulate, float* energy, float* scores, void* stream) {
  ffsplit_status s = check_score_args(ctx, shape, wt, X, T, mode, energy);
  if (s != FFSPLIT_OK) return s;
  if (!aligned16(X)) return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  const ScoreLayout L = score_layout(*shape, T);
  if (kCtrlBytes + L.end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this score call");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool need_w = scores && mode != FFSPLIT_SCORE_ACT_ONLY;
  if ((s = score_prepare(ctx, shape, wt, L, need_w, accumulate != 0, st)) != FFSPLIT_OK) return s;
  return score_batch(ctx, shape, L, X, T, mode, accumulate, energy, scores, st);
}

ffsplit_status ffsplit_score_host(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                  const void* X_host, int64_t T, int32_t mode, int32_t accumulate, float* energy,
                                  float* scores, void* stream) {
  ffsplit_status s = check_score_args(ctx, shape, wt, X_host, T, mode, energy);
  if (s != FFSPLIT_OK) return s;
  // The tokens pass through the workspace in chunks: behind the scoring buffers of a chunk of Tc tokens sits
  // the chunk itself.  Tc is the largest multiple of 128 (at most T) for which both fit.
  const size_t es = elem_size(shape->dtype);
  const size_t row = static_cast<size_t>(shape->d) * es;
  const size_t room = ctx->ws_bytes - kCtrlBytes;
  int64_t Tc = T;
  auto fits = [&](int64_t t) { return score_layout(*shape, t).end + align_up(static_cast<size_t>(t) * row) <= room; };
  if (!fits(Tc)) {
    int64_t lo = 0, hi = (T + 127) / 128;   // in units of 128 tokens: fits(128 lo) holds, fits(128 hi) does not
    if (!fits(128)) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small to stage 128 calibration tokens");
    lo = 1;
    while (hi - lo > 1) {
      const int64_t mid = (lo + hi) / 2;
      if (fits(128 * mid)) lo = mid; else hi = mid;
    }
    Tc = 128 * lo;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ScoreLayout L = score_layout(*shape, Tc);
  char* stage = ctx->ws + kCtrlBytes + L.end;
  const bool need_w = scores && mode != FFSPLIT_SCORE_ACT_ONLY;
  if ((s = score_prepare(ctx, shape, wt, L, need_w, accumulate != 0, st)) != FFSPLIT_OK) return s;
  const char* src = static_cast<const char*>(X_host);
  for (int64_t t0 = 0; t0 < T; t0 += Tc) {
    const int64_t tn = T - t0 < Tc ? T - t0 : Tc;
    cudaError_t e = cudaMemcpyAsync(stage, src + static_cast<size_t>(t0) * row, static_cast<size_t>(tn) * row,
                                    cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(calibration tokens)");
    const bool last = t0 + tn >= T;
    if ((s = score_batch(ctx, shape, L, stage, tn, mode, (accumulate || t0 > 0) ? 1 : 0, energy, last ? scores : nullptr,
                         st)) != FFSPLIT_OK)
      return s;
  }
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_score_finalize(ffsplit_ctx* ctx, const ffsplit_shape* shape, const void* W2, int32_t mode,
                                      float* energy, float* scores, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_shape(ctx, shape)) != FFSPLIT_OK) return s;
  if (!energy || !scores) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (mode < 0 || mode > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown score mode");
  const bool need_w = mode != FFSPLIT_SCORE_ACT_ONLY;
  if (need_w && !W2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "W2 is NULL");
  if (W2 && !aligned16(W2)) return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  const int m = shape->m;
  if (kCtrlBytes + align_up(static_cast<size_t>(m) * 4) > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small (needs 65536 + 4 m bytes)");
  ctx->score_prep.valid = false;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  float* w = reinterpret_cast<float*>(ctx->ws + kCtrlBytes);
  if (need_w && (s = launch_row_energy(ctx, shape->dtype, W2, m, shape->d, w, st)) != FFSPLIT_OK) return s;
  // no partials to add (groups = 0): the energy passes through unchanged and the scores are formed from it
  return launch_score_finalize(ctx, w, 0, m, w, energy, scores, mode, 1, st);
}

ffsplit_status ffsplit_score_activations(ffsplit_ctx* ctx, const ffsplit_shape* shape, const void* H, int64_t T,
                                         const void* W2, int32_t mode, int32_t accumulate, float* energy,
                                         float* scores, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_shape(ctx, shape)) != FFSPLIT_OK) return s;
  if (!H || !energy) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  if (mode < 0 || mode > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown score mode");
  const bool need_w = scores && mode != FFSPLIT_SCORE_ACT_ONLY;
  if (need_w && !W2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "W2 is NULL");
  if (!aligned16(H) || (W2 && !aligned16(W2))) return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  const int d = shape->d, m = shape->m, dt = shape->dtype;
  ctx->score_prep.valid = false;
  const int groups = column_energy_groups(T);
  const size_t w_off = 0, part_off = align_up((size_t)m * 4);
  const size_t end = part_off + align_up((size_t)groups * m * 4);
  if (kCtrlBytes + end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this score call");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = ctx->ws + kCtrlBytes;
  float* w = reinterpret_cast<float*>(base + w_off);
  float* partial = reinterpret_cast<float*>(base + part_off);
  if (need_w && (s = launch_row_energy(ctx, dt, W2, m, d, w, st)) != FFSPLIT_OK) return s;
  if ((s = launch_column_energy(ctx, dt, H, m, T, m, partial, mode == FFSPLIT_SCORE_SUM_NORM, st)) != FFSPLIT_OK) return s;
  return launch_score_finalize(ctx, partial, groups, m, w, energy, scores, mode, accumulate, st);
}

ffsplit_status ffsplit_select(ffsplit_ctx* ctx, const float* scores, int32_t m, int32_t k, int32_t* heavy_idx,
                              int32_t* light_idx, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if (!scores) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "scores is NULL");
  if (m < 1 || k < 0 || k > m) return fail(ctx, FFSPLIT_ERR_SHAPE, "need m >= 1 and 0 <= k <= m");
  if (k > 0 && !heavy_idx) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "heavy_idx is NULL");
  return launch_select(ctx, scores, m, k, heavy_idx, light_idx, static_cast<cudaStream_t>(stream));
}

ffsplit_status ffsplit_pack_size(const ffsplit_shape* shape, int32_t k, int32_t r, size_t* padded_bytes,
                                 size_t* logical_bytes) {
  ffsplit_status s = check_shape(nullptr, shape);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_split(nullptr, shape, k, r)) != FFSPLIT_OK) return s;
  BlobHeader h;
  layout_blob(*shape, make_dims(*shape, k, r), &h);
  if (padded_bytes) *padded_bytes = h.total_bytes;
  if (logical_bytes) *logical_bytes = h.logical_bytes;
  return FFSPLIT_OK;
}

static ffsplit_status pack_into(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                const int32_t* heavy_idx, int32_t k, const ffsplit_factors* f, const SplitDims& D,
                                const BlobHeader& h, void* blob, cudaStream_t st);

ffsplit_status ffsplit_pack(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                            const int32_t* heavy_idx, int32_t k, const ffsplit_factors* f, void* blob,
                            size_t blob_bytes, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_shape(ctx, shape)) != FFSPLIT_OK) return s;
  const int r = f ? f->r : 0;
  if ((s = check_split(ctx, shape, k, r)) != FFSPLIT_OK) return s;
  if (!wt || !wt->W1 || !wt->W2 || !blob) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (k > 0 && !heavy_idx) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "heavy_idx is NULL");
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  if (gated && (!wt->W1u || wt->b1)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "SwiGLU needs W1u and no b1");
  if (r > 0 && (!f->A1 || !f->B1 || !f->A2 || !f->B2 || (gated && (!f->A1u || !f->B1u))))
    return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL factor");
  if (!aligned16(wt->W1) || !aligned16(wt->W2) || (gated && !aligned16(wt->W1u)))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  if (reinterpret_cast<uintptr_t>(blob) % kAlign != 0) return fail(ctx, FFSPLIT_ERR_ALIGN, "blob must be 256-byte aligned");
  const SplitDims D = make_dims(*shape, k, r);
  BlobHeader h;
  layout_blob(*shape, D, &h);
  if (blob_bytes < h.total_bytes) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "blob buffer too small (ffsplit_pack_size)");
  return pack_into(ctx, shape, wt, heavy_idx, k, f, D, h, blob, static_cast<cudaStream_t>(stream));
}

// Fills a blob whose layout `h` has been worked out.  heavy_idx == nullptr with k == m stands for the
// identity 0 .. m-1 (the dense FFN): the heavy slices are then the whole matrices.
static ffsplit_status pack_into(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                const int32_t* heavy_idx, int32_t k, const ffsplit_factors* f, const SplitDims& D,
                                const BlobHeader& h, void* blob, cudaStream_t st) {
  ffsplit_status s;
  const int r = f ? f->r : 0;
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  char* b = static_cast<char*>(blob);
  const int d = shape->d, m = shape->m, dt = shape->dtype;
  const size_t es = elem_size(dt);
  // heavy slices: U1^T = (U[:, h2])^T, V1 = V[h2, :] -- plain copies of the inputs; all of the
  // gathers, transposes and bias conversions of the layer run as one batched launch
  prep_begin(ctx);
  if (heavy_idx || k == 0) {
    if ((s = launch_gather_cols_t(ctx, dt, wt->W1, m, d, heavy_idx, k, m, b + h.off[SEC_U1T], d, D.k_pad, st)) != FFSPLIT_OK)
      return s;
    if (gated &&
        (s = launch_gather_cols_t(ctx, dt, wt->W1u, m, d, heavy_idx, k, m, b + h.off[SEC_U1UT], d, D.k_pad, st)) != FFSPLIT_OK)
      return s;
  } else {
    // all columns, in order: U1^T is the transpose of the whole matrix
    if ((s = launch_transpose(ctx, dt, wt->W1, m, d, m, b + h.off[SEC_U1T], d, d, D.k_pad, nullptr, d, st)) != FFSPLIT_OK)
      return s;
    if (gated &&
        (s = launch_transpose(ctx, dt, wt->W1u, m, d, m, b + h.off[SEC_U1UT], d, d, D.k_pad, nullptr, d, st)) != FFSPLIT_OK)
      return s;
  }
  if ((s = launch_transpose(ctx, dt, wt->W2, d, k, d, b + h.off[SEC_V1B2T], D.kp_rp, D.k_pad, d, heavy_idx, m, st)) !=
      FFSPLIT_OK)
    return s;
  if (D.r_pad > 0) {
    const int ml = D.ml;
    if ((s = launch_transpose(ctx, dt, f->A1, r, d, r, b + h.off[SEC_A1T], d, d, D.r_pad, nullptr, d, st)) != FFSPLIT_OK) return s;
    if ((s = launch_transpose(ctx, dt, f->B1, ml, r, ml, b + h.off[SEC_B1T], D.r_pad, D.r_pad, D.ml_pad, nullptr, r, st)) != FFSPLIT_OK) return s;
    if (gated) {
      if ((s = launch_transpose(ctx, dt, f->A1u, r, d, r, b + h.off[SEC_A1UT], d, d, D.r_pad, nullptr, d, st)) != FFSPLIT_OK) return s;
      if ((s = launch_transpose(ctx, dt, f->B1u, ml, r, ml, b + h.off[SEC_B1UT], D.r_pad, D.r_pad, D.ml_pad, nullptr, r, st)) != FFSPLIT_OK) return s;
    }
    if ((s = launch_transpose(ctx, dt, f->A2, r, ml, r, b + h.off[SEC_A2T], D.ml_pad, D.ml_pad, D.r_pad, nullptr, ml, st)) != FFSPLIT_OK) return s;
    if ((s = launch_transpose(ctx, dt, f->B2, d, r, d, b + h.off[SEC_V1B2T] + (size_t)D.k_pad * es, D.kp_rp, D.r_pad, d,
                              nullptr, r, st)) != FFSPLIT_OK)
      return s;
  }
  if ((s = launch_pack_bias(ctx, dt, wt->b1, wt->b2, heavy_idx, m, k, d, reinterpret_cast<float*>(b + h.off[SEC_B1H]),
                            D.k_pad, reinterpret_cast<float*>(b + h.off[SEC_B1L]), D.ml_pad,
                            reinterpret_cast<float*>(b + h.off[SEC_B2]), st)) != FFSPLIT_OK)
    return s;
  if ((s = prep_flush(ctx, dt, st)) != FFSPLIT_OK) return s;
  ffsplit_ctx::BlobEntry& ent = ctx->blobs[blob];   // replaces whatever was registered at this address
  ent.h = h;
  ent.bytes = h.total_bytes;
  ent.hash = header_hash_host(&h);
  // the copy below reads this entry, which outlives the call
  cudaError_t e = cudaMemcpyAsync(blob, &ent.h, sizeof(h), cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(blob header)");
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_blob_open(ffsplit_ctx* ctx, const void* blob, size_t blob_bytes, void* stream) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  if (!blob) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "blob is NULL");
  if (reinterpret_cast<uintptr_t>(blob) % kAlign != 0) return fail(ctx, FFSPLIT_ERR_ALIGN, "blob must be 256-byte aligned");
  if (blob_bytes < sizeof(BlobHeader)) return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "blob_bytes is smaller than a header");
  ctx->blobs.erase(blob);   // whatever was registered at this address is stale from here on
  BlobHeader h;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(&h, blob, sizeof(h), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(blob header)");
  if (!header_valid(h, blob_bytes)) return fail(ctx, FFSPLIT_ERR_BAD_BLOB, "not a packed layer (bad header, or larger than blob_bytes)");
  ffsplit_ctx::BlobEntry& ent = ctx->blobs[blob];
  ent.h = h;
  ent.bytes = blob_bytes;
  ent.hash = header_hash_host(&h);
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_blob_close(ffsplit_ctx* ctx, const void* blob) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  if (ctx->blobs.erase(blob) == 0) return fail(ctx, FFSPLIT_ERR_BAD_BLOB, "blob not known to this context");
  ctx->tmaps.clear();   // tensor maps are keyed by address too
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_blob_section(ffsplit_ctx* ctx, const void* blob, int32_t which, size_t* offset, int64_t* rows,
                                    int64_t* cols, int64_t* ld) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  if (which < 0 || which >= kNumSections) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown section");
  const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blob, &s);
  if (!ent) return s;
  const BlobHeader* h = &ent->h;
  const SplitDims D = dims_of(*h);
  int64_t R = 0, C = 0, LD = 0;
  switch (which) {
    case SEC_U1T: R = D.k_pad; C = h->d; LD = h->d; break;
    case SEC_U1UT: R = D.n_in == 2 ? D.k_pad : 0; C = h->d; LD = h->d; break;
    case SEC_A1T: R = D.r_pad; C = h->d; LD = h->d; break;
    case SEC_A1UT: R = D.n_in == 2 ? D.r_pad : 0; C = h->d; LD = h->d; break;
    case SEC_B1T: R = D.ml_pad; C = D.r_pad; LD = D.r_pad; break;
    case SEC_B1UT: R = D.n_in == 2 ? D.ml_pad : 0; C = D.r_pad; LD = D.r_pad; break;
    case SEC_A2T: R = D.r_pad; C = D.ml_pad; LD = D.ml_pad; break;
    case SEC_V1B2T: R = h->d; C = D.kp_rp; LD = D.kp_rp; break;
    case SEC_B1H: R = 1; C = D.k_pad; LD = D.k_pad; break;
    case SEC_B1L: R = 1; C = D.ml_pad; LD = D.ml_pad; break;
    case SEC_B2: R = 1; C = h->d; LD = h->d; break;
  }
  if (offset) *offset = h->off[which];
  if (rows) *rows = R;
  if (cols) *cols = C;
  if (ld) *ld = LD;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_forward(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T, void* Y, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if (!blob || !X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  if (!aligned16(X) || !aligned16(Y)) return fail(ctx, FFSPLIT_ERR_ALIGN, "X and Y must be 16-byte aligned");
  const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blob, &s);
  if (!ent) return s;
  return run_forward(ctx, ent->h, static_cast<const char*>(blob), X, T, Y, static_cast<cudaStream_t>(stream), ent->hash);
}

ffsplit_status ffsplit_forward_dense(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                     const void* X, int64_t T, void* Y, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if ((s = check_shape(ctx, shape)) != FFSPLIT_OK) return s;
  if (!wt || !wt->W1 || !wt->W2 || !X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  if (gated && (!wt->W1u || wt->b1)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "SwiGLU needs W1u and no b1");
  if (!aligned16(X) || !aligned16(Y) || !aligned16(wt->W1) || !aligned16(wt->W2) || (gated && !aligned16(wt->W1u)))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "tensors must be 16-byte aligned");
  // the dense FFN is the split with every neuron heavy: its packed form goes behind the forward buffers
  const SplitDims D = make_dims(*shape, shape->m, 0);
  BlobHeader h;
  layout_blob(*shape, D, &h);
  const FwdLayout L = fwd_layout(D, shape->d, shape->dtype, shape->act, T);
  const size_t blob_off = align_up(kCtrlBytes + L.end);
  if (blob_off + h.total_bytes > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL,
                "workspace too small for ffsplit_forward_dense: ffsplit_workspace_size(T, 0, k = m, r = 0) + "
                "256 + the padded size of ffsplit_pack_size(k = m, r = 0)");
  char* blob = ctx->ws + blob_off;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if ((s = pack_into(ctx, shape, wt, nullptr, shape->m, nullptr, D, h, blob, st)) != FFSPLIT_OK) return s;
  return run_forward(ctx, h, blob, X, T, Y, st, 0);
}

ffsplit_status ffsplit_forward_host(ffsplit_ctx* ctx, const void* blob, const void* X_host, int64_t T, void* Y_host,
                                    void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if (!blob || !X_host || !Y_host) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (T < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "T must be >= 1");
  const ffsplit_ctx::BlobEntry* ent = find_blob(ctx, blob, &s);
  if (!ent) return s;
  const BlobHeader* h = &ent->h;
  const SplitDims D = dims_of(*h);
  const size_t es = elem_size(h->dtype);
  const FwdLayout L = fwd_layout(D, h->d, h->dtype, h->act, T);
  if (kCtrlBytes + L.end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this forward (ffsplit_workspace_size)");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = ctx->ws + kCtrlBytes;
  const size_t bytes = (size_t)T * h->d * es;
  cudaError_t e = cudaMemcpyAsync(base + L.xs, X_host, bytes, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(X)");
  if ((s = run_forward(ctx, *h, static_cast<const char*>(blob), base + L.xs, T, base + L.ys, st, ent->hash)) != FFSPLIT_OK) return s;
  e = cudaMemcpyAsync(Y_host, base + L.ys, bytes, cudaMemcpyDeviceToHost, st);
  return check_cuda(ctx, e, "cudaMemcpyAsync(Y)");
}

ffsplit_status ffsplit_forward_stack(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers, const void* X,
                                     int64_t T, void* Y, void* stream) {
  return forward_stack_impl(ctx, blobs, n_layers, X, T, Y, static_cast<cudaStream_t>(stream), false);
}

ffsplit_status ffsplit_forward_stack_host(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers,
                                          const void* X_host, int64_t T, void* Y_host, void* stream) {
  return forward_stack_impl(ctx, blobs, n_layers, X_host, T, Y_host, static_cast<cudaStream_t>(stream), true);
}

ffsplit_status ffsplit_stack_workspace_size(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers, int64_t T,
                                            size_t* bytes) {
  ffsplit_status s = check_ctx(ctx, false);
  if (s != FFSPLIT_OK) return s;
  if (!blobs || n_layers < 1 || !bytes || T < 1) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "bad argument");
  StackLayout SL;
  if ((s = stack_layout(ctx, blobs, n_layers, T, &SL)) != FFSPLIT_OK) return s;
  *bytes = kCtrlBytes + SL.end;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_debug_wait_timeout(ffsplit_ctx* ctx, int64_t limit_cycles, void* stream) {
  ffsplit_status s = check_ctx(ctx, true);
  if (s != FFSPLIT_OK) return s;
  if (limit_cycles < 1 || limit_cycles > 100000000)
    return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "limit_cycles must be in [1, 1e8] (well under a tenth of a second)");
  return launch_wait_timeout_probe(ctx, limit_cycles, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
