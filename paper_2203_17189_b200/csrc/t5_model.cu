// Host side of the library: configuration checks, parameter manifest, workspace
// plan, the forward/backward launch schedule of the T5.1.1 step, and the C ABI.
#include "../../include/t5_b200.h"
#include "common.cuh"

#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

namespace {

struct Tensor {
  std::string name;
  int64_t offset;
  int32_t shape[4];
  int32_t ndim;
  int64_t numel() const { int64_t n = 1; for (int i = 0; i < ndim; ++i) n *= shape[i]; return n; }
};

struct AttnP { int64_t norm, q, k, v, o; };
struct FfnP { int64_t norm, wi0, wi1, wo; };
struct EncLayerP { AttnP attn; FfnP ffn; };
struct DecLayerP { AttnP self, cross; FfnP ffn; };

// per-sub-layer saved activations
struct AttnWs { float* x; void* y; float* rstd; void* q; void* kv; void* ctx; float* ctx32; float* lse; };
struct FfnWs { float* x; void* y; float* rstd; void* h; void* hg; };

struct Workspace {
  std::vector<AttnWs> enc_attn, dec_self, dec_cross;
  std::vector<FfnWs> enc_ffn, dec_ffn;
  float *enc_x_final, *enc_rstd_f, *dec_x_final, *dec_rstd_f;
  void *enc_out, *dec_z, *logits;
  float* lse_tok;
  int *enc_code, *dec_code, *dec_in, *W_int, *status, *sk_flags;
  float* W_f;
  double* sums;
  float *bias_enc, *bias_dec, *dbias_enc, *dbias_dec, *norm_partial, *delta;
  float *dX_enc, *dX_dec, *dY32;
  void *dXb_enc, *dXb_dec, *dh, *dhg, *dy, *dctx, *dqkv, *dkv;
  void* ds_scratch;      // bf16 dS^T of one attention call (one-pass attention backward)
  int64_t ds_bytes;
  int64_t bytes;
};

char g_create_error[256] = "";
constexpr int kSkSlices = 2048, kSkSliceInts = 160;

}  // namespace

struct t5_handle {
  t5_config cfg;
  std::vector<Tensor> tensors;
  std::vector<std::pair<int64_t, int64_t>> gaps;   // [begin, end) element ranges not covered by tensors
  int64_t n_params;
  int64_t token_embed, enc_relbias, dec_relbias, enc_final_norm, dec_final_norm;
  std::vector<EncLayerP> enc;
  std::vector<DecLayerP> dec;
  BucketSpec spec_enc, spec_dec;
  std::string err;
  // opt-in per-kernel-family timing (CUDA events around each launch) and launch counting
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_events;      // pairs: start, stop
  std::vector<int> prof_cat;                 // category of each pair in use
  double prof_flops[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int64_t prof_launches[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int64_t launches_last_call = 0;
};

namespace {

int fail(t5_handle* h, int code, const char* fmt, ...) __attribute__((format(printf, 3, 4)));
int fail(t5_handle* h, int code, const char* fmt, ...) {
  char buf[256];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  if (h) h->err = buf; else snprintf(g_create_error, sizeof g_create_error, "%s", buf);
  return code;
}

inline size_t esize(const t5_handle* h) { return h->cfg.dtype == DT_F32 ? 4 : 2; }
inline const void* pptr(const t5_handle* h, const void* params, int64_t off) {
  return (const char*)params + off * (int64_t)esize(h);
}
inline void* eoff(const t5_handle* h, void* p, int64_t elems) { return (char*)p + elems * (int64_t)esize(h); }
inline const void* eoff(const t5_handle* h, const void* p, int64_t elems) {
  return (const char*)p + elems * (int64_t)esize(h);
}

int64_t add_tensor(t5_handle* h, const std::string& name, std::initializer_list<int32_t> shape) {
  Tensor t;
  t.name = name;
  t.ndim = (int32_t)shape.size();
  int i = 0;
  for (int32_t s : shape) t.shape[i++] = s;
  for (; i < 4; ++i) t.shape[i] = 1;
  int64_t off = (h->n_params + 63) / 64 * 64;      // 128-byte alignment in bf16
  if (off != h->n_params) h->gaps.push_back({h->n_params, off});
  t.offset = off;
  h->n_params = off + t.numel();
  h->tensors.push_back(t);
  return off;
}

void build_manifest(t5_handle* h) {
  const t5_config& c = h->cfg;
  int d = c.d_model, I = c.n_heads * c.d_kv, F = c.d_ff;
  h->n_params = 0;
  h->token_embed = add_tensor(h, "token_embed", {c.vocab, d});
  auto attn = [&](const std::string& p) {
    AttnP a;
    a.norm = add_tensor(h, p + ".norm", {d});
    a.q = add_tensor(h, p + ".q", {I, d});     // q, k, v are contiguous: one [3I, d] matrix
    a.k = add_tensor(h, p + ".k", {I, d});
    a.v = add_tensor(h, p + ".v", {I, d});
    a.o = add_tensor(h, p + ".o", {d, I});
    return a;
  };
  auto ffn = [&](const std::string& p) {
    FfnP f;
    f.norm = add_tensor(h, p + ".norm", {d});
    f.wi0 = add_tensor(h, p + ".wi0", {F, d});  // wi0, wi1 contiguous: one [2F, d] matrix
    f.wi1 = add_tensor(h, p + ".wi1", {F, d});
    f.wo = add_tensor(h, p + ".wo", {d, F});
    return f;
  };
  if (c.arch == 0) {
    h->enc_relbias = add_tensor(h, "enc.relbias", {c.rel_buckets, c.n_heads});
    for (int l = 0; l < c.n_enc_layers; ++l) {
      EncLayerP e;
      std::string p = "enc.L" + std::to_string(l);
      e.attn = attn(p + ".attn");
      e.ffn = ffn(p + ".ffn");
      h->enc.push_back(e);
    }
    h->enc_final_norm = add_tensor(h, "enc.final_norm", {d});
  }
  h->dec_relbias = add_tensor(h, "dec.relbias", {c.rel_buckets, c.n_heads});
  for (int l = 0; l < c.n_dec_layers; ++l) {
    DecLayerP e;
    std::string p = "dec.L" + std::to_string(l);
    e.self = attn(p + ".self");
    if (c.arch == 0) e.cross = attn(p + ".cross");
    e.ffn = ffn(p + ".ffn");
    h->dec.push_back(e);
  }
  h->dec_final_norm = add_tensor(h, "dec.final_norm", {d});
  int64_t end = (h->n_params + 63) / 64 * 64;
  if (end != h->n_params) h->gaps.push_back({h->n_params, end});
  h->n_params = end;
}

// Lays the workspace out for a batch of (B, Te, Td); base may be NULL (sizing only).
void plan_workspace(const t5_handle* h, int B, int Te, int Td, char* base, Workspace* w) {
  const t5_config& c = h->cfg;
  int64_t cur = 0;
  auto take = [&](int64_t bytes) -> void* {
    int64_t at = cur;
    cur += (bytes + 255) / 256 * 256;
    return base ? (void*)(base + at) : nullptr;
  };
  int64_t es = (int64_t)esize(h);
  int64_t d = c.d_model, I = (int64_t)c.n_heads * c.d_kv, F = c.d_ff, H = c.n_heads, V = c.vocab;
  bool encdec = c.arch == 0;
  if (!encdec) Te = 0;
  int64_t Ne = (int64_t)B * Te, Nd = (int64_t)B * Td, Nmax = Ne > Nd ? Ne : Nd;
  int Tmax = Te > Td ? Te : Td;
  // Activation policy 1: the normed activations y and the gated product hg are not kept per sub-layer; the
  // forward pass writes them into one shared buffer each (the next GEMM consumes them at once) and the backward
  // pass recomputes them from the saved x (and rstd) / pre-activations h right before the weight-gradient GEMMs.
  const bool recompute = c.recompute == 1;
  void* shared_y = nullptr;      // taken below, behind the status word
  void* shared_hg = nullptr;
  auto attn_ws = [&](int64_t Nq, int64_t Nk, int Tq, bool cross) {
    AttnWs a;
    a.x = (float*)take(Nq * d * 4);
    a.y = recompute ? shared_y : take(Nq * d * es);
    a.rstd = (float*)take(Nq * 4);
    a.q = take(Nq * (cross ? I : 3 * I) * es);
    a.kv = cross ? take(Nk * 2 * I * es) : nullptr;
    a.ctx = take(Nq * I * es);
    a.ctx32 = es == 2 ? (float*)take(Nq * I * 4) : nullptr;   // unrounded copy for the backward's delta
    a.lse = (float*)take((int64_t)B * H * Tq * 4);
    return a;
  };
  auto ffn_ws = [&](int64_t N) {
    FfnWs f;
    f.x = (float*)take(N * d * 4);
    f.y = recompute ? shared_y : take(N * d * es);
    f.rstd = (float*)take(N * 4);
    f.h = take(N * 2 * F * es);
    f.hg = recompute ? shared_hg : take(N * F * es);
    return f;
  };
  w->status = (int*)take(4);          // first, so its address does not depend on the batch shape
  w->sk_flags = (int*)take((int64_t)kSkSlices * kSkSliceInts * 4);   // per-GEMM flag slices of the stream-K tails
  if (recompute) {
    shared_y = take(Nmax * d * es);
    shared_hg = take(Nmax * F * es);
  }
  w->enc_attn.clear(); w->enc_ffn.clear(); w->dec_self.clear(); w->dec_cross.clear(); w->dec_ffn.clear();
  if (encdec) {
    for (int l = 0; l < c.n_enc_layers; ++l) {
      w->enc_attn.push_back(attn_ws(Ne, Ne, Te, false));
      w->enc_ffn.push_back(ffn_ws(Ne));
    }
  }
  w->enc_x_final = (float*)take(Ne * d * 4);
  w->enc_rstd_f = (float*)take(Ne * 4);
  w->enc_out = take(Ne * d * es);
  for (int l = 0; l < c.n_dec_layers; ++l) {
    w->dec_self.push_back(attn_ws(Nd, Nd, Td, false));
    if (encdec) w->dec_cross.push_back(attn_ws(Nd, Ne, Td, true));
    w->dec_ffn.push_back(ffn_ws(Nd));
  }
  w->dec_x_final = (float*)take(Nd * d * 4);
  w->dec_rstd_f = (float*)take(Nd * 4);
  w->dec_z = take(Nd * d * es);
  w->logits = take(Nd * V * es);
  w->lse_tok = (float*)take(Nd * 4);
  w->enc_code = (int*)take(Ne * 4);
  w->dec_code = (int*)take(Nd * 4);
  w->dec_in = (int*)take(Nd * 4);
  w->W_int = (int*)take(4);
  w->W_f = (float*)take(4);
  w->sums = (double*)take(16);
  int64_t span_e = Te > 0 ? 2 * Te - 1 : 0, span_d = 2 * Td - 1;
  w->bias_enc = (float*)take(H * span_e * 4);
  w->bias_dec = (float*)take(H * span_d * 4);
  w->dbias_enc = (float*)take(H * span_e * 4);
  w->dbias_dec = (float*)take(H * span_d * 4);
  w->norm_partial = (float*)take((int64_t)rmsnorm_bwd_parts((int)Nmax) * d * 4);
  w->delta = (float*)take((int64_t)B * H * Tmax * 4);
  w->dX_enc = (float*)take(Ne * d * 4);
  w->dX_dec = (float*)take(Nd * d * 4);
  w->dY32 = (float*)take(Ne * d * 4);
  w->dXb_enc = take(Ne * d * es);
  w->dXb_dec = take(Nd * d * es);
  w->dh = take(Nmax * 2 * F * es);
  w->dhg = take(Nmax * F * es);
  w->dy = take(Nmax * d * es);
  w->dctx = take(Nmax * I * es);
  w->dqkv = take(Nmax * 3 * I * es);
  w->dkv = take(Ne * 2 * I * es);
  w->ds_scratch = nullptr;
  w->ds_bytes = 0;
  if (c.dtype == DT_BF16 && (c.d_kv == 64 || c.d_kv == 128) && !(c.flags & (2 | (1 << 17)))) {
    int64_t need = attn_tc_ds_scratch_bytes(B, (int)H, Td, Td);
    if (encdec) {
      need = std::max(need, attn_tc_ds_scratch_bytes(B, (int)H, Te, Te));
      need = std::max(need, attn_tc_ds_scratch_bytes(B, (int)H, Td, Te));
    }
    w->ds_scratch = take(need);
    w->ds_bytes = need;
  }
  w->bytes = cur;
}

struct Ctx {
  t5_handle* h;
  const void* params;
  float* grads;
  cudaStream_t st;
  Workspace* w;
  int B, Te, Td;
  cudaError_t err;
  const char* where;
  int64_t launches;
  int sk_next;        // next unused flag slice
  int packed;         // the batch carries segment ids
};

enum { CAT_GEMM = 0, CAT_ATTN_FWD, CAT_ATTN_BWD, CAT_NORM, CAT_GEGLU, CAT_XENT, CAT_EMBED, CAT_MISC };

// Records a start/stop event pair around the launches made while it is alive (profiling mode only).
struct ProfScope {
  Ctx& cx;
  int idx = -1;
  ProfScope(Ctx& c, int cat, double flops, int n_kernels) : cx(c) {
    cx.launches += n_kernels;
    t5_handle* h = cx.h;
    if (!h->prof_on || cx.err != cudaSuccess) return;
    idx = (int)h->prof_cat.size();
    while ((int)h->prof_events.size() < 2 * (idx + 1)) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { idx = -1; return; }
      h->prof_events.push_back(e);
    }
    h->prof_cat.push_back(cat);
    h->prof_flops[cat] += flops;
    h->prof_launches[cat] += n_kernels;
    cudaEventRecord(h->prof_events[2 * idx], cx.st);
  }
  ~ProfScope() {
    if (idx >= 0) cudaEventRecord(cx.h->prof_events[2 * idx + 1], cx.st);
  }
};

// CK(call, what): plain runtime call.  CKL(cat, n, call, what): a launch of n kernels of family cat.
#define CK(call, what)                                            \
  do {                                                            \
    if (cx.err == cudaSuccess) {                                  \
      cudaError_t e_ = (call);                                    \
      if (e_ != cudaSuccess) { cx.err = e_; cx.where = what; }    \
    }                                                             \
  } while (0)
#define CKL(cat, n, call, what)                                   \
  do {                                                            \
    if (cx.err == cudaSuccess) {                                  \
      ProfScope ps_(cx, cat, 0.0, n);                             \
      cudaError_t e_ = (call);                                    \
      if (e_ != cudaSuccess) { cx.err = e_; cx.where = what; }    \
    }                                                             \
  } while (0)

void gemm(Ctx& cx, const GemmArgs& g0, const char* what) {
  int dt = cx.h->cfg.dtype;
  if (cx.err != cudaSuccess) return;
  GemmArgs g = g0;
  g.pair = ((cx.h->cfg.flags >> 2) & 1) ^ 1;      // CTA pairs unless flag bit 2 says otherwise
  if (g.out_f32 && cx.sk_next < kSkSlices) g.sk_flags = cx.w->sk_flags + (cx.sk_next++) * kSkSliceInts;
  ProfScope ps(cx, CAT_GEMM, 2.0 * g.M * g.N * g.K, 1);
  if (g.epi != 0 || (dt == DT_BF16 && !(cx.h->cfg.flags & 1) && gemm_tc_supported(g))) {
    CK(gemm_tc(g, cx.w->status, cx.st), what);
  } else {
    CK(gemm_simt(dt, g, cx.st), what);
  }
}

// Numerics debugging aid: in float32 mode, flag bit `bit` rounds one family of intermediates to
// bfloat16 precision in place, to attribute the bfloat16 mode's error to the buffer that causes it.
enum { RB_Y = 4, RB_QKV, RB_CTX, RB_H, RB_HG, RB_LOGITS, RB_DLOGITS, RB_DXB, RB_DY, RB_DCTX, RB_DQKV, RB_DHG, RB_DH };
void dbg_round(Ctx& cx, void* p, int64_t n, int bit) {
  if (cx.h->cfg.dtype != DT_F32 || !((cx.h->cfg.flags >> bit) & 1)) return;
  CK(launch_round_bf16((float*)p, n, cx.st), "debug rounding");
}

// Y[M,N] = alpha X[M,K] W[N,K]^T (+ resid)
void proj_fwd(Ctx& cx, const void* X, int ldx, int64_t w_off, int M, int N, int K, void* Y, int ldy, float alpha,
              const float* resid, const char* what) {
  GemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.alpha = alpha;
  g.A = X; g.lda = ldx; g.a_kmajor = 1;
  g.B = pptr(cx.h, cx.params, w_off); g.ldb = K; g.b_kmajor = 1;
  g.D = Y; g.ldd = ldy; g.out_f32 = resid != nullptr; g.resid = resid; g.ldr = ldy; g.accumulate = 0;
  gemm(cx, g, what);
}
// dX[M,K] = alpha dY[M,N] W[N,K]   (operand dtype out, or float32 with optional accumulate)
void proj_dgrad(Ctx& cx, const void* dY, int lddy, int64_t w_off, int M, int N, int K, void* dX, int lddx,
                float alpha, int out_f32, int accumulate, const char* what) {
  GemmArgs g{};
  g.M = M; g.N = K; g.K = N; g.alpha = alpha;
  g.A = dY; g.lda = lddy; g.a_kmajor = 1;
  g.B = pptr(cx.h, cx.params, w_off); g.ldb = K; g.b_kmajor = 0;
  g.D = dX; g.ldd = lddx; g.out_f32 = out_f32; g.accumulate = accumulate;
  gemm(cx, g, what);
}
// dW[N,K] = alpha dY[M,N]^T X[M,K]   (float32, overwrite)
void proj_wgrad(Ctx& cx, const void* dY, int lddy, const void* X, int ldx, int64_t w_off, int M, int N, int K,
                float alpha, const char* what) {
  GemmArgs g{};
  g.M = N; g.N = K; g.K = M; g.alpha = alpha;
  g.A = dY; g.lda = lddy; g.a_kmajor = 0;
  g.B = X; g.ldb = ldx; g.b_kmajor = 0;
  g.D = cx.grads + w_off; g.ldd = K; g.out_f32 = 1; g.accumulate = 0;
  gemm(cx, g, what);
}

// |key - query| from which the bucket no longer changes (the top bucket of that direction)
int saturation_distance(const BucketSpec& s) { return s.n_thr > 0 ? s.thr[s.n_thr - 1] : s.me; }

struct AttnGeom {
  int far;           // distance from which the relative-position bucket is saturated (0: no bias)
  int Tq, Tk;
  int64_t Nq, Nk;
  const int *code_q, *code_k;
  int causal;
  const float* bias;
  float* dbias;
};

void attn_args(Ctx& cx, const AttnWs& a, const AttnGeom& gm, bool cross, AttnArgs* out) {
  const t5_config& c = cx.h->cfg;
  int I = c.n_heads * c.d_kv;
  AttnArgs& t = *out;
  memset(&t, 0, sizeof t);
  if (cross) {
    t.Q = a.q; t.ldq = I;
    t.K = a.kv; t.V = eoff(cx.h, a.kv, I); t.ldk = t.ldv = 2 * I;
  } else {
    t.Q = a.q; t.K = eoff(cx.h, a.q, I); t.V = eoff(cx.h, a.q, 2 * I); t.ldq = t.ldk = t.ldv = 3 * I;
  }
  t.O = a.ctx; t.ldo = I; t.lse = a.lse; t.O32 = a.ctx32; t.ldo32 = I;
  t.B = cx.B; t.H = c.n_heads; t.Tq = gm.Tq; t.Tk = gm.Tk; t.dk = c.d_kv;
  t.code_q = gm.code_q; t.code_k = gm.code_k; t.causal = gm.causal;
  t.bias_delta = gm.bias; t.scale = c.attn_scale;
  t.packed = cx.packed;
}

// x_out = x + Attn(RMS(x))
void attn_forward(Ctx& cx, const AttnP& p, const AttnWs& a, float* x_out, const AttnGeom& gm, const void* kv_src) {
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, I = c.n_heads * c.d_kv, dt = c.dtype;
  bool cross = kv_src != nullptr;
  CKL(CAT_NORM, 1, launch_rmsnorm_fwd(dt, a.x, pptr(cx.h, cx.params, p.norm), a.y, a.rstd, (int)gm.Nq, d, c.rms_eps, cx.st),
     "rmsnorm_fwd");
  dbg_round(cx, a.y, gm.Nq * d, RB_Y);
  if (!cross) {
    proj_fwd(cx, a.y, d, p.q, (int)gm.Nq, 3 * I, d, a.q, 3 * I, 1.f, nullptr, "qkv proj");
    dbg_round(cx, a.q, gm.Nq * 3 * I, RB_QKV);
  } else {
    proj_fwd(cx, a.y, d, p.q, (int)gm.Nq, I, d, a.q, I, 1.f, nullptr, "q proj");
    proj_fwd(cx, kv_src, d, p.k, (int)gm.Nk, 2 * I, d, a.kv, 2 * I, 1.f, nullptr, "kv proj");
    dbg_round(cx, a.q, gm.Nq * I, RB_QKV);
    dbg_round(cx, a.kv, gm.Nk * 2 * I, RB_QKV);
  }
  AttnArgs t;
  attn_args(cx, a, gm, cross, &t);
  if (dt == DT_BF16 && !(c.flags & 2) && attn_tc_supported(t))
    CKL(CAT_ATTN_FWD, 1, attn_fwd_tc(t, cx.w->status, cx.st), "attn_fwd (tcgen05)");
  else
    CKL(CAT_ATTN_FWD, 1, attn_fwd_simt(dt, t, cx.st), "attn_fwd");
  dbg_round(cx, a.ctx, gm.Nq * I, RB_CTX);
  proj_fwd(cx, a.ctx, I, p.o, (int)gm.Nq, d, I, x_out, d, 1.f, a.x, "o proj");
}

// dX (in place) <- grad wrt sub-layer input; also refreshes dXb.  dY32: encoder-output gradient (cross only).
void attn_backward(Ctx& cx, const AttnP& p, const AttnWs& a, float* dX, void* dXb, const AttnGeom& gm,
                   const void* kv_src, float* dY32, int dY_accumulate) {
  const t5_config& c = cx.h->cfg;
  Workspace& w = *cx.w;
  int d = c.d_model, I = c.n_heads * c.d_kv, dt = c.dtype;
  bool cross = kv_src != nullptr;
  int Nq = (int)gm.Nq, Nk = (int)gm.Nk;
  proj_wgrad(cx, dXb, d, a.ctx, I, p.o, Nq, d, I, 1.f, "wgrad o");
  proj_dgrad(cx, dXb, d, p.o, Nq, d, I, w.dctx, I, 1.f, 0, 0, "dgrad o");
  dbg_round(cx, w.dctx, (int64_t)Nq * I, RB_DCTX);
  AttnArgs t;
  attn_args(cx, a, gm, cross, &t);
  t.dO = w.dctx; t.lddo = I; t.delta = w.delta; t.dbias_delta = gm.dbias; t.bias_far = gm.far;
  t.ds_scratch = w.ds_scratch; t.ds_bytes = w.ds_bytes;
  if (cross) {
    t.dQ = w.dqkv; t.lddq = I;
    t.dK = w.dkv; t.dV = eoff(cx.h, w.dkv, I); t.lddk = t.lddv = 2 * I;
  } else {
    t.dQ = w.dqkv; t.dK = eoff(cx.h, w.dqkv, I); t.dV = eoff(cx.h, w.dqkv, 2 * I);
    t.lddq = t.lddk = t.lddv = 3 * I;
  }
  if (dt == DT_BF16 && !(c.flags & 2) && attn_tc_supported(t))
    CKL(CAT_ATTN_BWD, 3, attn_bwd_tc(t, cx.w->status, cx.st), "attn_bwd (tcgen05)");
  else
    CKL(CAT_ATTN_BWD, 3, attn_bwd_simt(dt, t, cx.st), "attn_bwd");
  dbg_round(cx, w.dqkv, (int64_t)Nq * (cross ? I : 3 * I), RB_DQKV);
  if (cross) dbg_round(cx, w.dkv, (int64_t)Nk * 2 * I, RB_DQKV);
  if (c.recompute == 1) {
    CKL(CAT_NORM, 1, launch_rmsnorm_fwd(dt, a.x, pptr(cx.h, cx.params, p.norm), a.y, a.rstd, Nq, d, c.rms_eps, cx.st),
       "rmsnorm_fwd (recomputed)");
    dbg_round(cx, a.y, (int64_t)Nq * d, RB_Y);
  }
  if (!cross) {
    proj_wgrad(cx, w.dqkv, 3 * I, a.y, d, p.q, Nq, 3 * I, d, 1.f, "wgrad qkv");
    proj_dgrad(cx, w.dqkv, 3 * I, p.q, Nq, 3 * I, d, w.dy, d, 1.f, 0, 0, "dgrad qkv");
  } else {
    proj_wgrad(cx, w.dqkv, I, a.y, d, p.q, Nq, I, d, 1.f, "wgrad q");
    proj_dgrad(cx, w.dqkv, I, p.q, Nq, I, d, w.dy, d, 1.f, 0, 0, "dgrad q");
    proj_wgrad(cx, w.dkv, 2 * I, kv_src, d, p.k, Nk, 2 * I, d, 1.f, "wgrad kv");
    proj_dgrad(cx, w.dkv, 2 * I, p.k, Nk, 2 * I, d, dY32, d, 1.f, 1, dY_accumulate, "dgrad kv");
  }
  dbg_round(cx, w.dy, (int64_t)Nq * d, RB_DY);
  CKL(CAT_NORM, 2, launch_rmsnorm_bwd(dt, w.dy, 0, a.x, a.rstd, pptr(cx.h, cx.params, p.norm), dX, dX, dXb, cx.grads + p.norm,
                        w.norm_partial, Nq, d, cx.st),
     "rmsnorm_bwd");
  dbg_round(cx, dXb, (int64_t)Nq * d, RB_DXB);
}

// the gated-GELU epilogues run in the tensor-core GEMM on CTA pairs; flags bit 3 keeps the separate kernels
bool fused_geglu_ok(Ctx& cx, GemmArgs& g) {
  const t5_config& c = cx.h->cfg;
  if (c.dtype != DT_BF16 || (c.flags & (1 | 4 | 8))) return false;
  // measured: with a short contraction (d_model 512 / 768) the heavier epilogue costs more than the separate
  // bandwidth-bound kernels it replaces; from d_model ~1024 on the two are even and the fusion saves traffic
  if (c.d_model < 1024) return false;
  g.pair = 1;
  return gemm_tc_supported(g) && gemm_tc_epi_supported(g);
}

void ffn_forward(Ctx& cx, const FfnP& p, const FfnWs& f, float* x_out, int64_t N) {
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, F = c.d_ff, dt = c.dtype;
  CKL(CAT_NORM, 1, launch_rmsnorm_fwd(dt, f.x, pptr(cx.h, cx.params, p.norm), f.y, f.rstd, (int)N, d, c.rms_eps, cx.st),
     "rmsnorm_fwd");
  dbg_round(cx, f.y, N * d, RB_Y);
  GemmArgs gf{};
  gf.M = (int)N; gf.N = 2 * F; gf.K = d; gf.alpha = 1.f;
  gf.A = f.y; gf.lda = d; gf.a_kmajor = 1;
  gf.B = pptr(cx.h, cx.params, p.wi0); gf.ldb = d; gf.b_kmajor = 1;
  gf.D = f.h; gf.ldd = 2 * F; gf.epi = 1; gf.aux = f.hg; gf.ld_aux = F; gf.F = F;
  if (fused_geglu_ok(cx, gf)) {
    gemm(cx, gf, "wi proj + gated GELU");
  } else {
    proj_fwd(cx, f.y, d, p.wi0, (int)N, 2 * F, d, f.h, 2 * F, 1.f, nullptr, "wi proj");
    dbg_round(cx, f.h, N * 2 * F, RB_H);
    CKL(CAT_GEGLU, 1, launch_geglu_fwd(dt, f.h, f.hg, (int)N, F, cx.st), "geglu_fwd");
    dbg_round(cx, f.hg, N * F, RB_HG);
  }
  proj_fwd(cx, f.hg, F, p.wo, (int)N, d, F, x_out, d, 1.f, f.x, "wo proj");
}

void ffn_backward(Ctx& cx, const FfnP& p, const FfnWs& f, float* dX, void* dXb, int64_t N) {
  const t5_config& c = cx.h->cfg;
  Workspace& w = *cx.w;
  int d = c.d_model, F = c.d_ff, dt = c.dtype, n = (int)N;
  if (c.recompute == 1) {
    CKL(CAT_GEGLU, 1, launch_geglu_fwd(dt, f.h, f.hg, n, F, cx.st), "geglu_fwd (recomputed)");
    dbg_round(cx, f.hg, N * F, RB_HG);
  }
  proj_wgrad(cx, dXb, d, f.hg, F, p.wo, n, d, F, 1.f, "wgrad ffn.wo");
  GemmArgs gb{};
  gb.M = n; gb.N = F; gb.K = d; gb.alpha = 1.f;
  gb.A = dXb; gb.lda = d; gb.a_kmajor = 1;
  gb.B = pptr(cx.h, cx.params, p.wo); gb.ldb = F; gb.b_kmajor = 0;
  gb.D = w.dh; gb.ldd = 2 * F; gb.epi = 2; gb.aux = f.h; gb.ld_aux = 2 * F; gb.F = F;
  if (fused_geglu_ok(cx, gb)) {
    gemm(cx, gb, "dgrad ffn.wo + gated GELU backward");
  } else {
    proj_dgrad(cx, dXb, d, p.wo, n, d, F, w.dhg, F, 1.f, 0, 0, "dgrad ffn.wo");
    dbg_round(cx, w.dhg, N * F, RB_DHG);
    CKL(CAT_GEGLU, 1, launch_geglu_bwd(dt, w.dhg, f.h, w.dh, n, F, cx.st), "geglu_bwd");
    dbg_round(cx, w.dh, N * 2 * F, RB_DH);
  }
  if (c.recompute == 1) {
    CKL(CAT_NORM, 1, launch_rmsnorm_fwd(dt, f.x, pptr(cx.h, cx.params, p.norm), f.y, f.rstd, n, d, c.rms_eps, cx.st),
       "rmsnorm_fwd (recomputed)");
    dbg_round(cx, f.y, N * d, RB_Y);
  }
  proj_wgrad(cx, w.dh, 2 * F, f.y, d, p.wi0, n, 2 * F, d, 1.f, "wgrad ffn.wi");
  proj_dgrad(cx, w.dh, 2 * F, p.wi0, n, 2 * F, d, w.dy, d, 1.f, 0, 0, "dgrad ffn.wi");
  dbg_round(cx, w.dy, N * d, RB_DY);
  CKL(CAT_NORM, 2, launch_rmsnorm_bwd(dt, w.dy, 0, f.x, f.rstd, pptr(cx.h, cx.params, p.norm), dX, dX, dXb, cx.grads + p.norm,
                        w.norm_partial, n, d, cx.st),
     "rmsnorm_bwd");
  dbg_round(cx, dXb, N * d, RB_DXB);
}

AttnGeom enc_geom(Ctx& cx) {
  AttnGeom g;
  g.Tq = g.Tk = cx.Te; g.Nq = g.Nk = (int64_t)cx.B * cx.Te;
  g.code_q = g.code_k = cx.w->enc_code; g.causal = 0; g.bias = cx.w->bias_enc; g.dbias = cx.w->dbias_enc;
  g.far = saturation_distance(cx.h->spec_enc);
  return g;
}
AttnGeom self_geom(Ctx& cx) {
  AttnGeom g;
  g.Tq = g.Tk = cx.Td; g.Nq = g.Nk = (int64_t)cx.B * cx.Td;
  g.code_q = g.code_k = cx.w->dec_code; g.causal = 1; g.bias = cx.w->bias_dec; g.dbias = cx.w->dbias_dec;
  g.far = saturation_distance(cx.h->spec_dec);
  return g;
}
AttnGeom cross_geom(Ctx& cx) {
  AttnGeom g;
  g.Tq = cx.Td; g.Tk = cx.Te; g.Nq = (int64_t)cx.B * cx.Td; g.Nk = (int64_t)cx.B * cx.Te;
  g.code_q = cx.w->dec_code; g.code_k = cx.w->enc_code; g.causal = 0; g.bias = nullptr; g.dbias = nullptr;
  g.far = 0;
  return g;
}

void run_prep(Ctx& cx, const t5_batch* b) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  CK(cudaMemsetAsync(w.status, 0, 4, cx.st), "memset status");
  CK(cudaMemsetAsync(w.sk_flags, 0, (int64_t)kSkSlices * kSkSliceInts * 4, cx.st), "memset stream-K flags");
  CKL(CAT_MISC, 2, launch_prep(c.arch == 0 ? b->d_enc_tokens : nullptr, b->d_enc_segment_ids, b->d_dec_targets,
                 b->d_dec_segment_ids, cx.B, cx.Te, cx.Td, w.enc_code, w.dec_code, w.dec_in, w.W_int, w.W_f, cx.st),
     "prep");
  if (c.arch == 0 && cx.Te > 0)
    CKL(CAT_MISC, 1, launch_relbias_expand(c.dtype, cx.h->spec_enc, pptr(cx.h, cx.params, cx.h->enc_relbias), c.n_heads, cx.Te,
                             cx.Te, w.bias_enc, cx.st),
       "relbias_expand enc");
  CKL(CAT_MISC, 1, launch_relbias_expand(c.dtype, cx.h->spec_dec, pptr(cx.h, cx.params, cx.h->dec_relbias), c.n_heads, cx.Td,
                           cx.Td, w.bias_dec, cx.st),
     "relbias_expand dec");
}

void encoder_forward(Ctx& cx, const t5_batch* b) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int L = c.n_enc_layers, d = c.d_model;
  int64_t Ne = (int64_t)cx.B * cx.Te;
  float* x0 = L > 0 ? w.enc_attn[0].x : w.enc_x_final;
  CKL(CAT_EMBED, 1, launch_embed_gather(c.dtype, pptr(cx.h, cx.params, cx.h->token_embed), b->d_enc_tokens, x0, (int)Ne, d, cx.st),
     "embed enc");
  AttnGeom g = enc_geom(cx);
  for (int l = 0; l < L; ++l) {
    attn_forward(cx, cx.h->enc[l].attn, w.enc_attn[l], w.enc_ffn[l].x, g, nullptr);
    float* x_next = l + 1 < L ? w.enc_attn[l + 1].x : w.enc_x_final;
    ffn_forward(cx, cx.h->enc[l].ffn, w.enc_ffn[l], x_next, Ne);
  }
  CKL(CAT_NORM, 1, launch_rmsnorm_fwd(c.dtype, w.enc_x_final, pptr(cx.h, cx.params, cx.h->enc_final_norm), w.enc_out,
                        w.enc_rstd_f, (int)Ne, d, c.rms_eps, cx.st),
     "enc final norm");
  dbg_round(cx, w.enc_out, Ne * d, RB_Y);
}

// enc_y: encoder output used by cross-attention (NULL for decoder-only); logits_out: where logits go
void decoder_forward(Ctx& cx, const void* enc_y, void* logits_out) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int L = c.n_dec_layers, d = c.d_model;
  int64_t Nd = (int64_t)cx.B * cx.Td;
  float* x0 = L > 0 ? w.dec_self[0].x : w.dec_x_final;
  CKL(CAT_EMBED, 1, launch_embed_gather(c.dtype, pptr(cx.h, cx.params, cx.h->token_embed), w.dec_in, x0, (int)Nd, d, cx.st),
     "embed dec");
  AttnGeom gs = self_geom(cx), gc = cross_geom(cx);
  bool encdec = c.arch == 0;
  for (int l = 0; l < L; ++l) {
    float* after_self = encdec ? w.dec_cross[l].x : w.dec_ffn[l].x;
    attn_forward(cx, cx.h->dec[l].self, w.dec_self[l], after_self, gs, nullptr);
    if (encdec) attn_forward(cx, cx.h->dec[l].cross, w.dec_cross[l], w.dec_ffn[l].x, gc, enc_y);
    float* x_next = l + 1 < L ? w.dec_self[l + 1].x : w.dec_x_final;
    ffn_forward(cx, cx.h->dec[l].ffn, w.dec_ffn[l], x_next, Nd);
  }
  CKL(CAT_NORM, 1, launch_rmsnorm_fwd(c.dtype, w.dec_x_final, pptr(cx.h, cx.params, cx.h->dec_final_norm), w.dec_z, w.dec_rstd_f,
                        (int)Nd, d, c.rms_eps, cx.st),
     "dec final norm");
  dbg_round(cx, w.dec_z, Nd * d, RB_Y);
  proj_fwd(cx, w.dec_z, d, cx.h->token_embed, (int)Nd, c.vocab, d, logits_out, c.vocab, c.logit_scale, nullptr,
           "logits");
  dbg_round(cx, logits_out, Nd * c.vocab, RB_LOGITS);
}

void backward(Ctx& cx, const t5_batch* b) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, V = c.vocab, dt = c.dtype, H = c.n_heads;
  int64_t Nd = (int64_t)cx.B * cx.Td, Ne = (int64_t)cx.B * cx.Te;
  bool encdec = c.arch == 0;
  for (auto& gp : cx.h->gaps)
    CK(cudaMemsetAsync(cx.grads + gp.first, 0, (gp.second - gp.first) * 4, cx.st), "memset gaps");
  if (encdec && cx.Te > 0) CK(cudaMemsetAsync(w.dbias_enc, 0, (int64_t)H * (2 * cx.Te - 1) * 4, cx.st), "memset dbias");
  CK(cudaMemsetAsync(w.dbias_dec, 0, (int64_t)H * (2 * cx.Td - 1) * 4, cx.st), "memset dbias");
  // tied embedding: dE = logit_scale dlogits^T Z (overwrites), dZ = logit_scale dlogits E
  proj_wgrad(cx, w.logits, V, w.dec_z, d, cx.h->token_embed, (int)Nd, V, d, c.logit_scale, "wgrad logits");
  proj_dgrad(cx, w.logits, V, cx.h->token_embed, (int)Nd, V, d, w.dy, d, c.logit_scale, 0, 0, "dgrad logits");
  dbg_round(cx, w.dy, Nd * d, RB_DY);
  CKL(CAT_NORM, 2, launch_rmsnorm_bwd(dt, w.dy, 0, w.dec_x_final, w.dec_rstd_f, pptr(cx.h, cx.params, cx.h->dec_final_norm),
                        nullptr, w.dX_dec, w.dXb_dec, cx.grads + cx.h->dec_final_norm, w.norm_partial, (int)Nd, d,
                        cx.st),
     "dec final norm bwd");
  dbg_round(cx, w.dXb_dec, Nd * d, RB_DXB);
  AttnGeom gs = self_geom(cx), gc = cross_geom(cx);
  bool first_cross = true;
  for (int l = c.n_dec_layers - 1; l >= 0; --l) {
    ffn_backward(cx, cx.h->dec[l].ffn, w.dec_ffn[l], w.dX_dec, w.dXb_dec, Nd);
    if (encdec) {
      attn_backward(cx, cx.h->dec[l].cross, w.dec_cross[l], w.dX_dec, w.dXb_dec, gc, w.enc_out, w.dY32,
                    first_cross ? 0 : 1);
      first_cross = false;
    }
    attn_backward(cx, cx.h->dec[l].self, w.dec_self[l], w.dX_dec, w.dXb_dec, gs, nullptr, nullptr, 0);
  }
  CKL(CAT_EMBED, 1, launch_embed_scatter_add(w.dec_in, w.dX_dec, cx.grads + cx.h->token_embed, (int)Nd, d, cx.st),
     "embed scatter dec");
  CKL(CAT_MISC, 1, launch_relbias_fold(cx.h->spec_dec, w.dbias_dec, H, cx.Td, cx.Td, c.rel_buckets, cx.grads + cx.h->dec_relbias,
                         cx.st),
     "relbias fold dec");
  if (!encdec) return;
  CKL(CAT_NORM, 2, launch_rmsnorm_bwd(dt, w.dY32, 1, w.enc_x_final, w.enc_rstd_f, pptr(cx.h, cx.params, cx.h->enc_final_norm),
                        nullptr, w.dX_enc, w.dXb_enc, cx.grads + cx.h->enc_final_norm, w.norm_partial, (int)Ne, d,
                        cx.st),
     "enc final norm bwd");
  dbg_round(cx, w.dXb_enc, Ne * d, RB_DXB);
  AttnGeom ge = enc_geom(cx);
  for (int l = c.n_enc_layers - 1; l >= 0; --l) {
    ffn_backward(cx, cx.h->enc[l].ffn, w.enc_ffn[l], w.dX_enc, w.dXb_enc, Ne);
    attn_backward(cx, cx.h->enc[l].attn, w.enc_attn[l], w.dX_enc, w.dXb_enc, ge, nullptr, nullptr, 0);
  }
  CKL(CAT_EMBED, 1, launch_embed_scatter_add(b->d_enc_tokens, w.dX_enc, cx.grads + cx.h->token_embed, (int)Ne, d, cx.st),
     "embed scatter enc");
  CKL(CAT_MISC, 1, launch_relbias_fold(cx.h->spec_enc, w.dbias_enc, H, cx.Te, cx.Te, c.rel_buckets, cx.grads + cx.h->enc_relbias,
                         cx.st),
     "relbias fold enc");
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15) == 0; }

// Common argument checks; fills cx and lays out the workspace.
int begin_call(t5_handle* h, const void* params, const t5_batch* b, void* ws, int64_t ws_bytes, void* stream,
               Workspace* w, Ctx* cx, bool need_enc_tokens) {
  if (!h) return T5_ERR_NULL;
  if (!params || !b || !ws) return fail(h, T5_ERR_NULL, "null params, batch or workspace pointer");
  const t5_config& c = h->cfg;
  int Te = c.arch == 0 ? b->Te : 0;
  if (b->B < 1 || b->B > c.max_batch || b->Td < 1 || b->Td > c.max_dec_len ||
      (c.arch == 0 && (Te < 1 || Te > c.max_enc_len)))
    return fail(h, T5_ERR_SHAPE, "batch %dx(%d,%d) outside the configured maxima %dx(%d,%d)", b->B, b->Te, b->Td,
                c.max_batch, c.max_enc_len, c.max_dec_len);
  if (!b->d_dec_targets || (need_enc_tokens && c.arch == 0 && !b->d_enc_tokens))
    return fail(h, T5_ERR_NULL, "null token array in batch");
  if (!aligned16(params) || !aligned16(ws)) return fail(h, T5_ERR_ALIGN, "params/workspace not 16-byte aligned");
  plan_workspace(h, b->B, Te, b->Td, (char*)ws, w);
  if (w->bytes > ws_bytes)
    return fail(h, T5_ERR_WORKSPACE, "workspace of %lld bytes given, %lld needed", (long long)ws_bytes,
                (long long)w->bytes);
  cx->h = h; cx->params = params; cx->grads = nullptr; cx->st = (cudaStream_t)stream; cx->w = w;
  cx->B = b->B; cx->Te = Te; cx->Td = b->Td; cx->err = cudaSuccess; cx->where = ""; cx->launches = 0; cx->sk_next = 0;
  cx->packed = (b->d_enc_segment_ids != nullptr || b->d_dec_segment_ids != nullptr) ? 1 : 0;
  return T5_OK;
}

int end_call(t5_handle* h, Ctx& cx) {
  h->launches_last_call = cx.launches;
  if (cx.err != cudaSuccess)
    return fail(h, T5_ERR_CUDA, "%s: %s", cx.where, cudaGetErrorString(cx.err));
  return T5_OK;
}

}  // namespace

// =============================================================================== C ABI
extern "C" {

int t5_create(const t5_config* cfg, t5_handle** out) {
  if (!cfg || !out) return fail(nullptr, T5_ERR_NULL, "null config or output pointer");
  *out = nullptr;
  const t5_config& c = *cfg;
  if (c.abi_version != T5_ABI_VERSION) return fail(nullptr, T5_ERR_CONFIG, "abi_version %d != %d", c.abi_version, T5_ABI_VERSION);
  if (c.arch != 0 && c.arch != 1) return fail(nullptr, T5_ERR_CONFIG, "arch must be 0 or 1");
  if (c.dtype != DT_F32 && c.dtype != DT_BF16) return fail(nullptr, T5_ERR_CONFIG, "dtype must be 0 or 1");
  if (c.d_kv != 32 && c.d_kv != 64 && c.d_kv != 128) return fail(nullptr, T5_ERR_CONFIG, "d_kv must be 32, 64 or 128");
  if (c.d_model < 8 || c.d_model % 8 || c.d_ff < 8 || c.d_ff % 8 || c.vocab < 8 || c.vocab % 8)
    return fail(nullptr, T5_ERR_CONFIG, "d_model, d_ff and vocab must be positive multiples of 8");
  if (c.n_heads < 1 || c.n_heads > 256) return fail(nullptr, T5_ERR_CONFIG, "n_heads out of range");
  if (c.n_dec_layers < 1 || c.n_enc_layers < 0 || (c.arch == 1 && c.n_enc_layers != 0))
    return fail(nullptr, T5_ERR_CONFIG, "layer counts: need n_dec_layers >= 1; decoder-only has no encoder layers");
  if (c.max_batch < 1 || c.max_dec_len < 1 || (c.arch == 0 && c.max_enc_len < 1))
    return fail(nullptr, T5_ERR_CONFIG, "max_batch / max lengths must be positive");
  if ((int64_t)c.max_batch * (c.max_enc_len > c.max_dec_len ? c.max_enc_len : c.max_dec_len) > (1 << 24))
    return fail(nullptr, T5_ERR_CONFIG, "more than 2^24 tokens per step");
  if (c.recompute < 0 || c.recompute > 1) return fail(nullptr, T5_ERR_CONFIG, "recompute must be 0 or 1");
  t5_handle* h = new t5_handle();
  h->cfg = c;
  if (!build_bucket_spec(1, c.rel_buckets, c.rel_max_distance, &h->spec_enc) ||
      !build_bucket_spec(0, c.rel_buckets, c.rel_max_distance, &h->spec_dec)) {
    delete h;
    return fail(nullptr, T5_ERR_CONFIG, "unsupported rel_buckets / rel_max_distance");
  }
  build_manifest(h);
  *out = h;
  return T5_OK;
}

int t5_destroy(t5_handle* h) {
  if (h)
    for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
  delete h;
  return T5_OK;
}

const char* t5_last_error(const t5_handle* h) { return h ? h->err.c_str() : g_create_error; }

int t5_param_count(const t5_handle* h, int64_t* n) {
  if (!h || !n) return T5_ERR_NULL;
  *n = h->n_params;
  return T5_OK;
}

int t5_param_tensors(const t5_handle* h, int32_t* n) {
  if (!h || !n) return T5_ERR_NULL;
  *n = (int32_t)h->tensors.size();
  return T5_OK;
}

int t5_param_manifest(const t5_handle* h, int32_t idx, char name[64], int64_t* offset, int32_t shape[4],
                      int32_t* ndim) {
  if (!h || !name || !offset || !shape || !ndim) return T5_ERR_NULL;
  if (idx < 0 || idx >= (int32_t)h->tensors.size()) return T5_ERR_ARG;
  const Tensor& t = h->tensors[idx];
  snprintf(name, 64, "%s", t.name.c_str());
  *offset = t.offset;
  for (int i = 0; i < 4; ++i) shape[i] = t.shape[i];
  *ndim = t.ndim;
  return T5_OK;
}

int t5_workspace_bytes(const t5_handle* h, int64_t* bytes) {
  if (!h || !bytes) return T5_ERR_NULL;
  Workspace w;
  plan_workspace(h, h->cfg.max_batch, h->cfg.max_enc_len, h->cfg.max_dec_len, nullptr, &w);
  *bytes = w.bytes;
  return T5_OK;
}

int t5_init_params(t5_handle* h, void* d_params, uint64_t seed, float stddev, void* stream) {
  if (!h) return T5_ERR_NULL;
  if (!d_params) return fail(h, T5_ERR_NULL, "null parameter buffer");
  if (!aligned16(d_params)) return fail(h, T5_ERR_ALIGN, "parameter buffer not 16-byte aligned");
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(d_params, 0, h->n_params * esize(h), st);
  for (size_t i = 0; i < h->tensors.size() && e == cudaSuccess; ++i) {
    const Tensor& t = h->tensors[i];
    bool scale = t.ndim == 1;
    e = launch_fill_normal(h->cfg.dtype, eoff(h, d_params, t.offset), t.numel(), t.offset, seed,
                           scale ? 0.f : stddev, scale ? 1.f : 0.f, st);
  }
  if (e != cudaSuccess) return fail(h, T5_ERR_CUDA, "init_params: %s", cudaGetErrorString(e));
  return T5_OK;
}

int t5_train_step_fwd_bwd(t5_handle* h, const void* d_params, const t5_batch* batch, float* d_grads,
                          float* d_loss4, void* d_workspace, int64_t workspace_bytes, void* stream) {
  Workspace w;
  Ctx cx;
  int rc = begin_call(h, d_params, batch, d_workspace, workspace_bytes, stream, &w, &cx, true);
  if (rc != T5_OK) return rc;
  if (!d_grads || !d_loss4) return fail(h, T5_ERR_NULL, "null gradient or loss pointer");
  if (!aligned16(d_grads)) return fail(h, T5_ERR_ALIGN, "gradient buffer not 16-byte aligned");
  cx.grads = d_grads;
  const t5_config& c = h->cfg;
  run_prep(cx, batch);
  if (c.arch == 0) encoder_forward(cx, batch);
  decoder_forward(cx, c.arch == 0 ? w.enc_out : nullptr, w.logits);
  CK(cudaMemsetAsync(w.sums, 0, 16, cx.st), "memset sums");
  CKL(CAT_XENT, 1, launch_xent(c.dtype, w.logits, batch->d_dec_targets, cx.B * cx.Td, c.vocab, c.z_loss, w.W_f, w.sums, w.lse_tok,
                 cx.st),
     "xent");
  CKL(CAT_MISC, 1, launch_finalize_loss(w.sums, w.W_f, d_loss4, cx.st), "finalize loss");
  dbg_round(cx, w.logits, (int64_t)cx.B * cx.Td * c.vocab, RB_DLOGITS);
  backward(cx, batch);
  return end_call(h, cx);
}

int t5_encode(t5_handle* h, const void* d_params, const t5_batch* batch, void* d_enc_out, void* d_workspace,
              int64_t workspace_bytes, void* stream) {
  Workspace w;
  Ctx cx;
  int rc = begin_call(h, d_params, batch, d_workspace, workspace_bytes, stream, &w, &cx, true);
  if (rc != T5_OK) return rc;
  if (h->cfg.arch != 0) return fail(h, T5_ERR_CONFIG, "t5_encode needs the encoder-decoder architecture");
  if (!d_enc_out) return fail(h, T5_ERR_NULL, "null output pointer");
  run_prep(cx, batch);
  encoder_forward(cx, batch);
  CK(cudaMemcpyAsync(d_enc_out, w.enc_out, (int64_t)cx.B * cx.Te * h->cfg.d_model * esize(h),
                     cudaMemcpyDeviceToDevice, cx.st),
     "copy encoder output");
  return end_call(h, cx);
}

int t5_decode_logits(t5_handle* h, const void* d_params, const t5_batch* batch, const void* d_enc_out,
                     void* d_logits, void* d_workspace, int64_t workspace_bytes, void* stream) {
  Workspace w;
  Ctx cx;
  int rc = begin_call(h, d_params, batch, d_workspace, workspace_bytes, stream, &w, &cx, true);
  if (rc != T5_OK) return rc;
  if (!d_logits || (h->cfg.arch == 0 && !d_enc_out)) return fail(h, T5_ERR_NULL, "null logits or encoder output");
  if (!aligned16(d_logits) || !aligned16(d_enc_out)) return fail(h, T5_ERR_ALIGN, "logits/encoder output not aligned");
  run_prep(cx, batch);
  decoder_forward(cx, h->cfg.arch == 0 ? d_enc_out : nullptr, d_logits);
  return end_call(h, cx);
}

int t5_device_status(t5_handle* h, const void* d_workspace, void* stream) {
  if (!h || !d_workspace) return T5_ERR_NULL;
  int status = 0;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(&status, d_workspace, sizeof(int), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return fail(h, T5_ERR_CUDA, "device_status: %s", cudaGetErrorString(e));
  if (status != 0) return fail(h, T5_ERR_DEVICE_TIMEOUT, "a bounded device-side wait ran out (code %d)", status);
  return T5_OK;
}

int t5_profile_enable(t5_handle* h, int32_t on) {
  if (!h) return T5_ERR_NULL;
  h->prof_on = on != 0;
  h->prof_cat.clear();
  for (int i = 0; i < 8; ++i) { h->prof_flops[i] = 0; h->prof_launches[i] = 0; }
  return T5_OK;
}

int t5_profile_read(t5_handle* h, double ms[8], double flops[8], int64_t launches[8]) {
  if (!h || !ms || !flops || !launches) return T5_ERR_NULL;
  for (int i = 0; i < 8; ++i) { ms[i] = 0; flops[i] = h->prof_flops[i]; launches[i] = h->prof_launches[i]; }
  for (size_t i = 0; i < h->prof_cat.size(); ++i) {
    cudaError_t e = cudaEventSynchronize(h->prof_events[2 * i + 1]);
    float t = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, h->prof_events[2 * i], h->prof_events[2 * i + 1]);
    if (e != cudaSuccess) return fail(h, T5_ERR_CUDA, "profile_read: %s", cudaGetErrorString(e));
    ms[h->prof_cat[i]] += t;
  }
  h->prof_cat.clear();
  for (int i = 0; i < 8; ++i) { h->prof_flops[i] = 0; h->prof_launches[i] = 0; }
  return T5_OK;
}

int t5_launch_count(const t5_handle* h, int64_t* n) {
  if (!h || !n) return T5_ERR_NULL;
  *n = h->launches_last_call;
  return T5_OK;
}

int t5_relpos_buckets(int32_t bidirectional, int32_t num_buckets, int32_t max_distance, int32_t rel_lo, int32_t n,
                      int32_t* d_out, void* stream) {
  if (!d_out) return T5_ERR_NULL;
  BucketSpec s;
  if (!build_bucket_spec(bidirectional, num_buckets, max_distance, &s)) return T5_ERR_CONFIG;
  cudaError_t e = launch_buckets(s, rel_lo, n, d_out, (cudaStream_t)stream);
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

int t5_xent_zloss(int32_t dtype, void* d_logits, const int32_t* d_targets, int32_t n_rows, int32_t vocab,
                  float z_loss, const float* d_W, double* d_sums, float* d_lse, void* stream) {
  if (!d_logits || !d_targets || !d_W || !d_sums || !d_lse) return T5_ERR_NULL;
  if ((dtype != DT_F32 && dtype != DT_BF16) || vocab < 8 || vocab % 8 || n_rows < 0) return T5_ERR_ARG;
  cudaError_t e = launch_xent(dtype, d_logits, d_targets, n_rows, vocab, z_loss, d_W, d_sums, d_lse,
                              (cudaStream_t)stream);
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

int t5_attention(int32_t dtype, int32_t impl, int32_t backward, int32_t B, int32_t H, int32_t Tq, int32_t Tk,
                 int32_t d_kv, int32_t causal, float scale, const void* d_q, int32_t ldq, const void* d_k,
                 int32_t ldk, const void* d_v, int32_t ldv, void* d_o, int32_t ldo, float* d_o32, float* d_lse,
                 const int32_t* d_code_q, const int32_t* d_code_k, const float* d_bias_delta, const void* d_do,
                 int32_t lddo, void* d_dq, int32_t lddq, void* d_dk, int32_t lddk, void* d_dv, int32_t lddv,
                 float* d_delta, float* d_dbias_delta, void* stream) {
  if (!d_q || !d_k || !d_v || !d_o || !d_lse || !d_code_q || !d_code_k) return T5_ERR_NULL;
  if (backward && (!d_do || !d_dq || !d_dk || !d_dv || !d_delta)) return T5_ERR_NULL;
  if ((dtype != DT_F32 && dtype != DT_BF16) || B < 0 || H < 1 || Tq < 1 || Tk < 1) return T5_ERR_ARG;
  if (d_kv != 32 && d_kv != 64 && d_kv != 128) return T5_ERR_ARG;
  AttnArgs a;
  memset(&a, 0, sizeof a);
  a.O32 = d_o32; a.ldo32 = H * d_kv;
  a.Q = d_q; a.K = d_k; a.V = d_v; a.O = d_o; a.ldq = ldq; a.ldk = ldk; a.ldv = ldv; a.ldo = ldo; a.lse = d_lse;
  a.B = B; a.H = H; a.Tq = Tq; a.Tk = Tk; a.dk = d_kv; a.code_q = d_code_q; a.code_k = d_code_k; a.causal = causal;
  a.bias_delta = d_bias_delta; a.scale = scale; a.dO = d_do; a.lddo = lddo; a.dQ = d_dq; a.dK = d_dk; a.dV = d_dv;
  a.lddq = lddq; a.lddk = lddk; a.lddv = lddv; a.delta = d_delta; a.dbias_delta = d_dbias_delta;
  a.packed = 1;      // the codes may describe packed rows: keep the tile-skipping bookkeeping on
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (impl == 0) {
    e = backward ? attn_bwd_simt(dtype, a, st) : attn_fwd_simt(dtype, a, st);
  } else {
    if (dtype != DT_BF16 || !attn_tc_supported(a)) return T5_ERR_ARG;
    e = backward ? attn_bwd_tc(a, nullptr, st) : attn_fwd_tc(a, nullptr, st);
  }
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

int t5_attention_ds_scratch_bytes(int32_t B, int32_t H, int32_t Tq, int32_t Tk, int64_t* bytes) {
  if (!bytes) return T5_ERR_NULL;
  if (B < 0 || H < 1 || Tq < 1 || Tk < 1) return T5_ERR_ARG;
  *bytes = attn_tc_ds_scratch_bytes(B, H, Tq, Tk);
  return T5_OK;
}

int t5_attention_backward_onepass(int32_t B, int32_t H, int32_t Tq, int32_t Tk, int32_t d_kv, int32_t causal,
                                  float scale, const void* d_q, int32_t ldq, const void* d_k, int32_t ldk,
                                  const void* d_v, int32_t ldv, const void* d_o, int32_t ldo, const float* d_o32,
                                  const float* d_lse, const int32_t* d_code_q, const int32_t* d_code_k,
                                  const float* d_bias_delta, const void* d_do, int32_t lddo, void* d_dq,
                                  int32_t lddq, void* d_dk, int32_t lddk, void* d_dv, int32_t lddv, float* d_delta,
                                  float* d_dbias_delta, int32_t bias_far, void* d_ds_scratch,
                                  int64_t ds_scratch_bytes, void* stream) {
  if (!d_q || !d_k || !d_v || !d_o || !d_lse || !d_code_q || !d_code_k || !d_do || !d_dq || !d_dk || !d_dv ||
      !d_delta || !d_ds_scratch)
    return T5_ERR_NULL;
  if (B < 0 || H < 1 || Tq < 1 || Tk < 1 || (d_kv != 64 && d_kv != 128) || bias_far < 0) return T5_ERR_ARG;
  if (ds_scratch_bytes < attn_tc_ds_scratch_bytes(B, H, Tq, Tk) || ((uintptr_t)d_ds_scratch & 127)) return T5_ERR_ARG;
  AttnArgs a;
  memset(&a, 0, sizeof a);
  a.O32 = const_cast<float*>(d_o32); a.ldo32 = H * d_kv;
  a.Q = d_q; a.K = d_k; a.V = d_v; a.O = const_cast<void*>(d_o); a.ldq = ldq; a.ldk = ldk; a.ldv = ldv; a.ldo = ldo;
  a.lse = const_cast<float*>(d_lse);
  a.B = B; a.H = H; a.Tq = Tq; a.Tk = Tk; a.dk = d_kv; a.code_q = d_code_q; a.code_k = d_code_k; a.causal = causal;
  a.bias_delta = d_bias_delta; a.scale = scale; a.dO = d_do; a.lddo = lddo; a.dQ = d_dq; a.dK = d_dk; a.dV = d_dv;
  a.lddq = lddq; a.lddk = lddk; a.lddv = lddv; a.delta = d_delta; a.dbias_delta = d_dbias_delta;
  a.bias_far = bias_far; a.ds_scratch = d_ds_scratch; a.ds_bytes = ds_scratch_bytes;
  if (!attn_tc_supported(a) || !attn_tc_onepass_supported(a)) return T5_ERR_ARG;
  cudaError_t e = attn_bwd_tc(a, nullptr, (cudaStream_t)stream);
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

int t5_gemm(int32_t dtype, int32_t impl, int32_t M, int32_t N, int32_t K, float alpha, const void* d_A, int32_t lda,
            int32_t a_kmajor, const void* d_B, int32_t ldb, int32_t b_kmajor, void* d_D, int32_t ldd,
            int32_t out_f32, int32_t accumulate, int32_t* d_sk_flags, void* stream) {
  if (!d_A || !d_B || !d_D) return T5_ERR_NULL;
  if (M < 0 || N < 0 || K < 0 || (dtype != DT_F32 && dtype != DT_BF16)) return T5_ERR_ARG;
  GemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.alpha = alpha; g.A = d_A; g.lda = lda; g.a_kmajor = a_kmajor;
  g.B = d_B; g.ldb = ldb; g.b_kmajor = b_kmajor; g.D = d_D; g.ldd = ldd;
  g.out_f32 = (dtype == DT_F32) ? 1 : out_f32; g.accumulate = accumulate; g.sk_flags = d_sk_flags;
  cudaError_t e;
  if (impl == 0) {
    e = gemm_simt(dtype, g, (cudaStream_t)stream);
  } else {
    if (dtype != DT_BF16 || !gemm_tc_supported(g)) return T5_ERR_ARG;
    g.pair = impl == 2;
    e = gemm_tc(g, nullptr, (cudaStream_t)stream);
  }
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

}  // extern "C"
