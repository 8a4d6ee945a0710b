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

// per-sub-layer saved activations.  x: residual input (float32); xg = x * g (operand dtype), the A operand of the
// sub-layer's first projection, whose epilogue applies the RMSNorm factor from ssq = rowsum(x^2).
struct AttnWs { float* x; void* xg; float* ssq; void* q; void* kv; void* ctx; float* ctx32; float* lse; };
struct FfnWs { float* x; void* xg; float* ssq; void* h; void* hg; };
// where the kernel that produces a residual block writes its operand copy and statistics: the norm that reads it
struct NextNorm { void* xg; float* ssq; int64_t g_off; };

struct Workspace {
  std::vector<AttnWs> enc_attn, dec_self, dec_cross;
  std::vector<FfnWs> enc_ffn, dec_ffn;
  float *enc_x_final, *enc_ssq_f, *dec_x_final, *dec_ssq_f;
  void *enc_xg_f, *dec_xg_f, *logits;
  float* ssq_all;        // every ssq vector of the step, contiguous: zeroed once per call
  int64_t ssq_floats;
  float* lse_tok;
  int *enc_code, *dec_code, *dec_in, *W_int, *status, *sk_flags;
  float* dec_w;          // loss weight of every decoder position (0 / 1)
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
  int64_t lm_head = -1;      // separate output head (untied_head), else -1: the logits use token_embed
  std::vector<EncLayerP> enc;
  std::vector<DecLayerP> dec;
  BucketSpec spec_enc, spec_dec;
  std::string err;
  // opt-in per-kernel-family timing (CUDA events around each launch) and launch counting
  bool prof_on = false;
  std::vector<cudaEvent_t> prof_events;      // pairs: start, stop
  std::vector<int> prof_cat;                 // category of each pair in use
  struct ProfRec { const char* what; int M, N, K; };
  std::vector<ProfRec> prof_rec;             // what each pair brackets (GEMMs: their shape)
  double prof_flops[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int64_t prof_launches[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int64_t launches_last_call = 0;
  // second stream for the weight-gradient GEMMs of the backward pass (see Overlap below); owned by the handle
  cudaStream_t side = nullptr;
  int side_dev = -1;
  std::vector<cudaEvent_t> sync_events;      // fork / join events, reused round-robin
  size_t sync_next = 0;
  cudaEvent_t reader_events[8] = {};         // one per scratch buffer the side stream reads
  std::vector<cudaEvent_t> layer_events;     // per decoder layer: its cross-attention keys / values are projected
  // data-parallel training: called as ranges of the gradient buffer become final (see t5_set_grad_hook)
  t5_grad_ready_fn grad_hook = nullptr;
  void* grad_hook_user = nullptr;
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
    f.wi1 = c.ffn_act == 1 ? -1 : add_tensor(h, p + ".wi1", {F, d});      // the ReLU FFN has no gate
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
  if (c.untied_head) h->lm_head = add_tensor(h, "lm_head", {c.vocab, d});
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
  // Activation policy 1: the operand copies xg = x * g and the gated product hg are not kept per sub-layer; the
  // forward pass writes them into one shared buffer each (the next GEMM consumes them at once) and the backward
  // pass recomputes them from the saved x / pre-activations h right before the weight-gradient GEMMs.
  const bool recompute = c.recompute == 1;
  void* shared_y = nullptr;      // taken below, behind the status word
  void* shared_hg = nullptr;
  float* ssq_cur = nullptr;
  auto take_ssq = [&](int64_t n) {
    float* at = ssq_cur;
    ssq_cur += (n + 63) / 64 * 64;
    return base ? at : nullptr;
  };
  auto attn_ws = [&](int64_t Nq, int64_t Nk, int Tq, bool cross) {
    AttnWs a;
    a.x = (float*)take(Nq * d * 4);
    a.xg = recompute ? shared_y : take(Nq * d * es);
    a.ssq = take_ssq(Nq);
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
    f.xg = recompute ? shared_y : take(N * d * es);
    f.ssq = take_ssq(N);
    f.h = take(N * 2 * F * es);
    f.hg = recompute ? shared_hg : take(N * F * es);
    return f;
  };
  w->status = (int*)take(4);          // first, so its address does not depend on the batch shape
  w->sk_flags = (int*)take((int64_t)kSkSlices * kSkSliceInts * 4);   // per-GEMM flag slices of the stream-K tails
  {
    auto pad = [](int64_t n) { return (n + 63) / 64 * 64; };
    w->ssq_floats = (2 * (int64_t)c.n_enc_layers + 1) * pad(Ne) + (3 * (int64_t)c.n_dec_layers + 1) * pad(Nd);
    w->ssq_all = (float*)take(w->ssq_floats * 4);
    ssq_cur = w->ssq_all;
  }
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
  w->enc_ssq_f = take_ssq(Ne);
  w->enc_xg_f = take(Ne * d * es);      // always kept: every cross-attention block reads it
  for (int l = 0; l < c.n_dec_layers; ++l) {
    w->dec_self.push_back(attn_ws(Nd, Nd, Td, false));
    if (encdec) w->dec_cross.push_back(attn_ws(Nd, Ne, Td, true));
    w->dec_ffn.push_back(ffn_ws(Nd));
  }
  w->dec_x_final = (float*)take(Nd * d * 4);
  w->dec_ssq_f = take_ssq(Nd);
  w->dec_xg_f = take(Nd * d * es);
  w->logits = take(Nd * V * es);
  w->lse_tok = (float*)take(Nd * 4);
  w->enc_code = (int*)take(Ne * 4);
  w->dec_code = (int*)take(Nd * 4);
  w->dec_in = (int*)take(Nd * 4);
  w->dec_w = (float*)take(Nd * 4);
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

// Scratch buffers that a weight-gradient GEMM on the side stream reads and the main stream rewrites later
enum { BUF_DXB_DEC = 0, BUF_DXB_ENC, BUF_DH, BUF_DQKV, BUF_DKV, BUF_EMBED_GRAD, BUF_DY32, BUF_COUNT };

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
  int prefix;         // the batch carries prefix-LM flags (folded into the decoder's position codes)
  // Overlap: the weight-gradient GEMMs have no consumer before the end of the step, so they run on a second
  // stream and fill the SMs that the tails and launch gaps of the main stream's kernels leave idle.
  cudaStream_t side = nullptr;               // NULL: everything on the caller's stream
  cudaEvent_t reader[BUF_COUNT] = {};        // recorded on the side stream behind the last GEMM that reads the buffer
  bool reader_pending[BUF_COUNT] = {};
};

enum { CAT_GEMM = 0, CAT_ATTN_FWD, CAT_ATTN_BWD, CAT_NORM, CAT_GEGLU, CAT_XENT, CAT_EMBED, CAT_MISC };

// Records a start/stop event pair around the launches made while it is alive (profiling mode only).
struct ProfScope {
  Ctx& cx;
  int idx = -1;
  ProfScope(Ctx& c, int cat, double flops, int n_kernels, const char* what = "", int M = 0, int N = 0, int K = 0) : cx(c) {
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
    h->prof_rec.push_back({what, M, N, K});
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
      ProfScope ps_(cx, cat, 0.0, n, what);                       \
      cudaError_t e_ = (call);                                    \
      if (e_ != cudaSuccess) { cx.err = e_; cx.where = what; }    \
    }                                                             \
  } while (0)

cudaEvent_t next_sync_event(Ctx& cx) {
  t5_handle* h = cx.h;
  if (h->sync_events.size() < 64) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    h->sync_events.push_back(e);
    return e;
  }
  // reuse is safe: a wait refers to the record that preceded it, and 64 events span far more launches than are
  // ever in flight between a record and its wait
  return h->sync_events[h->sync_next++ % h->sync_events.size()];
}
// the side stream waits for everything enqueued on the main stream so far
void fork_to_side(Ctx& cx) {
  if (!cx.side || cx.err != cudaSuccess) return;
  cudaEvent_t e = next_sync_event(cx);
  if (!e) { cx.err = cudaErrorMemoryAllocation; cx.where = "sync event"; return; }
  CK(cudaEventRecord(e, cx.st), "fork record");
  CK(cudaStreamWaitEvent(cx.side, e, 0), "fork wait");
}
// a GEMM that reads scratch buffer `buf` has just been enqueued on the side stream
void mark_reader(Ctx& cx, int buf) {
  if (!cx.side || cx.err != cudaSuccess) return;
  if (!cx.reader[buf]) {
    cudaEvent_t& e = cx.h->reader_events[buf];
    if (!e && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) {
      e = nullptr;
      cx.err = cudaErrorMemoryAllocation; cx.where = "sync event";
      return;
    }
    cx.reader[buf] = e;
  }
  CK(cudaEventRecord(cx.reader[buf], cx.side), "reader record");
  cx.reader_pending[buf] = true;
}
// the main stream is about to rewrite `buf`: the side stream's reads of it must be done
void wait_readers(Ctx& cx, int buf) {
  if (!cx.side || !cx.reader_pending[buf] || cx.err != cudaSuccess) return;
  CK(cudaStreamWaitEvent(cx.st, cx.reader[buf], 0), "reader wait");
  cx.reader_pending[buf] = false;
}
// the main stream waits for all side-stream work (end of the call: the caller's stream then orders everything)
void join_side(Ctx& cx) {
  if (!cx.side) return;
  cudaEvent_t e = next_sync_event(cx);
  if (!e) return;
  cudaError_t r = cudaEventRecord(e, cx.side);
  if (r == cudaSuccess) r = cudaStreamWaitEvent(cx.st, e, 0);
  if (r != cudaSuccess && cx.err == cudaSuccess) { cx.err = r; cx.where = "join side stream"; }
}

void gemm(Ctx& cx, const GemmArgs& g0, const char* what, cudaStream_t st = nullptr) {
  int dt = cx.h->cfg.dtype;
  if (cx.err != cudaSuccess) return;
  if (!st) st = cx.st;
  GemmArgs g = g0;
  g.pair = ((cx.h->cfg.flags >> 2) & 1) ^ 1;      // CTA pairs unless flag bit 2 says otherwise
  if (g.out_f32 && cx.sk_next < kSkSlices) g.sk_flags = cx.w->sk_flags + (cx.sk_next++) * kSkSliceInts;
  ProfScope ps(cx, CAT_GEMM, 2.0 * g.M * g.N * g.K, 1, what, g.M, g.N, g.K);
  if (g.epi != 0 || (dt == DT_BF16 && !(cx.h->cfg.flags & 1) && gemm_tc_supported(g))) {
    CK(gemm_tc(g, cx.w->status, st), what);
  } else {
    CK(gemm_simt(dt, g, st), what);
  }
}

RowNorm row_norm(Ctx& cx, const float* ssq) {
  RowNorm r;
  r.ssq = ssq; r.inv_d = 1.f / (float)cx.h->cfg.d_model; r.eps = cx.h->cfg.rms_eps;
  return r;
}
const RowNorm kNoNorm = {nullptr, 0.f, 0.f};

// Y[M,N] = alpha (rn factor of the row) X[M,K] W[N,K]^T
void proj_fwd(Ctx& cx, const void* X, int ldx, int64_t w_off, int M, int N, int K, void* Y, int ldy, float alpha,
              RowNorm rn, const char* what, cudaStream_t st = nullptr) {
  GemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.alpha = alpha;
  g.A = X; g.lda = ldx; g.a_kmajor = 1;
  g.B = pptr(cx.h, cx.params, w_off); g.ldb = K; g.b_kmajor = 1;
  g.D = Y; g.ldd = ldy; g.out_f32 = 0; g.rn = rn;
  gemm(cx, g, what, st);
}
// Xout[M,N] = X[M,K] W[N,K]^T + resid (float32: the new residual rows); with nn also their operand copy
// Xout * g_next and sums of squares for the RMSNorm that reads them next
void proj_fwd_residual(Ctx& cx, const void* X, int ldx, int64_t w_off, int M, int N, int K, float* Xout,
                       const float* resid, const NextNorm* nn, const char* what) {
  GemmArgs g{};
  g.M = M; g.N = N; g.K = K; g.alpha = 1.f;
  g.A = X; g.lda = ldx; g.a_kmajor = 1;
  g.B = pptr(cx.h, cx.params, w_off); g.ldb = K; g.b_kmajor = 1;
  g.D = Xout; g.ldd = N; g.out_f32 = 1; g.resid = resid; g.ldr = N;
  if (nn) { g.xg_out = nn->xg; g.ld_xg = N; g.g_next = pptr(cx.h, cx.params, nn->g_off); g.ssq_out = nn->ssq; }
  gemm(cx, g, what);
}
// dX[M,K] = alpha dY[M,N] W[N,K]   (operand dtype out, or float32 with optional accumulate)
void proj_dgrad(Ctx& cx, const void* dY, int lddy, int64_t w_off, int M, int N, int K, void* dX, int lddx,
                float alpha, int out_f32, int accumulate, const char* what, cudaStream_t st = nullptr) {
  GemmArgs g{};
  g.M = M; g.N = K; g.K = N; g.alpha = alpha;
  g.A = dY; g.lda = lddy; g.a_kmajor = 1;
  g.B = pptr(cx.h, cx.params, w_off); g.ldb = K; g.b_kmajor = 0;
  g.D = dX; g.ldd = lddx; g.out_f32 = out_f32; g.accumulate = accumulate;
  gemm(cx, g, what, st);
}
// dW[N,K] = alpha dY[M,N]^T X[M,K]   (float32, overwrite).  Runs on the side stream when there is one; dY lives in
// scratch buffer `buf`, which the main stream must not rewrite before this GEMM has read it (wait_readers).
void proj_wgrad(Ctx& cx, const void* dY, int lddy, const void* X, int ldx, int64_t w_off, int M, int N, int K,
                float alpha, int buf, const char* what) {
  GemmArgs g{};
  g.M = N; g.N = K; g.K = M; g.alpha = alpha;
  g.A = dY; g.lda = lddy; g.a_kmajor = 0;
  g.B = X; g.ldb = ldx; g.b_kmajor = 0;
  g.D = cx.grads + w_off; g.ldd = K; g.out_f32 = 1; g.accumulate = 0;
  if (cx.side) {
    fork_to_side(cx);
    gemm(cx, g, what, cx.side);
    mark_reader(cx, buf);
  } else {
    gemm(cx, g, what);
  }
}

// |key - query| from which the bucket no longer changes (the top bucket of that direction)
int saturation_distance(const BucketSpec& s) { return s.n_thr > 0 ? s.thr[s.n_thr - 1] : s.me; }

struct AttnGeom {
  int prefix = 0;    // causal with a fully visible prefix (flag bit in the position codes)
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
  t = AttnArgs{};
  if (cross) {
    t.Q = a.q; t.ldq = I;
    t.K = a.kv; t.V = eoff(cx.h, a.kv, I); t.ldk = t.ldv = 2 * I;
  } else {
    t.Q = a.q; t.K = eoff(cx.h, a.q, I); t.V = eoff(cx.h, a.q, 2 * I); t.ldq = t.ldk = t.ldv = 3 * I;
  }
  t.O = a.ctx; t.ldo = I; t.lse = a.lse; t.O32 = a.ctx32; t.ldo32 = I;
  t.B = cx.B; t.H = c.n_heads; t.Tq = gm.Tq; t.Tk = gm.Tk; t.dk = c.d_kv;
  t.code_q = gm.code_q; t.code_k = gm.code_k; t.causal = gm.causal;
  t.bias_delta = gm.bias; t.scale = c.attn_scale; t.bias_far = gm.far;
  t.packed = cx.packed;
  t.prefix = gm.prefix;
}

// x_out = x + Attn(RMS(x)).  The norm is folded: the projections read a.xg = x * g and scale their rows by
// (a.ssq / d + eps)^-1/2.  Cross-attention: keys / values are projected from kv_src whose rows carry kv_rn.
// nn: where the output projection leaves the operand copy and statistics of x_out for the next norm.
// kv_done: the keys / values were projected on the side stream (cross_kv_forward); wait for that event instead.
void attn_forward(Ctx& cx, const AttnP& p, const AttnWs& a, float* x_out, const NextNorm& nn, const AttnGeom& gm,
                  const void* kv_src, RowNorm kv_rn, cudaEvent_t kv_done = nullptr) {
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, I = c.n_heads * c.d_kv, dt = c.dtype;
  bool cross = kv_src != nullptr;
  RowNorm rn = row_norm(cx, a.ssq);
  if (!cross) {
    proj_fwd(cx, a.xg, d, p.q, (int)gm.Nq, 3 * I, d, a.q, 3 * I, 1.f, rn, "qkv proj");
  } else {
    proj_fwd(cx, a.xg, d, p.q, (int)gm.Nq, I, d, a.q, I, 1.f, rn, "q proj");
    if (kv_done) CK(cudaStreamWaitEvent(cx.st, kv_done, 0), "wait for kv proj");
    else proj_fwd(cx, kv_src, d, p.k, (int)gm.Nk, 2 * I, d, a.kv, 2 * I, 1.f, kv_rn, "kv proj");
  }
  AttnArgs t;
  attn_args(cx, a, gm, cross, &t);
  if (dt == DT_BF16 && !(c.flags & 2) && attn_tc_supported(t))
    CKL(CAT_ATTN_FWD, 1, attn_fwd_tc(t, cx.w->status, cx.st), "attn_fwd (tcgen05)");
  else
    CKL(CAT_ATTN_FWD, 1, attn_fwd_simt(dt, t, cx.st), "attn_fwd");
  proj_fwd_residual(cx, a.ctx, I, p.o, (int)gm.Nq, d, I, x_out, a.x, &nn, "o proj");
}

// backward of the folded RMSNorm at the head of a sub-layer: w.dy holds t (see launch_rmsnorm_bwd)
void norm_backward(Ctx& cx, int64_t g_off, const float* x, const float* ssq, const void* t, int t_f32,
                   const float* dX_in, float* dX, void* dXb, int rows, const char* what) {
  const t5_config& c = cx.h->cfg;
  wait_readers(cx, dXb == cx.w->dXb_enc ? BUF_DXB_ENC : BUF_DXB_DEC);      // weight-gradient GEMMs still reading dXb
  CKL(CAT_NORM, 2, launch_rmsnorm_bwd(c.dtype, t, t_f32, x, row_norm(cx, ssq), pptr(cx.h, cx.params, g_off), dX_in, dX,
                                      dXb, cx.grads + g_off, cx.w->norm_partial, rows, c.d_model, cx.st),
      what);
}

// dX (in place) <- grad wrt sub-layer input; also refreshes dXb.  dY32: encoder-output gradient (cross only).
// The gradients of q, k, v leave the attention kernels with their rows multiplied by the RMSNorm factor of the
// projection that made them: that is what both the weight-gradient GEMM (against xg) and the data-gradient GEMM want.
void attn_backward(Ctx& cx, const AttnP& p, const AttnWs& a, float* dX, void* dXb, const AttnGeom& gm,
                   const void* kv_src, RowNorm kv_rn, float* dY32, int dY_accumulate) {
  const t5_config& c = cx.h->cfg;
  Workspace& w = *cx.w;
  int d = c.d_model, I = c.n_heads * c.d_kv, dt = c.dtype;
  bool cross = kv_src != nullptr;
  int Nq = (int)gm.Nq, Nk = (int)gm.Nk;
  const int buf_dxb = dXb == w.dXb_enc ? BUF_DXB_ENC : BUF_DXB_DEC;
  proj_wgrad(cx, dXb, d, a.ctx, I, p.o, Nq, d, I, 1.f, buf_dxb, "wgrad o");
  proj_dgrad(cx, dXb, d, p.o, Nq, d, I, w.dctx, I, 1.f, 0, 0, "dgrad o");
  AttnArgs t;
  attn_args(cx, a, gm, cross, &t);
  t.dO = w.dctx; t.lddo = I; t.delta = w.delta; t.dbias_delta = gm.dbias; t.bias_far = gm.far;
  t.ds_scratch = w.ds_scratch; t.ds_bytes = w.ds_bytes;
  t.rn_q = row_norm(cx, a.ssq);
  t.rn_k = cross ? kv_rn : t.rn_q;
  if (cross) {
    t.dQ = w.dqkv; t.lddq = I;
    t.dK = w.dkv; t.dV = eoff(cx.h, w.dkv, I); t.lddk = t.lddv = 2 * I;
  } else {
    t.dQ = w.dqkv; t.dK = eoff(cx.h, w.dqkv, I); t.dV = eoff(cx.h, w.dqkv, 2 * I);
    t.lddq = t.lddk = t.lddv = 3 * I;
  }
  wait_readers(cx, BUF_DQKV);
  if (cross) wait_readers(cx, BUF_DKV);
  if (dt == DT_BF16 && !(c.flags & 2) && attn_tc_supported(t))
    CKL(CAT_ATTN_BWD, 3, attn_bwd_tc(t, cx.w->status, cx.st), "attn_bwd (tcgen05)");
  else
    CKL(CAT_ATTN_BWD, 3, attn_bwd_simt(dt, t, cx.st), "attn_bwd");
  if (c.recompute == 1)
    CKL(CAT_NORM, 1, launch_scale_cols(dt, a.x, pptr(cx.h, cx.params, p.norm), a.xg, Nq, d, cx.st), "x * g (recomputed)");
  if (!cross) {
    proj_wgrad(cx, w.dqkv, 3 * I, a.xg, d, p.q, Nq, 3 * I, d, 1.f, BUF_DQKV, "wgrad qkv");
    proj_dgrad(cx, w.dqkv, 3 * I, p.q, Nq, 3 * I, d, w.dy, d, 1.f, 0, 0, "dgrad qkv");
  } else {
    proj_wgrad(cx, w.dqkv, I, a.xg, d, p.q, Nq, I, d, 1.f, BUF_DQKV, "wgrad q");
    proj_dgrad(cx, w.dqkv, I, p.q, Nq, I, d, w.dy, d, 1.f, 0, 0, "dgrad q");
    proj_wgrad(cx, w.dkv, 2 * I, kv_src, d, p.k, Nk, 2 * I, d, 1.f, BUF_DKV, "wgrad kv");
    // the encoder-output gradient has no reader before the decoder's backward pass is over: side stream as well
    // (its launches there run in order, so the accumulation over the layers stays sequential)
    proj_dgrad(cx, w.dkv, 2 * I, p.k, Nk, 2 * I, d, dY32, d, 1.f, 1, dY_accumulate, "dgrad kv", cx.side);
    if (cx.side) { mark_reader(cx, BUF_DKV); mark_reader(cx, BUF_DY32); }
  }
  norm_backward(cx, p.norm, a.x, a.ssq, w.dy, 0, dX, dX, dXb, Nq, "rmsnorm_bwd");
}

// the gated-GELU epilogues run in the tensor-core GEMM on CTA pairs; flags bit 3 keeps the separate kernels
bool fused_geglu_ok(Ctx& cx, GemmArgs& g) {
  const t5_config& c = cx.h->cfg;
  if (c.dtype != DT_BF16 || (c.flags & (1 | 4 | 8)) || c.ffn_act != 0) return false;
  // measured with the eight-warp epilogue: the fusion wins at every width the tensor-core path takes (small,
  // d_model 512: 19.3 -> 18.4 ms per step; base, 768: 87.0 -> 84.8 ms); below that the contraction is too short
  if (c.d_model < 512) return false;
  g.pair = 1;
  return gemm_tc_supported(g) && gemm_tc_epi_supported(g);
}

void ffn_forward(Ctx& cx, const FfnP& p, const FfnWs& f, float* x_out, const NextNorm& nn, int64_t N) {
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, F = c.d_ff, dt = c.dtype;
  RowNorm rn = row_norm(cx, f.ssq);
  GemmArgs gf{};
  gf.M = (int)N; gf.N = 2 * F; gf.K = d; gf.alpha = 1.f;
  gf.A = f.xg; gf.lda = d; gf.a_kmajor = 1;
  gf.B = pptr(cx.h, cx.params, p.wi0); gf.ldb = d; gf.b_kmajor = 1;
  gf.D = f.h; gf.ldd = 2 * F; gf.epi = 1; gf.aux = f.hg; gf.ld_aux = F; gf.F = F; gf.rn = rn;
  if (fused_geglu_ok(cx, gf)) {
    gemm(cx, gf, "wi proj + gated GELU");
  } else {
    const int Fh = c.ffn_act == 1 ? F : 2 * F;      // the ReLU FFN has one input matrix
    proj_fwd(cx, f.xg, d, p.wi0, (int)N, Fh, d, f.h, Fh, 1.f, rn, "wi proj");
    CKL(CAT_GEGLU, 1, launch_geglu_fwd(dt, c.ffn_act, f.h, f.hg, (int)N, F, cx.st), "ffn activation");
  }
  proj_fwd_residual(cx, f.hg, F, p.wo, (int)N, d, F, x_out, f.x, &nn, "wo proj");
}

void ffn_backward(Ctx& cx, const FfnP& p, const FfnWs& f, float* dX, void* dXb, int64_t N) {
  const t5_config& c = cx.h->cfg;
  Workspace& w = *cx.w;
  int d = c.d_model, F = c.d_ff, dt = c.dtype, n = (int)N;
  RowNorm rn = row_norm(cx, f.ssq);
  if (c.recompute == 1)
    CKL(CAT_GEGLU, 1, launch_geglu_fwd(dt, c.ffn_act, f.h, f.hg, n, F, cx.st), "ffn activation (recomputed)");
  const int Fh = c.ffn_act == 1 ? F : 2 * F;
  proj_wgrad(cx, dXb, d, f.hg, F, p.wo, n, d, F, 1.f, dXb == w.dXb_enc ? BUF_DXB_ENC : BUF_DXB_DEC, "wgrad ffn.wo");
  wait_readers(cx, BUF_DH);      // the previous sub-layer's weight-gradient GEMM may still read dh
  // dh = [da | db] leaves with its rows multiplied by the RMSNorm factor (see attn_backward)
  GemmArgs gb{};
  gb.M = n; gb.N = F; gb.K = d; gb.alpha = 1.f;
  gb.A = dXb; gb.lda = d; gb.a_kmajor = 1;
  gb.B = pptr(cx.h, cx.params, p.wo); gb.ldb = F; gb.b_kmajor = 0;
  gb.D = w.dh; gb.ldd = 2 * F; gb.epi = 2; gb.aux = f.h; gb.ld_aux = 2 * F; gb.F = F; gb.rn = rn;
  if (fused_geglu_ok(cx, gb)) {
    gemm(cx, gb, "dgrad ffn.wo + gated GELU backward");
  } else {
    proj_dgrad(cx, dXb, d, p.wo, n, d, F, w.dhg, F, 1.f, 0, 0, "dgrad ffn.wo");
    CKL(CAT_GEGLU, 1, launch_geglu_bwd(dt, c.ffn_act, w.dhg, f.h, w.dh, n, F, rn, cx.st), "ffn activation backward");
  }
  if (c.recompute == 1)
    CKL(CAT_NORM, 1, launch_scale_cols(dt, f.x, pptr(cx.h, cx.params, p.norm), f.xg, n, d, cx.st), "x * g (recomputed)");
  proj_wgrad(cx, w.dh, Fh, f.xg, d, p.wi0, n, Fh, d, 1.f, BUF_DH, "wgrad ffn.wi");
  proj_dgrad(cx, w.dh, Fh, p.wi0, n, Fh, d, w.dy, d, 1.f, 0, 0, "dgrad ffn.wi");
  norm_backward(cx, p.norm, f.x, f.ssq, w.dy, 0, dX, dX, dXb, n, "rmsnorm_bwd");
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
  g.prefix = cx.prefix;
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
  CK(cudaMemsetAsync(w.ssq_all, 0, w.ssq_floats * 4, cx.st), "memset row statistics");
  CKL(CAT_MISC, 2, launch_prep(c.arch == 0 ? b->d_enc_tokens : nullptr, b->d_enc_segment_ids, b->d_dec_targets,
                 b->d_dec_segment_ids, b->d_dec_prefix, cx.B, cx.Te, cx.Td, w.enc_code, w.dec_code, w.dec_in, w.dec_w,
                 w.W_int, w.W_f, cx.st),
     "prep");
  if (c.arch == 0 && cx.Te > 0)
    CKL(CAT_MISC, 1, launch_relbias_expand(c.dtype, cx.h->spec_enc, pptr(cx.h, cx.params, cx.h->enc_relbias), c.n_heads, cx.Te,
                             cx.Te, w.bias_enc, cx.st),
       "relbias_expand enc");
  CKL(CAT_MISC, 1, launch_relbias_expand(c.dtype, cx.h->spec_dec, pptr(cx.h, cx.params, cx.h->dec_relbias), c.n_heads, cx.Td,
                           cx.Td, w.bias_dec, cx.st),
     "relbias_expand dec");
}

// The norm that reads the residual block in front of encoder sub-layer (l, which): its operand copy, statistics, scale
NextNorm enc_norm_at(Ctx& cx, int l, int which) {      // which: 0 attention, 1 FFN; l == n_enc_layers: final norm
  Workspace& w = *cx.w;
  if (l >= cx.h->cfg.n_enc_layers) return {w.enc_xg_f, w.enc_ssq_f, cx.h->enc_final_norm};
  if (which == 0) return {w.enc_attn[l].xg, w.enc_attn[l].ssq, cx.h->enc[l].attn.norm};
  return {w.enc_ffn[l].xg, w.enc_ffn[l].ssq, cx.h->enc[l].ffn.norm};
}
NextNorm dec_norm_at(Ctx& cx, int l, int which) {      // which: 0 self, 1 cross, 2 FFN
  Workspace& w = *cx.w;
  if (l >= cx.h->cfg.n_dec_layers) return {w.dec_xg_f, w.dec_ssq_f, cx.h->dec_final_norm};
  if (which == 0) return {w.dec_self[l].xg, w.dec_self[l].ssq, cx.h->dec[l].self.norm};
  if (which == 1) return {w.dec_cross[l].xg, w.dec_cross[l].ssq, cx.h->dec[l].cross.norm};
  return {w.dec_ffn[l].xg, w.dec_ffn[l].ssq, cx.h->dec[l].ffn.norm};
}

void encoder_forward(Ctx& cx, const t5_batch* b) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int L = c.n_enc_layers, d = c.d_model;
  int64_t Ne = (int64_t)cx.B * cx.Te;
  float* x0 = L > 0 ? w.enc_attn[0].x : w.enc_x_final;
  NextNorm n0 = enc_norm_at(cx, 0, 0);
  CKL(CAT_EMBED, 1, launch_embed_gather(c.dtype, pptr(cx.h, cx.params, cx.h->token_embed), b->d_enc_tokens, x0,
                                        pptr(cx.h, cx.params, n0.g_off), n0.xg, n0.ssq, (int)Ne, d, cx.st),
     "embed enc");
  AttnGeom g = enc_geom(cx);
  for (int l = 0; l < L; ++l) {
    attn_forward(cx, cx.h->enc[l].attn, w.enc_attn[l], w.enc_ffn[l].x, enc_norm_at(cx, l, 1), g, nullptr, kNoNorm);
    float* x_next = l + 1 < L ? w.enc_attn[l + 1].x : w.enc_x_final;
    ffn_forward(cx, cx.h->enc[l].ffn, w.enc_ffn[l], x_next, enc_norm_at(cx, l + 1, 0), Ne);
  }
}

// enc_src: what the cross-attention projects keys and values from - the folded encoder output (enc_xg_f with the
// final norm's statistics) inside a training step, or a caller's normed encoder output (no factor); NULL for
// decoder-only.  logits_out: where the logits go.
void decoder_forward(Ctx& cx, const void* enc_src, RowNorm enc_rn, void* logits_out) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int L = c.n_dec_layers, d = c.d_model;
  int64_t Nd = (int64_t)cx.B * cx.Td;
  float* x0 = L > 0 ? w.dec_self[0].x : w.dec_x_final;
  NextNorm n0 = dec_norm_at(cx, 0, 0);
  CKL(CAT_EMBED, 1, launch_embed_gather(c.dtype, pptr(cx.h, cx.params, cx.h->token_embed), w.dec_in, x0,
                                        pptr(cx.h, cx.params, n0.g_off), n0.xg, n0.ssq, (int)Nd, d, cx.st),
     "embed dec");
  AttnGeom gs = self_geom(cx), gc = cross_geom(cx);
  bool encdec = c.arch == 0;
  // The keys / values of every cross-attention block depend on the encoder output only: with a side stream all
  // layers' projections go there at once (large GEMMs that fill the SMs the decoder's small kernels leave idle),
  // and each cross-attention block waits for its own.
  bool kv_ahead = encdec && cx.side != nullptr && cx.err == cudaSuccess;
  if (kv_ahead) {
    t5_handle* h = cx.h;
    while ((int)h->layer_events.size() < L && kv_ahead) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) kv_ahead = false;
      else h->layer_events.push_back(e);
    }
  }
  if (kv_ahead) {
    const int I = c.n_heads * c.d_kv;
    fork_to_side(cx);
    for (int l = 0; l < L; ++l) {
      proj_fwd(cx, enc_src, d, cx.h->dec[l].cross.k, (int)gc.Nk, 2 * I, d, w.dec_cross[l].kv, 2 * I, 1.f, enc_rn, "kv proj",
               cx.side);
      CK(cudaEventRecord(cx.h->layer_events[l], cx.side), "kv proj record");
    }
  }
  for (int l = 0; l < L; ++l) {
    float* after_self = encdec ? w.dec_cross[l].x : w.dec_ffn[l].x;
    attn_forward(cx, cx.h->dec[l].self, w.dec_self[l], after_self, dec_norm_at(cx, l, encdec ? 1 : 2), gs, nullptr, kNoNorm);
    if (encdec)
      attn_forward(cx, cx.h->dec[l].cross, w.dec_cross[l], w.dec_ffn[l].x, dec_norm_at(cx, l, 2), gc, enc_src, enc_rn,
                   kv_ahead ? cx.h->layer_events[l] : nullptr);
    float* x_next = l + 1 < L ? w.dec_self[l + 1].x : w.dec_x_final;
    ffn_forward(cx, cx.h->dec[l].ffn, w.dec_ffn[l], x_next, dec_norm_at(cx, l + 1, 0), Nd);
  }
  // logits = logit_scale RMS(x) E^T: the final norm is folded like the others
  const int64_t head = cx.h->lm_head >= 0 ? cx.h->lm_head : cx.h->token_embed;
  proj_fwd(cx, w.dec_xg_f, d, head, (int)Nd, c.vocab, d, logits_out, c.vocab, c.logit_scale,
           row_norm(cx, w.dec_ssq_f), "logits");
}

// Elements [begin, end) of the gradient buffer are final once the work enqueued so far is done: tell the caller's
// hook, with a stream that follows all of that work (the side stream, made to wait for the main stream first, when
// the weight-gradient GEMMs run there; else the caller's own stream).
void grads_ready(Ctx& cx, int64_t begin, int64_t end) {
  if (!cx.h->grad_hook || cx.err != cudaSuccess || end <= begin) return;
  cudaStream_t s = cx.st;
  if (cx.side) {
    fork_to_side(cx);
    s = cx.side;
  }
  if (cx.err == cudaSuccess) cx.h->grad_hook(cx.h->grad_hook_user, begin, end - begin, cx.w->W_f, (void*)s);
}

void backward(Ctx& cx, const t5_batch* b) {
  Workspace& w = *cx.w;
  const t5_config& c = cx.h->cfg;
  int d = c.d_model, V = c.vocab, H = c.n_heads;
  int64_t Nd = (int64_t)cx.B * cx.Td, Ne = (int64_t)cx.B * cx.Te;
  bool encdec = c.arch == 0;
  for (auto& gp : cx.h->gaps)
    CK(cudaMemsetAsync(cx.grads + gp.first, 0, (gp.second - gp.first) * 4, cx.st), "memset gaps");
  if (encdec && cx.Te > 0) CK(cudaMemsetAsync(w.dbias_enc, 0, (int64_t)H * (2 * cx.Te - 1) * 4, cx.st), "memset dbias");
  CK(cudaMemsetAsync(w.dbias_dec, 0, (int64_t)H * (2 * cx.Td - 1) * 4, cx.st), "memset dbias");
  // tied embedding (w.logits holds dlogits with the final norm's row factors): dE = logit_scale dlogits^T xg
  // (overwrites), t = logit_scale dlogits E
  const int64_t head = cx.h->lm_head >= 0 ? cx.h->lm_head : cx.h->token_embed;
  if (cx.h->lm_head >= 0)      // separate head: the embedding gradient only collects the gathered rows
    CK(cudaMemsetAsync(cx.grads + cx.h->token_embed, 0, (int64_t)V * d * 4, cx.st), "memset embedding gradient");
  proj_wgrad(cx, w.logits, V, w.dec_xg_f, d, head, (int)Nd, V, d, c.logit_scale, BUF_EMBED_GRAD, "wgrad logits");
  proj_dgrad(cx, w.logits, V, head, (int)Nd, V, d, w.dy, d, c.logit_scale, 0, 0, "dgrad logits");
  norm_backward(cx, cx.h->dec_final_norm, w.dec_x_final, w.dec_ssq_f, w.dy, 0, nullptr, w.dX_dec, w.dXb_dec, (int)Nd,
                "dec final norm bwd");
  AttnGeom gs = self_geom(cx), gc = cross_geom(cx);
  RowNorm enc_rn = row_norm(cx, w.enc_ssq_f);
  bool first_cross = true;
  for (int l = c.n_dec_layers - 1; l >= 0; --l) {
    ffn_backward(cx, cx.h->dec[l].ffn, w.dec_ffn[l], w.dX_dec, w.dXb_dec, Nd);
    if (encdec) {
      attn_backward(cx, cx.h->dec[l].cross, w.dec_cross[l], w.dX_dec, w.dXb_dec, gc, w.enc_xg_f, enc_rn, w.dY32,
                    first_cross ? 0 : 1);
      first_cross = false;
    }
    attn_backward(cx, cx.h->dec[l].self, w.dec_self[l], w.dX_dec, w.dXb_dec, gs, nullptr, kNoNorm, nullptr, 0);
    grads_ready(cx, cx.h->dec[l].self.norm, l + 1 < c.n_dec_layers ? cx.h->dec[l + 1].self.norm : cx.h->dec_final_norm);
  }
  wait_readers(cx, BUF_EMBED_GRAD);      // the embedding gradient must hold the logits' share before rows are added to it
  CKL(CAT_EMBED, 1, launch_embed_scatter_add(w.dec_in, w.dX_dec, cx.grads + cx.h->token_embed, (int)Nd, d, cx.st),
     "embed scatter dec");
  CKL(CAT_MISC, 1, launch_relbias_fold(cx.h->spec_dec, w.dbias_dec, H, cx.Td, cx.Td, c.rel_buckets, cx.grads + cx.h->dec_relbias,
                         cx.st),
     "relbias fold dec");
  if (!encdec) {
    grads_ready(cx, 0, cx.h->dec[0].self.norm);                       // embedding, bias table
    grads_ready(cx, cx.h->dec_final_norm, cx.h->n_params);            // final norm, separate output head
    return;
  }
  wait_readers(cx, BUF_DY32);      // the encoder-output gradient is complete
  norm_backward(cx, cx.h->enc_final_norm, w.enc_x_final, w.enc_ssq_f, w.dY32, 1, nullptr, w.dX_enc, w.dXb_enc, (int)Ne,
                "enc final norm bwd");
  AttnGeom ge = enc_geom(cx);
  for (int l = c.n_enc_layers - 1; l >= 0; --l) {
    ffn_backward(cx, cx.h->enc[l].ffn, w.enc_ffn[l], w.dX_enc, w.dXb_enc, Ne);
    attn_backward(cx, cx.h->enc[l].attn, w.enc_attn[l], w.dX_enc, w.dXb_enc, ge, nullptr, kNoNorm, nullptr, 0);
    grads_ready(cx, cx.h->enc[l].attn.norm, l + 1 < c.n_enc_layers ? cx.h->enc[l + 1].attn.norm : cx.h->enc_final_norm);
  }
  CKL(CAT_EMBED, 1, launch_embed_scatter_add(b->d_enc_tokens, w.dX_enc, cx.grads + cx.h->token_embed, (int)Ne, d, cx.st),
     "embed scatter enc");
  CKL(CAT_MISC, 1, launch_relbias_fold(cx.h->spec_enc, w.dbias_enc, H, cx.Te, cx.Te, c.rel_buckets, cx.grads + cx.h->enc_relbias,
                         cx.st),
     "relbias fold enc");
  grads_ready(cx, cx.h->dec_final_norm, cx.h->n_params);              // decoder final norm, separate output head
  grads_ready(cx, cx.h->enc_final_norm, cx.h->dec[0].self.norm);      // encoder final norm, decoder bias table
  grads_ready(cx, 0, cx.h->enc[0].attn.norm);                         // embedding, encoder bias table
}

// ---- incremental decoding: the caller's cache buffer holds, per decoder layer, the self-attention keys / values of the
// positions decoded so far and (encoder-decoder) the cross-attention keys / values of the encoder output
struct DecodeCache {
  std::vector<void*> self_kv;      // [B, Tmax, 2I] per layer (k | v)
  std::vector<void*> cross_kv;     // [B, Te, 2I] per layer
  int *self_code, *enc_code, *ones, *status;      // [B, Tmax] (1 = decoded), [B, Te], [B], [1]
  float* bias_step;                // [H, Tmax] bias of key j for the query at the current position
  int64_t bytes;
};
void plan_cache(const t5_handle* h, int B, int Te, int Tmax, char* base, DecodeCache* k) {
  const t5_config& c = h->cfg;
  int64_t cur = 0;
  auto take = [&](int64_t bytes) -> void* {
    int64_t at = cur;
    cur += (bytes + 255) / 256 * 256;
    return base ? (void*)(base + at) : nullptr;
  };
  const int64_t es = (int64_t)esize(h), I = (int64_t)c.n_heads * c.d_kv;
  if (c.arch != 0) Te = 0;
  k->status = (int*)take(4);
  k->self_kv.clear(); k->cross_kv.clear();
  for (int l = 0; l < c.n_dec_layers; ++l) {
    k->self_kv.push_back(take((int64_t)B * Tmax * 2 * I * es));
    k->cross_kv.push_back(take((int64_t)B * Te * 2 * I * es));
  }
  k->self_code = (int*)take((int64_t)B * Tmax * 4);
  k->enc_code = (int*)take((int64_t)B * Te * 4);
  k->ones = (int*)take((int64_t)B * 4);
  k->bias_step = (float*)take((int64_t)c.n_heads * Tmax * 4);
  k->bytes = cur;
}

// One decoder sub-layer of attention for a single new position per row: queries from the new row, keys / values
// from the cache (self-attention appends the new row's k, v first).
void attn_step(Ctx& cx, const AttnP& p, const AttnWs& a, float* x_out, const NextNorm& nn, void* kv_cache, int Tk,
               const int* code_k, const float* bias, const int* ones, bool self, int t, int Tmax) {
  const t5_config& c = cx.h->cfg;
  const int d = c.d_model, I = c.n_heads * c.d_kv, dt = c.dtype, B = cx.B;
  const int64_t es = (int64_t)esize(cx.h);
  RowNorm rn = row_norm(cx, a.ssq);
  if (self) {
    proj_fwd(cx, a.xg, d, p.q, B, 3 * I, d, a.q, 3 * I, 1.f, rn, "qkv proj (step)");
    // row b of [k | v] goes to position t of row b's cache
    CK(cudaMemcpy2DAsync((char*)kv_cache + (int64_t)t * 2 * I * es, (size_t)Tmax * 2 * I * es, (const char*)a.q + I * es,
                         (size_t)3 * I * es, (size_t)2 * I * es, B, cudaMemcpyDeviceToDevice, cx.st),
       "append k, v to the cache");
  } else {
    proj_fwd(cx, a.xg, d, p.q, B, I, d, a.q, I, 1.f, rn, "q proj (step)");
  }
  AttnArgs ta{};
  ta.Q = a.q; ta.ldq = self ? 3 * I : I;
  ta.K = kv_cache; ta.V = eoff(cx.h, kv_cache, I); ta.ldk = ta.ldv = 2 * I;
  ta.O = a.ctx; ta.ldo = I; ta.lse = a.lse; ta.O32 = a.ctx32; ta.ldo32 = I;
  ta.B = B; ta.H = c.n_heads; ta.Tq = 1; ta.Tk = Tk; ta.dk = c.d_kv;
  ta.code_q = ones; ta.code_k = code_k; ta.causal = 0;      // the cache holds no later position: no causal test needed
  ta.bias_delta = bias; ta.scale = c.attn_scale; ta.packed = 1;
  if (dt == DT_BF16 && !(c.flags & 2) && attn_tc_supported(ta))
    CKL(CAT_ATTN_FWD, 1, attn_fwd_tc(ta, cx.w->status, cx.st), "attn step (tcgen05)");
  else
    CKL(CAT_ATTN_FWD, 1, attn_fwd_simt(dt, ta, cx.st), "attn step");
  proj_fwd_residual(cx, a.ctx, I, p.o, B, d, I, x_out, a.x, &nn, "o proj (step)");
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
  cx->prefix = b->d_dec_prefix != nullptr ? 1 : 0;
  cx->side = nullptr;
  for (int i = 0; i < BUF_COUNT; ++i) { cx->reader[i] = nullptr; cx->reader_pending[i] = false; }
  return T5_OK;
}

// The side stream of the handle for the current device (created on first use); NULL if overlap is off for this call
// (activation policy 1 rewrites the buffers the weight-gradient GEMMs read; the per-launch timing mode wants one
// kernel at a time; flags bit 4 switches it off).
cudaStream_t side_stream_for_call(t5_handle* h) {
  const t5_config& c = h->cfg;
  if (c.recompute != 0 || h->prof_on || (c.flags & 16)) return nullptr;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return nullptr;
  if (h->side && h->side_dev != dev) {
    cudaStreamDestroy(h->side);
    h->side = nullptr;
  }
  if (!h->side) {
    if (cudaStreamCreateWithFlags(&h->side, cudaStreamNonBlocking) != cudaSuccess) { h->side = nullptr; return nullptr; }
    h->side_dev = dev;
  }
  return h->side;
}

int end_call(t5_handle* h, Ctx& cx) {
  join_side(cx);
  h->launches_last_call = cx.launches;
  if (cx.err != cudaSuccess)
    return fail(h, T5_ERR_CUDA, "%s: %s", cx.where, cudaGetErrorString(cx.err));
  return T5_OK;
}

}  // namespace

// =============================================================================== C ABI
// Status word of the kernel-level entry points below (t5_attention, t5_attention_backward_onepass, t5_gemm and the
// allocation-free attention backward): they have no workspace whose first word could serve.  NULL: no reporting.
int32_t* g_kernel_status = nullptr;

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
  if (c.ffn_act < 0 || c.ffn_act > 2) return fail(nullptr, T5_ERR_CONFIG, "ffn_act must be 0, 1 or 2");
  if (c.untied_head != 0 && c.untied_head != 1) return fail(nullptr, T5_ERR_CONFIG, "untied_head must be 0 or 1");
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
  if (h) {
    for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
    for (cudaEvent_t e : h->sync_events) cudaEventDestroy(e);
    for (cudaEvent_t e : h->reader_events)
      if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : h->layer_events) cudaEventDestroy(e);
    if (h->side) cudaStreamDestroy(h->side);
  }
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

int t5_adamw_update(t5_handle* h, void* d_params, float* d_master, float* d_m, float* d_v, const float* d_grads,
                    int64_t step, float lr, float beta1, float beta2, float eps, float weight_decay, float grad_scale,
                    void* stream) {
  if (!h) return T5_ERR_NULL;
  if (!d_params || !d_master || !d_m || !d_v || !d_grads) return fail(h, T5_ERR_NULL, "null optimizer buffer");
  if (!aligned16(d_params) || !aligned16(d_master) || !aligned16(d_m) || !aligned16(d_v) || !aligned16(d_grads))
    return fail(h, T5_ERR_ALIGN, "optimizer buffers must be 16-byte aligned");
  if (step < 1 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f))
    return fail(h, T5_ERR_ARG, "adamw: need step >= 1, 0 <= beta < 1, eps > 0");
  const float bc1 = 1.f - (float)pow((double)beta1, (double)step), bc2 = 1.f - (float)pow((double)beta2, (double)step);
  // runs of consecutive tensors with the same decay class (matrices decay, 1-D norm scales do not); the padding
  // between tensors rides along (its gradient is zero)
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaSuccess;
  size_t i = 0;
  const size_t nt = h->tensors.size();
  while (i < nt && e == cudaSuccess) {
    const bool decay = h->tensors[i].ndim > 1;
    size_t j = i;
    while (j + 1 < nt && (h->tensors[j + 1].ndim > 1) == decay) ++j;
    const int64_t lo = h->tensors[i].offset, hi = j + 1 < nt ? h->tensors[j + 1].offset : h->n_params;
    e = launch_adamw(h->cfg.dtype, eoff(h, d_params, lo), d_master + lo, d_m + lo, d_v + lo, d_grads + lo, hi - lo, lr, beta1,
                     beta2, eps, decay ? weight_decay : 0.f, grad_scale, bc1, bc2, st);
    i = j + 1;
  }
  if (e != cudaSuccess) return fail(h, T5_ERR_CUDA, "adamw: %s", cudaGetErrorString(e));
  return T5_OK;
}

int t5_set_grad_hook(t5_handle* h, t5_grad_ready_fn fn, void* user) {
  if (!h) return T5_ERR_NULL;
  h->grad_hook = fn;
  h->grad_hook_user = user;
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
  cx.side = side_stream_for_call(h);
  run_prep(cx, batch);
  if (c.arch == 0) encoder_forward(cx, batch);
  decoder_forward(cx, c.arch == 0 ? w.enc_xg_f : nullptr, row_norm(cx, w.enc_ssq_f), w.logits);
  CK(cudaMemsetAsync(w.sums, 0, 16, cx.st), "memset sums");
  // dlogits overwrite the logits, rows already multiplied by the final norm's factor (see backward())
  CKL(CAT_XENT, 1, launch_xent(c.dtype, w.logits, batch->d_dec_targets, w.dec_w, cx.B * cx.Td, c.vocab, c.z_loss, w.W_f, w.sums,
                 w.lse_tok, row_norm(cx, w.dec_ssq_f), cx.st),
     "xent");
  CKL(CAT_MISC, 1, launch_finalize_loss(w.sums, w.W_f, d_loss4, cx.st), "finalize loss");
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
  if (!aligned16(d_enc_out)) return fail(h, T5_ERR_ALIGN, "encoder output not 16-byte aligned");
  run_prep(cx, batch);
  encoder_forward(cx, batch);
  // the call's result is the normed output itself: one explicit RMSNorm pass over the final residual rows
  CKL(CAT_NORM, 1, launch_rmsnorm_fwd(h->cfg.dtype, w.enc_x_final, pptr(h, d_params, h->enc_final_norm), d_enc_out, nullptr,
                                      cx.B * cx.Te, h->cfg.d_model, h->cfg.rms_eps, cx.st),
      "enc final norm");
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
  decoder_forward(cx, h->cfg.arch == 0 ? d_enc_out : nullptr, kNoNorm, d_logits);
  return end_call(h, cx);
}

int t5_decode_cache_bytes(const t5_handle* h, int32_t B, int32_t Te, int32_t Tmax, int64_t* bytes) {
  if (!h || !bytes) return T5_ERR_NULL;
  if (B < 1 || Tmax < 1 || (h->cfg.arch == 0 && Te < 1)) return T5_ERR_ARG;
  DecodeCache k;
  plan_cache(h, B, Te, Tmax, nullptr, &k);
  *bytes = k.bytes;
  return T5_OK;
}

int t5_decode_begin(t5_handle* h, const void* d_params, int32_t B, int32_t Te, int32_t Tmax, const int32_t* d_enc_tokens,
                    const void* d_enc_out, void* d_cache, int64_t cache_bytes, void* stream) {
  if (!h) return T5_ERR_NULL;
  const t5_config& c = h->cfg;
  const bool encdec = c.arch == 0;
  if (!d_params || !d_cache || (encdec && (!d_enc_tokens || !d_enc_out))) return fail(h, T5_ERR_NULL, "null pointer");
  if (B < 1 || B > c.max_batch || Tmax < 1 || Tmax > c.max_dec_len || (encdec && (Te < 1 || Te > c.max_enc_len)))
    return fail(h, T5_ERR_SHAPE, "decode_begin: %d rows, %d encoder / %d decoder positions outside the configured maxima", B, Te,
                Tmax);
  if (!aligned16(d_params) || !aligned16(d_cache) || (encdec && !aligned16(d_enc_out)))
    return fail(h, T5_ERR_ALIGN, "params / cache / encoder output not 16-byte aligned");
  DecodeCache k;
  plan_cache(h, B, Te, Tmax, (char*)d_cache, &k);
  if (k.bytes > cache_bytes)
    return fail(h, T5_ERR_WORKSPACE, "cache of %lld bytes given, %lld needed", (long long)cache_bytes, (long long)k.bytes);
  Workspace w{};
  w.status = k.status;
  Ctx cx{};
  cx.h = h; cx.params = d_params; cx.st = (cudaStream_t)stream; cx.w = &w; cx.B = B; cx.Te = encdec ? Te : 0; cx.Td = 1;
  cx.err = cudaSuccess; cx.where = ""; cx.sk_next = kSkSlices;      // no stream-K flags in this call
  CK(cudaMemsetAsync(k.status, 0, 4, cx.st), "memset status");
  CK(cudaMemsetAsync(k.self_code, 0, (int64_t)B * Tmax * 4, cx.st), "memset cache codes");
  // positions not decoded yet are masked out of the softmax, but their value rows still enter P V with weight 0:
  // they must hold finite numbers
  for (int l = 0; l < c.n_dec_layers; ++l)
    CK(cudaMemsetAsync(k.self_kv[l], 0, (int64_t)B * Tmax * 2 * c.n_heads * c.d_kv * (int64_t)esize(h), cx.st), "memset cache");
  CK(launch_set_column(k.ones, 1, 0, B, 1, cx.st), "ones");
  if (encdec) {
    const int d = c.d_model, I = c.n_heads * c.d_kv;
    CK(launch_pad_codes(d_enc_tokens, k.enc_code, B * Te, cx.st), "encoder key codes");
    for (int l = 0; l < c.n_dec_layers; ++l)
      proj_fwd(cx, d_enc_out, d, h->dec[l].cross.k, B * Te, 2 * I, d, k.cross_kv[l], 2 * I, 1.f, kNoNorm, "kv proj (cache)");
  }
  return end_call(h, cx);
}

int t5_decode_step(t5_handle* h, const void* d_params, void* d_cache, int64_t cache_bytes, int32_t B, int32_t Te,
                   int32_t Tmax, int32_t t, const int32_t* d_tokens, void* d_logits, void* d_workspace,
                   int64_t workspace_bytes, void* stream) {
  if (!h) return T5_ERR_NULL;
  const t5_config& c = h->cfg;
  const bool encdec = c.arch == 0;
  if (!d_params || !d_cache || !d_tokens || !d_logits || !d_workspace) return fail(h, T5_ERR_NULL, "null pointer");
  if (B < 1 || B > c.max_batch || Tmax < 1 || Tmax > c.max_dec_len || t < 0 || t >= Tmax ||
      (encdec && (Te < 1 || Te > c.max_enc_len)))
    return fail(h, T5_ERR_SHAPE, "decode_step: position %d of %d, %d rows, %d encoder positions out of range", t, Tmax, B, Te);
  if (!aligned16(d_params) || !aligned16(d_cache) || !aligned16(d_logits) || !aligned16(d_workspace))
    return fail(h, T5_ERR_ALIGN, "params / cache / logits / workspace not 16-byte aligned");
  DecodeCache k;
  plan_cache(h, B, Te, Tmax, (char*)d_cache, &k);
  if (k.bytes > cache_bytes)
    return fail(h, T5_ERR_WORKSPACE, "cache of %lld bytes given, %lld needed", (long long)cache_bytes, (long long)k.bytes);
  // the step is the decoder on one position per row: the workspace is laid out for (B, no encoder rows, 1)
  Workspace w;
  plan_workspace(h, B, 0, 1, (char*)d_workspace, &w);
  if (w.bytes > workspace_bytes)
    return fail(h, T5_ERR_WORKSPACE, "workspace of %lld bytes given, %lld needed", (long long)workspace_bytes,
                (long long)w.bytes);
  Ctx cx{};
  cx.h = h; cx.params = d_params; cx.st = (cudaStream_t)stream; cx.w = &w; cx.B = B; cx.Te = 0; cx.Td = 1;
  cx.err = cudaSuccess; cx.where = "";
  const int L = c.n_dec_layers, d = c.d_model;
  CK(cudaMemsetAsync(w.status, 0, 4, cx.st), "memset status");
  CK(cudaMemsetAsync(w.ssq_all, 0, w.ssq_floats * 4, cx.st), "memset row statistics");
  CK(launch_set_column(k.self_code, Tmax, t, B, 1, cx.st), "mark position decoded");
  // bias of key j for the query at position t: distance j - t, entry j of a [t + 1 queries] x [Tmax - t keys] expansion
  CKL(CAT_MISC, 1, launch_relbias_expand(c.dtype, h->spec_dec, pptr(h, d_params, h->dec_relbias), c.n_heads, t + 1, Tmax - t,
                                         k.bias_step, cx.st),
      "relbias_expand (step)");
  float* x0 = L > 0 ? w.dec_self[0].x : w.dec_x_final;
  NextNorm n0 = dec_norm_at(cx, 0, 0);
  CKL(CAT_EMBED, 1, launch_embed_gather(c.dtype, pptr(h, d_params, h->token_embed), d_tokens, x0, pptr(h, d_params, n0.g_off),
                                        n0.xg, n0.ssq, B, d, cx.st),
      "embed (step)");
  for (int l = 0; l < L; ++l) {
    float* after_self = encdec ? w.dec_cross[l].x : w.dec_ffn[l].x;
    attn_step(cx, h->dec[l].self, w.dec_self[l], after_self, dec_norm_at(cx, l, encdec ? 1 : 2), k.self_kv[l], Tmax, k.self_code,
              k.bias_step, k.ones, true, t, Tmax);
    if (encdec)
      attn_step(cx, h->dec[l].cross, w.dec_cross[l], w.dec_ffn[l].x, dec_norm_at(cx, l, 2), k.cross_kv[l], Te, k.enc_code, nullptr,
                k.ones, false, t, Tmax);
    float* x_next = l + 1 < L ? w.dec_self[l + 1].x : w.dec_x_final;
    ffn_forward(cx, h->dec[l].ffn, w.dec_ffn[l], x_next, dec_norm_at(cx, l + 1, 0), B);
  }
  const int64_t head = h->lm_head >= 0 ? h->lm_head : h->token_embed;
  proj_fwd(cx, w.dec_xg_f, d, head, B, c.vocab, d, d_logits, c.vocab, c.logit_scale, row_norm(cx, w.dec_ssq_f), "logits (step)");
  return end_call(h, cx);
}

int t5_decode_step_workspace_bytes(const t5_handle* h, int32_t B, int64_t* bytes) {
  if (!h || !bytes) return T5_ERR_NULL;
  if (B < 1) return T5_ERR_ARG;
  Workspace w;
  plan_workspace(h, B, 0, 1, nullptr, &w);
  *bytes = w.bytes;
  return T5_OK;
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
  h->prof_rec.clear();
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
  h->prof_rec.clear();
  for (int i = 0; i < 8; ++i) { h->prof_flops[i] = 0; h->prof_launches[i] = 0; }
  return T5_OK;
}

int t5_profile_launches(t5_handle* h, t5_profile_launch* out, int32_t max_records, int32_t* n_records) {
  if (!h || !n_records || (max_records > 0 && !out)) return T5_ERR_NULL;
  *n_records = (int32_t)h->prof_cat.size();
  for (int32_t i = 0; i < *n_records && i < max_records; ++i) {
    cudaError_t e = cudaEventSynchronize(h->prof_events[2 * i + 1]);
    float t = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&t, h->prof_events[2 * i], h->prof_events[2 * i + 1]);
    if (e != cudaSuccess) return fail(h, T5_ERR_CUDA, "profile_launches: %s", cudaGetErrorString(e));
    t5_profile_launch& r = out[i];
    snprintf(r.what, sizeof r.what, "%s", h->prof_rec[i].what);
    r.family = h->prof_cat[i]; r.M = h->prof_rec[i].M; r.N = h->prof_rec[i].N; r.K = h->prof_rec[i].K; r.ms = t;
  }
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
  cudaError_t e = launch_xent(dtype, d_logits, d_targets, nullptr, n_rows, vocab, z_loss, d_W, d_sums, d_lse,
                              RowNorm{nullptr, 0.f, 0.f}, (cudaStream_t)stream);
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

int t5_kernel_status_word(int32_t* d_status) {
  g_kernel_status = d_status;
  return T5_OK;
}

int t5_selftest_bounded_wait(int32_t* d_status, int64_t limit_cycles, void* stream) {
  if (!d_status) return T5_ERR_NULL;
  if (limit_cycles < 1 || limit_cycles > 4000000000ll) return T5_ERR_ARG;
  cudaError_t e = launch_selftest_bounded_wait(d_status, limit_cycles, (cudaStream_t)stream);
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
    e = backward ? attn_bwd_tc(a, g_kernel_status, st) : attn_fwd_tc(a, g_kernel_status, st);
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
  a.packed = 1;      // the codes may describe packed rows: keep the tile-skipping bookkeeping on
  if (!attn_tc_supported(a) || !attn_tc_onepass_supported(a)) return T5_ERR_ARG;
  cudaError_t e = attn_bwd_tc(a, g_kernel_status, (cudaStream_t)stream);
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
    e = gemm_tc(g, g_kernel_status, (cudaStream_t)stream);
  }
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}

}  // extern "C"
