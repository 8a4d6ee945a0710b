// Shared declarations of the GPU library: element types, the relative-position
// bucket rule, and the launcher prototypes of every kernel family.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

// dtype codes of the C ABI
enum { DT_F32 = 0, DT_BF16 = 1 };

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------
// Relative-position bucket.  The closed form
//   bucket = me + floor( log(n/me) / log(MD/me) * (nb - me) ), capped at nb-1,
// is turned on the host into integer thresholds thr[q] = smallest n whose
// floor(...) is >= q+1 (exact comparison of integer powers), so the device
// only compares integers and both sides agree bit for bit.
// ---------------------------------------------------------------------------
#define T5_MAX_BUCKET_THR 128
struct BucketSpec {
  int bidirectional;
  int nb;      // buckets available per direction (num_buckets/2 if bidirectional)
  int me;      // nb/2: distances below this map to themselves
  int n_thr;   // number of thresholds (= nb - me - 1 useful ones)
  int thr[T5_MAX_BUCKET_THR];
};

__host__ __device__ inline int bucket_of(const BucketSpec& s, int rel) {
  int off = 0, n;
  if (s.bidirectional) {
    if (rel > 0) off = s.nb;
    n = rel < 0 ? -rel : rel;
  } else {
    n = rel < 0 ? -rel : 0;
  }
  if (n < s.me) return off + n;
  int q = 0;
  while (q < s.n_thr && n >= s.thr[q]) ++q;
  return off + s.me + q;
}

// Position codes: 0 for padding, else the segment id (1 if unpacked); in a prefix LM the positions of the fully
// visible prefix also carry T5_PREFIX_BIT.  Query (code cq, position i) may attend key (ck, j) iff both belong to
// the same segment and, when causal, j <= i or both lie in the prefix.
#define T5_PREFIX_BIT 0x40000000
__host__ __device__ __forceinline__ bool pair_valid(int cq, int ck, bool causal, int j, int i) {
  const int sk = ck & ~T5_PREFIX_BIT;
  return sk != 0 && (cq & ~T5_PREFIX_BIT) == sk && (!causal || j <= i || ((cq & ck) & T5_PREFIX_BIT) != 0);
}

// Builds the thresholds; returns false if the parameters are unsupported.
bool build_bucket_spec(int bidirectional, int num_buckets, int max_distance, BucketSpec* out);

// ---------------------------------------------------------------------------
// RMSNorm folded into the GEMMs around it.  y = x (mean(x^2) + eps)^-1/2 g feeds a projection y W^T; here the
// kernel that produces the residual row x also writes xg = x * g (operand dtype) and adds the row's sum of
// squares into ssq[row]; the projection runs on xg and its epilogue multiplies row m of the product by
// (ssq[m] / d + eps)^-1/2.  A RowNorm names such a statistics vector; ssq == NULL means "no factor".
// ---------------------------------------------------------------------------
struct RowNorm {
  const float* ssq;   // [rows] sum over the d columns of x^2, float32
  float inv_d, eps;
};
__device__ __forceinline__ float rn_factor(const RowNorm& r, int64_t row) {
  return r.ssq ? rsqrtf(r.ssq[row] * r.inv_d + r.eps) : 1.f;
}

// ---------------------------------------------------------------------------
// Programmatic dependent launch.  A kernel launched with launch_pdl may have its CTAs brought onto the SMs while the
// kernel before it in the stream is still draining; pdl_sync(), the first thing such a kernel executes, holds every
// thread until that earlier grid has completed and its writes are visible, and at once lets the kernel after this
// one start its own launch.  What overlaps is launch latency and CTA set-up, never any access to global memory.
// Under an ordinary launch both instructions do nothing.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void pdl_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
}

// ---------------------------------------------------------------------------
// Launchers.  `dtype` selects float / bf16 storage for "T" tensors; all
// reductions and accumulators are float32.  Every launcher returns the
// cudaError_t of its launch.
// ---------------------------------------------------------------------------
struct GemmArgs {
  int M, N, K;
  float alpha;
  const void* A; int lda; int a_kmajor;   // A stored [M,K] if a_kmajor else [K,M]
  const void* B; int ldb; int b_kmajor;   // B stored [N,K] if b_kmajor else [K,N]
  void* D; int ldd; int out_f32;          // D[M,N]; float32 or operand dtype
  const float* resid; int ldr;            // optional float32 addend (D may alias it)
  int accumulate;                         // D += (float32 output only)
  // fused gated-GELU epilogues (CTA-pair kernel, bf16):
  //   epi 1 (forward): B = [Wi0; Wi1] stored [2F, K]; D = h [M, 2F] receives a = A Wi0^T and b = A Wi1^T, aux = hg [M, F]
  //                    receives gelu(a) * b.  N must be 2F.
  //   epi 2 (backward): the product is d(hg) [M, F] (N = F); aux = h [M, 2F] (a | b); D = dh [M, 2F] receives
  //                    da = d(hg) * b * gelu'(a) and db = d(hg) * gelu(a).
  int epi; void* aux; int ld_aux; int F;
  int pair;                               // 1: 256 x 256 tiles on CTA pairs (cta_group::2) where M, N >= 256
  // RMSNorm fold, consumer side: row m of the product (epi 0, 1) or of d(hg) (epi 2) is multiplied by rn's factor
  RowNorm rn;
  // RMSNorm fold, producer side (float32 output with a residual addend only): besides D = alpha A B + resid the
  // epilogue writes xg[m, n] = D[m, n] * g_next[n] in the operand dtype and adds sum_n D[m, n]^2 of its columns
  // into ssq_out[m] (zeroed by the caller before the GEMM)
  void* xg_out; int ld_xg; const void* g_next; float* ssq_out;
  int* sk_flags;                          // optional: >= 160 zeroed ints; lets the tcgen05 kernel split the
                                          // tiles of a partial last wave along K over all SMs (float32 output)
};
cudaError_t gemm_simt(int dtype, const GemmArgs& g, cudaStream_t st);
// tcgen05 path: bf16 operands only.  `status` is a device int set non-zero if a
// bounded wait inside the kernel ran out.
cudaError_t gemm_tc(const GemmArgs& g, int* d_status, cudaStream_t st);
bool gemm_tc_supported(const GemmArgs& g);
bool gemm_tc_epi_supported(const GemmArgs& g);   // g.epi != 0 can run fused

struct AttnArgs {
  // rows of Q/O/dQ/dO are (b*Tq + i), rows of K/V/dK/dV are (b*Tk + j);
  // head h occupies columns [h*dk, (h+1)*dk) from each base pointer.
  const void *Q, *K, *V;
  void* O;
  int ldq, ldk, ldv, ldo;
  float* lse;               // [B,H,Tq]
  float* O32; int ldo32;    // optional float32 copy of O (written by forward, read by backward): delta =
                            // rowsum(dO * O) must see O unrounded, or a component shared by all values
                            // of a row no longer cancels in dS = P (dP - delta)
  int B, H, Tq, Tk, dk;
  const int* code_q;        // [B,Tq]
  const int* code_k;        // [B,Tk]
  int causal;
  const float* bias_delta;  // [H, Tq+Tk-1] indexed by (j - i + Tq - 1), or NULL
  float scale;
  // backward only
  const void* dO; int lddo;
  void *dQ, *dK, *dV; int lddq, lddk, lddv;
  float* delta;             // [B,H,Tq] scratch: sum_d dO*O
  float* dbias_delta;       // [H, Tq+Tk-1] float32, accumulated (+=), or NULL
  int bias_far;             // 0, or a distance F such that the bias is constant for (j - i) >= F and constant for
                            // (j - i) <= -F (the saturated buckets): the backward may then add the whole dS mass
                            // of such regions to the entries at +F / -F instead of to each distance
  // optional scratch of attn_tc_ds_scratch_bytes(B, H, Tq, Tk) bytes: with it the tcgen05 backward makes
  // one pass over the scores (dK, dV and a bf16 copy of dS^T in this buffer) and takes dQ from the stored dS
  void* ds_scratch = nullptr;
  int64_t ds_bytes = 0;
  // backward only: rows of dQ are multiplied by rn_q's factor, rows of dK and dV by rn_k's (the RMSNorm fold of
  // the projections that made q, k, v wants their gradients scaled that way; NULL statistics = factor 1)
  RowNorm rn_q = {nullptr, 0.f, 0.f}, rn_k = {nullptr, 0.f, 0.f};
  // non-zero: rows may hold several segments (packed examples).  The tcgen05 forward then leaves out key tiles whose
  // range of position codes does not meet the range of the CTA's query rows; 0 skips that bookkeeping.
  int packed = 0;
  // non-zero: causal attention whose position codes may carry T5_PREFIX_BIT (prefix LM): keys ahead of a query can
  // be valid, so the kernels walk every tile instead of stopping at the diagonal
  int prefix = 0;
};
int64_t attn_tc_ds_scratch_bytes(int B, int H, int Tq, int Tk);
bool attn_tc_onepass_supported(const AttnArgs& a);   // the backward will take the one-pass route
cudaError_t attn_fwd_simt(int dtype, const AttnArgs& a, cudaStream_t st);
cudaError_t attn_bwd_simt(int dtype, const AttnArgs& a, cudaStream_t st);
// tcgen05 path: bf16, d_kv 64 or 128.  The backward also needs O (for delta = rowsum(dO*O)).
bool attn_tc_supported(const AttnArgs& a);
cudaError_t attn_fwd_tc(const AttnArgs& a, int* d_status, cudaStream_t st);
cudaError_t attn_bwd_tc(const AttnArgs& a, int* d_status, cudaStream_t st);
// status word the kernel-level entry points of the C ABI hand to the tcgen05 kernels (NULL: none)
extern int32_t* g_kernel_status;
// One CTA waits, with the kernels' own bounded wait, on a barrier nothing ever arrives at: after limit_cycles it
// gives up, writes code 99 into *d_status and returns (exercises the give-up path without any hang)
cudaError_t launch_selftest_bounded_wait(int* d_status, long long limit_cycles, cudaStream_t st);

// element-wise / row kernels
// dec_prefix (optional 0/1 flags): flagged positions get T5_PREFIX_BIT in their code and loss weight 0
cudaError_t launch_prep(const int* enc_tok, const int* enc_seg, const int* dec_tgt, const int* dec_seg,
                        const int* dec_prefix, int B, int Te, int Td, int* enc_code, int* dec_code, int* dec_in,
                        float* dec_w, int* W_int, float* W_f, cudaStream_t st);
cudaError_t launch_pad_codes(const int* tok, int* code, int n, cudaStream_t st);      // code = tok != 0
cudaError_t launch_set_column(int* p, int ld, int col, int rows, int value, cudaStream_t st);
// X[t] = E[tok[t]] (float32); with g != NULL also XG[t] = X[t] * g (dtype T) and ssq[t] = sum X[t]^2
cudaError_t launch_embed_gather(int dtype, const void* E, const int* tok, float* X, const void* g, void* XG,
                                float* ssq, int n_tok, int d, cudaStream_t st);
cudaError_t launch_embed_scatter_add(const int* tok, const float* dX, float* dE, int n_tok, int d,
                                     cudaStream_t st);
cudaError_t launch_rmsnorm_fwd(int dtype, const float* X, const void* g, void* Y, float* rstd,
                               int rows, int d, float eps, cudaStream_t st);
// Backward of the folded RMSNorm.  t = gradient wrt xg = x * g, i.e. (row factor r) * (gradient wrt the normed
// activations): what the data-gradient GEMM of a projection leaves when its incoming gradient rows carry the
// factor r.  dx = g t - x (r^2 / d) sum_k (t g x)_k;  dg = sum_rows t x.
// dX_out = (dX_in ? dX_in : 0) + dx; writes float32 dX_out and a T copy dXb (if non-NULL).
// t is float32 if t_f32 else T.  dg (float32 [d]) is OVERWRITTEN; partial: scratch [n_part*d].
cudaError_t launch_rmsnorm_bwd(int dtype, const void* t, int t_f32, const float* X, RowNorm rn,
                               const void* g, const float* dX_in, float* dX_out, void* dXb, float* dg,
                               float* partial, int rows, int d, cudaStream_t st);
// XG = X * g (dtype T): recomputes the operand copy of a residual row block
cudaError_t launch_scale_cols(int dtype, const float* X, const void* g, void* XG, int rows, int d, cudaStream_t st);
int rmsnorm_bwd_parts(int rows);
// FFN non-linearity.  act 0 / 2: h [rows, 2F] = [a | b], hg = gelu(a) * b (tanh form / exact erf form);
// act 1: h [rows, F], hg = relu(h).
cudaError_t launch_geglu_fwd(int dtype, int act, const void* h, void* hg, int rows, int F, cudaStream_t st);
// its backward (dh has h's shape); rows of dh are multiplied by rn's factor
cudaError_t launch_geglu_bwd(int dtype, int act, const void* dhg, const void* h, void* dh, int rows, int F, RowNorm rn,
                             cudaStream_t st);
// weights: per-row loss weights (NULL: 1 where the target is not padding); rows of the gradient written over the
// logits are multiplied by rn's factor
cudaError_t launch_xent(int dtype, void* logits, const int* targets, const float* weights, int rows, int V, float z,
                        const float* W, double* sums, float* lse, RowNorm rn, cudaStream_t st);
cudaError_t launch_finalize_loss(const double* sums, const float* W, float* loss4, cudaStream_t st);
cudaError_t launch_fill_normal(int dtype, void* p, int64_t n, int64_t flat_offset, uint64_t seed,
                               float stddev, float mean, cudaStream_t st);
// AdamW on elements [0, n) of the given pointers (n a multiple of 4); see t5_adamw_update
cudaError_t launch_adamw(int dtype, void* params, float* master, float* m, float* v, const float* g, int64_t n,
                         float lr, float b1, float b2, float eps, float wd, float gscale, float bc1, float bc2,
                         cudaStream_t st);
cudaError_t launch_cast_f32_to(int dtype, const float* src, void* dst, int64_t n, cudaStream_t st);
// bias tables
cudaError_t launch_relbias_expand(int dtype, const BucketSpec& spec, const void* table, int H, int Tq,
                                  int Tk, float* bias_delta, cudaStream_t st);
cudaError_t launch_relbias_fold(const BucketSpec& spec, const float* dbias_delta, int H, int Tq, int Tk,
                                int num_buckets, float* dtable, cudaStream_t st);
cudaError_t launch_buckets(const BucketSpec& spec, int rel_lo, int n, int* out, cudaStream_t st);
