/*
 * t5_b200.h -- C ABI of the B200 (sm_100a) library that runs one training step
 * (forward and backward) of a T5.1.1-style Transformer, plus the two inference
 * calls a model must expose.
 *
 * Where the operations come from: the paper's "Example Models" section names
 * the models (T5 / T5.1.1 encoder-decoder, and a decoder-only configuration);
 * its "Model Implementation" section says a model is wrapped so that it exposes
 * a loss, an evaluation and an inference method; its "Task-based API" section
 * says feature converters hand the model raw integer arrays (encoder-decoder
 * or decoder-only layouts).  The paper prints no formula; the arithmetic is the
 * public T5.1.1 definition, restated beside each call below.
 *
 * Conventions for every call
 *  - Returns 0 on success or a negative T5_ERR_* code.  Nothing aborts, throws
 *    or traps.  t5_last_error() returns a message for the last failure on the
 *    handle (or for a failed t5_create when passed NULL).
 *  - Pointers named d_* are DEVICE pointers owned by the caller; they must be
 *    16-byte aligned.  Everything else is a host pointer.
 *  - The library allocates no device memory.  All work is ordered by the
 *    caller's stream (a cudaStream_t passed as void*): kernels are enqueued
 *    on it, except that the training step runs its weight-gradient GEMMs on
 *    a second stream owned by the handle, forked from the caller's stream
 *    and joined back into it before the call returns, so anything enqueued
 *    on the caller's stream afterwards sees the finished step.  No call
 *    synchronises the device.
 *  - Token id 0 is padding.  Segment ids are optional (NULL = one example per
 *    row); segment id 0 marks padding in packed rows.  A position's "code" is
 *    0 when its token is padding, else its segment id (1 if unpacked).  Query
 *    i attends key j iff code_k[j] != 0 and code_q[i] == code_k[j] (and
 *    j <= i in the decoder's self-attention).  A query with no valid key
 *    produces a zero attention output.  Decoder codes come from the targets.
 */
#ifndef T5_B200_H_
#define T5_B200_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define T5_ABI_VERSION 2

#if defined(__GNUC__)
#define T5_API __attribute__((visibility("default")))
#else
#define T5_API
#endif

enum {
  T5_OK = 0,
  T5_ERR_NULL = -1,         /* a required pointer is NULL */
  T5_ERR_CONFIG = -2,       /* unsupported or inconsistent configuration */
  T5_ERR_SHAPE = -3,        /* batch sizes outside the configured maxima */
  T5_ERR_ALIGN = -4,        /* device pointer not 16-byte aligned */
  T5_ERR_WORKSPACE = -5,    /* workspace smaller than t5_workspace_bytes() */
  T5_ERR_CUDA = -6,         /* a CUDA runtime/driver call failed (see message) */
  T5_ERR_DEVICE_TIMEOUT = -7, /* a bounded device-side wait ran out */
  T5_ERR_ARG = -8           /* bad scalar argument */
};

/* Model and execution configuration (plain data). */
typedef struct {
  int32_t abi_version;      /* T5_ABI_VERSION */
  int32_t arch;             /* 0 encoder-decoder, 1 decoder-only */
  int32_t n_enc_layers, n_dec_layers;
  int32_t d_model, n_heads, d_kv, d_ff, vocab;
  int32_t rel_buckets, rel_max_distance;        /* 32, 128 */
  int32_t max_batch, max_enc_len, max_dec_len;  /* workspace sizing */
  float z_loss, rms_eps, attn_scale, logit_scale; /* 1e-4, 1e-6, 1.0, d_model^-1/2 */
  int32_t dtype;            /* 0: float32 everywhere (validation mode);
                               1: bfloat16 parameters/operands, float32 accumulation */
  int32_t recompute;        /* activation policy: 0 keep everything; 1 do not keep the scaled
                               operand copy of the residual rows and the gated-GELU product of
                               each sub-layer but recompute them (one scaling pass, one
                               gated-GELU pass) in the backward pass right before the
                               weight-gradient GEMMs that read them: a smaller workspace for a
                               few per cent of step time */
  int32_t flags;            /* debugging aids for bfloat16 mode: bit 0 = use the plain SIMT
                               GEMM kernel, bit 1 = use the plain SIMT attention kernels,
                               bit 2 = do NOT run the GEMMs on CTA pairs (cta_group::2),
                               bit 3 = keep the gated GELU in separate kernels instead of the GEMM epilogues.
                               bit 4 = keep the weight-gradient GEMMs on the caller's stream (no second stream).
                               bit 17 = attention backward as two kernels that each recompute the scores
                               (no dS scratch in the workspace) instead of the one-pass pair. */
  /* Members of the model family the paper's "Example Models" section lists beside T5.1.1: */
  int32_t ffn_act;          /* 0: gated GELU, tanh form (T5.1.1; FFN(y) = (gelu(y Wi0) * (y Wi1)) Wo);
                               1: ReLU without a gate (T5 v1.0; FFN(y) = relu(y Wi0) Wo, no wi1 tensor);
                               2: gated GELU, exact (erf) form */
  int32_t untied_head;      /* 0: the logits use the token embedding (logit_scale d_model^-1/2 by convention);
                               1: they use a separate tensor lm_head [vocab, embed] (released T5.1.1;
                               logit_scale 1 by convention) */
} t5_config;

/* One batch.  All pointers are device pointers to int32 arrays. */
typedef struct {
  int32_t B, Te, Td;
  const int32_t* d_enc_tokens;       /* [B,Te]; NULL for decoder-only */
  const int32_t* d_enc_segment_ids;  /* [B,Te] or NULL */
  const int32_t* d_dec_targets;      /* [B,Td]; decoder inputs = targets shifted right
                                        (0 at a row or segment start) */
  const int32_t* d_dec_segment_ids;  /* [B,Td] or NULL */
  const int32_t* d_dec_prefix;       /* [B,Td] 0/1 or NULL.  Prefix LM (the decoder-only model with an
                                        "inputs" part): flagged positions of a segment see each other in
                                        full, the rest stay causal, and flagged positions carry no loss */
} t5_batch;

typedef struct t5_handle t5_handle;

/* Host-only: validates the configuration and builds the parameter manifest. */
T5_API int t5_create(const t5_config* cfg, t5_handle** out);
T5_API int t5_destroy(t5_handle* h);
T5_API const char* t5_last_error(const t5_handle* h);

/* Parameters live in ONE flat device buffer of t5_param_count() elements of
 * the configured dtype (gradients: the same layout in float32).  Tensor i of
 * t5_param_tensors() has `name`, element `offset`, and `shape`.  Names follow
 * the paper's logical-axis idea ("Model Implementation" section):
 *   token_embed [vocab, embed]; {enc,dec}.relbias [buckets, heads];
 *   *.norm / *.final_norm [embed];
 *   enc.L<i>.attn.{q,k,v} [heads*kv, embed]; .o [embed, heads*kv];
 *   *.ffn.{wi0,wi1} [mlp, embed]; .wo [embed, mlp];
 *   dec.L<i>.{self,cross}.* likewise; lm_head [vocab, embed] last when untied_head = 1;
 *   no *.ffn.wi1 when ffn_act = 1.
 * Dense weights are stored [out_features, in_features], row-major: a
 * projection computes y[t, o] = sum_i x[t, i] * W[o, i]. */
T5_API int t5_param_count(const t5_handle* h, int64_t* n_elements);
T5_API int t5_param_tensors(const t5_handle* h, int32_t* n_tensors);
T5_API int t5_param_manifest(const t5_handle* h, int32_t idx, char name[64], int64_t* offset,
                      int32_t shape[4], int32_t* ndim);

/* Bytes of scratch the step needs at the configured maxima. */
T5_API int t5_workspace_bytes(const t5_handle* h, int64_t* bytes);

/* Fills d_params: matrices, embedding and bias tables ~ N(0, stddev), norm
 * scales = 1.  Counter-based: element e of the flat buffer is a function of
 * (seed, e) only (splitmix64 hash -> two uniforms -> Box-Muller). */
T5_API int t5_init_params(t5_handle* h, void* d_params, uint64_t seed, float stddev, void* stream);

/* The loss method and its gradient ("Model Implementation" section: a model
 * defines its loss).  With w_t = [target_t != 0], W = sum w:
 *   x = E[tokens];  per layer: x += Attn(RMS(x)), x += FFN(RMS(x));
 *   RMS(x) = x * (mean(x^2)+eps)^-1/2 * g;
 *   Attn: softmax_j(attn_scale * q_i.k_j + table[bucket(j-i), head] + mask) v, then Wo;
 *         encoder: bidirectional buckets; decoder self: causal, one-sided buckets;
 *         cross-attention: keys/values from the encoder output, no bias;
 *   FFN(y) = (gelu_tanh(y Wi0) * (y Wi1)) Wo;
 *   logits = logit_scale * RMS(x_dec) E^T;  lse_t = log sum_v exp(logits_tv);
 *   L = (1/W) sum_t w_t (lse_t - logits_t[target_t] + z_loss * lse_t^2).
 * Writes d_loss4 = [L, cross-entropy part, z-loss part, W] (float32) and
 * OVERWRITES d_grads (float32, parameter layout) with dL/dparams.
 * W = 0 gives zero loss and zero gradients. */
T5_API int t5_train_step_fwd_bwd(t5_handle* h, const void* d_params, const t5_batch* batch,
                          float* d_grads, float* d_loss4, void* d_workspace,
                          int64_t workspace_bytes, void* stream);

/* The optimizer step that follows the gradients in the paper's training loop ("Overall structure" section; the paper
 * prints no update rule - this is AdamW with decoupled weight decay).  All buffers are flat, in the parameter layout:
 * d_master (float32 master weights), d_m, d_v (float32 moments, zero before the first step), d_grads (float32, as
 * written by t5_train_step_fwd_bwd); d_params receives the master weights rounded to the configured dtype.
 *   g = grad_scale * grad;  m = beta1 m + (1 - beta1) g;  v = beta2 v + (1 - beta2) g^2;
 *   master -= lr ( (m / (1 - beta1^step)) / (sqrt(v / (1 - beta2^step)) + eps) + weight_decay master ),  step >= 1.
 * Weight decay applies to matrices, embeddings and bias tables, not to the 1-D norm scales. */
T5_API int t5_adamw_update(t5_handle* h, void* d_params, float* d_master, float* d_m, float* d_v,
                           const float* d_grads, int64_t step, float lr, float beta1, float beta2, float eps,
                           float weight_decay, float grad_scale, void* stream);

/* Inference method, encoder half: d_enc_out [B,Te,d_model] in the configured
 * dtype = the encoder stack's output after its final norm. */
T5_API int t5_encode(t5_handle* h, const void* d_params, const t5_batch* batch, void* d_enc_out,
              void* d_workspace, int64_t workspace_bytes, void* stream);

/* Inference method, decoder half: teacher-forced logits [B,Td,vocab]
 * (configured dtype) for the whole target sequence given d_enc_out (ignored
 * for decoder-only).  batch->d_enc_tokens / segment ids supply the key mask of
 * the cross-attention. */
T5_API int t5_decode_logits(t5_handle* h, const void* d_params, const t5_batch* batch,
                     const void* d_enc_out, void* d_logits, void* d_workspace,
                     int64_t workspace_bytes, void* stream);

/* Incremental decoding (the inference method applied one position at a time, "Model Implementation" section; the
 * result at position t equals row t of t5_decode_logits on the same inputs).  One example per row (segment ids are
 * not used).  The caller owns a cache buffer of t5_decode_cache_bytes(B, Te, Tmax) bytes that holds, per decoder
 * layer, the self-attention keys / values of the positions decoded so far and the cross-attention keys / values.
 *  - t5_decode_begin: resets the cache and (encoder-decoder) projects every layer's cross-attention keys / values
 *    from d_enc_out [B, Te, d_model], the output of t5_encode; d_enc_tokens [B, Te] gives the key mask (id 0 = padding).
 *  - t5_decode_step: position t (0, 1, 2, ... in order) of all B rows.  d_tokens [B] is the decoder INPUT at that
 *    position (0 at t = 0, afterwards the token chosen at t - 1); writes d_logits [B, vocab] in the configured dtype
 *    and appends the position's keys / values to the cache.  d_workspace: t5_decode_step_workspace_bytes(B) bytes.
 * Te is ignored (may be 0) for the decoder-only architecture. */
T5_API int t5_decode_cache_bytes(const t5_handle* h, int32_t B, int32_t Te, int32_t Tmax, int64_t* bytes);
T5_API int t5_decode_step_workspace_bytes(const t5_handle* h, int32_t B, int64_t* bytes);
T5_API int t5_decode_begin(t5_handle* h, const void* d_params, int32_t B, int32_t Te, int32_t Tmax,
                           const int32_t* d_enc_tokens, const void* d_enc_out, void* d_cache, int64_t cache_bytes,
                           void* stream);
T5_API int t5_decode_step(t5_handle* h, const void* d_params, void* d_cache, int64_t cache_bytes, int32_t B, int32_t Te,
                          int32_t Tmax, int32_t t, const int32_t* d_tokens, void* d_logits, void* d_workspace,
                          int64_t workspace_bytes, void* stream);

/* Data-parallel training ("XLA GSPMD partitioning" section: data parallelism
 * with replicated parameters; the partitioner there inserts the gradient
 * all-reduce, here the caller does, overlapped with the backward pass).
 * While t5_train_step_fwd_bwd enqueues its backward pass it calls the hook, on
 * the calling host thread, each time a contiguous range of the gradient buffer
 * has received its last write - the decoder's layers from the last to the
 * first, then the encoder's, then the remaining tensors (embedding, bias
 * tables, final norms, output head):
 *   offset, count  element range of d_grads (float32) that is final;
 *   d_rank_weight  device float: W_r, this call's number of loss-carrying
 *                  target positions (the gradients are normalised by it);
 *   stream         a CUDA stream on which everything that writes the range
 *                  has been enqueued: work the hook enqueues behind an event
 *                  recorded on it (e.g. scaling by W_r and an all-reduce on a
 *                  communication stream) sees the final values while the rest
 *                  of the backward pass keeps running.  The stream belongs to
 *                  the library or the caller; the hook must not block on it.
 * The ranges of one call are disjoint and cover the whole buffer.  fn = NULL
 * removes the hook.  T5_ERR_NULL without a handle. */
typedef void (*t5_grad_ready_fn)(void* user, int64_t offset, int64_t count, const float* d_rank_weight, void* stream);
T5_API int t5_set_grad_hook(t5_handle* h, t5_grad_ready_fn fn, void* user);

/* Reads back the status word the kernels of the last call on this workspace
 * left behind (their waits on TMA/tensor-core barriers are bounded; one that
 * runs out records a code instead of spinning).  SYNCHRONISES the stream.
 * Returns T5_OK or T5_ERR_DEVICE_TIMEOUT. */
T5_API int t5_device_status(t5_handle* h, const void* d_workspace, void* stream);

/* Measurement aids (no counterpart in the paper).  With profiling enabled every
 * kernel launch of the following calls is bracketed by a CUDA event pair on the
 * caller's stream.  t5_profile_read() waits for those events, returns per kernel
 * family the summed device time (ms), the algorithmic FLOPs of its GEMMs and
 * the number of kernels, then clears the record.  Families: 0 GEMM,
 * 1 attention forward, 2 attention backward, 3 RMSNorm, 4 gated GELU,
 * 5 cross-entropy, 6 embedding, 7 other.  t5_launch_count(): kernels launched
 * by the most recent step/encode/decode call on this handle. */
T5_API int t5_profile_enable(t5_handle* h, int32_t on);
T5_API int t5_profile_read(t5_handle* h, double ms[8], double flops[8], int64_t launches[8]);
/* The same record launch by launch, in launch order (call it BEFORE t5_profile_read, which clears the record):
 * what the event pair brackets, its family, the GEMM's M, N, K (0 for other kernels) and its device time.
 * Fills at most max_records entries of `out` (host memory); *n_records receives how many exist. */
typedef struct {
  char what[40];
  int32_t family, M, N, K;
  float ms;
} t5_profile_launch;
T5_API int t5_profile_launches(t5_handle* h, t5_profile_launch* out, int32_t max_records, int32_t* n_records);
T5_API int t5_launch_count(const t5_handle* h, int64_t* n);

/* ---- single operations of the path, exported for element-wise parity tests ---- */

/* Relative-position bucket (closed form, exact integer thresholds):
 * d_out[i] = bucket(rel_lo + i) for i in [0, n), rel = key - query. */
T5_API int t5_relpos_buckets(int32_t bidirectional, int32_t num_buckets, int32_t max_distance,
                      int32_t rel_lo, int32_t n, int32_t* d_out, void* stream);

/* Softmax cross-entropy with z-loss over rows of logits [n_rows, vocab]
 * (dtype 0 float32 / 1 bfloat16), IN PLACE: on return d_logits holds
 * dL/dlogits = (w/W)(p (1 + 2 z lse) - onehot).  d_W: device float holding W.
 * d_sums[2] (float64, zeroed by the caller) accumulate sum w*ce and sum w*z*lse^2;
 * d_lse [n_rows] receives lse. */
T5_API int t5_xent_zloss(int32_t dtype, void* d_logits, const int32_t* d_targets, int32_t n_rows,
                  int32_t vocab, float z_loss, const float* d_W, double* d_sums, float* d_lse,
                  void* stream);

/* D[M,N] = alpha * A * B (+ D when accumulate), bf16/f32 operands, f32 accumulation.
 * a_kmajor: A is stored [M,K] (else [K,M]); b_kmajor: B is stored [N,K] (else [K,N]);
 * lda/ldb/ldd are row strides in elements.  out_f32: D is float32, else the operand
 * dtype.  impl 0 = SIMT kernel, 1 = tcgen05/TMEM/TMA kernel (bfloat16 only), 2 = the same on
 * CTA pairs (cta_group::2, 256 x 256 tiles) where M, N >= 256.
 * d_sk_flags: NULL, or 160 zeroed int32 that allow the tcgen05 kernel to cut the
 * tiles of a partial last wave along K over all SMs (float32 output only). */
T5_API int t5_gemm(int32_t dtype, int32_t impl, int32_t M, int32_t N, int32_t K, float alpha,
            const void* d_A, int32_t lda, int32_t a_kmajor, const void* d_B, int32_t ldb,
            int32_t b_kmajor, void* d_D, int32_t ldd, int32_t out_f32, int32_t accumulate,
            int32_t* d_sk_flags, void* stream);

/* One attention call on raw buffers (forward, or backward given the forward's
 * outputs):  S_ij = scale q_i.k_j + bias_delta[h, j - i + Tq - 1], masked by
 * the position codes (and j <= i when causal), P = softmax_j, O = P V,
 * lse = log sum_j exp S.  Rows of q/o/do/dq are (b*Tq + i), rows of k/v/dk/dv
 * are (b*Tk + j); head h occupies columns [h*d_kv, (h+1)*d_kv); ld* are row
 * strides in elements.  d_bias_delta [H, Tq+Tk-1] may be NULL.  d_o32 (may be
 * NULL) is a dense float32 [B*Tq, H*d_kv] copy of O that forward writes and
 * backward reads for delta = rowsum(dO * O).  Backward writes
 * dq, dk, dv, uses d_delta [B,H,Tq] as scratch and ADDS dS summed along
 * diagonals into d_dbias_delta (may be NULL).  impl 0 = SIMT kernels,
 * 1 = tcgen05 kernels (bfloat16, d_kv 64 or 128).  The tcgen05 forward leaves
 * out key tiles whose range of position codes does not meet the range of a
 * CTA's 128 query rows (packed rows); the training step switches that
 * bookkeeping off for batches without segment ids, this entry point keeps it on. */
T5_API int t5_attention(int32_t dtype, int32_t impl, int32_t backward, int32_t B, int32_t H, int32_t Tq,
                        int32_t Tk, int32_t d_kv, int32_t causal, float scale, const void* d_q, int32_t ldq,
                        const void* d_k, int32_t ldk, const void* d_v, int32_t ldv, void* d_o, int32_t ldo,
                        float* d_o32, float* d_lse, const int32_t* d_code_q, const int32_t* d_code_k,
                        const float* d_bias_delta, const void* d_do, int32_t lddo, void* d_dq, int32_t lddq,
                        void* d_dk, int32_t lddk, void* d_dv, int32_t lddv, float* d_delta,
                        float* d_dbias_delta, void* stream);

/* Attention backward in one pass over the scores (tcgen05 kernels, bfloat16,
 * d_kv 64 or 128): the same result as t5_attention(..., backward = 1, ...) - whose two
 * kernels each recompute the scores and the probabilities - from one kernel that
 * produces dK, dV and a bfloat16 copy of dS^T in d_ds_scratch, and a second that
 * takes dQ = scale dS K from that copy.  (Backward of the attention the
 * "Example Models" section's T5 family uses.)  d_ds_scratch: device buffer of at
 * least t5_attention_ds_scratch_bytes(B, H, Tq, Tk) bytes, 128-byte aligned,
 * owned by the caller, contents undefined on return.  bias_far: 0, or a distance
 * F such that the bias is constant for (j - i) >= F and for (j - i) <= -F; the
 * dS mass of those regions is then added to the entries at +F and -F of
 * d_dbias_delta.  Other arguments as in t5_attention.  T5_ERR_ARG if the shape is
 * not covered (d_kv not 64 or 128, or a query length whose per-CTA tables exceed shared
 * memory) or the scratch is too small. */
T5_API int t5_attention_ds_scratch_bytes(int32_t B, int32_t H, int32_t Tq, int32_t Tk, int64_t* bytes);
T5_API int t5_attention_backward_onepass(
    int32_t B, int32_t H, int32_t Tq, int32_t Tk, int32_t d_kv, int32_t causal, float scale, const void* d_q,
    int32_t ldq, const void* d_k, int32_t ldk, const void* d_v, int32_t ldv, const void* d_o, int32_t ldo,
    const float* d_o32, const float* d_lse, const int32_t* d_code_q, const int32_t* d_code_k,
    const float* d_bias_delta, const void* d_do, int32_t lddo, void* d_dq, int32_t lddq, void* d_dk, int32_t lddk,
    void* d_dv, int32_t lddv, float* d_delta, float* d_dbias_delta, int32_t bias_far, void* d_ds_scratch,
    int64_t ds_scratch_bytes, void* stream);

/* Status word for the kernel-level entry points (t5_attention,
 * t5_attention_backward_onepass, t5_attention_backward_noalloc, t5_gemm): they
 * have no workspace whose first word could carry it.  d_status: device int32,
 * zeroed by the caller, or NULL to switch reporting off (the default).  A
 * tensor-core kernel whose bounded wait on a TMA / MMA barrier runs out writes
 * its code there (first one wins), abandons its tile and returns normally; the
 * outputs of that call are then incomplete.  The pointer is process-wide and
 * read at launch time; the caller owns the word and reads it after
 * synchronising the stream.  ("Model Implementation" section: the methods a
 * model exposes must report failure to the training loop; the paper names no
 * mechanism.)  Returns T5_OK. */
T5_API int t5_kernel_status_word(int32_t* d_status);

/* Exercises the give-up path of the kernels' bounded waits without hanging
 * anything: one small CTA waits, with the same wait routine the tensor-core
 * kernels use, on a barrier that nothing ever arrives at.  After limit_cycles
 * SM cycles (1 .. 4e9) the wait gives up, writes code 99 into *d_status (device
 * int32, zeroed by the caller) and the kernel returns in the ordinary way; the
 * context stays usable.  No memory traffic, no tensor memory.
 * T5_ERR_NULL / T5_ERR_ARG for bad arguments. */
T5_API int t5_selftest_bounded_wait(int32_t* d_status, int64_t limit_cycles, void* stream);

/* Attention backward without caller-provided scratch.  The paper has no
 * counterpart; this exists for callers that cannot allocate device memory:
 * code in a region where cudaMalloc is illegal or must be avoided, plug-ins
 * that are handed only their inputs and outputs by a framework that owns the
 * allocator, processes whose device memory pool is committed at start-up.
 * Same computation and arguments as t5_attention(..., backward = 1, ...),
 * except that the delta[B,H,Tq] scratch lives in a fixed array inside the
 * library (T5_NOALLOC_MAX_ROWS floats = 4 MiB, held by every GPU that loads
 * the library until the process exits).  The call allocates nothing.
 *  - B*H*Tq must not exceed T5_NOALLOC_MAX_ROWS, else T5_ERR_SHAPE.
 *  - The first call on each device looks up the array's device address (with
 *    that device current); make that first call before any stream capture.
 *  - All calls share the one array per device and it keeps the previous
 *    call's contents.  Nothing in it needs clearing: every element a call
 *    reads is first written by that call.  Two calls whose kernels overlap on
 *    the same GPU (different streams) race on it; serialise them.
 *  - d_dbias_delta is ADDED to, as in t5_attention. */
#define T5_NOALLOC_MAX_ROWS (1 << 20)
T5_API int t5_attention_backward_noalloc(
    int32_t dtype, int32_t impl, int32_t B, int32_t H, int32_t Tq, int32_t Tk, int32_t d_kv, int32_t causal,
    float scale, const void* d_q, int32_t ldq, const void* d_k, int32_t ldk, const void* d_v, int32_t ldv,
    const void* d_o, int32_t ldo, const float* d_o32, const float* d_lse, const int32_t* d_code_q,
    const int32_t* d_code_k, const float* d_bias_delta, const void* d_do, int32_t lddo, void* d_dq,
    int32_t lddq, void* d_dk, int32_t lddk, void* d_dv, int32_t lddv, float* d_dbias_delta, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* T5_B200_H_ */
