// Bandwidth-bound kernels of the step: input preparation, embedding gather and
// scatter-add, RMSNorm forward/backward, gated-GELU forward/backward, the
// vocabulary cross-entropy with z-loss, parameter initialisation.
#include "common.cuh"

#include <math.h>

namespace {

constexpr int kWarp = 32;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// 4 consecutive elements as floats (16-byte load for float, 8-byte for bf16)
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const bf16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// ------------------------------------------------------------------ input prep
// code = 0 for padding else segment id (1 if unpacked); decoder input = target
// shifted right inside a segment; W = number of non-pad targets.
__global__ void prep_kernel(const int* __restrict__ enc_tok, const int* __restrict__ enc_seg,
                            const int* __restrict__ dec_tgt, const int* __restrict__ dec_seg,
                            const int* __restrict__ dec_prefix, int B,
                            int Te, int Td, int* __restrict__ enc_code, int* __restrict__ dec_code,
                            int* __restrict__ dec_in, float* __restrict__ dec_w, int* __restrict__ W_int) {
  int b = blockIdx.x;
  if (enc_tok != nullptr) {
    for (int t = threadIdx.x; t < Te; t += blockDim.x) {
      int i = b * Te + t;
      int tok = enc_tok[i];
      enc_code[i] = tok != 0 ? (enc_seg ? enc_seg[i] : 1) : 0;
    }
  }
  int cnt = 0;
  for (int t = threadIdx.x; t < Td; t += blockDim.x) {
    int i = b * Td + t;
    int tok = dec_tgt[i];
    const int pre = (dec_prefix != nullptr && dec_prefix[i] != 0) ? 1 : 0;      // prefix LM: given, not predicted
    const int code = tok != 0 ? (dec_seg ? dec_seg[i] : 1) : 0;
    dec_code[i] = (code != 0 && pre) ? (code | T5_PREFIX_BIT) : code;
    int u = 0;
    if (t > 0 && (dec_seg == nullptr || dec_seg[i] == dec_seg[i - 1])) u = dec_tgt[i - 1];
    dec_in[i] = u;
    const int wt = (tok != 0 && !pre) ? 1 : 0;
    dec_w[i] = (float)wt;
    cnt += wt;
  }
  cnt = __reduce_add_sync(0xffffffffu, cnt);
  if ((threadIdx.x & 31) == 0 && cnt) atomicAdd(W_int, cnt);
}
// position codes without the decoder's bookkeeping: 0 for padding, else 1 (one example per row)
__global__ void pad_codes_kernel(const int* __restrict__ tok, int* __restrict__ code, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) code[i] = tok[i] != 0 ? 1 : 0;
}
// p[r * ld + col] = value for r in [0, rows)
__global__ void set_column_kernel(int* __restrict__ p, int ld, int col, int rows, int value) {
  int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < rows) p[(int64_t)r * ld + col] = value;
}
__global__ void w_to_float_kernel(const int* W_int, float* W_f) { *W_f = (float)(*W_int); }

// ------------------------------------------------------------------ embedding
template <typename T>
__global__ void embed_gather_kernel(const T* __restrict__ E, const int* __restrict__ tok,
                                    float* __restrict__ X, int n_tok, int d) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // one float4 each
  int per_row = d >> 2;
  if (idx >= (int64_t)n_tok * per_row) return;
  int r = (int)(idx / per_row), c = (int)(idx % per_row) << 2;
  store4(X + (int64_t)r * d + c, load4(E + (int64_t)tok[r] * d + c));
}

// The same gather for a residual stream whose RMSNorm is folded into the next projection: one warp per token also
// writes XG = X * g and the row's sum of squares.
template <typename T>
__global__ void embed_gather_norm_kernel(const T* __restrict__ E, const int* __restrict__ tok, float* __restrict__ X,
                                         const T* __restrict__ g, T* __restrict__ XG, float* __restrict__ ssq,
                                         int n_tok, int d) {
  const int row = blockIdx.x * (blockDim.x / kWarp) + threadIdx.x / kWarp, lane = threadIdx.x & 31;
  if (row >= n_tok) return;
  const T* e = E + (int64_t)tok[row] * d;
  float ss = 0.f;
  for (int c = lane * 4; c < d; c += 128) {
    const float4 v = load4(e + c), gg = load4(g + c);
    store4(X + (int64_t)row * d + c, v);
    store4(XG + (int64_t)row * d + c, make_float4(v.x * gg.x, v.y * gg.y, v.z * gg.z, v.w * gg.w));
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if (lane == 0) ssq[row] = ss;
}

// XG = X * g (the operand copy of residual rows, recomputed)
template <typename T>
__global__ void scale_cols_kernel(const float* __restrict__ X, const T* __restrict__ g, T* __restrict__ XG,
                                  int64_t n4, int d4) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= n4) return;
  const int c = (int)(idx % d4) * 4;
  const float4 v = load4(X + idx * 4), gg = load4(g + c);
  store4(XG + idx * 4, make_float4(v.x * gg.x, v.y * gg.y, v.z * gg.z, v.w * gg.w));
}

__global__ void embed_scatter_add_kernel(const int* __restrict__ tok, const float* __restrict__ dX,
                                         float* __restrict__ dE, int n_tok, int d) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)n_tok * d) return;
  int r = (int)(idx / d), c = (int)(idx % d);
  float v = dX[idx];
  if (v != 0.f) atomicAdd(dE + (int64_t)tok[r] * d + c, v);
}

// ------------------------------------------------------------------ RMSNorm
// y = x * (mean(x^2)+eps)^-1/2 * g.  One warp per row, float4 accesses.
template <typename T>
__global__ void rmsnorm_fwd_kernel(const float* __restrict__ X, const T* __restrict__ g,
                                   T* __restrict__ Y, float* __restrict__ rstd, int rows, int d,
                                   float eps) {
  int row = blockIdx.x * (blockDim.x / kWarp) + threadIdx.x / kWarp;
  int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const float* x = X + (int64_t)row * d;
  float ss = 0.f;
#pragma unroll 4
  for (int c = lane * 4; c < d; c += 128) {
    float4 v = load4(x + c);
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  float r = rsqrtf(ss / (float)d + eps);
  if (lane == 0 && rstd != nullptr) rstd[row] = r;
  T* y = Y + (int64_t)row * d;
#pragma unroll 4
  for (int c = lane * 4; c < d; c += 128) {
    float4 v = load4(x + c);
    float4 gg = load4(g + c);
    store4(y + c, make_float4(v.x * r * gg.x, v.y * r * gg.y, v.z * r * gg.z, v.w * r * gg.w));
  }
}

// Backward of the folded RMSNorm: dY holds t = r * (gradient wrt the normed activations), r^2 = 1 / (ssq/d + eps).
// dx = g t - x (r^2 / d) sum_k (t g x)_k;  dg = sum_rows t x.
// Each warp walks rows with stride; per-CTA partial dg goes to partial[cta, d].
template <typename T, typename TDY>
__global__ void rmsnorm_bwd_kernel(const TDY* __restrict__ dY, const float* __restrict__ X,
                                   RowNorm rn, const T* __restrict__ g,
                                   const float* __restrict__ dX_in, float* __restrict__ dX_out,
                                   T* __restrict__ dXb, float* __restrict__ partial, int rows, int d) {
  extern __shared__ float s_dg[];   // [d]
  for (int c = threadIdx.x; c < d; c += blockDim.x) s_dg[c] = 0.f;
  __syncthreads();
  int lane = threadIdx.x & 31;
  int warps = blockDim.x / kWarp;
  int w = threadIdx.x / kWarp;
  constexpr int kMaxChunks = 16;     // d <= 2048 keeps dg in registers; larger d loops via smem
  float acc[kMaxChunks][4];
#pragma unroll
  for (int i = 0; i < kMaxChunks; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
  for (int row = blockIdx.x * warps + w; row < rows; row += gridDim.x * warps) {
    const float* x = X + (int64_t)row * d;
    const TDY* dy = dY + (int64_t)row * d;
    const float r2 = 1.f / (rn.ssq[row] * rn.inv_d + rn.eps);
    float m = 0.f;
#pragma unroll 4
    for (int c = lane * 4; c < d; c += 128) {
      float4 xv = load4(x + c), dv = load4(dy + c), gv = load4(g + c);
      m += dv.x * gv.x * xv.x + dv.y * gv.y * xv.y + dv.z * gv.z * xv.z + dv.w * gv.w * xv.w;
    }
    m = warp_sum(m) / (float)d;
    float r3m = r2 * m;
    auto body = [&](int c, float* a4) {
      float4 xv = load4(x + c), dv = load4(dy + c), gv = load4(g + c);
      float4 o;
      o.x = dv.x * gv.x - xv.x * r3m;
      o.y = dv.y * gv.y - xv.y * r3m;
      o.z = dv.z * gv.z - xv.z * r3m;
      o.w = dv.w * gv.w - xv.w * r3m;
      if (dX_in != nullptr) {
        float4 p = load4(dX_in + (int64_t)row * d + c);
        o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
      }
      store4(dX_out + (int64_t)row * d + c, o);
      if (dXb != nullptr) store4(dXb + (int64_t)row * d + c, o);
      a4[0] = dv.x * xv.x; a4[1] = dv.y * xv.y; a4[2] = dv.z * xv.z; a4[3] = dv.w * xv.w;
    };
#pragma unroll
    for (int ch = 0; ch < kMaxChunks; ++ch) {
      int c = lane * 4 + ch * 128;
      if (c < d) {
        float a4[4];
        body(c, a4);
        acc[ch][0] += a4[0]; acc[ch][1] += a4[1]; acc[ch][2] += a4[2]; acc[ch][3] += a4[3];
      }
    }
    for (int c = lane * 4 + kMaxChunks * 128; c < d; c += 128) {
      float a4[4];
      body(c, a4);
      atomicAdd(&s_dg[c + 0], a4[0]); atomicAdd(&s_dg[c + 1], a4[1]);
      atomicAdd(&s_dg[c + 2], a4[2]); atomicAdd(&s_dg[c + 3], a4[3]);
    }
  }
#pragma unroll
  for (int ch = 0; ch < kMaxChunks; ++ch) {
    int c = lane * 4 + ch * 128;
    if (c < d) {
      atomicAdd(&s_dg[c + 0], acc[ch][0]); atomicAdd(&s_dg[c + 1], acc[ch][1]);
      atomicAdd(&s_dg[c + 2], acc[ch][2]); atomicAdd(&s_dg[c + 3], acc[ch][3]);
    }
  }
  __syncthreads();
  for (int c = threadIdx.x; c < d; c += blockDim.x) partial[(int64_t)blockIdx.x * d + c] = s_dg[c];
}

// Same arithmetic, one row per CTA pass (d <= 1024 * NCH): thread t owns columns [4t, 4t + 4) of each 1024-column
// chunk for every row its CTA visits, so g and the dg partial sums of those columns live in registers (no shared
// atomics) and a row's x, t and incoming dx are each read exactly once.  The loads of the CTA's next row go out
// before the current row's block-wide reduction, so the CTA has memory requests in flight the whole time.
template <typename T, typename TDY, int NCH>
__global__ void __launch_bounds__(256, 2)
rmsnorm_bwd_rows_kernel(const TDY* __restrict__ dY, const float* __restrict__ X, RowNorm rn,
                        const T* __restrict__ g, const float* dX_in, float* dX_out, T* __restrict__ dXb,
                        float* __restrict__ partial, int rows, int d) {
  pdl_sync();
  __shared__ float red[2][8];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  float4 gv[NCH], acc[NCH];
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
    const int c = ch * 1024 + tid * 4;
    gv[ch] = c < d ? load4(g + c) : make_float4(0.f, 0.f, 0.f, 0.f);
    acc[ch] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const float inv_d = 1.f / (float)d;
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 xv[NCH], dv[NCH], pv[NCH], xn[NCH], dn[NCH], pn[NCH];
  float ssq = 0.f, ssq_n = 0.f;
  auto fetch = [&](int row, float4 (&x4)[NCH], float4 (&d4)[NCH], float4 (&p4)[NCH], float& sq) {
    const int64_t off = (int64_t)row * d;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c = ch * 1024 + tid * 4;
      x4[ch] = c < d ? load4(X + off + c) : z;
      d4[ch] = c < d ? load4(dY + off + c) : z;
      p4[ch] = (c < d && dX_in != nullptr) ? load4(dX_in + off + c) : z;
    }
    sq = rn.ssq[row];
  };
  int row = blockIdx.x;
  if (row < rows) fetch(row, xv, dv, pv, ssq);
  int par = 0;
  for (; row < rows; row += gridDim.x, par ^= 1) {
    const int next = row + gridDim.x;
    if (next < rows) fetch(next, xn, dn, pn, ssq_n);
    const int64_t off = (int64_t)row * d;
    const float r2 = 1.f / (ssq * rn.inv_d + rn.eps);
    float m = 0.f;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch)
      m += dv[ch].x * gv[ch].x * xv[ch].x + dv[ch].y * gv[ch].y * xv[ch].y + dv[ch].z * gv[ch].z * xv[ch].z +
           dv[ch].w * gv[ch].w * xv[ch].w;
    m = warp_sum(m);
    if (lane == 0) red[par][w] = m;
    __syncthreads();      // red[par] is rewritten two rows later, behind the next row's barrier
    float tot = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) tot += red[par][i];
    const float r3m = r2 * tot * inv_d;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c = ch * 1024 + tid * 4;
      if (c < d) {
        float4 o;
        o.x = dv[ch].x * gv[ch].x - xv[ch].x * r3m + pv[ch].x;
        o.y = dv[ch].y * gv[ch].y - xv[ch].y * r3m + pv[ch].y;
        o.z = dv[ch].z * gv[ch].z - xv[ch].z * r3m + pv[ch].z;
        o.w = dv[ch].w * gv[ch].w - xv[ch].w * r3m + pv[ch].w;
        store4(dX_out + off + c, o);
        if (dXb != nullptr) store4(dXb + off + c, o);
        acc[ch].x += dv[ch].x * xv[ch].x; acc[ch].y += dv[ch].y * xv[ch].y;
        acc[ch].z += dv[ch].z * xv[ch].z; acc[ch].w += dv[ch].w * xv[ch].w;
      }
    }
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) { xv[ch] = xn[ch]; dv[ch] = dn[ch]; pv[ch] = pn[ch]; }
    ssq = ssq_n;
  }
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
    const int c = ch * 1024 + tid * 4;
    if (c < d) store4(partial + (int64_t)blockIdx.x * d + c, acc[ch]);
  }
}

__global__ void colsum_kernel(const float* __restrict__ partial, int n_part, int d, float* __restrict__ out) {
  pdl_sync();
  // block (32, 16): 32 columns, the partial rows split over 16 groups, then a shared-memory tree
  __shared__ float red[16][33];
  int c = blockIdx.x * 32 + threadIdx.x;
  float s = 0.f;
  if (c < d)
    for (int p = threadIdx.y; p < n_part; p += 16) s += partial[(int64_t)p * d + c];
  red[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0 && c < d) {
    float t = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) t += red[i][threadIdx.x];
    out[c] = t;
  }
}

// ------------------------------------------------------------------ gated GELU
// FAST = true uses the hardware tanh approximation (relative error ~2^-11: below bfloat16 resolution);
// the float32 validation mode keeps tanhf.
template <bool FAST>
__device__ __forceinline__ float tanh_sel(float x) {
  if (FAST) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
  }
  return tanhf(x);
}
// gelu(u) and its derivative from one tanh
template <bool FAST>
__device__ __forceinline__ void gelu_both(float u, float& g, float& dg) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  float u2 = u * u;
  float t = tanh_sel<FAST>(c * (u + a * u * u2));
  g = 0.5f * u * (1.f + t);
  dg = 0.5f * (1.f + t) + 0.5f * u * (1.f - t * t) * c * (1.f + 3.f * a * u2);
}
template <bool FAST>
__device__ __forceinline__ float gelu_tanh_f(float u) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  return 0.5f * u * (1.f + tanh_sel<FAST>(c * (u + a * u * u * u)));
}

// 8 consecutive elements as floats: one 16-byte access for bf16, two for float
struct F8 { float v[8]; };
__device__ __forceinline__ F8 load8(const float* p) {
  float4 a = load4(p), b = load4(p + 4);
  return {{a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w}};
}
__device__ __forceinline__ F8 load8(const bf16* p) {
  uint4 u = *reinterpret_cast<const uint4*>(p);
  F8 r;
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    r.v[2 * i] = __uint_as_float(w[i] << 16);
    r.v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
  return r;
}
__device__ __forceinline__ void store8(float* p, const F8& f) {
  store4(p, make_float4(f.v[0], f.v[1], f.v[2], f.v[3]));
  store4(p + 4, make_float4(f.v[4], f.v[5], f.v[6], f.v[7]));
}
__device__ __forceinline__ void store8(bf16* p, const F8& f) {
  uint4 u;
  __nv_bfloat162 t;
  t = __floats2bfloat162_rn(f.v[0], f.v[1]); u.x = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f.v[2], f.v[3]); u.y = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f.v[4], f.v[5]); u.z = *reinterpret_cast<uint32_t*>(&t);
  t = __floats2bfloat162_rn(f.v[6], f.v[7]); u.w = *reinterpret_cast<uint32_t*>(&t);
  *reinterpret_cast<uint4*>(p) = u;
}

// exact GELU u Phi(u) and its derivative Phi(u) + u phi(u)
__device__ __forceinline__ void gelu_erf_both(float u, float& g, float& dg) {
  const float cdf = 0.5f * (1.f + erff(u * 0.7071067811865476f));
  g = u * cdf;
  dg = cdf + u * 0.3989422804014327f * __expf(-0.5f * u * u);
}
// ACT 0: gated GELU (tanh form), 1: ReLU without a gate, 2: gated GELU (erf form)
template <int ACT, bool FAST>
__device__ __forceinline__ void act_both(float u, float& g, float& dg) {
  if (ACT == 1) { g = fmaxf(u, 0.f); dg = u > 0.f ? 1.f : 0.f; }
  else if (ACT == 2) gelu_erf_both(u, g, dg);
  else gelu_both<FAST>(u, g, dg);
}

// ACT 0 / 2: h [rows, 2F] = [a | b]; hg = act(a) * b.  ACT 1: h [rows, F]; hg = relu(h).   (8 elements per thread)
template <typename T, int ACT>
__global__ void geglu_fwd_kernel(const T* __restrict__ h, T* __restrict__ hg, int rows, int F) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int per_row = F >> 3;
  if (idx >= (int64_t)rows * per_row) return;
  int r = (int)(idx / per_row), c = (int)(idx % per_row) << 3;
  constexpr bool FAST = sizeof(T) == 2;
  const int ldh = ACT == 1 ? F : 2 * F;
  F8 a = load8(h + (int64_t)r * ldh + c), o;
  if (ACT == 1) {
#pragma unroll
    for (int i = 0; i < 8; ++i) o.v[i] = fmaxf(a.v[i], 0.f);
  } else {
    F8 b = load8(h + (int64_t)r * ldh + F + c);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float ge, dge;
      if (ACT == 0) ge = gelu_tanh_f<FAST>(a.v[i]); else gelu_erf_both(a.v[i], ge, dge);
      o.v[i] = ge * b.v[i];
    }
  }
  store8(hg + (int64_t)r * F + c, o);
}
// da = f dhg * b * act'(a); db = f dhg * act(a) (gated);  dh = f dhg * relu'(h) (ReLU);  f = rn's factor of the row
template <typename T, int ACT>
__global__ void geglu_bwd_kernel(const T* __restrict__ dhg, const T* __restrict__ h, T* __restrict__ dh,
                                 int rows, int F, RowNorm rn) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int per_row = F >> 3;
  if (idx >= (int64_t)rows * per_row) return;
  int r = (int)(idx / per_row), c = (int)(idx % per_row) << 3;
  constexpr bool FAST = sizeof(T) == 2;
  const int ldh = ACT == 1 ? F : 2 * F;
  const float f = rn_factor(rn, r);
  F8 a = load8(h + (int64_t)r * ldh + c), g = load8(dhg + (int64_t)r * F + c), da, db;
  if (ACT == 1) {
#pragma unroll
    for (int i = 0; i < 8; ++i) da.v[i] = a.v[i] > 0.f ? f * g.v[i] : 0.f;
    store8(dh + (int64_t)r * ldh + c, da);
    return;
  }
  F8 b = load8(h + (int64_t)r * ldh + F + c);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float ge, dge;
    act_both<ACT, FAST>(a.v[i], ge, dge);
    da.v[i] = f * g.v[i] * b.v[i] * dge;
    db.v[i] = f * g.v[i] * ge;
  }
  store8(dh + (int64_t)r * ldh + c, da);
  store8(dh + (int64_t)r * ldh + F + c, db);
}

// ------------------------------------------------------------------ cross-entropy + z-loss
// One CTA per row.  The row is staged in shared memory (as T) when it fits, so
// global memory sees one read and one write per logit.
template <typename T>
__global__ void xent_kernel(T* __restrict__ logits, const int* __restrict__ targets,
                            const float* __restrict__ weights, int V, float z,
                            const float* __restrict__ Wp, double* __restrict__ sums,
                            float* __restrict__ lse_out, int staged, RowNorm rn) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  T* srow = reinterpret_cast<T*>(smem_raw);
  __shared__ float red[33];
  int row = blockIdx.x;
  T* grow = logits + (int64_t)row * V;
  int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  int V4 = V & ~3;
  float mx = -INFINITY;
  for (int c = tid * 4; c < V4; c += blockDim.x * 4) {
    float4 v = load4(grow + c);
    if (staged) store4(srow + c, v);
    mx = fmaxf(fmaxf(mx, fmaxf(v.x, v.y)), fmaxf(v.z, v.w));
  }
  for (int c = V4 + tid; c < V; c += blockDim.x) {
    float v = to_f(grow[c]);
    if (staged) srow[c] = grow[c];
    mx = fmaxf(mx, v);
  }
  mx = warp_max(mx);
  if (lane == 0) red[wid] = mx;
  __syncthreads();
  if (wid == 0) {
    float v = lane < nw ? red[lane] : -INFINITY;
    v = warp_max(v);
    if (lane == 0) red[32] = v;
  }
  __syncthreads();
  mx = red[32];
  const T* src = staged ? srow : grow;
  float se = 0.f;
  for (int c = tid * 4; c < V4; c += blockDim.x * 4) {
    float4 v = load4(src + c);
    se += __expf(v.x - mx) + __expf(v.y - mx) + __expf(v.z - mx) + __expf(v.w - mx);
  }
  for (int c = V4 + tid; c < V; c += blockDim.x) se += __expf(to_f(src[c]) - mx);
  se = warp_sum(se);
  __syncthreads();
  if (lane == 0) red[wid] = se;
  __syncthreads();
  if (wid == 0) {
    float v = lane < nw ? red[lane] : 0.f;
    v = warp_sum(v);
    if (lane == 0) red[32] = v;
  }
  __syncthreads();
  se = red[32];
  float lse = logf(se) + mx;
  int tgt = targets[row];
  float W = *Wp;
  float w = ((weights ? weights[row] != 0.f : tgt != 0) && W > 0.f) ? 1.f : 0.f;
  if (tid == 0) {
    lse_out[row] = lse;
    if (w != 0.f) {
      float tl = to_f(src[tgt]);
      atomicAdd(&sums[0], (double)(lse - tl));
      atomicAdd(&sums[1], (double)(z * lse * lse));
    }
  }
  const float rf = rn_factor(rn, row);      // the gradient rows carry the factor of a folded RMSNorm
  float coef = w != 0.f ? rf * (1.f + 2.f * z * lse) / (se * W) : 0.f;   // p = exp(v-mx)/se
  float sub = w != 0.f ? rf / W : 0.f;
  for (int c = tid * 4; c < V4; c += blockDim.x * 4) {
    float4 v = load4(src + c);
    float4 o = make_float4(__expf(v.x - mx) * coef, __expf(v.y - mx) * coef, __expf(v.z - mx) * coef,
                           __expf(v.w - mx) * coef);
    if (tgt >= c && tgt < c + 4) (&o.x)[tgt - c] -= sub;
    store4(grow + c, o);
  }
  for (int c = V4 + tid; c < V; c += blockDim.x) {
    float o = __expf(to_f(src[c]) - mx) * coef;
    if (c == tgt) o -= sub;
    grow[c] = from_f<T>(o);
  }
}

__global__ void finalize_loss_kernel(const double* sums, const float* Wp, float* loss4) {
  float W = *Wp;
  if (W > 0.f) {
    double ce = sums[0] / W, zl = sums[1] / W;
    loss4[0] = (float)(ce + zl); loss4[1] = (float)ce; loss4[2] = (float)zl; loss4[3] = W;
  } else {
    loss4[0] = loss4[1] = loss4[2] = loss4[3] = 0.f;
  }
}

// ------------------------------------------------------------------ init
__device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ull;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
// element e (flat index) <- mean + stddev * sqrt(-2 ln u1) cos(2 pi u2), (u1,u2) from splitmix64(seed, e)
template <typename T>
__global__ void fill_normal_kernel(T* p, int64_t n, int64_t flat_offset, uint64_t seed, float stddev,
                                   float mean) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float v = mean;
  if (stddev != 0.f) {
    uint64_t h = splitmix64(seed ^ splitmix64((uint64_t)(flat_offset + i)));
    float u1 = ((float)(uint32_t)(h >> 40) + 1.0f) * (1.0f / 16777216.0f);   // (0,1]
    float u2 = (float)(uint32_t)((h >> 8) & 0xFFFFFFu) * (1.0f / 16777216.0f);
    v += stddev * sqrtf(-2.f * logf(u1)) * cospif(2.f * u2);
  }
  p[i] = from_f<T>(v);
}

// One AdamW step on a range of the flat buffers (float32 master weights, moments and gradients; the operand-dtype
// copy of the parameters is refreshed from the master weights).  bc1 = 1 - b1^t, bc2 = 1 - b2^t.
template <typename T>
__global__ void adamw_kernel(T* __restrict__ params, float* __restrict__ master, float* __restrict__ m,
                             float* __restrict__ v, const float* __restrict__ g, int64_t n, float lr, float b1, float b2,
                             float eps, float wd, float gscale, float bc1, float bc2) {
  const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i >= n) return;      // n is a multiple of 4 (tensors are padded to 64 elements)
  const float4 g4 = load4(g + i), m4 = load4(m + i), v4 = load4(v + i), t4 = load4(master + i);
  float gg[4] = {g4.x * gscale, g4.y * gscale, g4.z * gscale, g4.w * gscale};
  float mm[4] = {m4.x, m4.y, m4.z, m4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w}, tt[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    mm[k] = b1 * mm[k] + (1.f - b1) * gg[k];
    vv[k] = b2 * vv[k] + (1.f - b2) * gg[k] * gg[k];
    tt[k] -= lr * ((mm[k] / bc1) / (sqrtf(vv[k] / bc2) + eps) + wd * tt[k]);
  }
  store4(m + i, make_float4(mm[0], mm[1], mm[2], mm[3]));
  store4(v + i, make_float4(vv[0], vv[1], vv[2], vv[3]));
  store4(master + i, make_float4(tt[0], tt[1], tt[2], tt[3]));
  store4(params + i, make_float4(tt[0], tt[1], tt[2], tt[3]));
}

template <typename T>
__global__ void cast_kernel(const float* __restrict__ s, T* __restrict__ d, int64_t n) {
  int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i + 3 < n) {
    store4(d + i, load4(s + i));
  } else {
    for (; i < n; ++i) d[i] = from_f<T>(s[i]);
  }
}

inline unsigned blocks_for(int64_t n, int per) { return (unsigned)((n + per - 1) / per); }

}  // namespace

// =========================================================================== launchers
cudaError_t launch_prep(const int* enc_tok, const int* enc_seg, const int* dec_tgt, const int* dec_seg,
                        const int* dec_prefix, int B, int Te, int Td, int* enc_code, int* dec_code, int* dec_in,
                        float* dec_w, int* W_int, float* W_f, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(W_int, 0, sizeof(int), st);
  if (e != cudaSuccess) return e;
  prep_kernel<<<B, 128, 0, st>>>(enc_tok, enc_seg, dec_tgt, dec_seg, dec_prefix, B, Te, Td, enc_code, dec_code,
                                 dec_in, dec_w, W_int);
  w_to_float_kernel<<<1, 1, 0, st>>>(W_int, W_f);
  return cudaGetLastError();
}

cudaError_t launch_pad_codes(const int* tok, int* code, int n, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  pad_codes_kernel<<<blocks_for(n, 256), 256, 0, st>>>(tok, code, n);
  return cudaGetLastError();
}
cudaError_t launch_set_column(int* p, int ld, int col, int rows, int value, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  set_column_kernel<<<blocks_for(rows, 128), 128, 0, st>>>(p, ld, col, rows, value);
  return cudaGetLastError();
}

cudaError_t launch_embed_gather(int dtype, const void* E, const int* tok, float* X, const void* g, void* XG,
                                float* ssq, int n_tok, int d, cudaStream_t st) {
  int64_t n = (int64_t)n_tok * (d / 4);
  if (n == 0) return cudaSuccess;
  if (g != nullptr) {
    if (dtype == DT_F32)
      embed_gather_norm_kernel<float><<<blocks_for(n_tok, 8), 256, 0, st>>>((const float*)E, tok, X, (const float*)g,
                                                                           (float*)XG, ssq, n_tok, d);
    else
      embed_gather_norm_kernel<bf16><<<blocks_for(n_tok, 8), 256, 0, st>>>((const bf16*)E, tok, X, (const bf16*)g,
                                                                          (bf16*)XG, ssq, n_tok, d);
    return cudaGetLastError();
  }
  if (dtype == DT_F32)
    embed_gather_kernel<float><<<blocks_for(n, 256), 256, 0, st>>>((const float*)E, tok, X, n_tok, d);
  else
    embed_gather_kernel<bf16><<<blocks_for(n, 256), 256, 0, st>>>((const bf16*)E, tok, X, n_tok, d);
  return cudaGetLastError();
}

cudaError_t launch_embed_scatter_add(const int* tok, const float* dX, float* dE, int n_tok, int d,
                                     cudaStream_t st) {
  int64_t n = (int64_t)n_tok * d;
  if (n == 0) return cudaSuccess;
  embed_scatter_add_kernel<<<blocks_for(n, 256), 256, 0, st>>>(tok, dX, dE, n_tok, d);
  return cudaGetLastError();
}

cudaError_t launch_rmsnorm_fwd(int dtype, const float* X, const void* g, void* Y, float* rstd, int rows,
                               int d, float eps, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  int wpb = 8;
  if (dtype == DT_F32)
    rmsnorm_fwd_kernel<float><<<blocks_for(rows, wpb), wpb * 32, 0, st>>>(X, (const float*)g, (float*)Y,
                                                                          rstd, rows, d, eps);
  else
    rmsnorm_fwd_kernel<bf16><<<blocks_for(rows, wpb), wpb * 32, 0, st>>>(X, (const bf16*)g, (bf16*)Y, rstd,
                                                                         rows, d, eps);
  return cudaGetLastError();
}

int rmsnorm_bwd_parts(int rows) {
  int p = rows < 592 ? rows : 592;      // upper bound of the grid (narrow rows: four resident CTAs per SM)
  if (p < 1) p = 1;
  return p;
}

cudaError_t launch_scale_cols(int dtype, const float* X, const void* g, void* XG, int rows, int d, cudaStream_t st) {
  const int64_t n4 = (int64_t)rows * (d / 4);
  if (n4 == 0) return cudaSuccess;
  if (dtype == DT_F32)
    scale_cols_kernel<float><<<blocks_for(n4, 256), 256, 0, st>>>(X, (const float*)g, (float*)XG, n4, d / 4);
  else
    scale_cols_kernel<bf16><<<blocks_for(n4, 256), 256, 0, st>>>(X, (const bf16*)g, (bf16*)XG, n4, d / 4);
  return cudaGetLastError();
}

cudaError_t launch_rmsnorm_bwd(int dtype, const void* dy, int dy_f32, const float* X, RowNorm rn,
                               const void* g, const float* dX_in, float* dX_out, void* dXb, float* dg,
                               float* partial, int rows, int d, cudaStream_t st) {
  int parts = rmsnorm_bwd_parts(rows);
  // rows wider than 1024 columns cost ~100 registers per thread: two resident CTAs per SM, each with two rows' loads
  // in flight; narrower rows fit four
  if (d > 1024 && parts > 296) parts = 296;
  if (d <= 4096) {
#define RBR(T, TDY, NCH)                                                                                          \
  launch_pdl(rmsnorm_bwd_rows_kernel<T, TDY, NCH>, dim3(parts), dim3(256), 0, st, (const TDY*)dy, X, rn, (const T*)g, \
             dX_in, dX_out, (T*)dXb, partial, rows, d)
#define RBR_N(T, TDY)                                                     \
  do {                                                                    \
    if (d <= 1024) RBR(T, TDY, 1); else if (d <= 2048) RBR(T, TDY, 2);    \
    else RBR(T, TDY, 4);                                                  \
  } while (0)
    if (dtype == DT_F32) {
      RBR_N(float, float);
    } else if (dy_f32) {
      RBR_N(bf16, float);
    } else {
      RBR_N(bf16, bf16);
    }
#undef RBR_N
#undef RBR
  } else {
    if (parts > 296) parts = 296;
    size_t sm = (size_t)d * sizeof(float);
#define RB(T, TDY)                                                                                     \
  rmsnorm_bwd_kernel<T, TDY><<<parts, 256, sm, st>>>((const TDY*)dy, X, rn, (const T*)g, dX_in, dX_out, \
                                                     (T*)dXb, partial, rows, d)
    if (dtype == DT_F32) {
      RB(float, float);
    } else if (dy_f32) {
      RB(bf16, float);
    } else {
      RB(bf16, bf16);
    }
#undef RB
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  return launch_pdl(colsum_kernel, dim3(blocks_for(d, 32)), dim3(32, 16), 0, st, (const float*)partial, parts, d, dg);
}

cudaError_t launch_geglu_fwd(int dtype, int act, const void* h, void* hg, int rows, int F, cudaStream_t st) {
  int64_t n = (int64_t)rows * (F / 8);
  if (n == 0) return cudaSuccess;
#define GF(T, ACT) geglu_fwd_kernel<T, ACT><<<blocks_for(n, 256), 256, 0, st>>>((const T*)h, (T*)hg, rows, F)
  if (dtype == DT_F32) { if (act == 1) GF(float, 1); else if (act == 2) GF(float, 2); else GF(float, 0); }
  else { if (act == 1) GF(bf16, 1); else if (act == 2) GF(bf16, 2); else GF(bf16, 0); }
#undef GF
  return cudaGetLastError();
}

cudaError_t launch_geglu_bwd(int dtype, int act, const void* dhg, const void* h, void* dh, int rows, int F, RowNorm rn,
                             cudaStream_t st) {
  int64_t n = (int64_t)rows * (F / 8);
  if (n == 0) return cudaSuccess;
#define GB(T, ACT) geglu_bwd_kernel<T, ACT><<<blocks_for(n, 256), 256, 0, st>>>((const T*)dhg, (const T*)h, (T*)dh, rows, F, rn)
  if (dtype == DT_F32) { if (act == 1) GB(float, 1); else if (act == 2) GB(float, 2); else GB(float, 0); }
  else { if (act == 1) GB(bf16, 1); else if (act == 2) GB(bf16, 2); else GB(bf16, 0); }
#undef GB
  return cudaGetLastError();
}

cudaError_t launch_xent(int dtype, void* logits, const int* targets, const float* weights, int rows, int V, float z,
                        const float* W, double* sums, float* lse, RowNorm rn, cudaStream_t st) {
  if (rows == 0) return cudaSuccess;
  size_t esz = dtype == DT_F32 ? 4 : 2;
  size_t row_bytes = ((size_t)V * esz + 15) & ~(size_t)15;
  int staged = row_bytes <= 160 * 1024 && ((V * esz) % 8 == 0);
  size_t sm = staged ? row_bytes : 16;
  cudaError_t e;
  if (dtype == DT_F32) {
    if (sm > 48 * 1024) {
      e = cudaFuncSetAttribute(xent_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
    }
    xent_kernel<float><<<rows, 512, sm, st>>>((float*)logits, targets, weights, V, z, W, sums, lse, staged, rn);
  } else {
    if (sm > 48 * 1024) {
      e = cudaFuncSetAttribute(xent_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
    }
    xent_kernel<bf16><<<rows, 512, sm, st>>>((bf16*)logits, targets, weights, V, z, W, sums, lse, staged, rn);
  }
  return cudaGetLastError();
}

cudaError_t launch_finalize_loss(const double* sums, const float* W, float* loss4, cudaStream_t st) {
  finalize_loss_kernel<<<1, 1, 0, st>>>(sums, W, loss4);
  return cudaGetLastError();
}

cudaError_t launch_fill_normal(int dtype, void* p, int64_t n, int64_t flat_offset, uint64_t seed,
                               float stddev, float mean, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    fill_normal_kernel<float><<<blocks_for(n, 256), 256, 0, st>>>((float*)p, n, flat_offset, seed, stddev, mean);
  else
    fill_normal_kernel<bf16><<<blocks_for(n, 256), 256, 0, st>>>((bf16*)p, n, flat_offset, seed, stddev, mean);
  return cudaGetLastError();
}

cudaError_t launch_adamw(int dtype, void* params, float* master, float* m, float* v, const float* g, int64_t n,
                         float lr, float b1, float b2, float eps, float wd, float gscale, float bc1, float bc2,
                         cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    adamw_kernel<float><<<blocks_for(n, 1024), 256, 0, st>>>((float*)params, master, m, v, g, n, lr, b1, b2, eps, wd,
                                                             gscale, bc1, bc2);
  else
    adamw_kernel<bf16><<<blocks_for(n, 1024), 256, 0, st>>>((bf16*)params, master, m, v, g, n, lr, b1, b2, eps, wd,
                                                            gscale, bc1, bc2);
  return cudaGetLastError();
}

cudaError_t launch_cast_f32_to(int dtype, const float* src, void* dst, int64_t n, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    cast_kernel<float><<<blocks_for(n, 1024), 256, 0, st>>>(src, (float*)dst, n);
  else
    cast_kernel<bf16><<<blocks_for(n, 1024), 256, 0, st>>>(src, (bf16*)dst, n);
  return cudaGetLastError();
}

