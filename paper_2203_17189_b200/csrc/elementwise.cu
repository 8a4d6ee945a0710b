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
                            const int* __restrict__ dec_tgt, const int* __restrict__ dec_seg, int B,
                            int Te, int Td, int* __restrict__ enc_code, int* __restrict__ dec_code,
                            int* __restrict__ dec_in, int* __restrict__ W_int) {
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
    dec_code[i] = tok != 0 ? (dec_seg ? dec_seg[i] : 1) : 0;
    int u = 0;
    if (t > 0 && (dec_seg == nullptr || dec_seg[i] == dec_seg[i - 1])) u = dec_tgt[i - 1];
    dec_in[i] = u;
    cnt += tok != 0;
  }
  cnt = __reduce_add_sync(0xffffffffu, cnt);
  if ((threadIdx.x & 31) == 0 && cnt) atomicAdd(W_int, cnt);
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
  if (lane == 0) rstd[row] = r;
  T* y = Y + (int64_t)row * d;
#pragma unroll 4
  for (int c = lane * 4; c < d; c += 128) {
    float4 v = load4(x + c);
    float4 gg = load4(g + c);
    store4(y + c, make_float4(v.x * r * gg.x, v.y * r * gg.y, v.z * r * gg.z, v.w * r * gg.w));
  }
}

// dx = r (dy*g) - x r^3 mean(dy*g*x);  dg = sum_rows dy x r.
// Each warp walks rows with stride; per-CTA partial dg goes to partial[cta, d].
template <typename T, typename TDY>
__global__ void rmsnorm_bwd_kernel(const TDY* __restrict__ dY, const float* __restrict__ X,
                                   const float* __restrict__ rstd, const T* __restrict__ g,
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
    float r = rstd[row];
    float m = 0.f;
#pragma unroll 4
    for (int c = lane * 4; c < d; c += 128) {
      float4 xv = load4(x + c), dv = load4(dy + c), gv = load4(g + c);
      m += dv.x * gv.x * xv.x + dv.y * gv.y * xv.y + dv.z * gv.z * xv.z + dv.w * gv.w * xv.w;
    }
    m = warp_sum(m) / (float)d;
    float r3m = r * r * r * m;
    auto body = [&](int c, float* a4) {
      float4 xv = load4(x + c), dv = load4(dy + c), gv = load4(g + c);
      float4 o;
      o.x = r * dv.x * gv.x - xv.x * r3m;
      o.y = r * dv.y * gv.y - xv.y * r3m;
      o.z = r * dv.z * gv.z - xv.z * r3m;
      o.w = r * dv.w * gv.w - xv.w * r3m;
      if (dX_in != nullptr) {
        float4 p = load4(dX_in + (int64_t)row * d + c);
        o.x += p.x; o.y += p.y; o.z += p.z; o.w += p.w;
      }
      store4(dX_out + (int64_t)row * d + c, o);
      if (dXb != nullptr) store4(dXb + (int64_t)row * d + c, o);
      a4[0] = dv.x * xv.x * r; a4[1] = dv.y * xv.y * r; a4[2] = dv.z * xv.z * r; a4[3] = dv.w * xv.w * r;
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
// atomics), a row's x, dy and incoming dx are each read exactly once, and all of a row's loads are in flight before
// the one block-wide reduction it needs.
template <typename T, typename TDY, int NCH>
__global__ void __launch_bounds__(256)
rmsnorm_bwd_rows_kernel(const TDY* __restrict__ dY, const float* __restrict__ X, const float* __restrict__ rstd,
                        const T* __restrict__ g, const float* dX_in, float* dX_out, T* __restrict__ dXb,
                        float* __restrict__ partial, int rows, int d) {
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
  int par = 0;
  for (int row = blockIdx.x; row < rows; row += gridDim.x, par ^= 1) {
    const int64_t off = (int64_t)row * d;
    float4 xv[NCH], dv[NCH], pv[NCH];
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c = ch * 1024 + tid * 4;
      const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
      xv[ch] = c < d ? load4(X + off + c) : z;
      dv[ch] = c < d ? load4(dY + off + c) : z;
      pv[ch] = (c < d && dX_in != nullptr) ? load4(dX_in + off + c) : z;
    }
    const float r = rstd[row];
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
    const float r3m = r * r * r * tot * inv_d;
#pragma unroll
    for (int ch = 0; ch < NCH; ++ch) {
      const int c = ch * 1024 + tid * 4;
      if (c < d) {
        float4 o;
        o.x = r * dv[ch].x * gv[ch].x - xv[ch].x * r3m + pv[ch].x;
        o.y = r * dv[ch].y * gv[ch].y - xv[ch].y * r3m + pv[ch].y;
        o.z = r * dv[ch].z * gv[ch].z - xv[ch].z * r3m + pv[ch].z;
        o.w = r * dv[ch].w * gv[ch].w - xv[ch].w * r3m + pv[ch].w;
        store4(dX_out + off + c, o);
        if (dXb != nullptr) store4(dXb + off + c, o);
        acc[ch].x += dv[ch].x * xv[ch].x * r; acc[ch].y += dv[ch].y * xv[ch].y * r;
        acc[ch].z += dv[ch].z * xv[ch].z * r; acc[ch].w += dv[ch].w * xv[ch].w * r;
      }
    }
  }
#pragma unroll
  for (int ch = 0; ch < NCH; ++ch) {
    const int c = ch * 1024 + tid * 4;
    if (c < d) store4(partial + (int64_t)blockIdx.x * d + c, acc[ch]);
  }
}

__global__ void colsum_kernel(const float* __restrict__ partial, int n_part, int d, float* __restrict__ out) {
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

// h [rows, 2F] = [a | b]; hg = gelu(a) * b     (8 elements per thread)
template <typename T>
__global__ void geglu_fwd_kernel(const T* __restrict__ h, T* __restrict__ hg, int rows, int F) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int per_row = F >> 3;
  if (idx >= (int64_t)rows * per_row) return;
  int r = (int)(idx / per_row), c = (int)(idx % per_row) << 3;
  F8 a = load8(h + (int64_t)r * 2 * F + c), b = load8(h + (int64_t)r * 2 * F + F + c), o;
  constexpr bool FAST = sizeof(T) == 2;
#pragma unroll
  for (int i = 0; i < 8; ++i) o.v[i] = gelu_tanh_f<FAST>(a.v[i]) * b.v[i];
  store8(hg + (int64_t)r * F + c, o);
}
// da = dhg * b * gelu'(a); db = dhg * gelu(a)
template <typename T>
__global__ void geglu_bwd_kernel(const T* __restrict__ dhg, const T* __restrict__ h, T* __restrict__ dh,
                                 int rows, int F) {
  int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  int per_row = F >> 3;
  if (idx >= (int64_t)rows * per_row) return;
  int r = (int)(idx / per_row), c = (int)(idx % per_row) << 3;
  F8 a = load8(h + (int64_t)r * 2 * F + c), b = load8(h + (int64_t)r * 2 * F + F + c);
  F8 g = load8(dhg + (int64_t)r * F + c), da, db;
  constexpr bool FAST = sizeof(T) == 2;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    float ge, dge;
    gelu_both<FAST>(a.v[i], ge, dge);
    da.v[i] = g.v[i] * b.v[i] * dge;
    db.v[i] = g.v[i] * ge;
  }
  store8(dh + (int64_t)r * 2 * F + c, da);
  store8(dh + (int64_t)r * 2 * F + F + c, db);
}

// ------------------------------------------------------------------ cross-entropy + z-loss
// One CTA per row.  The row is staged in shared memory (as T) when it fits, so
// global memory sees one read and one write per logit.
template <typename T>
__global__ void xent_kernel(T* __restrict__ logits, const int* __restrict__ targets, int V, float z,
                            const float* __restrict__ Wp, double* __restrict__ sums,
                            float* __restrict__ lse_out, int staged) {
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
  float w = (tgt != 0 && W > 0.f) ? 1.f : 0.f;
  if (tid == 0) {
    lse_out[row] = lse;
    if (w != 0.f) {
      float tl = to_f(src[tgt]);
      atomicAdd(&sums[0], (double)(lse - tl));
      atomicAdd(&sums[1], (double)(z * lse * lse));
    }
  }
  float coef = w != 0.f ? (1.f + 2.f * z * lse) / (se * W) : 0.f;   // p = exp(v-mx)/se
  float sub = w != 0.f ? 1.f / W : 0.f;
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

template <typename T>
__global__ void cast_kernel(const float* __restrict__ s, T* __restrict__ d, int64_t n) {
  int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (i + 3 < n) {
    store4(d + i, load4(s + i));
  } else {
    for (; i < n; ++i) d[i] = from_f<T>(s[i]);
  }
}

__global__ void round_bf16_kernel(float* p, int64_t n) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) p[i] = __bfloat162float(__float2bfloat16_rn(p[i]));
}

inline unsigned blocks_for(int64_t n, int per) { return (unsigned)((n + per - 1) / per); }

}  // namespace

// =========================================================================== launchers
cudaError_t launch_prep(const int* enc_tok, const int* enc_seg, const int* dec_tgt, const int* dec_seg,
                        int B, int Te, int Td, int* enc_code, int* dec_code, int* dec_in, int* W_int,
                        float* W_f, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(W_int, 0, sizeof(int), st);
  if (e != cudaSuccess) return e;
  prep_kernel<<<B, 128, 0, st>>>(enc_tok, enc_seg, dec_tgt, dec_seg, B, Te, Td, enc_code, dec_code, dec_in,
                                 W_int);
  w_to_float_kernel<<<1, 1, 0, st>>>(W_int, W_f);
  return cudaGetLastError();
}

cudaError_t launch_embed_gather(int dtype, const void* E, const int* tok, float* X, int n_tok, int d,
                                cudaStream_t st) {
  int64_t n = (int64_t)n_tok * (d / 4);
  if (n == 0) return cudaSuccess;
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
  int p = rows < 592 ? rows : 592;      // four resident CTAs per SM
  if (p < 1) p = 1;
  return p;
}

cudaError_t launch_rmsnorm_bwd(int dtype, const void* dy, int dy_f32, const float* X, const float* rstd,
                               const void* g, const float* dX_in, float* dX_out, void* dXb, float* dg,
                               float* partial, int rows, int d, cudaStream_t st) {
  int parts = rmsnorm_bwd_parts(rows);
  if (d <= 4096) {
#define RBR(T, TDY, NCH)                                                                                          \
  rmsnorm_bwd_rows_kernel<T, TDY, NCH><<<parts, 256, 0, st>>>((const TDY*)dy, X, rstd, (const T*)g, dX_in, dX_out, \
                                                              (T*)dXb, partial, rows, d)
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
  rmsnorm_bwd_kernel<T, TDY><<<parts, 256, sm, st>>>((const TDY*)dy, X, rstd, (const T*)g, dX_in, dX_out, \
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
  colsum_kernel<<<blocks_for(d, 32), dim3(32, 16), 0, st>>>(partial, parts, d, dg);
  return cudaGetLastError();
}

cudaError_t launch_geglu_fwd(int dtype, const void* h, void* hg, int rows, int F, cudaStream_t st) {
  int64_t n = (int64_t)rows * (F / 8);
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    geglu_fwd_kernel<float><<<blocks_for(n, 256), 256, 0, st>>>((const float*)h, (float*)hg, rows, F);
  else
    geglu_fwd_kernel<bf16><<<blocks_for(n, 256), 256, 0, st>>>((const bf16*)h, (bf16*)hg, rows, F);
  return cudaGetLastError();
}

cudaError_t launch_geglu_bwd(int dtype, const void* dhg, const void* h, void* dh, int rows, int F,
                             cudaStream_t st) {
  int64_t n = (int64_t)rows * (F / 8);
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    geglu_bwd_kernel<float><<<blocks_for(n, 256), 256, 0, st>>>((const float*)dhg, (const float*)h,
                                                                (float*)dh, rows, F);
  else
    geglu_bwd_kernel<bf16><<<blocks_for(n, 256), 256, 0, st>>>((const bf16*)dhg, (const bf16*)h, (bf16*)dh,
                                                               rows, F);
  return cudaGetLastError();
}

cudaError_t launch_xent(int dtype, void* logits, const int* targets, int rows, int V, float z,
                        const float* W, double* sums, float* lse, cudaStream_t st) {
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
    xent_kernel<float><<<rows, 512, sm, st>>>((float*)logits, targets, V, z, W, sums, lse, staged);
  } else {
    if (sm > 48 * 1024) {
      e = cudaFuncSetAttribute(xent_kernel<bf16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm);
      if (e != cudaSuccess) return e;
    }
    xent_kernel<bf16><<<rows, 512, sm, st>>>((bf16*)logits, targets, V, z, W, sums, lse, staged);
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

cudaError_t launch_cast_f32_to(int dtype, const float* src, void* dst, int64_t n, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  if (dtype == DT_F32)
    cast_kernel<float><<<blocks_for(n, 1024), 256, 0, st>>>(src, (float*)dst, n);
  else
    cast_kernel<bf16><<<blocks_for(n, 1024), 256, 0, st>>>(src, (bf16*)dst, n);
  return cudaGetLastError();
}

cudaError_t launch_round_bf16(float* p, int64_t n, cudaStream_t st) {
  if (n == 0) return cudaSuccess;
  round_bf16_kernel<<<blocks_for(n, 256), 256, 0, st>>>(p, n);
  return cudaGetLastError();
}
