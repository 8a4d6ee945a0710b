// SIMT attention (forward and backward) with float32 arithmetic: the float32
// validation mode's kernels and the cross-check for the tensor-core path.
//   S_ij = scale q_i.k_j + bias_delta[h, j-i];  masked entries excluded;
//   P = softmax_j(S) (online max/sum);  O = P V;  lse_i = log sum_j exp(S_ij).
// Backward recomputes P from lse:  dV = P^T dO, dP = dO V^T,
//   dS = P (dP - delta_i), delta_i = dO_i.O_i,  dQ = scale dS K,  dK = scale dS^T Q,
//   dbias_delta[h, j-i] += dS_ij.
#include "common.cuh"

#include <math.h>

namespace {

__device__ __forceinline__ float wsum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float wmax(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

struct P {   // plain-pointer copy of AttnArgs for the kernels
  const void *Q, *K, *V, *dO;
  void *O, *dQ, *dK, *dV;
  int ldq, ldk, ldv, ldo, lddo, lddq, lddk, lddv;
  float *lse, *delta, *dbias_delta, *O32;
  int ldo32;
  const float* bias_delta;
  const int *code_q, *code_k;
  int B, H, Tq, Tk, causal;
  int prefix;      // see AttnArgs::prefix: tiles are not cut at the diagonal
  float scale;
  RowNorm rn_q, rn_k;      // row factors of dQ and of dK / dV (folded RMSNorm), see AttnArgs
};

template <typename T, int DK>
__global__ void __launch_bounds__(128) attn_fwd_kernel(P a) {
  extern __shared__ float sm[];
  float* Qs = sm;                       // [32][DK]
  float* Ks = Qs + 32 * DK;             // [32][DK+1]
  float* Vs = Ks + 32 * (DK + 1);       // [32][DK+1]
  int* cks = reinterpret_cast<int*>(Vs + 32 * (DK + 1));   // [32]
  constexpr int C = DK / 32;
  int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * 32;
  int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* Q = (const T*)a.Q; const T* K = (const T*)a.K; const T* V = (const T*)a.V;
  for (int idx = tid; idx < 32 * DK; idx += 128) {
    int i = idx / DK, d = idx % DK, gi = q0 + i;
    Qs[i * DK + d] = gi < a.Tq ? to_f(Q[(int64_t)(b * a.Tq + gi) * a.ldq + h * DK + d]) : 0.f;
  }
  int cq[8];
  float m[8], l[8], o[8][C];
#pragma unroll
  for (int qq = 0; qq < 8; ++qq) {
    int gi = q0 + warp * 8 + qq;
    cq[qq] = gi < a.Tq ? a.code_q[b * a.Tq + gi] : 0;
    m[qq] = -INFINITY; l[qq] = 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) o[qq][c] = 0.f;
  }
  int span = a.Tq + a.Tk - 1;
  int k_end = (a.causal && !a.prefix) ? min(a.Tk, q0 + 32) : a.Tk;
  for (int k0 = 0; k0 < k_end; k0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * DK; idx += 128) {
      int j = idx / DK, d = idx % DK, gj = k0 + j;
      bool in = gj < a.Tk;
      Ks[j * (DK + 1) + d] = in ? to_f(K[(int64_t)(b * a.Tk + gj) * a.ldk + h * DK + d]) : 0.f;
      Vs[j * (DK + 1) + d] = in ? to_f(V[(int64_t)(b * a.Tk + gj) * a.ldv + h * DK + d]) : 0.f;
    }
    if (tid < 32) cks[tid] = (k0 + tid) < a.Tk ? a.code_k[b * a.Tk + k0 + tid] : 0;
    __syncthreads();
    int j = k0 + lane;
    int ck = cks[lane];
#pragma unroll
    for (int qq = 0; qq < 8; ++qq) {
      int il = warp * 8 + qq, i = q0 + il;
      float s = 0.f;
#pragma unroll 8
      for (int d = 0; d < DK; ++d) s = fmaf(Qs[il * DK + d], Ks[lane * (DK + 1) + d], s);
      bool valid = pair_valid(cq[qq], ck, a.causal != 0, j, i) && j < a.Tk && i < a.Tq;
      s *= a.scale;
      if (valid && a.bias_delta) s += a.bias_delta[h * span + (j - i + a.Tq - 1)];
      s = valid ? s : -INFINITY;
      float m_new = fmaxf(m[qq], wmax(s));
      if (m_new == -INFINITY) continue;
      float p = valid ? __expf(s - m_new) : 0.f;
      float corr = m[qq] == -INFINITY ? 0.f : __expf(m[qq] - m_new);
      l[qq] = l[qq] * corr + wsum(p);
#pragma unroll
      for (int c = 0; c < C; ++c) o[qq][c] *= corr;
      for (int jj = 0; jj < 32; ++jj) {
        float pj = __shfl_sync(0xffffffffu, p, jj);
#pragma unroll
        for (int c = 0; c < C; ++c) o[qq][c] = fmaf(pj, Vs[jj * (DK + 1) + lane + 32 * c], o[qq][c]);
      }
      m[qq] = m_new;
    }
  }
  T* O = (T*)a.O;
#pragma unroll
  for (int qq = 0; qq < 8; ++qq) {
    int i = q0 + warp * 8 + qq;
    if (i >= a.Tq) continue;
    float inv = l[qq] > 0.f ? 1.f / l[qq] : 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c)
      O[(int64_t)(b * a.Tq + i) * a.ldo + h * DK + lane + 32 * c] = from_f<T>(o[qq][c] * inv);
    if (a.O32)
#pragma unroll
      for (int c = 0; c < C; ++c) a.O32[(int64_t)(b * a.Tq + i) * a.ldo32 + h * DK + lane + 32 * c] = o[qq][c] * inv;
    if (lane == 0) a.lse[(int64_t)(b * a.H + h) * a.Tq + i] = l[qq] > 0.f ? m[qq] + logf(l[qq]) : -INFINITY;
  }
}

// delta[b,h,i] = sum_d dO[i,d] O[i,d]; one warp per (b,i,h)
template <typename T, int DK>
__global__ void attn_delta_kernel(P a) {
  int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  int total = a.B * a.Tq * a.H;
  if (gw >= total) return;
  int h = gw % a.H, row = gw / a.H;    // row = b*Tq + i
  int b = row / a.Tq, i = row % a.Tq;
  const T* O = (const T*)a.O; const T* dO = (const T*)a.dO;
  float s = 0.f;
#pragma unroll
  for (int c = 0; c < DK / 32; ++c)
    s += (a.O32 ? a.O32[(int64_t)row * a.ldo32 + h * DK + lane + 32 * c]
                : to_f(O[(int64_t)row * a.ldo + h * DK + lane + 32 * c])) *
         to_f(dO[(int64_t)row * a.lddo + h * DK + lane + 32 * c]);
  s = wsum(s);
  if (lane == 0) a.delta[(int64_t)(b * a.H + h) * a.Tq + i] = s;
}

// dQ and dbias: CTA = 32 queries of one (b,h); lane = key inside a 32-key tile.
template <typename T, int DK>
__global__ void __launch_bounds__(128) attn_bwd_dq_kernel(P a) {
  extern __shared__ float sm[];
  float* Qs = sm;                        // [32][DK]
  float* dOs = Qs + 32 * DK;             // [32][DK]
  float* Ks = dOs + 32 * DK;             // [32][DK+1]
  float* Vs = Ks + 32 * (DK + 1);        // [32][DK+1]
  int* cks = reinterpret_cast<int*>(Vs + 32 * (DK + 1));   // [32]
  float* dbs = reinterpret_cast<float*>(cks + 32);          // [Tk + 31]
  constexpr int C = DK / 32;
  int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * 32;
  int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* Q = (const T*)a.Q; const T* K = (const T*)a.K; const T* V = (const T*)a.V;
  const T* dO = (const T*)a.dO;
  for (int idx = tid; idx < 32 * DK; idx += 128) {
    int i = idx / DK, d = idx % DK, gi = q0 + i;
    bool in = gi < a.Tq;
    Qs[idx] = in ? to_f(Q[(int64_t)(b * a.Tq + gi) * a.ldq + h * DK + d]) : 0.f;
    dOs[idx] = in ? to_f(dO[(int64_t)(b * a.Tq + gi) * a.lddo + h * DK + d]) : 0.f;
  }
  bool want_db = a.dbias_delta != nullptr;
  if (want_db)
    for (int idx = tid; idx < a.Tk + 31; idx += 128) dbs[idx] = 0.f;
  int cq[8];
  float lse[8], dl[8], dq[8][C];
#pragma unroll
  for (int qq = 0; qq < 8; ++qq) {
    int gi = q0 + warp * 8 + qq;
    bool in = gi < a.Tq;
    cq[qq] = in ? a.code_q[b * a.Tq + gi] : 0;
    lse[qq] = in ? a.lse[(int64_t)(b * a.H + h) * a.Tq + gi] : -INFINITY;
    dl[qq] = in ? a.delta[(int64_t)(b * a.H + h) * a.Tq + gi] : 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) dq[qq][c] = 0.f;
  }
  int span = a.Tq + a.Tk - 1;
  int k_end = (a.causal && !a.prefix) ? min(a.Tk, q0 + 32) : a.Tk;
  for (int k0 = 0; k0 < k_end; k0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * DK; idx += 128) {
      int j = idx / DK, d = idx % DK, gj = k0 + j;
      bool in = gj < a.Tk;
      Ks[j * (DK + 1) + d] = in ? to_f(K[(int64_t)(b * a.Tk + gj) * a.ldk + h * DK + d]) : 0.f;
      Vs[j * (DK + 1) + d] = in ? to_f(V[(int64_t)(b * a.Tk + gj) * a.ldv + h * DK + d]) : 0.f;
    }
    if (tid < 32) cks[tid] = (k0 + tid) < a.Tk ? a.code_k[b * a.Tk + k0 + tid] : 0;
    __syncthreads();
    int j = k0 + lane;
    int ck = cks[lane];
#pragma unroll
    for (int qq = 0; qq < 8; ++qq) {
      int il = warp * 8 + qq, i = q0 + il;
      float s = 0.f, dp = 0.f;
#pragma unroll 8
      for (int d = 0; d < DK; ++d) {
        s = fmaf(Qs[il * DK + d], Ks[lane * (DK + 1) + d], s);
        dp = fmaf(dOs[il * DK + d], Vs[lane * (DK + 1) + d], dp);
      }
      bool valid = pair_valid(cq[qq], ck, a.causal != 0, j, i) && j < a.Tk && i < a.Tq &&
                   lse[qq] != -INFINITY;
      s *= a.scale;
      if (valid && a.bias_delta) s += a.bias_delta[h * span + (j - i + a.Tq - 1)];
      float p = valid ? __expf(s - lse[qq]) : 0.f;
      float ds = p * (dp - dl[qq]);
      if (want_db && valid) atomicAdd(&dbs[j - il + 31 - 0], ds);   // local index: (j - i) + q0 + 31
      for (int jj = 0; jj < 32; ++jj) {
        float dsj = __shfl_sync(0xffffffffu, ds, jj);
#pragma unroll
        for (int c = 0; c < C; ++c) dq[qq][c] = fmaf(dsj, Ks[jj * (DK + 1) + lane + 32 * c], dq[qq][c]);
      }
    }
  }
  T* dQ = (T*)a.dQ;
#pragma unroll
  for (int qq = 0; qq < 8; ++qq) {
    int i = q0 + warp * 8 + qq;
    if (i >= a.Tq) continue;
    const float f = a.scale * rn_factor(a.rn_q, (int64_t)b * a.Tq + i);
#pragma unroll
    for (int c = 0; c < C; ++c)
      dQ[(int64_t)(b * a.Tq + i) * a.lddq + h * DK + lane + 32 * c] = from_f<T>(f * dq[qq][c]);
  }
  if (want_db) {
    __syncthreads();
    // dbs index x holds distance (j - i) = x - 31 - q0  ->  global index x - 31 - q0 + Tq - 1
    for (int x = tid; x < a.Tk + 31; x += 128) {
      float v = dbs[x];
      int gidx = x - 31 - q0 + a.Tq - 1;
      if (v != 0.f && gidx >= 0 && gidx < span) atomicAdd(&a.dbias_delta[(int64_t)h * span + gidx], v);
    }
  }
}

// dK and dV: CTA = 32 keys of one (b,h), 8 per warp; lane = query inside a 32-query tile.
template <typename T, int DK>
__global__ void __launch_bounds__(128) attn_bwd_dkv_kernel(P a) {
  extern __shared__ float sm[];
  float* Ks = sm;                        // [32][DK]
  float* Vs = Ks + 32 * DK;              // [32][DK]
  float* Qs = Vs + 32 * DK;              // [32][DK+1]
  float* dOs = Qs + 32 * (DK + 1);       // [32][DK+1]
  float* lses = dOs + 32 * (DK + 1);     // [32]
  float* dls = lses + 32;                // [32]
  int* cqs = reinterpret_cast<int*>(dls + 32);   // [32]
  constexpr int C = DK / 32;
  int b = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * 32;
  int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const T* Q = (const T*)a.Q; const T* K = (const T*)a.K; const T* V = (const T*)a.V;
  const T* dO = (const T*)a.dO;
  for (int idx = tid; idx < 32 * DK; idx += 128) {
    int j = idx / DK, d = idx % DK, gj = k0 + j;
    bool in = gj < a.Tk;
    Ks[idx] = in ? to_f(K[(int64_t)(b * a.Tk + gj) * a.ldk + h * DK + d]) : 0.f;
    Vs[idx] = in ? to_f(V[(int64_t)(b * a.Tk + gj) * a.ldv + h * DK + d]) : 0.f;
  }
  int ck[8];
  float dk[8][C], dv[8][C];
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    int gj = k0 + warp * 8 + kk;
    ck[kk] = gj < a.Tk ? a.code_k[b * a.Tk + gj] : 0;
#pragma unroll
    for (int c = 0; c < C; ++c) dk[kk][c] = dv[kk][c] = 0.f;
  }
  int span = a.Tq + a.Tk - 1;
  int q_begin = (a.causal && !a.prefix) ? k0 : 0;     // k0 is a multiple of 32: queries before it see none of these keys
  for (int q0 = q_begin; q0 < a.Tq; q0 += 32) {
    __syncthreads();
    for (int idx = tid; idx < 32 * DK; idx += 128) {
      int i = idx / DK, d = idx % DK, gi = q0 + i;
      bool in = gi < a.Tq;
      Qs[i * (DK + 1) + d] = in ? to_f(Q[(int64_t)(b * a.Tq + gi) * a.ldq + h * DK + d]) : 0.f;
      dOs[i * (DK + 1) + d] = in ? to_f(dO[(int64_t)(b * a.Tq + gi) * a.lddo + h * DK + d]) : 0.f;
    }
    if (tid < 32) {
      int gi = q0 + tid;
      bool in = gi < a.Tq;
      lses[tid] = in ? a.lse[(int64_t)(b * a.H + h) * a.Tq + gi] : -INFINITY;
      dls[tid] = in ? a.delta[(int64_t)(b * a.H + h) * a.Tq + gi] : 0.f;
      cqs[tid] = in ? a.code_q[b * a.Tq + gi] : 0;
    }
    __syncthreads();
    int i = q0 + lane;
    int cq = cqs[lane];
    float lse = lses[lane], dl = dls[lane];
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      int jl = warp * 8 + kk, j = k0 + jl;
      float s = 0.f, dp = 0.f;
#pragma unroll 8
      for (int d = 0; d < DK; ++d) {
        s = fmaf(Qs[lane * (DK + 1) + d], Ks[jl * DK + d], s);
        dp = fmaf(dOs[lane * (DK + 1) + d], Vs[jl * DK + d], dp);
      }
      bool valid = pair_valid(cq, ck[kk], a.causal != 0, j, i) && j < a.Tk && i < a.Tq &&
                   lse != -INFINITY;
      s *= a.scale;
      if (valid && a.bias_delta) s += a.bias_delta[h * span + (j - i + a.Tq - 1)];
      float p = valid ? __expf(s - lse) : 0.f;
      float ds = p * (dp - dl);
      for (int ii = 0; ii < 32; ++ii) {
        float pi = __shfl_sync(0xffffffffu, p, ii);
        float dsi = __shfl_sync(0xffffffffu, ds, ii);
#pragma unroll
        for (int c = 0; c < C; ++c) {
          dv[kk][c] = fmaf(pi, dOs[ii * (DK + 1) + lane + 32 * c], dv[kk][c]);
          dk[kk][c] = fmaf(dsi, Qs[ii * (DK + 1) + lane + 32 * c], dk[kk][c]);
        }
      }
    }
  }
  T* dK = (T*)a.dK; T* dV = (T*)a.dV;
#pragma unroll
  for (int kk = 0; kk < 8; ++kk) {
    int j = k0 + warp * 8 + kk;
    if (j >= a.Tk) continue;
    const float f = rn_factor(a.rn_k, (int64_t)b * a.Tk + j);
#pragma unroll
    for (int c = 0; c < C; ++c) {
      dK[(int64_t)(b * a.Tk + j) * a.lddk + h * DK + lane + 32 * c] = from_f<T>(f * a.scale * dk[kk][c]);
      dV[(int64_t)(b * a.Tk + j) * a.lddv + h * DK + lane + 32 * c] = from_f<T>(f * dv[kk][c]);
    }
  }
}

P to_p(const AttnArgs& a) {
  P p;
  p.Q = a.Q; p.K = a.K; p.V = a.V; p.dO = a.dO; p.O = a.O; p.dQ = a.dQ; p.dK = a.dK; p.dV = a.dV;
  p.ldq = a.ldq; p.ldk = a.ldk; p.ldv = a.ldv; p.ldo = a.ldo; p.lddo = a.lddo; p.lddq = a.lddq;
  p.lddk = a.lddk; p.lddv = a.lddv; p.lse = a.lse; p.delta = a.delta; p.dbias_delta = a.dbias_delta;
  p.O32 = a.O32; p.ldo32 = a.ldo32;
  p.bias_delta = a.bias_delta; p.code_q = a.code_q; p.code_k = a.code_k; p.B = a.B; p.H = a.H;
  p.Tq = a.Tq; p.Tk = a.Tk; p.causal = a.causal; p.scale = a.scale;
  p.rn_q = a.rn_q; p.rn_k = a.rn_k;
  p.prefix = a.prefix;
  return p;
}

template <typename T, int DK>
cudaError_t fwd_t(const AttnArgs& a, cudaStream_t st) {
  size_t smem = (32 * DK + 2 * 32 * (DK + 1) + 32) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_kernel<T, DK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.Tq + 31) / 32, a.H, a.B);
  attn_fwd_kernel<T, DK><<<grid, 128, smem, st>>>(to_p(a));
  return cudaGetLastError();
}

template <typename T, int DK>
cudaError_t bwd_t(const AttnArgs& a, cudaStream_t st) {
  P p = to_p(a);
  int total_warps = a.B * a.Tq * a.H;
  attn_delta_kernel<T, DK><<<(total_warps + 7) / 8, 256, 0, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  size_t smem_q = (2 * 32 * DK + 2 * 32 * (DK + 1) + 32 + a.Tk + 32) * sizeof(float);
  e = cudaFuncSetAttribute(attn_bwd_dq_kernel<T, DK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_q);
  if (e != cudaSuccess) return e;
  dim3 gq((a.Tq + 31) / 32, a.H, a.B);
  attn_bwd_dq_kernel<T, DK><<<gq, 128, smem_q, st>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  size_t smem_k = (2 * 32 * DK + 2 * 32 * (DK + 1) + 96) * sizeof(float);
  e = cudaFuncSetAttribute(attn_bwd_dkv_kernel<T, DK>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           (int)smem_k);
  if (e != cudaSuccess) return e;
  dim3 gk((a.Tk + 31) / 32, a.H, a.B);
  attn_bwd_dkv_kernel<T, DK><<<gk, 128, smem_k, st>>>(p);
  return cudaGetLastError();
}

}  // namespace

#define DISPATCH(fn)                                                      \
  if (dtype == DT_F32) {                                                  \
    if (a.dk == 32) return fn<float, 32>(a, st);                          \
    if (a.dk == 64) return fn<float, 64>(a, st);                          \
    if (a.dk == 128) return fn<float, 128>(a, st);                        \
  } else {                                                                \
    if (a.dk == 32) return fn<bf16, 32>(a, st);                           \
    if (a.dk == 64) return fn<bf16, 64>(a, st);                           \
    if (a.dk == 128) return fn<bf16, 128>(a, st);                         \
  }                                                                       \
  return cudaErrorInvalidValue;

cudaError_t attn_fwd_simt(int dtype, const AttnArgs& a, cudaStream_t st) {
  if (a.B == 0 || a.Tq == 0) return cudaSuccess;
  DISPATCH(fwd_t)
}
cudaError_t attn_bwd_simt(int dtype, const AttnArgs& a, cudaStream_t st) {
  if (a.B == 0 || a.Tq == 0) return cudaSuccess;
  DISPATCH(bwd_t)
}
