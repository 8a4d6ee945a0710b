// Plain shared-memory-tiled SIMT GEMM with float32 accumulation.  It is the
// arithmetic of the float32 validation mode and the cross-check for the
// tcgen05 kernel; it handles any shape, stride and operand orientation.
#include "common.cuh"

namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <typename T, typename TD, bool AK, bool BK>
__global__ void __launch_bounds__(256) gemm_simt_kernel(int M, int N, int K, float alpha,
                                                        const T* __restrict__ A, int lda,
                                                        const T* __restrict__ B, int ldb, TD* D, int ldd,
                                                        const float* resid, int ldr, int accumulate, RowNorm rn,
                                                        T* xg_out, int ld_xg, const T* g_next, float* ssq_out) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  int tid = threadIdx.x;
  int tx = tid & 15, ty = tid >> 4;
  int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int m, k;
      if (AK) { k = tid & 15; m = (tid >> 4) + 16 * i; } else { m = tid & 63; k = (tid >> 6) + 4 * i; }
      int gm = m0 + m, gk = k0 + k;
      float v = 0.f;
      if (gm < M && gk < K) v = to_f(AK ? A[(int64_t)gm * lda + gk] : A[(int64_t)gk * lda + gm]);
      As[k][m] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int n, k;
      if (BK) { k = tid & 15; n = (tid >> 4) + 16 * i; } else { n = tid & 63; k = (tid >> 6) + 4 * i; }
      int gn = n0 + n, gk = k0 + k;
      float v = 0.f;
      if (gn < N && gk < K) v = to_f(BK ? B[(int64_t)gn * ldb + gk] : B[(int64_t)gk * ldb + gn]);
      Bs[k][n] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < TK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    int gm = m0 + ty * 4 + i;
    if (gm >= M) continue;
    const float arow = alpha * rn_factor(rn, gm);      // folded RMSNorm: factor of the product's row
    float ss = 0.f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      int gn = n0 + tx * 4 + j;
      if (gn >= N) continue;
      float v = arow * acc[i][j];
      if (resid != nullptr) v += resid[(int64_t)gm * ldr + gn];
      TD* dp = D + (int64_t)gm * ldd + gn;
      if (accumulate) v += to_f(*dp);
      *dp = from_f<TD>(v);
      if (xg_out != nullptr) {      // producer side of the fold: operand copy x * g and the row's sum of squares
        xg_out[(int64_t)gm * ld_xg + gn] = from_f<T>(v * to_f(g_next[gn]));
        ss += v * v;
      }
    }
    if (xg_out != nullptr) atomicAdd(ssq_out + gm, ss);
  }
}

template <typename T, typename TD>
cudaError_t launch(const GemmArgs& g, cudaStream_t st) {
  dim3 grid((g.N + TN - 1) / TN, (g.M + TM - 1) / TM);
  if (g.M <= 0 || g.N <= 0) return cudaSuccess;
#define GO(AK, BK)                                                                                   \
  gemm_simt_kernel<T, TD, AK, BK><<<grid, 256, 0, st>>>(g.M, g.N, g.K, g.alpha, (const T*)g.A, g.lda, \
                                                        (const T*)g.B, g.ldb, (TD*)g.D, g.ldd, g.resid, \
                                                        g.ldr, g.accumulate, g.rn, (T*)g.xg_out, g.ld_xg,    \
                                                        (const T*)g.g_next, g.ssq_out)
  if (g.a_kmajor && g.b_kmajor) GO(true, true);
  else if (g.a_kmajor) GO(true, false);
  else if (g.b_kmajor) GO(false, true);
  else GO(false, false);
#undef GO
  return cudaGetLastError();
}

}  // namespace

cudaError_t gemm_simt(int dtype, const GemmArgs& g, cudaStream_t st) {
  if (dtype == DT_F32) return launch<float, float>(g, st);
  if (g.out_f32) return launch<bf16, float>(g, st);
  return launch<bf16, bf16>(g, st);
}
