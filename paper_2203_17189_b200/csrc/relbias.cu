// Relative-position bias: integer bucket thresholds (host, exact), expansion of
// the [buckets, heads] table into a per-head vector indexed by the signed
// distance, and the backward fold of the distance-indexed gradient into the
// table.
#include "common.cuh"

#include <math.h>

#include <vector>

namespace {

// Minimal unsigned big integer: enough to compare n^p * me^q with MD^q * me^p.
struct BigU {
  std::vector<uint32_t> w;   // little endian
  explicit BigU(uint32_t v = 1) : w(1, v) {}
  void mul(uint32_t m) {
    uint64_t carry = 0;
    for (size_t i = 0; i < w.size(); ++i) {
      uint64_t t = (uint64_t)w[i] * m + carry;
      w[i] = (uint32_t)t;
      carry = t >> 32;
    }
    if (carry) w.push_back((uint32_t)carry);
  }
  void mul_pow(uint32_t base, int e) { for (int i = 0; i < e; ++i) mul(base); }
  bool ge(const BigU& o) const {
    if (w.size() != o.w.size()) return w.size() > o.w.size();
    for (size_t i = w.size(); i-- > 0;)
      if (w[i] != o.w[i]) return w[i] > o.w[i];
    return true;
  }
};

// floor( log(n/me)/log(MD/me) * p ) reaches q  <=>  n^p * me^q >= MD^q * me^p
bool reaches(int n, int me, int md, int p, int q) {
  long double t = (long double)p * logl((long double)n / me) / logl((long double)md / me);
  if (fabsl(t - (long double)q) > 1e-6L) return t > (long double)q;
  BigU l(1), r(1);
  l.mul_pow((uint32_t)n, p);
  l.mul_pow((uint32_t)me, q);
  r.mul_pow((uint32_t)md, q);
  r.mul_pow((uint32_t)me, p);
  return l.ge(r);
}

template <typename T>
__global__ void relbias_expand_kernel(BucketSpec spec, const T* __restrict__ table, int H, int Tq, int Tk,
                                      float* __restrict__ bias_delta) {
  int span = Tq + Tk - 1;
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= H * span) return;
  int h = idx / span, r = idx % span;
  int rel = r - (Tq - 1);
  bias_delta[idx] = to_f(table[bucket_of(spec, rel) * H + h]);
}

// dtable[bucket, h] = sum over distances of that bucket; one CTA per head.
__global__ void relbias_fold_kernel(BucketSpec spec, const float* __restrict__ dbias_delta, int H, int Tq,
                                    int Tk, int num_buckets, float* __restrict__ dtable) {
  extern __shared__ float acc[];   // [num_buckets]
  int h = blockIdx.x;
  int span = Tq + Tk - 1;
  for (int b = threadIdx.x; b < num_buckets; b += blockDim.x) acc[b] = 0.f;
  __syncthreads();
  for (int r = threadIdx.x; r < span; r += blockDim.x) {
    float v = dbias_delta[(int64_t)h * span + r];
    if (v != 0.f) atomicAdd(&acc[bucket_of(spec, r - (Tq - 1))], v);
  }
  __syncthreads();
  for (int b = threadIdx.x; b < num_buckets; b += blockDim.x) dtable[b * H + h] = acc[b];
}

__global__ void buckets_kernel(BucketSpec spec, int rel_lo, int n, int* __restrict__ out) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = bucket_of(spec, rel_lo + i);
}

}  // namespace

bool build_bucket_spec(int bidirectional, int num_buckets, int max_distance, BucketSpec* out) {
  if (num_buckets < 4 || num_buckets > 2 * T5_MAX_BUCKET_THR || (num_buckets & 3)) return false;
  int nb = bidirectional ? num_buckets / 2 : num_buckets;
  int me = nb / 2;
  int p = nb - me;
  if (max_distance <= me || max_distance > 65536) return false;
  out->bidirectional = bidirectional ? 1 : 0;
  out->nb = nb;
  out->me = me;
  // thr[q-1] = smallest n >= me whose floor(...) >= q, for q = 1 .. p-1 (q >= p is capped at nb-1)
  out->n_thr = p - 1;
  int n = me;
  for (int q = 1; q <= p - 1; ++q) {
    while (n < max_distance && !reaches(n, me, max_distance, p, q)) ++n;
    out->thr[q - 1] = n;
  }
  for (int q = p - 1; q < T5_MAX_BUCKET_THR; ++q) out->thr[q] = 0x7fffffff;
  return true;
}

cudaError_t launch_relbias_expand(int dtype, const BucketSpec& spec, const void* table, int H, int Tq, int Tk,
                                  float* bias_delta, cudaStream_t st) {
  int n = H * (Tq + Tk - 1);
  if (n <= 0) return cudaSuccess;
  if (dtype == DT_F32)
    relbias_expand_kernel<float><<<(n + 255) / 256, 256, 0, st>>>(spec, (const float*)table, H, Tq, Tk,
                                                                  bias_delta);
  else
    relbias_expand_kernel<bf16><<<(n + 255) / 256, 256, 0, st>>>(spec, (const bf16*)table, H, Tq, Tk,
                                                                 bias_delta);
  return cudaGetLastError();
}

cudaError_t launch_relbias_fold(const BucketSpec& spec, const float* dbias_delta, int H, int Tq, int Tk,
                                int num_buckets, float* dtable, cudaStream_t st) {
  relbias_fold_kernel<<<H, 256, num_buckets * sizeof(float), st>>>(spec, dbias_delta, H, Tq, Tk, num_buckets,
                                                                   dtable);
  return cudaGetLastError();
}

cudaError_t launch_buckets(const BucketSpec& spec, int rel_lo, int n, int* out, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  buckets_kernel<<<(n + 255) / 256, 256, 0, st>>>(spec, rel_lo, n, out);
  return cudaGetLastError();
}
