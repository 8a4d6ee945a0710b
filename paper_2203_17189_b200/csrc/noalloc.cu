// Attention backward for callers that cannot allocate device memory.
//
// The regular backward call needs a scratch vector delta[B, H, Tq] (one float per
// query row and head) that the caller allocates.  Some callers cannot do that:
// code running in a region where cudaMalloc is illegal or must be avoided,
// plug-ins handed only their input and output buffers by a host framework that
// owns the allocator, and processes whose device memory pool is fully committed
// at start-up.  For them the scratch lives in a fixed-size array that is part of
// the library image.
#include "../../include/t5_b200.h"
#include "common.cuh"

#include <string.h>

namespace {

constexpr int64_t kMaxDeltaFloats = T5_NOALLOC_MAX_ROWS;   // B * H * Tq of one call

// Every GPU that loads the library holds this array (4 MiB) until the process exits.
static __device__ __align__(256) float g_delta_scratch[kMaxDeltaFloats];

constexpr int kMaxDevices = 64;
float* g_scratch_ptr[kMaxDevices];      // device address of g_delta_scratch, per device (0 = not set up)

// In host code the array's name is only a handle; kernels need its device address, which differs
// per device.  Looked up once per device, with that device current.
cudaError_t scratch_for_current_device(float** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (g_scratch_ptr[dev] == nullptr) {
    float* p = nullptr;
    e = cudaGetSymbolAddress((void**)&p, g_delta_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int t5_attention_backward_noalloc(
    int32_t dtype, int32_t impl, int32_t B, int32_t H, int32_t Tq, int32_t Tk, int32_t d_kv, int32_t causal,
    float scale, const void* d_q, int32_t ldq, const void* d_k, int32_t ldk, const void* d_v, int32_t ldv,
    const void* d_o, int32_t ldo, const float* d_o32, const float* d_lse, const int32_t* d_code_q,
    const int32_t* d_code_k, const float* d_bias_delta, const void* d_do, int32_t lddo, void* d_dq, int32_t lddq,
    void* d_dk, int32_t lddk, void* d_dv, int32_t lddv, float* d_dbias_delta, void* stream) {
  if (!d_q || !d_k || !d_v || !d_o || !d_lse || !d_code_q || !d_code_k || !d_do || !d_dq || !d_dk || !d_dv)
    return T5_ERR_NULL;
  if ((dtype != DT_F32 && dtype != DT_BF16) || B < 1 || H < 1 || Tq < 1 || Tk < 1) return T5_ERR_ARG;
  if (d_kv != 32 && d_kv != 64 && d_kv != 128) return T5_ERR_ARG;
  if ((int64_t)B * H * Tq > kMaxDeltaFloats) return T5_ERR_SHAPE;   // B*H*Tq beyond the built-in scratch
  float* delta = nullptr;
  if (scratch_for_current_device(&delta) != cudaSuccess) return T5_ERR_CUDA;
  AttnArgs a;
  memset(&a, 0, sizeof a);
  a.Q = d_q; a.K = d_k; a.V = d_v; a.O = const_cast<void*>(d_o); a.ldq = ldq; a.ldk = ldk; a.ldv = ldv; a.ldo = ldo;
  a.O32 = const_cast<float*>(d_o32); a.ldo32 = H * d_kv; a.lse = const_cast<float*>(d_lse);
  a.B = B; a.H = H; a.Tq = Tq; a.Tk = Tk; a.dk = d_kv; a.code_q = d_code_q; a.code_k = d_code_k; a.causal = causal;
  a.bias_delta = d_bias_delta; a.scale = scale; a.dO = d_do; a.lddo = lddo; a.dQ = d_dq; a.dK = d_dk; a.dV = d_dv;
  a.lddq = lddq; a.lddk = lddk; a.lddv = lddv; a.delta = delta; a.dbias_delta = d_dbias_delta;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e;
  if (impl == 0) {
    e = attn_bwd_simt(dtype, a, st);
  } else {
    if (dtype != DT_BF16 || !attn_tc_supported(a)) return T5_ERR_ARG;
    e = attn_bwd_tc(a, g_kernel_status, st);
  }
  return e == cudaSuccess ? T5_OK : T5_ERR_CUDA;
}
