// bf16 GEMM on the 5th-generation tensor cores: D[M,N] = alpha * A * B (+resid / +D)
// with float32 accumulation in tensor memory.
//
// One persistent CTA per SM walks 128 x BN output tiles.  Warp roles:
//   warp 0  : TMA producer  - cp.async.bulk.tensor loads of 64-deep K slices of A and B
//             into a ring of 128-byte-swizzled shared-memory stages (mbarrier full/empty)
//   warp 1  : MMA issuer    - one thread issues tcgen05.mma (M=128, N=BN, K=16) from
//             shared-memory descriptors; tcgen05.commit releases stages and publishes
//             accumulators
//   warp 2  : allocates / frees tensor memory (2 accumulator buffers of BN columns)
//   warps 4-7: epilogue     - tcgen05.ld of the accumulator (one row per thread),
//             scaling / residual / accumulate, vector stores to global memory;
//             runs on buffer a while the MMA warp fills buffer a^1.
// Either operand may be K-major (contraction dimension contiguous) or MN-major; the
// latter is loaded as 64x64 boxes and described to the tensor core as a transposed
// operand, so backward GEMMs need no transposed copies.
// Every mbarrier wait is bounded: when the limit runs out the kernel records a code in
// *status, drains its own TMA loads, frees tensor memory and returns.
#include "common.cuh"
#include "tc_common.cuh"

namespace {

using namespace tc;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int kThreads = 256;

struct Params {
  int M, N, K;
  float alpha;
  void* D;
  int ldd;
  int out_f32;
  const float* resid;
  int ldr;
  int accumulate;
  int tiles_m, tiles_n;
  int* status;
};

template <int BN, int STAGES>
struct Smem {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarOffset = STAGES * kStageBytes;
  static constexpr int kTotal = kBarOffset + 256 + 1024;   // barriers + slack for 1024-byte alignment
};

template <int BN, int STAGES, bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, Params p) {
  using S = Smem<BN, STAGES>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + S::kBarOffset);
  uint64_t* empty = full + STAGES;
  uint64_t* tfull = empty + STAGES;      // [2]
  uint64_t* tempty = tfull + 2;          // [2]
  uint32_t* tmem_holder = (uint32_t*)(tempty + 2);
  volatile int* abort_flag = (volatile int*)(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_tiles = p.tiles_m * p.tiles_n;
  const int k_blocks = (p.K + BK - 1) / BK;
  constexpr uint32_t kTmemCols = 2 * BN;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) tmem_alloc(tmem_holder, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      uint32_t issued[STAGES];
#pragma unroll
      for (int i = 0; i < STAGES; ++i) issued[i] = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
        const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag, p.status, 1)) { ok = false; break; }
          unsigned char* sa = smem + s * S::kStageBytes;
          unsigned char* sb = sa + S::kABytes;
          mbar_arrive_expect_tx(&full[s], S::kStageBytes);
          const int k0 = kb * BK;
          if (!A_MN) {
            tma_load_2d(sa, &map_a, k0, m0, &full[s]);
          } else {
#pragma unroll
            for (int c = 0; c < BM / 64; ++c) tma_load_2d(sa + c * 8192, &map_a, m0 + c * 64, k0, &full[s]);
          }
          if (!B_MN) {
            tma_load_2d(sb, &map_b, k0, n0, &full[s]);
          } else {
#pragma unroll
            for (int c = 0; c < BN / 64; ++c) tma_load_2d(sb + c * 8192, &map_b, n0 + c * 64, k0, &full[s]);
          }
#pragma unroll
          for (int i = 0; i < STAGES; ++i)
            if (i == s) issued[i] += 1;
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
      }
      if (!ok) {
        // drain: every load this thread issued must land before the CTA gives up its shared memory
#pragma unroll
        for (int i = 0; i < STAGES; ++i) {
          if (issued[i] == 0) continue;
          uint32_t par = (issued[i] - 1) & 1;
          long long t0 = clock64();
          while (!mbar_try_wait(&full[i], par) && clock64() - t0 < kWaitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BM, BN, A_MN, B_MN);
      int s = 0;
      uint32_t ph = 0;
      int it = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
        const int ab = it & 1;
        const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(&tempty[ab], aph ^ 1, abort_flag, p.status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + ab * BN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!mbar_wait(&full[s], ph, abort_flag, p.status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * S::kStageBytes);
          const uint32_t sb = sa + S::kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            // K-major: 16 elements = 32 bytes further inside the 128-byte swizzled row;
            // MN-major: 16 K-rows = two 8-row groups of 1024 bytes further.
            uint64_t da = A_MN ? make_desc(sa + k * 2048, 8192, 1024) : make_desc(sa + k * 32, 16, 1024);
            uint64_t db = B_MN ? make_desc(sb + k * 2048, 8192, 1024) : make_desc(sb + k * 32, 16, 1024);
            umma_bf16(tacc, da, db, idesc, (kb | k) != 0);
          }
          umma_commit(&empty[s]);
          if (++s == STAGES) { s = 0; ph ^= 1; }
        }
        if (ok) umma_commit(&tfull[ab]);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue
    const int quad = warp & 3;
    int it = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
      const int m0 = (tile % p.tiles_m) * BM, n0 = (tile / p.tiles_m) * BN;
      const int ab = it & 1;
      const uint32_t aph = (it >> 1) & 1;
      if (p.out_f32 && (p.resid || p.accumulate)) {
        // the float32 addend of this thread's row: pull its cache lines into L2 while the MMAs of the tile run
        const int prow = m0 + quad * 32 + lane;
        if (prow < p.M) {
          const float* pr = p.resid ? p.resid + (int64_t)prow * p.ldr + n0 : (const float*)p.D + (int64_t)prow * p.ldd + n0;
#pragma unroll
          for (int c = 0; c < BN / 32; ++c)
            if (n0 + c * 32 < p.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(pr + c * 32));
        }
      }
      ok = mbar_wait(&tfull[ab], aph, abort_flag, p.status, 4);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const int row = m0 + quad * 32 + lane;
      const uint32_t tacc = tmem_base + ab * BN + ((uint32_t)(quad * 32) << 16);
#pragma unroll 1
      for (int c = 0; c < BN / 32; ++c) {
        const int col = n0 + c * 32;
        if (col >= p.N) break;               // uniform across the warp
        uint32_t r[32];
        tmem_ld_32x32b_x32(tacc + c * 32, r);
        tmem_wait_ld_dep(r);
        if (row < p.M) {
          const bool full_chunk = col + 32 <= p.N;
          if (p.out_f32) {
            float* d = (float*)p.D + (int64_t)row * p.ldd + col;
            const float* rs = p.resid ? p.resid + (int64_t)row * p.ldr + col : (p.accumulate ? d : nullptr);
            if (full_chunk) {
#pragma unroll
              for (int j = 0; j < 32; j += 4) {
                float4 v = make_float4(p.alpha * __uint_as_float(r[j]), p.alpha * __uint_as_float(r[j + 1]),
                                       p.alpha * __uint_as_float(r[j + 2]), p.alpha * __uint_as_float(r[j + 3]));
                if (rs) {
                  float4 a = *reinterpret_cast<const float4*>(rs + j);
                  v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
                }
                *reinterpret_cast<float4*>(d + j) = v;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (col + j < p.N) {
                  float v = p.alpha * __uint_as_float(r[j]);
                  if (rs) v += rs[j];
                  d[j] = v;
                }
              }
            }
          } else {
            bf16* d = (bf16*)p.D + (int64_t)row * p.ldd + col;
            if (full_chunk) {
#pragma unroll
              for (int j = 0; j < 32; j += 8) {
                uint4 o;
                __nv_bfloat162 b0 = __floats2bfloat162_rn(p.alpha * __uint_as_float(r[j]), p.alpha * __uint_as_float(r[j + 1]));
                __nv_bfloat162 b1 = __floats2bfloat162_rn(p.alpha * __uint_as_float(r[j + 2]), p.alpha * __uint_as_float(r[j + 3]));
                __nv_bfloat162 b2 = __floats2bfloat162_rn(p.alpha * __uint_as_float(r[j + 4]), p.alpha * __uint_as_float(r[j + 5]));
                __nv_bfloat162 b3 = __floats2bfloat162_rn(p.alpha * __uint_as_float(r[j + 6]), p.alpha * __uint_as_float(r[j + 7]));
                o.x = *reinterpret_cast<uint32_t*>(&b0); o.y = *reinterpret_cast<uint32_t*>(&b1);
                o.z = *reinterpret_cast<uint32_t*>(&b2); o.w = *reinterpret_cast<uint32_t*>(&b3);
                *reinterpret_cast<uint4*>(d + j) = o;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (col + j < p.N) d[j] = __float2bfloat16_rn(p.alpha * __uint_as_float(r[j]));
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tempty[ab]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- host side
// 2-D bf16 tensor [outer, inner] (inner contiguous, row stride ld elements); box = [box_outer, 64]
bool make_map(CUtensorMap* m, const void* base, int64_t inner, int64_t outer, int64_t ld, int box_outer) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int g_num_sms = 0;

template <int BN, int STAGES, bool A_MN, bool B_MN>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, int* status, cudaStream_t st) {
  using S = Smem<BN, STAGES>;
  static bool configured = false;
  auto kern = gemm_tc_kernel<BN, STAGES, A_MN, B_MN>;
  if (!configured) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal);
    if (e != cudaSuccess) return e;
    configured = true;
  }
  Params p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.alpha = g.alpha; p.D = g.D; p.ldd = g.ldd; p.out_f32 = g.out_f32;
  p.resid = g.resid; p.ldr = g.ldr; p.accumulate = g.accumulate;
  p.tiles_m = (g.M + BM - 1) / BM; p.tiles_n = (g.N + BN - 1) / BN; p.status = status;
  int tiles = p.tiles_m * p.tiles_n;
  int grid = tiles < g_num_sms ? tiles : g_num_sms;
  kern<<<grid, kThreads, S::kTotal, st>>>(ma, mb, p);
  return cudaGetLastError();
}

template <int BN, int STAGES>
cudaError_t dispatch(const GemmArgs& g, int* status, cudaStream_t st) {
  CUtensorMap ma, mb;
  bool ok;
  // A: K-major stored [M,K] -> box [128 rows, 64 k]; MN-major stored [K,M] -> box [64 k, 64 m]
  ok = g.a_kmajor ? make_map(&ma, g.A, g.K, g.M, g.lda, BM) : make_map(&ma, g.A, g.M, g.K, g.lda, 64);
  ok = ok && (g.b_kmajor ? make_map(&mb, g.B, g.K, g.N, g.ldb, BN) : make_map(&mb, g.B, g.N, g.K, g.ldb, 64));
  if (!ok) return cudaErrorInvalidValue;
  if (g.a_kmajor && g.b_kmajor) return launch<BN, STAGES, false, false>(g, ma, mb, status, st);
  if (g.a_kmajor) return launch<BN, STAGES, false, true>(g, ma, mb, status, st);
  if (g.b_kmajor) return launch<BN, STAGES, true, false>(g, ma, mb, status, st);
  return launch<BN, STAGES, true, true>(g, ma, mb, status, st);
}

}  // namespace

bool gemm_tc_supported(const GemmArgs& g) {
  if (g.M < 1 || g.N < 1 || g.K < 1) return false;
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (!al16(g.A) || !al16(g.B) || !al16(g.D)) return false;
  if (g.lda % 8 || g.ldb % 8) return false;
  if (g.out_f32 ? (g.ldd % 4) : (g.ldd % 8)) return false;
  if (g.resid && (!al16(g.resid) || g.ldr % 4)) return false;
  if (g.accumulate && !g.out_f32) return false;
  return tc::get_encode() != nullptr;
}

cudaError_t gemm_tc(const GemmArgs& g, int* d_status, cudaStream_t st) {
  if (g_num_sms == 0) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
  }
  // wide tiles unless N is small enough that they would mostly compute padding
  if (g.N > 128) return dispatch<256, 4>(g, d_status, st);
  return dispatch<128, 6>(g, d_status, st);
}
