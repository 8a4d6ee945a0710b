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
  int epi;            // 0 plain, 1 gated-GELU forward, 2 gated-GELU backward (see GemmArgs)
  void* aux;
  int ld_aux, F;
  // stream-K tail: the first sk_full * gridDim.x tiles are walked tile by tile; the remaining sk_rem tiles
  // (a partial wave) are cut along K into gridDim.x equal ranges of k-blocks.  sk_rem = 0 turns it off.
  int sk_full, sk_rem;
  int* sk_flags;      // [sk_rem], zeroed: counts the epilogue warps of the storing segment that are done
  // RMSNorm fold (see GemmArgs): row factor of the product; operand copy + sum of squares of the new residual rows
  RowNorm rn;
  bf16* xg_out;
  int ld_xg;
  const bf16* g_next;
  float* ssq_out;
};

// alpha times the RMSNorm factor of the accumulator row this thread holds (tensor-memory lane = row)
__device__ __forceinline__ float row_alpha(const Params& p, int row) {
  return (p.rn.ssq != nullptr && row < p.M) ? p.alpha * rsqrtf(p.rn.ssq[row] * p.rn.inv_d + p.rn.eps) : p.alpha;
}

// One unit of work of a CTA: k-blocks [kb0, kb1) of a tile.
//   kind 0: the whole tile;  1: the segment that reaches the tile's last k-block (it stores, then raises
//   the tile's flag);  2: an earlier segment (waits for the flag, then adds atomically).
struct Work { int tile, kb0, kb1, kind, flag; };

struct WorkIter {
  int it = 0;
  int n_tiles, k_blocks, sk_full, sk_rem;
  long long cur, u1;
  int unit, n_units;        // this scheduling unit (a CTA, or a CTA pair) and how many there are
  __device__ WorkIter(const Params& p, int kb, int unit_, int n_units_)
      : n_tiles(p.tiles_m * p.tiles_n), k_blocks(kb), sk_full(p.sk_full), sk_rem(p.sk_rem), unit(unit_), n_units(n_units_) {
    long long U = (long long)sk_rem * kb;
    cur = U * unit / n_units;
    u1 = U * (unit + 1) / n_units;
  }
  __device__ bool next(Work& w) {
    if (sk_rem == 0) {
      int tile = unit + it * n_units;
      if (tile >= n_tiles) return false;
      w = {tile, 0, k_blocks, 0, 0};
      ++it;
      return true;
    }
    if (it < sk_full) {
      w = {unit + it * n_units, 0, k_blocks, 0, 0};
      ++it;
      return true;
    }
    if (cur >= u1) return false;
    int t = (int)(cur / k_blocks), kb0 = (int)(cur % k_blocks);
    long long left = u1 - cur;
    int kb1 = left < k_blocks - kb0 ? kb0 + (int)left : k_blocks;
    cur += kb1 - kb0;
    w = {sk_full * n_units + t, kb0, kb1, (kb0 == 0 && kb1 == k_blocks) ? 0 : (kb1 == k_blocks ? 1 : 2), t};
    ++it;
    return true;
  }
};

// Tile order: groups of kGroupM tile rows are swept column by column, so that the tiles in flight at one time
// share a few A row-blocks and a few B column-blocks (both stay in L2) instead of streaming all of A per wave.
constexpr int kGroupM = 8;
__device__ __forceinline__ void tile_coords(int tile, int tiles_m, int tiles_n, int& tm, int& tn) {
  const int per_group = kGroupM * tiles_n;
  const int g = tile / per_group, r = tile - g * per_group;
  const int first = g * kGroupM;
  const int gsz = min(kGroupM, tiles_m - first);
  tm = first + r % gsz;
  tn = r / gsz;
}
__device__ __forceinline__ void store_bf16x4(bf16* d, float4 v) {
  __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x, v.y), b1 = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<uint32_t*>(&b0);
  o.y = *reinterpret_cast<uint32_t*>(&b1);
  *reinterpret_cast<uint2*>(d) = o;
}
__device__ __forceinline__ float4 load_bf16x4(const bf16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}
// Epilogue of one 128-row x BN-column accumulator tile for one warp (rows quad*32 .. +31 of the tile).
// Each thread holds one accumulator row; going through a per-warp shared-memory tile turns the stores (and the
// loads of the float32 addend) into 128-byte row segments instead of 32 scattered pieces.
// Chunks (32 columns each) [c_begin, c_end) of the tile are this warp's share.
// What an epilogue warp can fetch before its tile's accumulator is ready (while it waits for the MMAs): the row's
// RMSNorm factor, the first chunk of the float32 addend and the first chunk's norm scales.
struct EpiPre {
  float arow;
  float4 add0[8];
  float4 gn0;
};
__device__ __forceinline__ const float* epi_addend(const Params& p, bool add_atomic) {
  return (!p.out_f32 || add_atomic) ? nullptr : (p.resid ? p.resid : (p.accumulate ? (const float*)p.D : nullptr));
}
__device__ __forceinline__ void epi_fetch_addend(const Params& p, const float* addend, int m0, int n0, int quad, int lane,
                                                 int c, float4 (&dst)[8]) {
  const int rr0 = lane >> 3, col = n0 + c * 32 + (lane & 7) * 4;
  const int ld_add = p.resid ? p.ldr : p.ldd;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = m0 + quad * 32 + i * 4 + rr0;
    dst[i] = (addend && row < p.M && col < p.N) ? *reinterpret_cast<const float4*>(addend + (int64_t)row * ld_add + col)
                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
  }
}
__device__ __forceinline__ float4 epi_fetch_gn(const Params& p, int n0, int lane, int c) {
  const int col = n0 + c * 32 + (lane & 7) * 4;
  return (p.xg_out != nullptr && col < p.N) ? load_bf16x4(p.g_next + col) : make_float4(0.f, 0.f, 0.f, 0.f);
}
__device__ __forceinline__ void epi_prefetch(const Params& p, int m0, int n0, int quad, int lane, bool add_atomic,
                                             int c_begin, EpiPre& pre) {
  pre.arow = row_alpha(p, m0 + quad * 32 + lane);
  if (p.epi == 0) {
    epi_fetch_addend(p, epi_addend(p, add_atomic), m0, n0, quad, lane, c_begin, pre.add0);
    pre.gn0 = epi_fetch_gn(p, n0, lane, c_begin);
  }
}

template <int BN>
__device__ __forceinline__ void store_tile(const Params& p, float* tbuf, uint32_t tacc, int m0, int n0, int quad,
                                           int lane, bool add_atomic, const EpiPre& pre, int c_begin = 0,
                                           int c_end = BN / 32) {
  const int rr0 = lane >> 3, cc = (lane & 7) * 4;
  const float arow = pre.arow;
  const bool fold_out = p.xg_out != nullptr && !add_atomic;      // also write x * g and the rows' sums of squares
  float ss[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  // float32 addend (residual input, or D itself when accumulating) and the next norm's scales, fetched one chunk
  // ahead of their use (the first chunk's before the accumulator was ready)
  const float* addend = epi_addend(p, add_atomic);
  float4 add_next[8], gn_next = pre.gn0;
#pragma unroll
  for (int i = 0; i < 8; ++i) add_next[i] = pre.add0[i];
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    const int col0 = n0 + c * 32;
    if (col0 >= p.N) break;               // uniform across the warp
    float4 add_cur[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) add_cur[i] = add_next[i];
    const float4 gn = gn_next;
    uint32_t r[32];
    tmem_ld_32x32b_x32(tacc + c * 32, r);
    tmem_wait_ld_dep(r);
#pragma unroll
    for (int j = 0; j < 8; ++j)
      *reinterpret_cast<float4*>(tbuf + lane * 36 + j * 4) =
          make_float4(arow * __uint_as_float(r[4 * j]), arow * __uint_as_float(r[4 * j + 1]),
                      arow * __uint_as_float(r[4 * j + 2]), arow * __uint_as_float(r[4 * j + 3]));
    __syncwarp();
    if (c + 1 < c_end) {                                               // in flight while this chunk is stored
      if (addend) epi_fetch_addend(p, addend, m0, n0, quad, lane, c + 1, add_next);
      if (fold_out) gn_next = epi_fetch_gn(p, n0, lane, c + 1);
    }
    const int col = col0 + cc;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int rr = i * 4 + rr0;
      const int row = m0 + quad * 32 + rr;
      float4 v = *reinterpret_cast<const float4*>(tbuf + rr * 36 + cc);
      if (row < p.M && col < p.N) {        // N is a multiple of 4: a float4 never straddles the edge
        if (add_atomic) {
          float* d = (float*)p.D + (int64_t)row * p.ldd + col;
          asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(d), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w)
                       : "memory");
        } else if (p.out_f32) {
          v.x += add_cur[i].x; v.y += add_cur[i].y; v.z += add_cur[i].z; v.w += add_cur[i].w;
          *reinterpret_cast<float4*>((float*)p.D + (int64_t)row * p.ldd + col) = v;
          if (fold_out) {
            store_bf16x4(p.xg_out + (int64_t)row * p.ld_xg + col, make_float4(v.x * gn.x, v.y * gn.y, v.z * gn.z, v.w * gn.w));
            ss[i] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
          }
        } else {
          bf16* d = (bf16*)p.D + (int64_t)row * p.ldd + col;
          __nv_bfloat162 b0 = __floats2bfloat162_rn(v.x, v.y), b1 = __floats2bfloat162_rn(v.z, v.w);
          uint2 o;
          o.x = *reinterpret_cast<uint32_t*>(&b0);
          o.y = *reinterpret_cast<uint32_t*>(&b1);
          *reinterpret_cast<uint2*>(d) = o;
        }
      }
    }
    __syncwarp();                          // the tile is rewritten by the next chunk
  }
  if (fold_out) {
    // the eight lanes that share a row (same lane >> 3) add up their columns' squares; one atomic per row
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float t = ss[i];
      t += __shfl_xor_sync(0xffffffffu, t, 1);
      t += __shfl_xor_sync(0xffffffffu, t, 2);
      t += __shfl_xor_sync(0xffffffffu, t, 4);
      const int row = m0 + quad * 32 + i * 4 + rr0;
      if ((lane & 7) == 0 && row < p.M) atomicAdd(p.ssq_out + row, t);
    }
  }
}

// ---- gated-GELU epilogues (tanh approximation through the hardware tanh; outputs are bf16)
__device__ __forceinline__ void gelu_both_fast(float u, float& g, float& dg) {
  const float c = 0.7978845608028654f, a = 0.044715f;
  float u2 = u * u, t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(c * (u + a * u * u2)));
  g = 0.5f * u * (1.f + t);
  dg = 0.5f * (1.f + t) + 0.5f * u * (1.f - t * t) * c * (1.f + 3.f * a * u2);
}
// one accumulator chunk (32 columns of this thread's row) -> the warp's coalesced layout (8 x float4 per lane)
__device__ __forceinline__ void transpose_chunk(float* tbuf, int lane, const uint32_t (&r)[32], float alpha, float4 (&v)[8]) {
  const int rr0 = lane >> 3, cc = (lane & 7) * 4;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    *reinterpret_cast<float4*>(tbuf + lane * 36 + j * 4) =
        make_float4(alpha * __uint_as_float(r[4 * j]), alpha * __uint_as_float(r[4 * j + 1]),
                    alpha * __uint_as_float(r[4 * j + 2]), alpha * __uint_as_float(r[4 * j + 3]));
  __syncwarp();
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = *reinterpret_cast<const float4*>(tbuf + (i * 4 + rr0) * 36 + cc);
  __syncwarp();
}
// forward: accumulator columns [0,128) = a, [128,256) = b of feature block tn; writes h = [a | b] and hg = gelu(a) b
__device__ __forceinline__ void store_tile_geglu_fwd(const Params& p, float* tbuf, uint32_t tacc, int m0, int tn, int quad,
                                                     int lane, float arow, int c_begin = 0, int c_end = 4) {
  const int rr0 = lane >> 3, cc = (lane & 7) * 4;
  bf16* H = (bf16*)p.D;
  bf16* HG = (bf16*)p.aux;
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    uint32_t ra[32], rb[32];
    tmem_ld_32x32b_x32(tacc + c * 32, ra);
    tmem_ld_32x32b_x32(tacc + 128 + c * 32, rb);
    tmem_wait_ld_dep(ra);
    tmem_wait_ld_dep(rb);
    float4 va[8], vb[8];
    transpose_chunk(tbuf, lane, ra, arow, va);
    transpose_chunk(tbuf, lane, rb, arow, vb);
    const int col = tn * 128 + c * 32 + cc;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = m0 + quad * 32 + i * 4 + rr0;
      if (row < p.M && col < p.F) {
        store_bf16x4(H + (int64_t)row * p.ldd + col, va[i]);
        store_bf16x4(H + (int64_t)row * p.ldd + p.F + col, vb[i]);
        // the product uses a and b as stored (rounded to bf16): the backward pass recomputes from those
        auto rb = [](float x) { return __bfloat162float(__float2bfloat16_rn(x)); };
        const float4 a = make_float4(rb(va[i].x), rb(va[i].y), rb(va[i].z), rb(va[i].w));
        const float4 b = make_float4(rb(vb[i].x), rb(vb[i].y), rb(vb[i].z), rb(vb[i].w));
        float g0, g1, g2, g3, t;
        gelu_both_fast(a.x, g0, t); gelu_both_fast(a.y, g1, t); gelu_both_fast(a.z, g2, t); gelu_both_fast(a.w, g3, t);
        store_bf16x4(HG + (int64_t)row * p.ld_aux + col, make_float4(g0 * b.x, g1 * b.y, g2 * b.z, g3 * b.w));
      }
    }
  }
}
// backward: the accumulator is d(hg); aux = h = [a | b]; writes dh = [d(hg) b gelu'(a) | d(hg) gelu(a)]
template <int BN>
__device__ __forceinline__ void store_tile_geglu_bwd(const Params& p, float* tbuf, uint32_t tacc, int m0, int n0, int quad,
                                                     int lane, float arow, int c_begin = 0, int c_end = BN / 32) {
  const int rr0 = lane >> 3, cc = (lane & 7) * 4;      // arow: d(hg) rows carry the norm factor, da and db are linear in it
  const bf16* Hh = (const bf16*)p.aux;
  bf16* DH = (bf16*)p.D;
#pragma unroll 1
  for (int c = c_begin; c < c_end; ++c) {
    if (n0 + c * 32 >= p.N) break;
    uint32_t r[32];
    tmem_ld_32x32b_x32(tacc + c * 32, r);
    tmem_wait_ld_dep(r);
    const int col = n0 + c * 32 + cc;
    float4 av[8], bv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {      // a and b of the same elements, in flight while the chunk is transposed
      const int row = m0 + quad * 32 + i * 4 + rr0;
      const bool in = row < p.M && col < p.N;
      av[i] = in ? load_bf16x4(Hh + (int64_t)row * p.ld_aux + col) : make_float4(0.f, 0.f, 0.f, 0.f);
      bv[i] = in ? load_bf16x4(Hh + (int64_t)row * p.ld_aux + p.F + col) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    float4 v[8];
    transpose_chunk(tbuf, lane, r, arow, v);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int row = m0 + quad * 32 + i * 4 + rr0;
      if (row < p.M && col < p.N) {
        // d(hg) is rounded to bf16 first, as when it is stored between two kernels
        float4 g = make_float4(__bfloat162float(__float2bfloat16_rn(v[i].x)), __bfloat162float(__float2bfloat16_rn(v[i].y)),
                               __bfloat162float(__float2bfloat16_rn(v[i].z)), __bfloat162float(__float2bfloat16_rn(v[i].w)));
        float ge[4], dge[4];
        gelu_both_fast(av[i].x, ge[0], dge[0]); gelu_both_fast(av[i].y, ge[1], dge[1]);
        gelu_both_fast(av[i].z, ge[2], dge[2]); gelu_both_fast(av[i].w, ge[3], dge[3]);
        store_bf16x4(DH + (int64_t)row * p.ldd + col,
                     make_float4(g.x * bv[i].x * dge[0], g.y * bv[i].y * dge[1], g.z * bv[i].z * dge[2], g.w * bv[i].w * dge[3]));
        store_bf16x4(DH + (int64_t)row * p.ldd + p.F + col, make_float4(g.x * ge[0], g.y * ge[1], g.z * ge[2], g.w * ge[3]));
      }
    }
  }
}

template <int BN, int STAGES>
struct Smem {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = BN * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarOffset = STAGES * kStageBytes;
  static constexpr int kEpiOffset = kBarOffset + 256;       // 4 epilogue warps x [32][36] floats (transpose buffers)
  static constexpr int kEpiBytes = 4 * 32 * 36 * 4;
  static constexpr int kTotal = kEpiOffset + kEpiBytes + 1024;   // + slack for 1024-byte alignment
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
      WorkIter wi(p, k_blocks, blockIdx.x, gridDim.x);
      Work w;
      while (ok && wi.next(w)) {
        int tm, tn;
        tile_coords(w.tile, p.tiles_m, p.tiles_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
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
      WorkIter wi(p, k_blocks, blockIdx.x, gridDim.x);
      Work w;
      for (; ok && wi.next(w); ++it) {
        const int ab = it & 1;
        const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(&tempty[ab], aph ^ 1, abort_flag, p.status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + ab * BN;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
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
            umma_bf16(tacc, da, db, idesc, ((kb - w.kb0) | k) != 0);
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
    WorkIter wi(p, k_blocks, blockIdx.x, gridDim.x);
    Work w;
    for (; ok && wi.next(w); ++it) {
      int tm, tn;
        tile_coords(w.tile, p.tiles_m, p.tiles_n, tm, tn);
        const int m0 = tm * BM, n0 = tn * BN;
      const int ab = it & 1;
      const uint32_t aph = (it >> 1) & 1;
      EpiPre pre;
      epi_prefetch(p, m0, n0, quad, lane, w.kind == 2, 0, pre);
      ok = mbar_wait(&tfull[ab], aph, abort_flag, p.status, 4);
      if (ok && w.kind == 2) {
        // an earlier K-segment of a split tile: the segment that stores must be done first
        volatile int* flag = p.sk_flags + w.flag;
        long long t0 = clock64();
        while (*flag < 4) {
          if (clock64() - t0 > kWaitCycles) {
            if (p.status) atomicCAS(p.status, 0, 5);
            ok = false;
            break;
          }
          __nanosleep(200);
        }
        __threadfence();
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      const bool add_atomic = w.kind == 2;
      store_tile<BN>(p, reinterpret_cast<float*>(smem + S::kEpiOffset) + quad * (32 * 36),
                     tmem_base + ab * BN + ((uint32_t)(quad * 32) << 16), m0, n0, quad, lane, add_atomic, pre);
      if (w.kind == 1) {          // publish this warp's part of the stored tile to the adding segments
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(p.sk_flags + w.flag, 1);
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


// ============================================================================ two-CTA variant
// A cluster of two CTAs computes one 256 x 256 tile: CTA r loads rows [128 r, 128 r + 128) of A and of the B tile
// into its own shared memory (plain TMA, completion counted on the leader's barrier), the leader's MMA thread issues
// tcgen05.mma.cta_group::2 (M = 256, N = 256), each CTA's tensor memory receives its 128 rows of the result and each
// CTA runs the epilogue of its half.  Per CTA a K slice costs 32 KB of loads instead of 48 KB.
// Twelve warps: producer, MMA issuer, tensor-memory owner, one idle, and EIGHT epilogue warps - two per tensor-memory
// lane quarter, each with half of the tile's columns.  With four, every epilogue warp sat alone on its scheduler and
// the heavier epilogues (gated-GELU backward, float32 residual) ran at the pace of one warp's instruction latencies,
// longer than the tile's MMAs; a second warp per scheduler hides them.  The transpose buffers of the extra warps
// take the room of the sixth stage.
constexpr int kThreads2 = 384;          // 4 + kEpiWarps2 warps
constexpr int kEpiWarps2 = 8;
constexpr int STAGES2 = 5;
struct Smem2 {
  static constexpr int kABytes = 128 * BK * 2, kBBytes = 128 * BK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarOffset = STAGES2 * kStageBytes;
  static constexpr int kEpiOffset = kBarOffset + 256;
  static constexpr int kEpiBytes = kEpiWarps2 * 32 * 36 * 4;
  static constexpr int kTotal = kEpiOffset + kEpiBytes + 1024;
};
static_assert(Smem2::kTotal <= 227 * 1024, "shared memory of the CTA-pair kernel");

template <bool A_MN, bool B_MN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads2, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, Params p) {
  using S = Smem2;
  constexpr int BN = 256;
  extern __shared__ unsigned char smem_raw[];
  // both CTAs of a pair must use identical offsets: the dynamic shared-memory base is the same in both
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + S::kBarOffset);
  uint64_t* empty = full + STAGES2;
  uint64_t* tfull = empty + STAGES2;      // [2]
  uint64_t* tempty = tfull + 2;           // [2]
  uint32_t* tmem_holder = (uint32_t*)(tempty + 2);
  volatile int* abort_flag = (volatile int*)(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int n_tiles = p.tiles_m * p.tiles_n;             // 256 x 256 tiles
  const int k_blocks = (p.K + BK - 1) / BK;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  constexpr uint32_t kTmemCols = 512;
  // epilogue warps: n_epi / 4 per tensor-memory lane quarter, each with a share of the tile's eight 32-column chunks
  const int n_epi = (int)(blockDim.x >> 5) - 4, n_col_groups = n_epi >> 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES2; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 2 * n_epi); }  // the epilogue warps of both CTAs
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 2) tmem_alloc_pair(tmem_holder, kTmemCols);
  tc_fence_before();
  cluster_sync_all();                 // barriers of both CTAs exist before anything signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // Programmatic dependent launch: the next kernel of the stream (if it was launched that way) may bring its CTAs
  // in and run its own set-up while this grid drains; the threads of this kernel that touch global memory wait here
  // for the grid before it (no-ops under an ordinary launch).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      WorkIter wi(p, k_blocks, pair, n_pairs);
      Work w;
      while (ok && wi.next(w)) {
        int tm, tn;
        tile_coords(w.tile, p.tiles_m, p.tiles_n, tm, tn);
        const int m0 = tm * 256 + (int)rank * 128;
        // B rows of this CTA: its half of the 256-column tile, or (gated-GELU forward) the Wi0 / Wi1 block
        const int n0 = p.epi == 1 ? (int)rank * p.F + tn * 128 : tn * 256 + (int)rank * 128;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait(&empty[s], ph ^ 1, abort_flag, p.status, 6)) { ok = false; break; }
          unsigned char* sa = smem + s * S::kStageBytes;
          unsigned char* sb = sa + S::kABytes;
          if (leader) mbar_arrive_expect_tx(&full[s], 2 * S::kStageBytes);     // both CTAs' bytes land on this barrier
          const int k0 = kb * BK;
          if (!A_MN) {
            tma_load_2d_pair(sa, &map_a, k0, m0, &full[s]);
          } else {
#pragma unroll
            for (int c = 0; c < 2; ++c) tma_load_2d_pair(sa + c * 8192, &map_a, m0 + c * 64, k0, &full[s]);
          }
          if (!B_MN) {
            tma_load_2d_pair(sb, &map_b, k0, n0, &full[s]);
          } else {
#pragma unroll
            for (int c = 0; c < 2; ++c) tma_load_2d_pair(sb + c * 8192, &map_b, n0 + c * 64, k0, &full[s]);
          }
          if (++s == STAGES2) { s = 0; ph ^= 1; }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader CTA only)
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = make_idesc(256, 256, A_MN, B_MN);
      int s = 0;
      uint32_t ph = 0;
      int it = 0;
      bool ok = true;
      WorkIter wi(p, k_blocks, pair, n_pairs);
      Work w;
      for (; ok && wi.next(w); ++it) {
        const int ab = it & 1;
        const uint32_t aph = (it >> 1) & 1;
        if (!mbar_wait(&tempty[ab], aph ^ 1, abort_flag, p.status, 7)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tacc = tmem_base + ab * BN;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait(&full[s], ph, abort_flag, p.status, 8)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + s * S::kStageBytes);
          const uint32_t sb = sa + S::kABytes;
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            uint64_t da = A_MN ? make_desc(sa + k * 2048, 8192, 1024) : make_desc(sa + k * 32, 16, 1024);
            uint64_t db = B_MN ? make_desc(sb + k * 2048, 8192, 1024) : make_desc(sb + k * 32, 16, 1024);
            umma_bf16_pair(tacc, da, db, idesc, ((kb - w.kb0) | k) != 0);
          }
          umma_commit_pair(&empty[s]);            // frees the stage in both CTAs
          if (++s == STAGES2) { s = 0; ph ^= 1; }
        }
        if (ok) umma_commit_pair(&tfull[ab]);     // both CTAs' epilogues may read their half
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ epilogue (both CTAs, own 128 rows)
    const int quad = warp & 3, ew = warp - 4, ch = ew >> 2;      // ch: which share of the tile's columns
    const int c0 = ch * 8 / n_col_groups, c1 = (ch + 1) * 8 / n_col_groups;
    // gated-GELU forward: four chunk pairs (a and b of the same features), split over at most two groups
    const int g0 = ch < 2 ? ch * 2 : 4, g1 = ch < 2 ? ch * 2 + 2 : 4;
    int it = 0;
    bool ok = true;
    asm volatile("griddepcontrol.wait;" ::: "memory");
    WorkIter wi(p, k_blocks, pair, n_pairs);
    Work w;
    for (; ok && wi.next(w); ++it) {
      int tm, tn;
      tile_coords(w.tile, p.tiles_m, p.tiles_n, tm, tn);
      const int m0 = tm * 256 + (int)rank * 128, n0 = tn * 256;
      const int ab = it & 1;
      const uint32_t aph = (it >> 1) & 1;
      EpiPre pre;
      epi_prefetch(p, m0, n0, quad, lane, w.kind == 2, c0, pre);
      ok = mbar_wait(&tfull[ab], aph, abort_flag, p.status, 9);
      if (ok && w.kind == 2) {
        // an earlier K-segment of a split tile: the storing pair (16 epilogue warps) must be done first
        volatile int* flag = p.sk_flags + w.flag;
        long long t0 = clock64();
        while (*flag < 2 * n_epi) {
          if (clock64() - t0 > kWaitCycles) {
            if (p.status) atomicCAS(p.status, 0, 10);
            ok = false;
            break;
          }
          __nanosleep(200);
        }
        __threadfence();
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      float* tb = reinterpret_cast<float*>(smem + S::kEpiOffset) + ew * (32 * 36);
      const uint32_t tacc = tmem_base + ab * BN + ((uint32_t)(quad * 32) << 16);
      if (p.epi == 1) store_tile_geglu_fwd(p, tb, tacc, m0, tn, quad, lane, pre.arow, g0, g1);
      else if (p.epi == 2) store_tile_geglu_bwd<BN>(p, tb, tacc, m0, n0, quad, lane, pre.arow, c0, c1);
      else store_tile<BN>(p, tb, tacc, m0, n0, quad, lane, w.kind == 2, pre, c0, c1);
      if (w.kind == 1) {
        __threadfence();
        __syncwarp();
        if (lane == 0) atomicAdd(p.sk_flags + w.flag, 1);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_leader(&tempty[ab]);
    }
  }

  tc_fence_before();
  cluster_sync_all();                 // the peer's shared memory and barriers stay alive until both are done
  if (warp == 2) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
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

// SM count of the current device (cached per device ordinal)
int g_num_sms = 0;
int num_sms_of_current_device() {
  static int cache[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  if (cache[dev] == 0) cudaDeviceGetAttribute(&cache[dev], cudaDevAttrMultiProcessorCount, dev);
  return cache[dev];
}
// cudaFuncSetAttribute has to be repeated on every device that runs the kernel
bool first_use_on_device(bool (&seen)[64]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
  bool first = !seen[dev];
  seen[dev] = true;
  return first;
}

template <int BN, int STAGES, bool A_MN, bool B_MN>
cudaError_t launch(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, int* status, cudaStream_t st) {
  using S = Smem<BN, STAGES>;
  static bool configured[64] = {false};
  auto kern = gemm_tc_kernel<BN, STAGES, A_MN, B_MN>;
  if (first_use_on_device(configured)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, S::kTotal);
    if (e != cudaSuccess) return e;
  }
  Params p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.alpha = g.alpha; p.D = g.D; p.ldd = g.ldd; p.out_f32 = g.out_f32;
  p.resid = g.resid; p.ldr = g.ldr; p.accumulate = g.accumulate;
  p.tiles_m = (g.M + BM - 1) / BM; p.tiles_n = (g.N + BN - 1) / BN; p.status = status;
  p.epi = 0; p.aux = nullptr; p.ld_aux = 0; p.F = 0;
  p.rn = g.rn; p.xg_out = (bf16*)g.xg_out; p.ld_xg = g.ld_xg; p.g_next = (const bf16*)g.g_next; p.ssq_out = g.ssq_out;
  int tiles = p.tiles_m * p.tiles_n;
  int grid = tiles < g_num_sms ? tiles : g_num_sms;
  p.sk_full = 0; p.sk_rem = 0; p.sk_flags = nullptr;
  const int k_blocks = (g.K + BK - 1) / BK;
  const int rem = tiles % g_num_sms;
  // split the tiles of a partial last wave along K when that wave would leave a good part of the GPU idle
  // (measured: pays only for long K and after at least one full wave; short-K tiles lose more in the extra
  // atomic epilogues than the idle SMs cost)
  if (g.sk_flags && g.out_f32 && !g.xg_out && rem > 0 && k_blocks >= 128 && tiles >= g_num_sms && g_num_sms <= 160 &&
      (g_num_sms - rem) * 8 > g_num_sms * (tiles / g_num_sms + 1)) {
    grid = g_num_sms;
    p.sk_full = tiles / g_num_sms; p.sk_rem = rem; p.sk_flags = g.sk_flags;
  } else if (g.sk_flags && g.out_f32 && !g.xg_out && k_blocks >= 32 && tiles * 2 <= g_num_sms && tiles <= 160 &&
             (long long)k_blocks * tiles >= 4ll * g_num_sms) {
    // fewer tiles than half the SMs and a long contraction (weight gradients of narrow layers): every tile is cut
    // along K over all SMs - the same segments and flags as the tail above, with no full wave before them
    grid = g_num_sms;
    p.sk_full = 0; p.sk_rem = tiles; p.sk_flags = g.sk_flags;
  }
  kern<<<grid, kThreads, S::kTotal, st>>>(ma, mb, p);
  return cudaGetLastError();
}

template <bool A_MN, bool B_MN>
cudaError_t launch2(const GemmArgs& g, const CUtensorMap& ma, const CUtensorMap& mb, int* status, cudaStream_t st) {
  static bool configured[64] = {false};
  auto kern = gemm_tc2_kernel<A_MN, B_MN>;
  if (first_use_on_device(configured)) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem2::kTotal);
    if (e != cudaSuccess) return e;
  }
  Params p;
  p.M = g.M; p.N = g.N; p.K = g.K; p.alpha = g.alpha; p.D = g.D; p.ldd = g.ldd; p.out_f32 = g.out_f32;
  p.resid = g.resid; p.ldr = g.ldr; p.accumulate = g.accumulate;
  p.tiles_m = (g.M + 255) / 256; p.tiles_n = g.epi == 1 ? g.F / 128 : (g.N + 255) / 256; p.status = status;
  p.epi = g.epi; p.aux = g.aux; p.ld_aux = g.ld_aux; p.F = g.F;
  p.rn = g.rn; p.xg_out = (bf16*)g.xg_out; p.ld_xg = g.ld_xg; p.g_next = (const bf16*)g.g_next; p.ssq_out = g.ssq_out;
  p.sk_full = 0; p.sk_rem = 0; p.sk_flags = nullptr;
  int tiles = p.tiles_m * p.tiles_n;
  int pairs = g_num_sms / 2;
  const int k_blocks = (g.K + BK - 1) / BK, rem = tiles % pairs;
  // long-K float32-output GEMMs: split the tiles of a partial last wave along K over all pairs
  if (g.epi == 0 && g.sk_flags && g.out_f32 && !g.xg_out && rem > 0 && k_blocks >= 128 && tiles >= pairs && pairs <= 160 &&
      (pairs - rem) * 8 > pairs * (tiles / pairs + 1)) {
    p.sk_full = tiles / pairs; p.sk_rem = rem; p.sk_flags = g.sk_flags;
  } else if (g.epi == 0 && g.sk_flags && g.out_f32 && !g.xg_out && k_blocks >= 32 && tiles * 2 <= pairs && tiles <= 160 &&
             (long long)k_blocks * tiles >= 4ll * pairs) {
    // fewer tiles than half the pairs and a long contraction: every tile is cut along K over all pairs
    p.sk_full = 0; p.sk_rem = tiles; p.sk_flags = g.sk_flags;
  } else if (tiles < pairs) {
    pairs = tiles;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs); cfg.blockDim = dim3(kThreads2); cfg.dynamicSmemBytes = Smem2::kTotal; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, ma, mb, p);
}

// 256 x 256 tiles on CTA pairs: boxes are 128 rows (K-major) or 64 x 64 (MN-major), as for BN = 128
cudaError_t dispatch2(const GemmArgs& g, int* status, cudaStream_t st) {
  CUtensorMap ma, mb;
  bool ok = g.a_kmajor ? make_map(&ma, g.A, g.K, g.M, g.lda, 128) : make_map(&ma, g.A, g.M, g.K, g.lda, 64);
  ok = ok && (g.b_kmajor ? make_map(&mb, g.B, g.K, g.N, g.ldb, 128) : make_map(&mb, g.B, g.N, g.K, g.ldb, 64));
  if (!ok) return cudaErrorInvalidValue;
  if (g.a_kmajor && g.b_kmajor) return launch2<false, false>(g, ma, mb, status, st);
  if (g.a_kmajor) return launch2<false, true>(g, ma, mb, status, st);
  if (g.b_kmajor) return launch2<true, false>(g, ma, mb, status, st);
  return launch2<true, true>(g, ma, mb, status, st);
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
  if (g.N % 4) return false;
  if (g.resid && (!al16(g.resid) || g.ldr % 4)) return false;
  if (g.accumulate && !g.out_f32) return false;
  if (g.xg_out && (!g.out_f32 || !g.resid || g.accumulate || !g.g_next || !g.ssq_out || !al16(g.xg_out) ||
                   ((uintptr_t)g.g_next & 7) || g.ld_xg % 4))
    return false;
  return tc::get_encode() != nullptr;
}

bool gemm_tc_epi_supported(const GemmArgs& g) {
  if (g.epi != 1 && g.epi != 2) return false;
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (!g.pair || g.out_f32 || g.resid || g.accumulate || g.M < 256 || !g.aux || !al16(g.aux)) return false;
  if (g.F < 128 || g.F % 128 || g.ld_aux % 8 || g.ldd % 8) return false;
  if (g.epi == 1) return g.a_kmajor && g.b_kmajor && g.N == 2 * g.F && g.ldd >= 2 * g.F && g.ld_aux >= g.F;
  return g.N == g.F && g.ldd >= 2 * g.F && g.ld_aux >= 2 * g.F;
}

cudaError_t gemm_tc(const GemmArgs& g, int* d_status, cudaStream_t st) {
  g_num_sms = num_sms_of_current_device();
  if (g_num_sms <= 0) return cudaErrorInvalidDevice;
  if (g.epi != 0) return gemm_tc_epi_supported(g) ? dispatch2(g, d_status, st) : cudaErrorInvalidValue;
  if (g.pair && g.M >= 256 && g.N >= 256) return dispatch2(g, d_status, st);
  // wide tiles unless N is small enough that they would mostly compute padding
  if (g.N > 128) return dispatch<256, 4>(g, d_status, st);
  return dispatch<128, 6>(g, d_status, st);
}
