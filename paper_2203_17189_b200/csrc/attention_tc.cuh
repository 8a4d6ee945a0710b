// Declarations shared by the tcgen05 attention kernels: the kernel parameter block, small device helpers and the
// host-side tensor-map builder.  Everything sits in an unnamed namespace (one private copy per translation unit).
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

#include <math.h>

#include <algorithm>
#include <type_traits>

namespace {

using namespace tc;
using std::max;

constexpr float kLog2e = 1.4426950408889634f;

struct TcParams {
  float* o32;           // forward: optional float32 copy of the output rows
  int ldo32;
  void* out0;           // forward: O; dQ kernel: dQ; dKV kernel: dK
  void* out1;           // dKV kernel: dV
  int ld0, ld1;
  float* lse;           // [B,H,Tq] written by forward, read by backward
  const float* delta;   // [B,H,Tq]
  const int* code_q;
  const int* code_k;
  const float* bias_delta;   // [H, Tq+Tk-1] or NULL
  float* dbias_delta;        // [H, Tq+Tk-1] or NULL
  int B, H, Tq, Tk, causal;
  float scale;
  int* status;
  int bias_far;              // see AttnArgs::bias_far
  int packed;                // see AttnArgs::packed
  int prefix;                // see AttnArgs::prefix: no tile is cut off at the diagonal
  RowNorm rn_q, rn_k;        // see AttnArgs: row factors of dQ and of dK / dV
};


// Writes 8 consecutive bf16 of row `row` (columns [col8*8, col8*8+8) of a 64-column chunk) into a
// 128-byte-swizzled K-major tile: 16-byte piece index is XORed with (row % 8).
__device__ __forceinline__ void store_swizzled_16B(unsigned char* tile, int row, int piece, uint4 v) {
  *reinterpret_cast<uint4*>(tile + row * 128 + ((piece ^ (row & 7)) << 4)) = v;
}
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&t);
}

// Common position code of 64 consecutive keys/queries (one int2 per lane), or -1 if they differ.  A tile
// whose code equals every row's code (and lies on the allowed side of the diagonal) needs no per-element mask.
__device__ __forceinline__ int tile_code64(const int* codes, int lane) {
  int2 c = *reinterpret_cast<const int2*>(codes + lane * 2);
  int first = __shfl_sync(0xffffffffu, c.x, 0);
  bool same = c.x == first && c.y == first;
  return __all_sync(0xffffffffu, same) ? first : -1;
}
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }

// dst[i] = f(i) for i in [0, n) by NT threads; four loads are in flight before their stores, so the
// set-up of a CTA costs a couple of global-memory round trips instead of one per element.
template <int NT, typename T, typename F, int U = 4>
__device__ __forceinline__ void fill_batched(T* dst, int n, int tid, F f) {
  for (int base = tid; base < n; base += U * NT) {
    T v[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int i = base + u * NT;
      if (i < n) v[u] = f(i);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      int i = base + u * NT;
      if (i < n) dst[i] = v[u];
    }
  }
}

struct Bars {
  uint64_t ld[4];      // TMA barriers (meaning per kernel)
  uint64_t mma[2];     // MMA completion barriers
  uint32_t tmem;
  int abort_flag;
};


// Packed rows: which 64-row tiles of the "other" side (queries for a key block, keys for a query block) can hold a
// valid pair with this CTA's 128 "own" rows.  A pair is valid only if both positions carry the same non-zero
// segment code, so a 128-row block of the other side whose range of non-zero codes does not meet the range of the
// own rows holds none; its two tiles are left out.  The rule is taken per pair of 128-row blocks so that the kernel
// that walks key blocks and the kernel that walks query blocks leave out exactly the same (query, key) regions (the
// second one reads what the first one stored).
// Writes the kept tiles of [t_begin, t_end) (t_begin even) in increasing order to list_s (shared memory, t_end ints)
// and returns their number in every lane.  Run by ONE warp (all 32 lanes): every global load of the codes is
// independent of the others, so the whole list costs about one round trip to L2; the caller publishes the list to
// the other warps (an mbarrier arrive after __syncwarp).
__device__ __forceinline__ int packed_tile_list_warp(const int* own_codes, int T_own, int own0, const int* other_codes,
                                                     int T_other, int t_begin, int t_end, int* list_s, int lane) {
  auto load4 = [&](const int* codes, int T, int r0, int (&c)[4]) {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int r = r0 + lane + 32 * k;
      c[k] = r < T ? (codes[r] & ~T5_PREFIX_BIT) : 0;
    }
  };
  auto range = [&](const int (&c)[4], int& lo, int& hi) {
    lo = 0x7fffffff; hi = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (c[k]) { lo = min(lo, c[k]); hi = ::max(hi, c[k]); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = ::max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
  };
  int own[4], slo, shi;
  load4(own_codes, T_own, own0, own);
  int n = 0;
  // four 128-row blocks of the other side per round: sixteen loads per lane in flight
  for (int pb0 = t_begin / 2; 2 * pb0 < t_end; pb0 += 4) {
    int c[4][4];
#pragma unroll
    for (int q = 0; q < 4; ++q) load4(other_codes, T_other, (pb0 + q) * 128, c[q]);
    if (pb0 == t_begin / 2) range(own, slo, shi);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      int lo, hi;
      range(c[q], lo, hi);
      const bool act = shi > 0 && hi > 0 && hi >= slo && lo <= shi;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int t = 2 * (pb0 + q) + e;
        if (act && t < t_end) {
          if (lane == 0) list_s[n] = t;
          ++n;
        }
      }
    }
  }
  return n;
}

// ----------------------------------------------------------------------------- host side
// 3-D view [B][T][cols] of a row-major token matrix with row stride ld; box = [1][rows][64 cols]
bool make_map3(CUtensorMap* m, const void* base, int cols, int T, int B, int ld, int box_rows) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)T, (cuuint64_t)B};
  cuuint64_t strides[2] = {(cuuint64_t)ld * 2, (cuuint64_t)T * ld * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

TcParams base_params(const AttnArgs& a, int* status) {
  TcParams p{};
  p.lse = a.lse; p.delta = a.delta; p.code_q = a.code_q; p.code_k = a.code_k; p.bias_delta = a.bias_delta;
  p.bias_far = a.bias_far;
  p.packed = a.packed;
  p.dbias_delta = a.dbias_delta; p.B = a.B; p.H = a.H; p.Tq = a.Tq; p.Tk = a.Tk; p.causal = a.causal;
  p.scale = a.scale; p.status = status;
  p.rn_q = a.rn_q; p.rn_k = a.rn_k;
  p.prefix = a.prefix;
  return p;
}

}  // namespace
