// Attention on the tcgen05 tensor cores (bf16 operands, float32 accumulation in
// tensor memory), forward and backward, with the relative-position bias and the
// padding / segment / causal masks applied inside the softmax.
//
//   S_ij = scale q_i.k_j + bias_delta[h, j-i];  P = softmax_j over valid keys;  O = P V.
//   backward (P recomputed from the saved log-sum-exp):
//     dP = dO V^T,  dS = P (dP - delta_i),  dQ = scale dS K,  dK = scale dS^T Q,  dV = P^T dO,
//     dbias_delta[h, j-i] += dS_ij.
//
// Every kernel loads its operands with TMA into 128-byte-swizzled tiles, keeps scores and accumulators in tensor
// memory (thread r of a softmax warp group owns tensor-memory lane r = one row of the score tile), lets one
// thread (or one elected lane) issue the MMAs, and bounds every mbarrier wait.  Several CTAs share an SM so that
// one CTA's softmax overlaps another CTA's MMAs.
//   attn_fwd_tc_kernel        128 threads, CTA = 128 queries x all keys in 64-key tiles; S and the output
//                             accumulator in tensor memory, the accumulator rescaled in place and only when a row
//                             maximum grew by more than 2^8; key tiles without a valid pair (packed rows) left out.
//   backward, one pass over the scores (default whenever the caller provides the dS scratch: the training step
//   and t5_attention_backward_onepass):
//     attn_bwd_kvf_tc_kernel    320 threads (eight softmax warps, one MMA warp, one load / store warp), CTA = 128
//                               keys x all queries in 64-query tiles: dK, dV, the bias gradient and a bf16 copy
//                               of dS^T in the scratch [B*H, Tk^128, Tq^64].
//     attn_bwd_dq_ds_tc_kernel  192 threads, CTA = 128 queries: dQ = scale dS K from the stored dS^T.
//   backward, two kernels that each recompute the scores (t5_attention with backward = 1,
//   t5_attention_backward_noalloc, configuration flag bit 17: no scratch needed):
//     attn_bwd_dq_tc_kernel     256 threads, CTA = 128 queries x 64-key tiles; dQ in tensor memory; bias gradient.
//     attn_bwd_dkv_tc_kernel    256 threads, CTA = 128 keys x 64-query tiles, transposed scores; dK, dV.
//   attn_delta_tc_kernel      delta = rowsum(dO * O) from the float32 copy of O, ahead of either backward.
#include "attention_tc.cuh"

namespace {

// ============================================================================ forward
// 64-key tiles.  Tensor memory: S in columns [0,64), the output accumulator O in [64, 64+DK).
// Per tile one wait: thread 0 issues PV(t) and right behind it S(t+1) with a single commit, so the
// softmax of tile t+1 starts as soon as both are done.  O stays in tensor memory and is rescaled in
// place (tcgen05.ld / st) only when a row maximum of the warp changed; this keeps the register count
// low enough for four CTAs per SM, which is what hides the MMA and TMA latencies.
template <int DK>
struct FwdLayout {
  static constexpr int kQBytes = 128 * DK * 2;
  static constexpr int kKVBytes = 64 * DK * 2;          // one K or V tile
  static constexpr int kP = 128 * 64 * 2;
  static constexpr int kQ = 0, kK = kQBytes, kV = kK + kKVBytes, kPo = kV + kKVBytes, kMisc = kPo + kP;
  static int bytes(int Tk) {
    int tkp = (Tk + 63) / 64 * 64;
    return kMisc + (tkp + 128) * 4 + tkp * 4 + (tkp / 64 + 9) * 4 + (int)sizeof(Bars) + 1024 + 64;
  }
};

template <int DK>
__global__ void __launch_bounds__(128)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mk,
                   const __grid_constant__ CUtensorMap mv, TcParams p) {
  pdl_sync();
  using L = FwdLayout<DK>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int tkp = (p.Tk + 63) / 64 * 64;
  float* bias_s = (float*)(smem + L::kMisc);          // [tkp + 128], entry (key - row + 127), log2 units
  int* codes_s = (int*)(bias_s + tkp + 128);          // [tkp]
  int* tiles_s = codes_s + tkp;                       // [tkp / 64] key tiles this CTA visits, then 8 + 1 scratch words
  const int n_tiles_cap = tkp / 64;
  Bars* bars = (Bars*)(((uintptr_t)(tiles_s + n_tiles_cap + 9) + 15) & ~(uintptr_t)15);
  volatile int* abort_flag = &bars->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * 128;
  int n_kt = (p.Tk + 63) / 64;
  if (p.causal && !p.prefix) n_kt = min(n_kt, (q0 + 127) / 64 + 1);
  constexpr uint32_t kTmemCols = DK == 64 ? 128 : 256;

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(&bars->ld[i], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&bars->mma[i], 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 0) tmem_alloc(&bars->tmem, kTmemCols);
  const int span = p.Tq + p.Tk - 1;
  fill_batched<128>(bias_s, tkp + 128, tid, [&](int w) {
    int g = w - 127 - q0 + p.Tq - 1;
    return (p.bias_delta && g >= 0 && g < span) ? p.bias_delta[(int64_t)h * span + g] * kLog2e : 0.f;
  });
  fill_batched<128>(codes_s, tkp, tid, [&](int j) { return j < p.Tk ? p.code_k[b * p.Tk + j] : 0; });
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem;
  // low words of the operand descriptors (K-major Q, K, P; MN-major V)
  const uint32_t lQ = desc_lo_k(smem_u32(smem + L::kQ)), lK = desc_lo_k(smem_u32(smem + L::kK)),
                 lV = desc_lo_mn(smem_u32(smem + L::kV)), lP = desc_lo_k(smem_u32(smem + L::kPo));
  uint64_t* bar_k = &bars->ld[0];
  uint64_t* bar_v = &bars->ld[1];
  uint64_t* bar_m = &bars->mma[0];
  constexpr uint32_t idesc_s = make_idesc(128, 64, false, false);
  constexpr uint32_t idesc_pv = make_idesc(128, DK, false, true);
  uint32_t ph_k = 0, ph_v = 0, ph_m = 0;
  bool ok = true, pend_k = false, pend_v = false;      // pend_*: a load of that tile is in flight (thread 0 only)

  auto load_k = [&](int t) {
    pend_k = true;
    mbar_arrive_expect_tx(bar_k, L::kKVBytes);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) tma_load_3d(smem + L::kK + c * 8192, &mk, h * DK + c * 64, t * 64, b, bar_k);
  };
  auto load_v = [&](int t) {
    pend_v = true;
    mbar_arrive_expect_tx(bar_v, L::kKVBytes);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) tma_load_3d(smem + L::kV + c * 8192, &mv, h * DK + c * 64, t * 64, b, bar_v);
  };
  auto issue_s = [&]() {      // S = Q K^T of the tile in the K buffer; returns false if its load never arrived
    if (!mbar_wait(bar_k, ph_k, abort_flag, p.status, 11)) return false;
    ph_k ^= 1;
    pend_k = false;
    tc_fence_after();
#pragma unroll
    for (int kk = 0; kk < DK / 16; ++kk)
      umma_bf16_lo(tmem_base, lQ + (((kk >> 2) * 16384 + (kk & 3) * 32) >> 4), lK + (((kk >> 2) * 8192 + (kk & 3) * 32) >> 4),
                   idesc_s, kk != 0);
    return true;
  };

  if (tid == 0) {
    pend_k = true;
    mbar_arrive_expect_tx(bar_k, L::kQBytes + L::kKVBytes);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(smem + L::kQ + c * 16384, &mq, h * DK + c * 64, q0, b, bar_k);
      tma_load_3d(smem + L::kK + c * 8192, &mk, h * DK + c * 64, 0, b, bar_k);
    }
    load_v(0);
  }

  const int i = q0 + tid;
  const int cq = i < p.Tq ? p.code_q[b * p.Tq + i] : 0;
  // Key tiles worth visiting (packed rows only; done while the first loads are in flight).  A pair (query, key) is valid only if both carry the same non-zero
  // position code, so a key tile whose range of non-zero codes does not meet the range of this CTA's rows holds no
  // valid pair (other segments) and is left out.  Tile 0 always stays: its loads and S = Q K^T went out during the
  // set-up.  Every warp counts the list, warp 0 writes it.
  int n_act = n_kt;
  if (p.packed) {
    int* rng = tiles_s + n_tiles_cap;                  // [8]: (lo, hi) of each warp's rows
    const int cqs = cq & ~T5_PREFIX_BIT;               // segment part of the code
    int lo = cqs ? cqs : 0x7fffffff, hi = cqs;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = min(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = ::max(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((tid & 31) == 0) { rng[2 * warp] = lo; rng[2 * warp + 1] = hi; }
    __syncthreads();
    const int lane = tid & 31;
    int qlo = 0x7fffffff, qhi = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      qlo = min(qlo, rng[2 * w]);
      qhi = ::max(qhi, rng[2 * w + 1]);
    }
    n_act = 0;
    for (int base = 0; base < n_kt; base += 2) {       // 16 lanes per tile, one 16-byte load each
      const int t = base + (lane >> 4);
      int klo = 0x7fffffff, khi = 0;
      if (t < n_kt) {
        int4 c = *reinterpret_cast<const int4*>(codes_s + t * 64 + (lane & 15) * 4);
        c.x &= ~T5_PREFIX_BIT; c.y &= ~T5_PREFIX_BIT; c.z &= ~T5_PREFIX_BIT; c.w &= ~T5_PREFIX_BIT;
        klo = min(min(c.x ? c.x : 0x7fffffff, c.y ? c.y : 0x7fffffff), min(c.z ? c.z : 0x7fffffff, c.w ? c.w : 0x7fffffff));
        khi = ::max(::max(c.x, c.y), ::max(c.z, c.w));
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) {
        klo = min(klo, __shfl_xor_sync(0xffffffffu, klo, o));
        khi = ::max(khi, __shfl_xor_sync(0xffffffffu, khi, o));
      }
      const bool active = t < n_kt && (t == 0 || (khi > 0 && khi >= qlo && klo <= qhi));
      const unsigned m = __ballot_sync(0xffffffffu, active) & 0x00010001u;      // one vote per half warp
      if (warp == 0 && active && (lane & 15) == 0) tiles_s[n_act + ((lane >> 4) & (m & 1u))] = t;
      n_act += __popc(m);
    }
    __syncthreads();                                   // warp 0's list is visible to the thread that issues loads
  }
  if (tid == 0 && issue_s()) umma_commit(bar_m);       // S of tile 0 as soon as Q and K(0) have landed
  float m_run = -INFINITY, l_run = 0.f;
  const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
  const float sc2 = p.scale * kLog2e;
  const bool has_bias = p.bias_delta != nullptr;

  for (int u = 0; u < n_act && ok; ++u) {
    const int t = p.packed ? tiles_s[u] : u, k0 = t * 64;
    ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 12);      // S of this tile ready, PV of the previous one done
    ph_m ^= 1;
    if (!ok) break;
    tc_fence_after();
    if (tid == 0) {
      if (u + 1 < n_act) load_k(p.packed ? tiles_s[u + 1] : u + 1);   // K buffer: S of this tile has consumed it
      if (u > 0) load_v(t);                        // V buffer: PV of the previous tile has consumed it
    }
    // ---- softmax of this 64-key tile (scores in log2 units)
    const int tcode = tile_code64(codes_s + k0, tid & 31);
    const bool fast = tcode > 0 && __all_sync(0xffffffffu, cq == tcode) &&
                      (!p.causal || k0 + 63 <= q0 + (warp << 5));          // warp-uniform: no mask needed
    // All keys of the tile carry one code and none lies ahead of a row of this warp: a row then sees the whole tile
    // or nothing of it (padding rows, rows of another segment), so no entry needs a test of its own
    const bool by_row = !fast && tcode > 0 && (!p.causal || k0 + 63 <= q0 + (warp << 5));
    const bool row_ok = !by_row || ((cq ^ tcode) & ~T5_PREFIX_BIT) == 0;
    const float* brow = bias_s + (k0 - tid + 127);
    // the whole tile lies where the bias no longer depends on the distance (saturated bucket): one value, no loads
    const bool flat = has_bias && p.bias_far > 0 && (k0 - (q0 + 127) >= p.bias_far || q0 - (k0 + 63) >= p.bias_far);
    float sc[2][32];
    {
      uint32_t r[2][32];
      tmem_ld_32x32b_x32(tmem_base + lane_off, r[0]);
      tmem_ld_32x32b_x32(tmem_base + lane_off + 32, r[1]);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        tmem_wait_ld_dep(r[c]);
        if (flat) {
          const float b0 = brow[0];
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) sc[c][jj] = fmaf(__uint_as_float(r[c][jj]), sc2, b0);
        } else if (has_bias) {
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) sc[c][jj] = fmaf(__uint_as_float(r[c][jj]), sc2, brow[c * 32 + jj]);
        } else {
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) sc[c][jj] = __uint_as_float(r[c][jj]) * sc2;
        }
        if (!fast && !by_row) {
#pragma unroll
          for (int jj = 0; jj < 32; ++jj) {
            int j = k0 + c * 32 + jj;
            int ck = codes_s[j];
            bool valid = pair_valid(cq, ck, p.causal != 0, j, i);
            sc[c][jj] = valid ? sc[c][jj] : -INFINITY;
          }
        }
      }
    }
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int jj = 0; jj < 32; jj += 4) {
        mx[0] = fmaxf(mx[0], sc[c][jj]); mx[1] = fmaxf(mx[1], sc[c][jj + 1]);
        mx[2] = fmaxf(mx[2], sc[c][jj + 2]); mx[3] = fmaxf(mx[3], sc[c][jj + 3]);
      }
    // The reference point m_run of a row only follows its true maximum when that has grown by more than
    // kLazy (log2 units): until then exp2(score - m_run) <= 2^kLazy, which float32 sums and bfloat16
    // probabilities hold as well as values below one, and the accumulator rows need no rescaling.  The result
    // O = acc / l and lse = m_run + log2(l) do not depend on which reference point was used.
    constexpr float kLazy = 8.f;
    // a row that sees nothing of the tile (see by_row): no maximum, and below every probability becomes 2^-inf = 0
    const float m_tile = row_ok ? fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) : -INFINITY;
    const bool grow = m_tile > m_run + kLazy || (m_run == -INFINITY && m_tile != -INFINITY);
    const bool warp_moves = __any_sync(0xffffffffu, grow);
    const float m_new = warp_moves ? fmaxf(m_run, m_tile) : m_run;      // a warp that rescales moves all its rows
    const float m_eff = m_new == -INFINITY ? 0.f : m_new;      // a row with no valid key so far: exp2(-inf - 0) = 0
    const float m_exp = row_ok ? m_eff : INFINITY;
    const float corr = ex2_approx(m_run - m_eff);
    // rescale the accumulator rows of this warp if any of their reference points moved
    if (u > 0 && warp_moves) {
#pragma unroll
      for (int c = 0; c < DK / 32; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32(tmem_base + lane_off + 64 + c * 32, r);
        tmem_wait_ld_dep(r);
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) r[jj] = __float_as_uint(__uint_as_float(r[jj]) * corr);
        tmem_st_32x32b_x32(tmem_base + lane_off + 64 + c * 32, r);
      }
      tmem_wait_st();
    }
    float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int c = 0; c < 2; ++c)
#pragma unroll
      for (int q8 = 0; q8 < 4; ++q8) {
        uint32_t u[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          u[e] = pack_bf16(ex2_approx(sc[c][q8 * 8 + 2 * e] - m_exp), ex2_approx(sc[c][q8 * 8 + 2 * e + 1] - m_exp));
          // the row sum uses the bf16-rounded probabilities, so the weights the MMA applies sum to one
          ls[e] += bf16_lo(u[e]) + bf16_hi(u[e]);
        }
        store_swizzled_16B(smem + L::kPo, tid, c * 4 + q8, make_uint4(u[0], u[1], u[2], u[3]));
      }
    l_run = l_run * corr + ((ls[0] + ls[1]) + (ls[2] + ls[3]));
    m_run = m_new;
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      bool good = mbar_wait(bar_v, ph_v, abort_flag, p.status, 13);
      if (good) {
        ph_v ^= 1;
        pend_v = false;
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          umma_bf16_lo(tmem_base + 64, lP + ((ks * 32) >> 4), lV + ((ks * 2048) >> 4), idesc_pv, (u | ks) != 0);
        if (u + 1 < n_act) good = issue_s();
        if (good) umma_commit(bar_m);
      }
    }
  }
  if (ok) ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 14);   // last PV done
  if (ok) {
    tc_fence_after();
    const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
    bf16* orow = (bf16*)p.out0 + (int64_t)(b * p.Tq + i) * p.ld0 + h * DK;
    float* o32 = p.o32 ? p.o32 + (int64_t)(b * p.Tq + i) * p.ldo32 + h * DK : nullptr;
#pragma unroll
    for (int c = 0; c < DK / 32; ++c) {
      uint32_t r[32];
      tmem_ld_32x32b_x32(tmem_base + lane_off + 64 + c * 32, r);
      tmem_wait_ld_dep(r);
      if (i < p.Tq) {
#pragma unroll
        for (int d = 0; d < 32; d += 8) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(r[d]) * inv, __uint_as_float(r[d + 1]) * inv);
          v.y = pack_bf16(__uint_as_float(r[d + 2]) * inv, __uint_as_float(r[d + 3]) * inv);
          v.z = pack_bf16(__uint_as_float(r[d + 4]) * inv, __uint_as_float(r[d + 5]) * inv);
          v.w = pack_bf16(__uint_as_float(r[d + 6]) * inv, __uint_as_float(r[d + 7]) * inv);
          *reinterpret_cast<uint4*>(orow + c * 32 + d) = v;
        }
        if (o32) {
#pragma unroll
          for (int d = 0; d < 32; d += 4)
            *reinterpret_cast<float4*>(o32 + c * 32 + d) =
                make_float4(__uint_as_float(r[d]) * inv, __uint_as_float(r[d + 1]) * inv,
                            __uint_as_float(r[d + 2]) * inv, __uint_as_float(r[d + 3]) * inv);
        }
      }
    }
    // natural-log log-sum-exp of the scores
    if (i < p.Tq) p.lse[(int64_t)(b * p.H + h) * p.Tq + i] = l_run > 0.f ? (m_run + log2f(l_run)) / kLog2e : -INFINITY;
  }
  if (!ok && tid == 0) {   // let TMA loads that are still in flight land before the CTA exits
    long long t0 = clock64();
    while (pend_k && !mbar_try_wait(bar_k, ph_k) && clock64() - t0 < kWaitCycles) {}
    while (pend_v && !mbar_try_wait(bar_v, ph_v) && clock64() - t0 < kWaitCycles) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ============================================================================ backward: dQ (+ dbias)
template <int DK>
struct DqLayout {
  static constexpr int kQ = 0, kDO = 128 * DK * 2, kKV0 = 2 * 128 * DK * 2;
  static constexpr int kKVTile = 64 * DK * 2;                   // one K or V tile (64 keys)
  static constexpr int kStage = 2 * kKVTile;                    // K then V
  static constexpr int kDS = kKV0 + 3 * kStage;                 // [128 x 64] bf16
  static constexpr int kMisc = kDS + 128 * 64 * 2;
  static int bytes(int Tk) {
    int tkp = (Tk + 63) / 64 * 64;
    return kMisc + (tkp + 128) * 4 + 4 * (tkp + 32) * 4 + tkp * 4 + (int)sizeof(Bars) + 1024 + 64;
  }
};

template <int DK>
__global__ void __launch_bounds__(256, DK == 64 ? 2 : 1)
attn_bwd_dq_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mdo,
                      const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv, TcParams p) {
  using L = DqLayout<DK>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int tkp = (p.Tk + 63) / 64 * 64;
  float* bias_s = (float*)(smem + L::kMisc);          // [tkp + 128]
  // bias gradient: one window per warp, indexed by (key - lane + 31); a warp's lanes touch distinct
  // entries in one instruction, so plain read-modify-write (no atomics) is enough
  const int wlen = tkp + 32;
  float* dbias_s = bias_s + tkp + 128;                // [4][tkp + 32]
  int* codes_s = (int*)(dbias_s + 4 * wlen);          // [tkp]
  Bars* bars = (Bars*)(((uintptr_t)(codes_s + tkp) + 15) & ~(uintptr_t)15);
  volatile int* abort_flag = &bars->abort_flag;

  // 256 threads: thread (row, half) owns tensor-memory lane `row` and one 32-column half of each score tile
  const int tid = threadIdx.x, warp = tid >> 5, row = tid & 127, half = tid >> 7, quad = warp & 3;
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * 128;
  int n_kt = (p.Tk + 63) / 64;
  if (p.causal && !p.prefix) n_kt = min(n_kt, (q0 + 127) / 64 + 1);
  constexpr uint32_t kTmemCols = 256;
  const bool want_db = p.dbias_delta != nullptr;

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(&bars->ld[i], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&bars->mma[i], 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  uint64_t* bar_q = &bars->ld[0];        // Q and dO
  uint64_t* bar_kv = &bars->ld[1];       // [3] stages: ld[1..3]
  uint64_t* bar_m = &bars->mma[0];       // S(t), dP(t) ready and dQ(t-1) done
  auto load_kv = [&](int t) {
    int st = t % 3;
    unsigned char* base = smem + L::kKV0 + st * L::kStage;
    mbar_arrive_expect_tx(&bar_kv[st], L::kStage);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(base + c * 8192, &mk, h * DK + c * 64, t * 64, b, &bar_kv[st]);
      tma_load_3d(base + L::kKVTile + c * 8192, &mv, h * DK + c * 64, t * 64, b, &bar_kv[st]);
    }
  };
  if (tid == 0) {      // loads go out before the rest of the set-up so that their latency overlaps it
    mbar_arrive_expect_tx(bar_q, 2 * 128 * DK * 2);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(smem + L::kQ + c * 16384, &mq, h * DK + c * 64, q0, b, bar_q);
      tma_load_3d(smem + L::kDO + c * 16384, &mdo, h * DK + c * 64, q0, b, bar_q);
    }
    load_kv(0);
    if (n_kt > 1) load_kv(1);
  }
  if (warp == 0) tmem_alloc(&bars->tmem, kTmemCols);
  const int span = p.Tq + p.Tk - 1;
  fill_batched<256>(bias_s, tkp + 128, tid, [&](int w) {
    int g = w - 127 - q0 + p.Tq - 1;
    return (p.bias_delta && g >= 0 && g < span) ? p.bias_delta[(int64_t)h * span + g] * kLog2e : 0.f;
  });
  for (int w = tid; w < 4 * wlen; w += 256) dbias_s[w] = 0.f;
  fill_batched<256>(codes_s, tkp, tid, [&](int j) { return j < p.Tk ? p.code_k[b * p.Tk + j] : 0; });
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem;
  const uint32_t lQ = desc_lo_k(smem_u32(smem + L::kQ)), lDO = desc_lo_k(smem_u32(smem + L::kDO)),
                 lDS = desc_lo_k(smem_u32(smem + L::kDS));      // low words of the operand descriptors

  const int i = q0 + row;
  const bool row_in = i < p.Tq;
  const int cq = row_in ? p.code_q[b * p.Tq + i] : 0;
  const float lse2 = row_in ? p.lse[(int64_t)(b * p.H + h) * p.Tq + i] * kLog2e : -INFINITY;
  const float dl = row_in ? p.delta[(int64_t)(b * p.H + h) * p.Tq + i] : 0.f;
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  const float sc2 = p.scale * kLog2e;
  uint32_t ph_kv[3] = {0, 0, 0}, ph_m = 0;
  bool ok = true;
  float far_pos = 0.f, far_neg = 0.f;      // dS mass of blocks wholly beyond +bias_far / -bias_far
  constexpr uint32_t idesc_s = make_idesc(128, 64, false, false);
  constexpr uint32_t idesc_dq = make_idesc(128, DK, false, true);

  // S = Q K^T and dP = dO V^T of tile t (thread 0); false if the tile's load never arrived
  auto issue_s_dp = [&](int t) {
    const int st = t % 3;
    if (!mbar_wait(&bar_kv[st], ph_kv[st], abort_flag, p.status, 22)) return false;
    ph_kv[st] ^= 1;
    tc_fence_after();
    const uint32_t lK = desc_lo_k(smem_u32(smem + L::kKV0 + st * L::kStage)), lV = lK + (L::kKVTile >> 4);
#pragma unroll
    for (int kk = 0; kk < DK / 16; ++kk) {
      uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
      umma_bf16_lo(tmem_base, lQ + (oa >> 4), lK + (ob >> 4), idesc_s, kk != 0);
    }
#pragma unroll
    for (int kk = 0; kk < DK / 16; ++kk) {
      uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
      umma_bf16_lo(tmem_base + 64, lDO + (oa >> 4), lV + (ob >> 4), idesc_s, kk != 0);
    }
    return true;
  };
  if (tid == 0) {
    ok = mbar_wait(bar_q, 0, abort_flag, p.status, 21);
    if (ok && issue_s_dp(0)) umma_commit(bar_m);
  }

  for (int t = 0; t < n_kt && ok; ++t) {
    const int k0 = t * 64;
    ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 23);
    ph_m ^= 1;
    if (!ok) break;
    tc_fence_after();
    if (tid == 0 && t + 2 < n_kt) load_kv(t + 2);      // its stage held tile t-1, whose MMAs are all done
    const int tcode = tile_code64(codes_s + k0, tid & 31);
    const bool fast = tcode > 0 && __all_sync(0xffffffffu, cq == tcode) &&
                      (!p.causal || k0 + 63 <= q0 + (quad << 5));           // warp-uniform: no mask needed
    const float* brow = bias_s + (k0 - row + 127);
    const int lane = tid & 31;
    float* dbwin = dbias_s + quad * wlen + k0;        // window of this row quarter; entry = key - (row in quarter) + 31
    const bool has_bias = p.bias_delta != nullptr;
    uint32_t rs[32], rp[32];
    const int c = half;                                // this thread's 32 keys of the tile
    tmem_ld_32x32b_x32(tmem_base + lane_off + c * 32, rs);
    tmem_ld_32x32b_x32(tmem_base + lane_off + 64 + c * 32, rp);
    tmem_wait_ld_dep(rs);
    tmem_wait_ld_dep(rp);
    {
      float ds[32];
      // four compiled variants (mask needed or not, bias or not) chosen by one warp-uniform branch, so the common
      // unmasked case carries no mask or select instructions
      auto compute = [&](auto fast_c, auto bias_c) {
        constexpr bool FAST = decltype(fast_c)::value, BIAS = decltype(bias_c)::value;
#pragma unroll
        for (int jj = 0; jj < 32; ++jj) {
          float sv = BIAS ? fmaf(__uint_as_float(rs[jj]), sc2, brow[c * 32 + jj]) : __uint_as_float(rs[jj]) * sc2;
          float pr = ex2_approx(sv - lse2);
          if (!FAST) {
            int j = k0 + c * 32 + jj;
            int ck = codes_s[j];
            bool valid = pair_valid(cq, ck, p.causal != 0, j, i) && lse2 != -INFINITY;
            pr = valid ? pr : 0.f;
          }
          ds[jj] = pr * (__uint_as_float(rp[jj]) - dl);
        }
      };
      if (fast) {
        if (has_bias) compute(std::true_type{}, std::true_type{}); else compute(std::true_type{}, std::false_type{});
      } else {
        if (has_bias) compute(std::false_type{}, std::true_type{}); else compute(std::false_type{}, std::false_type{});
      }
      if (want_db) {
        const int kk0 = k0 + c * 32, i_lo = q0 + (quad << 5);       // this warp's 32 keys x 32 rows
        if (p.bias_far > 0 && kk0 - (i_lo + 31) >= p.bias_far) {
          // every (row, key) of the block is at least bias_far to the right: one bucket, plain sums
          float t0 = 0.f, t1 = 0.f;
#pragma unroll
          for (int jj = 0; jj < 32; jj += 2) { t0 += ds[jj]; t1 += ds[jj + 1]; }
          far_pos += t0 + t1;
        } else if (p.bias_far > 0 && i_lo - (kk0 + 31) >= p.bias_far) {
          float t0 = 0.f, t1 = 0.f;
#pragma unroll
          for (int jj = 0; jj < 32; jj += 2) { t0 += ds[jj]; t1 += ds[jj + 1]; }
          far_neg += t0 + t1;
        } else {
          // Diagonal sums of the block: at step t lane l takes column t of row (l + t) mod 32, which lies on
          // diagonal (col - row) = -l when l + t < 32 and 32 - l otherwise.
          float tot = 0.f, a1 = 0.f;
#pragma unroll
          for (int t2 = 0; t2 < 32; ++t2) {
            float v = __shfl_sync(0xffffffffu, ds[t2], (lane + t2) & 31);
            tot += v;
            a1 += (lane >= 32 - t2) ? v : 0.f;
          }
          // window entry (col - row + 31); the two column halves of a row quarter overlap there: atomics
          atomicAdd(&dbwin[c * 32 + 31 - lane], tot - a1);
          atomicAdd(&dbwin[c * 32 + 63 - lane], a1);
        }
      }
#pragma unroll
      for (int q8 = 0; q8 < 4; ++q8) {
        uint4 v;
        v.x = pack_bf16(ds[q8 * 8 + 0], ds[q8 * 8 + 1]);
        v.y = pack_bf16(ds[q8 * 8 + 2], ds[q8 * 8 + 3]);
        v.z = pack_bf16(ds[q8 * 8 + 4], ds[q8 * 8 + 5]);
        v.w = pack_bf16(ds[q8 * 8 + 6], ds[q8 * 8 + 7]);
        store_swizzled_16B(smem + L::kDS, row, c * 4 + q8, v);
      }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t lKm = desc_lo_mn(smem_u32(smem + L::kKV0 + (t % 3) * L::kStage));
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16_lo(tmem_base + 128, lDS + ((ks * 32) >> 4), lKm + ((ks * 2048) >> 4), idesc_dq, (t | ks) != 0);
      bool good = true;
      if (t + 1 < n_kt) good = issue_s_dp(t + 1);      // the scores of tile t are in registers by now
      if (good) umma_commit(bar_m);
    }
  }
  if (ok) ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 24);   // last dQ MMA done

  if (ok) {
    tc_fence_after();
    bf16* drow = (bf16*)p.out0 + (int64_t)(b * p.Tq + i) * p.ld0 + h * DK + half * (DK / 2);
    const float fq = row_in ? p.scale * rn_factor(p.rn_q, (int64_t)b * p.Tq + i) : 0.f;
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      uint32_t r[32];
      tmem_ld_32x32b_x32(tmem_base + lane_off + 128 + half * (DK / 2) + c * 32, r);
      tmem_wait_ld_dep(r);
      if (row_in) {
#pragma unroll
        for (int d = 0; d < 32; d += 8) {
          uint4 v;
          v.x = pack_bf16(fq * __uint_as_float(r[d]), fq * __uint_as_float(r[d + 1]));
          v.y = pack_bf16(fq * __uint_as_float(r[d + 2]), fq * __uint_as_float(r[d + 3]));
          v.z = pack_bf16(fq * __uint_as_float(r[d + 4]), fq * __uint_as_float(r[d + 5]));
          v.w = pack_bf16(fq * __uint_as_float(r[d + 6]), fq * __uint_as_float(r[d + 7]));
          *reinterpret_cast<uint4*>(drow + c * 32 + d) = v;
        }
      }
    }
  }
  if (!ok && tid == 0) {   // a wait ran out: give loads still in flight a bounded time to land
    long long t0 = clock64();
    while (clock64() - t0 < 4000000ll) {}
  }
  tc_fence_before();
  __syncthreads();
  if (ok && want_db && p.bias_far > 0) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      far_pos += __shfl_xor_sync(0xffffffffu, far_pos, o);
      far_neg += __shfl_xor_sync(0xffffffffu, far_neg, o);
    }
    if ((tid & 31) == 0) {
      const int gp = p.bias_far + p.Tq - 1, gn = -p.bias_far + p.Tq - 1;
      if (far_pos != 0.f && gp < span) atomicAdd(&p.dbias_delta[(int64_t)h * span + gp], far_pos);
      if (far_neg != 0.f && gn >= 0) atomicAdd(&p.dbias_delta[(int64_t)h * span + gn], far_neg);
    }
  }
  if (ok && want_db) {
    // CTA-level index (key - row + 127) = warp-level index + 96 - 32 * warp
    for (int w = tid; w < tkp + 128; w += 256) {
      float v = 0.f;
#pragma unroll
      for (int wp = 0; wp < 4; ++wp) {
        int x = w - 96 + 32 * wp;
        if (x >= 0 && x < wlen) v += dbias_s[wp * wlen + x];
      }
      int g = w - 127 - q0 + p.Tq - 1;
      if (v != 0.f && g >= 0 && g < span) atomicAdd(&p.dbias_delta[(int64_t)h * span + g], v);
    }
  }
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ============================================================================ backward: dK, dV
template <int DK>
struct DkvLayout {
  static constexpr int kK = 0, kV = 128 * DK * 2, kQD0 = 2 * 128 * DK * 2;
  static constexpr int kQTile = 64 * DK * 2;                    // one Q or dO tile (64 queries)
  static constexpr int kStage = 2 * kQTile;                     // Q then dO
  static constexpr int kPt = kQD0 + 2 * kStage;                 // [128 keys x 64 queries] bf16
  static constexpr int kDSt = kPt + 128 * 64 * 2;
  static constexpr int kMisc = kDSt + 128 * 64 * 2;
  static int bytes(int Tq) {
    int tqp = (Tq + 63) / 64 * 64;
    return kMisc + (tqp + 128) * 4 + 3 * tqp * 4 + (int)sizeof(Bars) + 1024 + 64;
  }
};

template <int DK>
__global__ void __launch_bounds__(256, DK == 64 ? 2 : 1)
attn_bwd_dkv_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mdo,
                       const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv, TcParams p) {
  using L = DkvLayout<DK>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int tqp = (p.Tq + 63) / 64 * 64;
  float* bias_s = (float*)(smem + L::kMisc);          // [tqp + 128], entry (key row - query + tqp), log2 units
  float* lse_s = bias_s + tqp + 128;                  // [tqp]  (log2 units)
  float* dl_s = lse_s + tqp;                          // [tqp]
  int* codes_s = (int*)(dl_s + tqp);                  // [tqp] query codes
  Bars* bars = (Bars*)(((uintptr_t)(codes_s + tqp) + 15) & ~(uintptr_t)15);
  volatile int* abort_flag = &bars->abort_flag;

  // 256 threads: thread (row, half) owns tensor-memory lane `row` (a key) and 32 of the 64 queries of each tile
  const int tid = threadIdx.x, warp = tid >> 5, row = tid & 127, half = tid >> 7, quad = warp & 3;
  const int b = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * 128;
  const int n_qt = (p.Tq + 63) / 64;
  const int t_begin = (p.causal && !p.prefix) ? k0 / 64 : 0;          // queries before k0 see none of these keys
  constexpr uint32_t kTmemCols = DK == 64 ? 256 : 512;

  if (tid == 0) {
    for (int i = 0; i < 4; ++i) mbar_init(&bars->ld[i], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&bars->mma[i], 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  uint64_t* bar_kv = &bars->ld[0];
  uint64_t* bar_qd = &bars->ld[1];       // [2] stages
  uint64_t* bar_m = &bars->mma[0];       // S^T(t), dP^T(t) ready and the accumulating MMAs of tile t-1 done
  auto load_qd = [&](int t) {
    int st = t & 1;
    unsigned char* base = smem + L::kQD0 + st * L::kStage;
    mbar_arrive_expect_tx(&bar_qd[st], L::kStage);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(base + c * 8192, &mq, h * DK + c * 64, t * 64, b, &bar_qd[st]);
      tma_load_3d(base + L::kQTile + c * 8192, &mdo, h * DK + c * 64, t * 64, b, &bar_qd[st]);
    }
  };
  if (tid == 0 && t_begin < n_qt) {      // loads go out before the rest of the set-up so that their latency overlaps it
    mbar_arrive_expect_tx(bar_kv, 2 * 128 * DK * 2);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(smem + L::kK + c * 16384, &mk, h * DK + c * 64, k0, b, bar_kv);
      tma_load_3d(smem + L::kV + c * 16384, &mv, h * DK + c * 64, k0, b, bar_kv);
    }
    load_qd(t_begin);
    if (t_begin + 1 < n_qt) load_qd(t_begin + 1);
  }
  if (warp == 0) tmem_alloc(&bars->tmem, kTmemCols);
  const int span = p.Tq + p.Tk - 1;
  // distance of (key j = k0 + row, query i): j - i ; window index w = row - i + tqp  in [1, tqp + 127]
  fill_batched<256>(bias_s, tqp + 128, tid, [&](int w) {
    int g = (w - tqp) + k0 + p.Tq - 1;
    return (p.bias_delta && g >= 0 && g < span) ? p.bias_delta[(int64_t)h * span + g] * kLog2e : 0.f;
  });
  fill_batched<256>(lse_s, tqp, tid, [&](int q) {
    return q < p.Tq ? p.lse[(int64_t)(b * p.H + h) * p.Tq + q] * kLog2e : -INFINITY;
  });
  fill_batched<256>(dl_s, tqp, tid, [&](int q) { return q < p.Tq ? p.delta[(int64_t)(b * p.H + h) * p.Tq + q] : 0.f; });
  fill_batched<256>(codes_s, tqp, tid, [&](int q) { return q < p.Tq ? p.code_q[b * p.Tq + q] : 0; });
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem;
  const uint32_t lK = desc_lo_k(smem_u32(smem + L::kK)), lV = desc_lo_k(smem_u32(smem + L::kV)),
                 lPt = desc_lo_k(smem_u32(smem + L::kPt)), lDSt = desc_lo_k(smem_u32(smem + L::kDSt));
  const int j = k0 + row;
  const bool row_in = j < p.Tk;
  const int ck = row_in ? p.code_k[b * p.Tk + j] : 0;
  const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
  const float sc2 = p.scale * kLog2e;
  uint32_t ph_qd[2] = {0, 0}, ph_m = 0;
  bool ok = true;
  constexpr uint32_t idesc_s = make_idesc(128, 64, false, false);
  constexpr uint32_t idesc_acc = make_idesc(128, DK, false, true);
  // S^T = K Q^T and dP^T = V dO^T of query tile t (thread 0); false if the tile's load never arrived
  auto issue_st = [&](int t) {
    const int st = t & 1;
    if (!mbar_wait(&bar_qd[st], ph_qd[st], abort_flag, p.status, 32)) return false;
    ph_qd[st] ^= 1;
    tc_fence_after();
    const uint32_t lQ = desc_lo_k(smem_u32(smem + L::kQD0 + st * L::kStage)), lDO = lQ + (L::kQTile >> 4);
#pragma unroll
    for (int kk = 0; kk < DK / 16; ++kk) {
      uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
      umma_bf16_lo(tmem_base, lK + (oa >> 4), lQ + (ob >> 4), idesc_s, kk != 0);
    }
#pragma unroll
    for (int kk = 0; kk < DK / 16; ++kk) {
      uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
      umma_bf16_lo(tmem_base + 64, lV + (oa >> 4), lDO + (ob >> 4), idesc_s, kk != 0);
    }
    return true;
  };
  if (tid == 0 && t_begin < n_qt) {
    ok = mbar_wait(bar_kv, 0, abort_flag, p.status, 31);
    if (ok && issue_st(t_begin)) umma_commit(bar_m);
  }

  for (int t = t_begin; t < n_qt && ok; ++t) {
    const int qb = t * 64;
    const uint32_t lQm = desc_lo_mn(smem_u32(smem + L::kQD0 + (t & 1) * L::kStage)), lDOm = lQm + (L::kQTile >> 4);
    ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 33);
    ph_m ^= 1;
    if (!ok) break;
    tc_fence_after();
    // the stage of tile t-1 is free (all MMAs that read it are done): fetch tile t+1 into it
    if (tid == 0 && t > t_begin && t + 1 < n_qt) load_qd(t + 1);
    const int tcode = tile_code64(codes_s + qb, tid & 31);
    const bool fast = tcode > 0 && __all_sync(0xffffffffu, ck == tcode) &&
                      (!p.causal || k0 + (quad << 5) + 31 <= qb);           // warp-uniform: no mask needed
    const float* brow = bias_s + (row - qb + tqp);       // element q of the tile: brow[-(q - qb)]
    const bool has_bias = p.bias_delta != nullptr;
    uint32_t rs[32], rp[32];
    const int c = half;                                // this thread's 32 queries of the tile
    tmem_ld_32x32b_x32(tmem_base + lane_off + c * 32, rs);
    tmem_ld_32x32b_x32(tmem_base + lane_off + 64 + c * 32, rp);
    tmem_wait_ld_dep(rs);
    tmem_wait_ld_dep(rp);
    {
      float pt[32], ds[32];
      auto compute = [&](auto fast_c, auto bias_c) {
        constexpr bool FAST = decltype(fast_c)::value, BIAS = decltype(bias_c)::value;
#pragma unroll
        for (int i4 = 0; i4 < 8; ++i4) {
          const float4 l4 = *reinterpret_cast<const float4*>(lse_s + qb + c * 32 + i4 * 4);
          const float4 d4 = *reinterpret_cast<const float4*>(dl_s + qb + c * 32 + i4 * 4);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int ii = i4 * 4 + e;
            const float lse2 = e == 0 ? l4.x : e == 1 ? l4.y : e == 2 ? l4.z : l4.w;
            const float dlq = e == 0 ? d4.x : e == 1 ? d4.y : e == 2 ? d4.z : d4.w;
            float sv = BIAS ? fmaf(__uint_as_float(rs[ii]), sc2, brow[-(c * 32 + ii)]) : __uint_as_float(rs[ii]) * sc2;
            float pr = ex2_approx(sv - lse2);
            if (!FAST) {
              int q = qb + c * 32 + ii;
              int cq = codes_s[q];
              bool valid = pair_valid(cq, ck, p.causal != 0, j, q) && lse2 != -INFINITY;
              pr = valid ? pr : 0.f;
            }
            pt[ii] = pr;
            ds[ii] = pr * (__uint_as_float(rp[ii]) - dlq);
          }
        }
      };
      if (fast) {
        if (has_bias) compute(std::true_type{}, std::true_type{}); else compute(std::true_type{}, std::false_type{});
      } else {
        if (has_bias) compute(std::false_type{}, std::true_type{}); else compute(std::false_type{}, std::false_type{});
      }
#pragma unroll
      for (int q8 = 0; q8 < 4; ++q8) {
        uint4 v;
        v.x = pack_bf16(pt[q8 * 8 + 0], pt[q8 * 8 + 1]);
        v.y = pack_bf16(pt[q8 * 8 + 2], pt[q8 * 8 + 3]);
        v.z = pack_bf16(pt[q8 * 8 + 4], pt[q8 * 8 + 5]);
        v.w = pack_bf16(pt[q8 * 8 + 6], pt[q8 * 8 + 7]);
        store_swizzled_16B(smem + L::kPt, row, c * 4 + q8, v);
        v.x = pack_bf16(ds[q8 * 8 + 0], ds[q8 * 8 + 1]);
        v.y = pack_bf16(ds[q8 * 8 + 2], ds[q8 * 8 + 3]);
        v.z = pack_bf16(ds[q8 * 8 + 4], ds[q8 * 8 + 5]);
        v.w = pack_bf16(ds[q8 * 8 + 6], ds[q8 * 8 + 7]);
        store_swizzled_16B(smem + L::kDSt, row, c * 4 + q8, v);
      }
    }
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    if (tid == 0) {
      tc_fence_after();
      const uint32_t first = (t == t_begin) ? 0u : 1u;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16_lo(tmem_base + 128, lPt + ((ks * 32) >> 4), lDOm + ((ks * 2048) >> 4), idesc_acc, first | ks);
#pragma unroll
      for (int ks = 0; ks < 4; ++ks)
        umma_bf16_lo(tmem_base + 128 + DK, lDSt + ((ks * 32) >> 4), lQm + ((ks * 2048) >> 4), idesc_acc, first | ks);
      bool good = true;
      if (t + 1 < n_qt) good = issue_st(t + 1);        // the scores of tile t are in registers by now
      if (good) umma_commit(bar_m);
    }
  }
  if (ok && t_begin < n_qt) ok = mbar_wait(bar_m, ph_m, abort_flag, p.status, 34);   // last accumulating MMAs done

  if (ok) {
    tc_fence_after();
    bf16* krow = (bf16*)p.out0 + (int64_t)(b * p.Tk + j) * p.ld0 + h * DK + half * (DK / 2);
    bf16* vrow = (bf16*)p.out1 + (int64_t)(b * p.Tk + j) * p.ld1 + h * DK + half * (DK / 2);
    const bool any = t_begin < n_qt;
    const float fv = row_in ? rn_factor(p.rn_k, (int64_t)b * p.Tk + j) : 0.f, fk = p.scale * fv;
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      uint32_t rv[32], rk[32];
      if (any) {
        tmem_ld_32x32b_x32(tmem_base + lane_off + 128 + half * (DK / 2) + c * 32, rv);
        tmem_ld_32x32b_x32(tmem_base + lane_off + 128 + DK + half * (DK / 2) + c * 32, rk);
        tmem_wait_ld_dep(rv);
        tmem_wait_ld_dep(rk);
      } else {
#pragma unroll
        for (int d = 0; d < 32; ++d) rv[d] = rk[d] = 0u;
      }
      if (row_in) {
#pragma unroll
        for (int d = 0; d < 32; d += 8) {
          uint4 v;
          v.x = pack_bf16(fv * __uint_as_float(rv[d]), fv * __uint_as_float(rv[d + 1]));
          v.y = pack_bf16(fv * __uint_as_float(rv[d + 2]), fv * __uint_as_float(rv[d + 3]));
          v.z = pack_bf16(fv * __uint_as_float(rv[d + 4]), fv * __uint_as_float(rv[d + 5]));
          v.w = pack_bf16(fv * __uint_as_float(rv[d + 6]), fv * __uint_as_float(rv[d + 7]));
          *reinterpret_cast<uint4*>(vrow + c * 32 + d) = v;
          v.x = pack_bf16(fk * __uint_as_float(rk[d]), fk * __uint_as_float(rk[d + 1]));
          v.y = pack_bf16(fk * __uint_as_float(rk[d + 2]), fk * __uint_as_float(rk[d + 3]));
          v.z = pack_bf16(fk * __uint_as_float(rk[d + 4]), fk * __uint_as_float(rk[d + 5]));
          v.w = pack_bf16(fk * __uint_as_float(rk[d + 6]), fk * __uint_as_float(rk[d + 7]));
          *reinterpret_cast<uint4*>(krow + c * 32 + d) = v;
        }
      }
    }
  }
  if (!ok && tid == 0) {   // a wait ran out: give loads still in flight a bounded time to land
    long long t0 = clock64();
    while (clock64() - t0 < 4000000ll) {}
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ----------------------------------------------------------------------------- delta = rowsum(dO * O)
// Thread = 8 consecutive columns of one token row (16 bytes of dO, 32 bytes of the float32 O copy); the DK / 8
// threads of a head reduce with shuffles.
template <int DK>
__global__ void __launch_bounds__(256)
attn_delta_tc_kernel(const bf16* __restrict__ O, int ldo, const float* __restrict__ O32, int ldo32,
                     const bf16* __restrict__ dO, int lddo, float* __restrict__ delta, int B, int H, int Tq) {
  pdl_sync();
  const int per_row = H * DK / 8;
  const int64_t gt = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t n_rows = (int64_t)B * Tq;
  const bool in = gt < n_rows * per_row;        // per_row is a multiple of DK / 8, so a head never straddles the end
  const int64_t row = in ? gt / per_row : 0;
  const int col = in ? (int)(gt - row * per_row) * 8 : 0;
  float s = 0.f;
  if (in) {
    const uint4 g = *reinterpret_cast<const uint4*>(dO + row * lddo + col);
    const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
    float a[8];
    if (O32) {
      const float4 a0 = *reinterpret_cast<const float4*>(O32 + row * ldo32 + col);
      const float4 a1 = *reinterpret_cast<const float4*>(O32 + row * ldo32 + col + 4);
      a[0] = a0.x; a[1] = a0.y; a[2] = a0.z; a[3] = a0.w; a[4] = a1.x; a[5] = a1.y; a[6] = a1.z; a[7] = a1.w;
    } else {
      const uint4 o = *reinterpret_cast<const uint4*>(O + row * ldo + col);
      const uint32_t ow[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[2 * i] = bf16_lo(ow[i]); a[2 * i + 1] = bf16_hi(ow[i]); }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) s += a[2 * i] * bf16_lo(gw[i]) + a[2 * i + 1] * bf16_hi(gw[i]);
  }
#pragma unroll
  for (int o = DK / 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (in && (threadIdx.x & (DK / 8 - 1)) == 0) {
    const int h = col / DK;
    const int b = (int)(row / Tq), i = (int)(row - (int64_t)b * Tq);
    delta[(int64_t)(b * H + h) * Tq + i] = s;
  }
}

// ============================================================================ backward in one pass over the scores
// Kernel A (dK, dV and dS): CTA = 128 keys x all queries (64-query tiles), warp-specialised, two CTAs per SM.
//   warps 0-7 : softmax.  Warp (quad, half) has 32 keys (its tensor-memory lanes) x 32 of the tile's 64 queries,
//               walked as two passes of 16: P^T and dS^T from the transposed scores S^T = K Q^T and dP^T = V dO^T
//               in tensor memory, written as bf16 tiles to shared memory; the bias gradient is reduced along
//               diagonals as in the dQ kernel above.  As soon as a tile's scores are in registers the warps release
//               the tensor-memory buffer, so the next tile's S^T / dP^T run during this tile's arithmetic.
//   warp 8    : issues every MMA (all lanes walk the loop, one elected lane executes): S^T / dP^T of tile t+1, then
//               the accumulating dV += P^T dO and dK += dS^T Q of tile t.
//   warp 9    : one thread loads the Q / dO tiles (TMA ring) and stores each dS^T tile to global memory (TMA store
//               out of the same shared-memory tile the dK MMA reads).
// The second CTA of the SM is at another point of its life: its set-up, its waits and its epilogue overlap this
// one's arithmetic.
// Kernel B (dQ): dQ = scale dS K, a plain TMA -> MMA pipeline over the stored dS^T (an MN-major A operand).
// The scores, the exponentials and dS are computed once instead of once per kernel; the price is one write and
// one read of dS (bf16) through global memory.
template <int DK>
struct KvfLayout {
  static constexpr int kStages = 2;                             // Q / dO ring
  static constexpr int kKVBytes = 128 * DK * 2;
  static constexpr int kK = 0, kV = kKVBytes, kQD0 = 2 * kKVBytes;
  static constexpr int kQTile = 64 * DK * 2;                    // one Q or dO tile (64 queries)
  static constexpr int kStage = 2 * kQTile;                     // Q then dO
  static constexpr int kP0 = kQD0 + kStages * kStage;           // [128 keys x 64 queries] bf16
  static constexpr int kDS0 = kP0 + 16384;                      // [128 keys x 64 queries] bf16
  static constexpr int kMisc = kDS0 + 16384;
  static constexpr int kBarBytes = 128;
  static int bytes(int Tq, bool want_db) {
    int tqp = (Tq + 63) / 64 * 64;
    return kMisc + (tqp + 128) * 4 + 3 * tqp * 4 + (want_db ? (tqp + 128) * 4 : 0) + (tqp / 64 + 4) * 4 + kBarBytes + 1024 + 64;
  }
};

struct KvfBars {
  uint64_t kv;
  uint64_t qd_full[2], qd_free[2];
  uint64_t s_full, s_free, p_full, p_free;
  uint64_t acc;
  uint64_t list;       // packed rows: the list of query tiles is in shared memory
  uint32_t tmem;
  int abort_flag;
};
static_assert(sizeof(KvfBars) <= 128, "barrier block");

constexpr int kKvfThreads = 10 * 32;
constexpr int kKvfSoftmaxThreads = 8 * 32;

template <int DK>
__global__ void __launch_bounds__(kKvfThreads, DK == 64 ? 2 : 1)
attn_bwd_kvf_tc_kernel(const __grid_constant__ CUtensorMap mq, const __grid_constant__ CUtensorMap mdo,
                       const __grid_constant__ CUtensorMap mk, const __grid_constant__ CUtensorMap mv,
                       const __grid_constant__ CUtensorMap mds, const __grid_constant__ CUtensorMap mdk_out,
                       const __grid_constant__ CUtensorMap mdv_out, TcParams p) {
  pdl_sync();
  using L = KvfLayout<DK>;
  constexpr int NST = L::kStages;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  const int tqp = (p.Tq + 63) / 64 * 64;
  const bool want_db = p.dbias_delta != nullptr;
  float* bias_s = (float*)(smem + L::kMisc);          // [tqp + 128], entry (key row - query + tqp), log2 units
  float* lse_s = bias_s + tqp + 128;                  // [tqp]  (log2 units)
  float* dl_s = lse_s + tqp;                          // [tqp]
  int* codes_s = (int*)(dl_s + tqp);                  // [tqp] query codes
  float* dbias_s = (float*)(codes_s + tqp);           // [tqp + 128], entry (key row - query + tqp)
  int* qt_s = (int*)(dbias_s + (want_db ? tqp + 128 : 0));      // [tqp / 64 + 2] query tiles this CTA walks (packed rows)
  KvfBars* bars = (KvfBars*)(((uintptr_t)(qt_s + tqp / 64 + 4) + 15) & ~(uintptr_t)15);
  volatile int* abort_flag = &bars->abort_flag;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.z, h = blockIdx.y, k0 = blockIdx.x * 128;
  const int n_qt = (p.Tq + 63) / 64;
  const int t_begin = (p.causal && !p.prefix) ? k0 / 64 : 0;          // queries before k0 see none of these keys
  int n = n_qt - t_begin;                              // tiles this CTA walks (fewer on packed rows, see below)
  auto tile_of = [&](int i) { return p.packed ? qt_s[i] : t_begin + i; };
  constexpr uint32_t kTmemCols = DK == 64 ? 256 : 512;
  constexpr uint32_t kColS = 0, kColDP = 64, kColDV = 128, kColDK = 128 + DK;

  auto load_qd = [&](int i) {
    const int st = i % NST, t = tile_of(i);
    unsigned char* base = smem + L::kQD0 + st * L::kStage;
    mbar_arrive_expect_tx(&bars->qd_full[st], L::kStage);
#pragma unroll
    for (int c = 0; c < DK / 64; ++c) {
      tma_load_3d(base + c * 8192, &mq, h * DK + c * 64, t * 64, b, &bars->qd_full[st]);
      tma_load_3d(base + L::kQTile + c * 8192, &mdo, h * DK + c * 64, t * 64, b, &bars->qd_full[st]);
    }
  };
  if (tid == 9 * 32) {      // the loading thread: its first loads go out before the rest of the set-up
    mbar_init(&bars->kv, 1);
    for (int i = 0; i < NST; ++i) { mbar_init(&bars->qd_full[i], 1); mbar_init(&bars->qd_free[i], 1); }
    mbar_init(&bars->s_full, 1);
    mbar_init(&bars->s_free, 8);         // the softmax warps have the tile's scores in registers
    mbar_init(&bars->p_full, 8);         // one arrival per softmax warp
    mbar_init(&bars->p_free, 2);         // the accumulating MMAs are done + the dS store has read the tile
    mbar_init(&bars->acc, 1);
    mbar_init(&bars->list, 1);
    bars->abort_flag = 0;
    fence_barrier_init();
  }
  // The loading warp, ahead of the CTA-wide barrier: K and V go out at once; on packed rows it then makes the list of
  // query tiles (those whose 128-query block shares a segment with this CTA's keys: the dQ kernel applies the same
  // rule, so the regions of the dS scratch that stay unwritten are never read), sends the first Q / dO tiles and
  // publishes the list; the other warps pick it up when they need it.
  const bool kv_loaded = n > 0;
  if (warp == 9) {
    if (lane == 0 && kv_loaded) {
      mbar_arrive_expect_tx(&bars->kv, 2 * L::kKVBytes);
#pragma unroll
      for (int c = 0; c < DK / 64; ++c) {
        tma_load_3d(smem + L::kK + c * 16384, &mk, h * DK + c * 64, k0, b, &bars->kv);
        tma_load_3d(smem + L::kV + c * 16384, &mv, h * DK + c * 64, k0, b, &bars->kv);
      }
    }
    __syncwarp();
    if (p.packed) {
      n = packed_tile_list_warp(p.code_k + (int64_t)b * p.Tk, p.Tk, k0, p.code_q + (int64_t)b * p.Tq, p.Tq, t_begin, n_qt,
                                qt_s, lane);
      if (lane == 0) qt_s[n_qt] = n;
      __syncwarp();
    }
    if (lane == 0) {
      for (int i = 0; i < NST && i < n; ++i) load_qd(i);
      if (p.packed) mbar_arrive(&bars->list);
    }
  }
  if (warp == 8) tmem_alloc(&bars->tmem, kTmemCols);
  const int span = p.Tq + p.Tk - 1;
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem;
  bool ok = true;
  if (p.packed && warp == 8) {
    ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->list, 0, abort_flag, p.status, 39));
    n = ok ? qt_s[n_qt] : 0;
  }

  if (warp == 9) {
    // ------------------------------------------------------------------ loads and the dS store
    if (lane == 0 && n == 0 && kv_loaded)      // every tile was left out: K and V must still land before the CTA ends
      mbar_wait_relaxed(&bars->kv, 0, abort_flag, p.status, 38);
    if (lane == 0 && n > 0) {
      for (int i = 0; i < n && ok; ++i) {
        ok = mbar_wait_relaxed(&bars->p_full, i & 1, abort_flag, p.status, 41);
        if (!ok) break;
        tma_store_3d(&mds, smem + L::kDS0, tile_of(i) * 64, k0, b * p.H + h);
        bulk_commit_group();
        if (i + NST < n) {    // the reload goes out before the store's read is waited for: its latency is the longer one
          ok = mbar_wait_relaxed(&bars->qd_free[i % NST], (i / NST) & 1, abort_flag, p.status, 42);
          if (ok) load_qd(i + NST);
        }
        bulk_wait_group_read<0>();                      // the store has read the tile: the softmax warps may refill it
        mbar_arrive(&bars->p_free);
      }
      bulk_wait_group<0>();
      if (!ok) {   // a wait ran out: give loads still in flight a bounded time to land
        long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) {}
      }
    }
  } else if (warp == 8) {
    // ------------------------------------------------------------------ MMA issue
    // All 32 lanes walk the loop (waits included) so that its counters and the descriptor words are warp-uniform;
    // the elected lane alone executes the MMAs and commits.
    if (n > 0) {
      const uint32_t lead = elect_one_lane();
      constexpr uint32_t idesc_s = make_idesc(128, 64, false, false);
      constexpr uint32_t idesc_acc = make_idesc(128, DK, false, true);
      // low words of the operand descriptors: K and V (K-major), the Q / dO ring, the P^T / dS^T tiles
      const uint32_t lK = desc_lo_k(smem_u32(smem + L::kK)), lV = desc_lo_k(smem_u32(smem + L::kV));
      const uint32_t lQ0 = desc_lo_k(smem_u32(smem + L::kQD0)), lPt = desc_lo_k(smem_u32(smem + L::kP0)),
                     lDSt = desc_lo_k(smem_u32(smem + L::kDS0));
      constexpr uint32_t kToMn = ((8192u >> 4) << 16) - ((16u >> 4) << 16);   // K-major low word -> MN-major
      // S^T = K Q^T and dP^T = V dO^T of tile i
      auto issue_sdp = [&](int i) {
        const int st = i % NST;
        if (!__all_sync(0xffffffffu, mbar_wait_relaxed(&bars->qd_full[st], (i / NST) & 1, abort_flag, p.status, 43))) return false;
        tc_fence_after();
        const uint32_t lQ = lQ0 + st * (L::kStage >> 4), lDO = lQ + (L::kQTile >> 4);
#pragma unroll
        for (int kk = 0; kk < DK / 16; ++kk) {
          uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
          umma_bf16_lo_lead(tmem_base + kColS, lK + (oa >> 4), lQ + (ob >> 4), idesc_s, kk != 0, lead);
        }
#pragma unroll
        for (int kk = 0; kk < DK / 16; ++kk) {
          uint32_t oa = (kk >> 2) * 16384 + (kk & 3) * 32, ob = (kk >> 2) * 8192 + (kk & 3) * 32;
          umma_bf16_lo_lead(tmem_base + kColDP, lV + (oa >> 4), lDO + (ob >> 4), idesc_s, kk != 0, lead);
        }
        umma_commit_lead(&bars->s_full, lead);
        return true;
      };
      ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->kv, 0, abort_flag, p.status, 44));
      if (ok) ok = issue_sdp(0);
      for (int i = 0; i < n && ok; ++i) {
        const int st = i % NST;
        if (i + 1 < n) {      // the softmax warps have the scores of tile i in registers: S^T / dP^T of tile i+1 go first
          ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->s_free, i & 1, abort_flag, p.status, 49));
          if (!ok) break;
          tc_fence_after();
          ok = issue_sdp(i + 1);
          if (!ok) break;
        }
        ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->p_full, i & 1, abort_flag, p.status, 45));
        if (!ok) break;
        tc_fence_after();
        const uint32_t lQm = lQ0 + st * (L::kStage >> 4) + kToMn, lDOm = lQm + (L::kQTile >> 4);
        const uint32_t first = i == 0 ? 0u : 1u;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          umma_bf16_lo_lead(tmem_base + kColDV, lPt + ((ks * 32) >> 4), lDOm + ((ks * 2048) >> 4), idesc_acc, first | ks, lead);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          umma_bf16_lo_lead(tmem_base + kColDK, lDSt + ((ks * 32) >> 4), lQm + ((ks * 2048) >> 4), idesc_acc, first | ks, lead);
        umma_commit_lead(&bars->p_free, lead);
        umma_commit_lead(&bars->qd_free[st], lead);
      }
      if (ok) umma_commit_lead(&bars->acc, lead);
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int quad = warp & 3, half = warp >> 2, row = quad * 32 + lane;
    const int j = k0 + row;
    const int ck = j < p.Tk ? p.code_k[b * p.Tk + j] : 0;
    // row factor of this key's dK / dV rows (folded RMSNorm), fetched now so that the epilogue does not wait for it
    const float fv_row = j < p.Tk ? rn_factor(p.rn_k, (int64_t)b * p.Tk + j) : 0.f;
    {
      // The per-CTA tables are filled here, by the softmax warps alone and behind their own barrier: the loads
      // and the first S^T / dP^T MMAs of the other two warps run meanwhile.  One batched fill of the four tables
      // (contiguous in shared memory), every global load in flight at once.  Bias: distance of (key j = k0 + row, query q) is j - q, window index w = row - q + tqp in [1, tqp + 127].
      const int64_t bh = (int64_t)(b * p.H + h) * p.Tq;
      const int nb = tqp + 128;
      auto table = [&](int x) -> uint32_t {
        if (x < nb) {
          int g = (x - tqp) + k0 + p.Tq - 1;
          return __float_as_uint((p.bias_delta && g >= 0 && g < span) ? p.bias_delta[(int64_t)h * span + g] * kLog2e : 0.f);
        }
        x -= nb;
        if (x < tqp) return __float_as_uint(x < p.Tq ? p.lse[bh + x] * kLog2e : -INFINITY);
        x -= tqp;
        if (x < tqp) return __float_as_uint(x < p.Tq ? p.delta[bh + x] : 0.f);
        x -= tqp;
        return (uint32_t)(x < p.Tq ? p.code_q[b * p.Tq + x] : 0);
      };
      fill_batched<kKvfSoftmaxThreads, uint32_t, decltype(table), 9>((uint32_t*)bias_s, nb + 3 * tqp, tid, table);
      if (want_db)
        for (int w = tid; w < nb; w += kKvfSoftmaxThreads) dbias_s[w] = 0.f;
      asm volatile("bar.sync 1, 256;" ::: "memory");
    }
    if (p.packed) {
      ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->list, 0, abort_flag, p.status, 40));
      n = ok ? qt_s[n_qt] : 0;
    }
    const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
    const float sc2 = p.scale * kLog2e;
    const bool has_bias = p.bias_delta != nullptr;
    float far_pos = 0.f, far_neg = 0.f;
    // `ok` is kept warp-uniform (every wait's answer goes through a vote): the warp-level barriers below are
    // reached by all 32 lanes or by none
    unsigned char* tP = smem + L::kP0;
    unsigned char* tD = smem + L::kDS0;
    for (int i = 0; i < n && ok; ++i) {
      const int qb = tile_of(i) * 64;
      const uint32_t par = i & 1;
      ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->s_full, par, abort_flag, p.status, 46));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        const int cc = half * 32 + c * 16;                 // first of this pass's 16 queries within the tile
        const int qq0 = qb + cc;
        int cmine = codes_s[qq0 + (lane & 15)];
        const bool fast = __all_sync(0xffffffffu, cmine == ck) && ck != 0 &&
                          (!p.causal || k0 + quad * 32 + 31 <= qq0);           // warp-uniform: no mask needed
        const float* brow = bias_s + (row - qq0 + tqp);    // element e: brow[-e]
        uint32_t rs[16], rp[16];
        tmem_ld_32x32b_x16(tmem_base + lane_off + kColS + cc, rs);
        tmem_ld_32x32b_x16(tmem_base + lane_off + kColDP + cc, rp);
        tmem_wait_ld_dep16(rs);
        tmem_wait_ld_dep16(rp);
        if (c == 1) {      // both passes are out of tensor memory: the MMA warp may overwrite the buffer (tile i+1)
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&bars->s_free);
        }
        float pt[16], ds[16];
        // bias_c: 0 none, 1 per distance, 2 one value for the whole pass (saturated bucket)
        auto compute = [&](auto fast_c, auto bias_c) {
          constexpr bool FAST = decltype(fast_c)::value;
          constexpr int BIAS = decltype(bias_c)::value;
          const float bflat = BIAS == 2 ? brow[0] : 0.f;
#pragma unroll
          for (int i4 = 0; i4 < 4; ++i4) {
            const float4 l4 = *reinterpret_cast<const float4*>(lse_s + qq0 + i4 * 4);
            const float4 d4 = *reinterpret_cast<const float4*>(dl_s + qq0 + i4 * 4);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int ii = i4 * 4 + e;
              const float lse2 = e == 0 ? l4.x : e == 1 ? l4.y : e == 2 ? l4.z : l4.w;
              const float dlq = e == 0 ? d4.x : e == 1 ? d4.y : e == 2 ? d4.z : d4.w;
              float sv = BIAS == 1 ? fmaf(__uint_as_float(rs[ii]), sc2, brow[-ii])
                                   : BIAS == 2 ? fmaf(__uint_as_float(rs[ii]), sc2, bflat) : __uint_as_float(rs[ii]) * sc2;
              float pr = ex2_approx(sv - lse2);
              if (!FAST) {
                int q = qq0 + ii;
                int cqv = codes_s[q];
                bool valid = pair_valid(cqv, ck, p.causal != 0, j, q) && lse2 != -INFINITY;
                pr = valid ? pr : 0.f;
              }
              pt[ii] = pr;
              ds[ii] = pr * (__uint_as_float(rp[ii]) - dlq);
            }
          }
        };
        using B0 = std::integral_constant<int, 0>;
        using B1 = std::integral_constant<int, 1>;
        using B2 = std::integral_constant<int, 2>;
        const int kk0b = k0 + quad * 32;                 // this pass: keys [kk0b, kk0b + 32) x queries [qq0, qq0 + 16)
        const bool flat = has_bias && p.bias_far > 0 && (kk0b - (qq0 + 15) >= p.bias_far || qq0 - (kk0b + 31) >= p.bias_far);
        if (fast) {
          if (flat) compute(std::true_type{}, B2{});
          else if (has_bias) compute(std::true_type{}, B1{});
          else compute(std::true_type{}, B0{});
        } else {
          if (has_bias) compute(std::false_type{}, B1{}); else compute(std::false_type{}, B0{});
        }
        if (want_db) {
          const int kk0 = k0 + quad * 32;                  // this pass: 32 keys x 16 queries
          if (p.bias_far > 0 && kk0 - (qq0 + 15) >= p.bias_far) {
            float t0 = 0.f, t1 = 0.f;
#pragma unroll
            for (int e = 0; e < 16; e += 2) { t0 += ds[e]; t1 += ds[e + 1]; }
            far_pos += t0 + t1;
          } else if (p.bias_far > 0 && qq0 - (kk0 + 31) >= p.bias_far) {
            float t0 = 0.f, t1 = 0.f;
#pragma unroll
            for (int e = 0; e < 16; e += 2) { t0 += ds[e]; t1 += ds[e + 1]; }
            far_neg += t0 + t1;
          } else {
            // Diagonal sums of the 32 x 16 block: at step e lane l takes query e of key row (l + e) mod 32, which
            // lies on diagonal (key - query) = l when l + e < 32 and l - 32 otherwise.
            float tot = 0.f, a1 = 0.f;
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              float v = __shfl_sync(0xffffffffu, ds[e], lane + e);      // source lane taken modulo 32
              tot += v;
              a1 += (lane + e >= 32) ? v : 0.f;
            }
            // window entry (key row - query + tqp); warps and passes overlap there: atomics
            float* win = dbias_s + (quad * 32 + lane - qq0 + tqp);
            atomicAdd(win, tot - a1);
            if (lane >= 17) atomicAdd(win - 32, a1);
          }
        }
        if (c == 0) {
          // the tile buffers are free once the accumulating MMAs of tile i-1 are done and its dS store has read them
          ok = __all_sync(0xffffffffu, mbar_wait_relaxed(&bars->p_free, par ^ 1, abort_flag, p.status, 47));
        }
        if (ok) {
#pragma unroll
          for (int q8 = 0; q8 < 2; ++q8) {
            uint4 v;
            v.x = pack_bf16(pt[q8 * 8 + 0], pt[q8 * 8 + 1]);
            v.y = pack_bf16(pt[q8 * 8 + 2], pt[q8 * 8 + 3]);
            v.z = pack_bf16(pt[q8 * 8 + 4], pt[q8 * 8 + 5]);
            v.w = pack_bf16(pt[q8 * 8 + 6], pt[q8 * 8 + 7]);
            store_swizzled_16B(tP, row, (cc >> 3) + q8, v);
            v.x = pack_bf16(ds[q8 * 8 + 0], ds[q8 * 8 + 1]);
            v.y = pack_bf16(ds[q8 * 8 + 2], ds[q8 * 8 + 3]);
            v.z = pack_bf16(ds[q8 * 8 + 4], ds[q8 * 8 + 5]);
            v.w = pack_bf16(ds[q8 * 8 + 6], ds[q8 * 8 + 7]);
            store_swizzled_16B(tD, row, (cc >> 3) + q8, v);
          }
        }
      }
      if (!ok) break;
      fence_proxy_async();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->p_full);
    }
    if (n > 0) ok = __all_sync(0xffffffffu, ok && mbar_wait_relaxed(&bars->acc, 0, abort_flag, p.status, 48));
    // the last dS store must have read its tile before the tile buffers are reused for the output rows
    if (n > 0) ok = __all_sync(0xffffffffu, ok && mbar_wait_relaxed(&bars->p_free, (n - 1) & 1, abort_flag, p.status, 50));
    // every softmax thread gets here whatever happened; behind this barrier the abort flag gives the whole group
    // one answer, so the barrier inside the epilogue is reached by all of them or by none
    asm volatile("bar.sync 1, 256;" ::: "memory");
    ok = *abort_flag == 0;
    if (ok) {
      tc_fence_after();
      // dV and dK rows go through idle operand tiles as 128-byte-swizzled [128 keys x 64] bf16 tiles (one per 64
      // columns) and leave with one TMA store per tile: full 128-byte row segments, rows beyond Tk clipped by the
      // tensor map.  dV uses the P^T / dS^T tiles, dK the dS^T tile (d_kv 64) or the Q / dO ring (d_kv 128).
      unsigned char* tV = smem + L::kP0;
      unsigned char* tK = DK == 64 ? smem + L::kDS0 : smem + L::kQD0;
      const float fv = fv_row, fk = p.scale * fv;
#pragma unroll
      for (int c = 0; c < DK / 32; ++c) {
        const int col = half * (DK / 2) + c * 16;          // this pass's 16 output columns
        const int chunk = col >> 6, piece0 = (col & 63) >> 3;
        uint32_t rv[16], rk[16];
        if (n > 0) {
          tmem_ld_32x32b_x16(tmem_base + lane_off + kColDV + col, rv);
          tmem_ld_32x32b_x16(tmem_base + lane_off + kColDK + col, rk);
          tmem_wait_ld_dep16(rv);
          tmem_wait_ld_dep16(rk);
        } else {
#pragma unroll
          for (int d = 0; d < 16; ++d) rv[d] = rk[d] = 0u;
        }
#pragma unroll
        for (int q8 = 0; q8 < 2; ++q8) {
          const int d = q8 * 8;
          uint4 v;
          v.x = pack_bf16(fv * __uint_as_float(rv[d]), fv * __uint_as_float(rv[d + 1]));
          v.y = pack_bf16(fv * __uint_as_float(rv[d + 2]), fv * __uint_as_float(rv[d + 3]));
          v.z = pack_bf16(fv * __uint_as_float(rv[d + 4]), fv * __uint_as_float(rv[d + 5]));
          v.w = pack_bf16(fv * __uint_as_float(rv[d + 6]), fv * __uint_as_float(rv[d + 7]));
          store_swizzled_16B(tV + chunk * 16384, row, piece0 + q8, v);
          v.x = pack_bf16(fk * __uint_as_float(rk[d]), fk * __uint_as_float(rk[d + 1]));
          v.y = pack_bf16(fk * __uint_as_float(rk[d + 2]), fk * __uint_as_float(rk[d + 3]));
          v.z = pack_bf16(fk * __uint_as_float(rk[d + 4]), fk * __uint_as_float(rk[d + 5]));
          v.w = pack_bf16(fk * __uint_as_float(rk[d + 6]), fk * __uint_as_float(rk[d + 7]));
          store_swizzled_16B(tK + chunk * 16384, row, piece0 + q8, v);
        }
      }
      fence_proxy_async();
      asm volatile("bar.sync 1, 256;" ::: "memory");      // the eight softmax warps
      if (tid == 0) {
#pragma unroll
        for (int c = 0; c < DK / 64; ++c) {
          tma_store_3d(&mdv_out, tV + c * 16384, h * DK + c * 64, k0, b);
          tma_store_3d(&mdk_out, tK + c * 16384, h * DK + c * 64, k0, b);
        }
        bulk_commit_group();
        bulk_wait_group_read<0>();
      }
      if (want_db && p.bias_far > 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          far_pos += __shfl_xor_sync(0xffffffffu, far_pos, o);
          far_neg += __shfl_xor_sync(0xffffffffu, far_neg, o);
        }
        if (lane == 0) {
          const int gp = p.bias_far + p.Tq - 1, gn = -p.bias_far + p.Tq - 1;
          if (far_pos != 0.f && gp < span) atomicAdd(&p.dbias_delta[(int64_t)h * span + gp], far_pos);
          if (far_neg != 0.f && gn >= 0) atomicAdd(&p.dbias_delta[(int64_t)h * span + gn], far_neg);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (want_db && !*abort_flag) {
    // window index w = (key row - query + tqp); distance = k0 + w - tqp
    for (int w = tid; w < tqp + 128; w += kKvfThreads) {
      const float v = dbias_s[w];
      const int g = k0 + w - tqp + p.Tq - 1;
      if (v != 0.f && g >= 0 && g < span) atomicAdd(&p.dbias_delta[(int64_t)h * span + g], v);
    }
  }
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Kernel B: dQ[128 queries x DK] = scale * sum over 64-key tiles of dS[128 x 64] K[64 x DK], with dS read from the
// key-major copy kernel A stored (so it is an MN-major A operand: two 64 x 64 boxes per tile).
template <int DK>
struct DqsLayout {
  static constexpr int kStages = 4;
  static constexpr int kABytes = 2 * 8192, kBBytes = 64 * DK * 2;
  static constexpr int kStage = kABytes + kBBytes;
  static constexpr int kBar = kStages * kStage;
  static constexpr int kList = kBar + 256;                       // key tiles this CTA walks (packed rows): up to 130 ints
  static constexpr int kTotal = kList + 1024 + 1024;
};

template <int DK>
__global__ void __launch_bounds__(192)
attn_bwd_dq_ds_tc_kernel(const __grid_constant__ CUtensorMap mds, const __grid_constant__ CUtensorMap mk, TcParams p) {
  pdl_sync();
  using L = DqsLayout<DK>;
  constexpr int NST = L::kStages;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(smem + L::kBar);
  uint64_t* empty = full + NST;
  uint64_t* done = empty + NST;
  uint64_t* list_bar = done + 1;      // packed rows: the list of key tiles is in shared memory
  uint32_t* tmem_holder = (uint32_t*)(list_bar + 1);
  volatile int* abort_flag = (volatile int*)(tmem_holder + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int b = blockIdx.z, h = blockIdx.y, q0 = blockIdx.x * 128;
  int n_kt = (p.Tk + 63) / 64;
  if (p.causal && !p.prefix) n_kt = min(n_kt, (q0 + 127) / 64 + 1);
  constexpr uint32_t kTmemCols = DK;
  int* kt_s = (int*)(smem + L::kList);
  auto tile_of = [&](int u) { return p.packed ? kt_s[u] : u; };

  if (tid == 0) {
    for (int s = 0; s < NST; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(done, 1);
    mbar_init(list_bar, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  // packed rows: the key tiles the dK / dV kernel left out for these queries hold nothing it stored.  The loading
  // warp makes the list while the rest of the set-up runs and publishes it; the others pick it up behind the barrier.
  const int t_end = n_kt;
  if (p.packed && warp == 0) {
    __syncwarp();
    n_kt = packed_tile_list_warp(p.code_q + (int64_t)b * p.Tq, p.Tq, q0, p.code_k + (int64_t)b * p.Tk, p.Tk, 0, t_end, kt_s, lane);
    if (lane == 0) kt_s[t_end] = n_kt;
    __syncwarp();
    if (lane == 0) mbar_arrive(list_bar);
  }
  if (warp == 1) tmem_alloc(tmem_holder, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  bool ok = true;
  if (p.packed && warp != 0) {
    ok = __all_sync(0xffffffffu, mbar_wait(list_bar, 0, abort_flag, p.status, 54));
    n_kt = ok ? kt_s[t_end] : 0;
  }

  if (warp == 0) {
    if (lane == 0) {
      int issued = 0;
      for (int u = 0; u < n_kt; ++u) {
        const int s = u % NST, t = tile_of(u);
        if (!mbar_wait(&empty[s], ((u / NST) & 1) ^ 1, abort_flag, p.status, 51)) { ok = false; break; }
        unsigned char* sa = smem + s * L::kStage;
        mbar_arrive_expect_tx(&full[s], L::kStage);
        tma_load_3d(sa, &mds, q0, t * 64, b * p.H + h, &full[s]);
        tma_load_3d(sa + 8192, &mds, q0 + 64, t * 64, b * p.H + h, &full[s]);
#pragma unroll
        for (int c = 0; c < DK / 64; ++c)
          tma_load_3d(sa + L::kABytes + c * 8192, &mk, h * DK + c * 64, t * 64, b, &full[s]);
        ++issued;
      }
      if (!ok && issued > 0) {   // a wait ran out: give loads still in flight a bounded time to land
        long long t0 = clock64();
        while (clock64() - t0 < 4000000ll) {}
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(128, DK, true, true);
      for (int t = 0; t < n_kt; ++t) {      // t counts the tiles walked, not key positions
        const int s = t % NST;
        if (!mbar_wait(&full[s], (t / NST) & 1, abort_flag, p.status, 52)) { ok = false; break; }
        tc_fence_after();
        const uint32_t la = desc_lo_mn(smem_u32(smem + s * L::kStage)), lb = la + (L::kABytes >> 4);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          umma_bf16_lo(tmem_base, la + ((ks * 2048) >> 4), lb + ((ks * 2048) >> 4), idesc, (t | ks) != 0);
        umma_commit(&empty[s]);
      }
      if (ok) umma_commit(done);
    }
  } else {
    // epilogue: warps 2-5; warp w may touch tensor-memory lanes 32 (w % 4) ..
    const int quad = warp & 3, row = quad * 32 + lane, i = q0 + row;
    const float fq = i < p.Tq ? p.scale * rn_factor(p.rn_q, (int64_t)b * p.Tq + i) : 0.f;      // before the wait
    ok = mbar_wait(done, 0, abort_flag, p.status, 53);
    if (ok) {
      tc_fence_after();
      bf16* drow = (bf16*)p.out0 + (int64_t)(b * p.Tq + i) * p.ld0 + h * DK;
      const uint32_t lane_off = (uint32_t)(quad * 32) << 16;
#pragma unroll
      for (int c = 0; c < DK / 32; ++c) {
        uint32_t r[32];
        if (n_kt > 0) {
          tmem_ld_32x32b_x32(tmem_base + lane_off + c * 32, r);
          tmem_wait_ld_dep(r);
        } else {
#pragma unroll
          for (int d = 0; d < 32; ++d) r[d] = 0u;
        }
        if (i < p.Tq) {
#pragma unroll
          for (int d = 0; d < 32; d += 8) {
            uint4 v;
            v.x = pack_bf16(fq * __uint_as_float(r[d]), fq * __uint_as_float(r[d + 1]));
            v.y = pack_bf16(fq * __uint_as_float(r[d + 2]), fq * __uint_as_float(r[d + 3]));
            v.z = pack_bf16(fq * __uint_as_float(r[d + 4]), fq * __uint_as_float(r[d + 5]));
            v.w = pack_bf16(fq * __uint_as_float(r[d + 6]), fq * __uint_as_float(r[d + 7]));
            *reinterpret_cast<uint4*>(drow + c * 32 + d) = v;
          }
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

template <int DK>
cudaError_t fwd_launch(const AttnArgs& a, int* status, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  int I = a.H * DK;
  if (!make_map3(&mq, a.Q, I, a.Tq, a.B, a.ldq, 128) || !make_map3(&mk, a.K, I, a.Tk, a.B, a.ldk, 64) ||
      !make_map3(&mv, a.V, I, a.Tk, a.B, a.ldv, 64))
    return cudaErrorInvalidValue;
  int smem = FwdLayout<DK>::bytes(a.Tk);
  cudaError_t e = cudaFuncSetAttribute(attn_fwd_tc_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  TcParams p = base_params(a, status);
  p.out0 = a.O; p.ld0 = a.ldo; p.o32 = a.O32; p.ldo32 = a.ldo32;
  dim3 grid((a.Tq + 127) / 128, a.H, a.B);
  return launch_pdl(attn_fwd_tc_kernel<DK>, grid, dim3(128), smem, st, mq, mk, mv, p);
}

// One pass over the scores: kernel A (dK, dV, dS^T to scratch) then kernel B (dQ from the stored dS^T).
template <int DK>
cudaError_t bwd_fused_launch(const AttnArgs& a, int* status, cudaStream_t st) {
  const int I = a.H * DK;
  const int tqp = (a.Tq + 63) / 64 * 64, tkp = (a.Tk + 127) / 128 * 128;
  TcParams p = base_params(a, status);
  CUtensorMap mq, mdo, mk, mv, mds_st, mds_ld, mk64, mdk_out, mdv_out;
  if (!make_map3(&mq, a.Q, I, a.Tq, a.B, a.ldq, 64) || !make_map3(&mdo, a.dO, I, a.Tq, a.B, a.lddo, 64) ||
      !make_map3(&mk, a.K, I, a.Tk, a.B, a.ldk, 128) || !make_map3(&mv, a.V, I, a.Tk, a.B, a.ldv, 128) ||
      !make_map3(&mk64, a.K, I, a.Tk, a.B, a.ldk, 64) ||
      !make_map3(&mdk_out, a.dK, I, a.Tk, a.B, a.lddk, 128) || !make_map3(&mdv_out, a.dV, I, a.Tk, a.B, a.lddv, 128) ||
      !make_map3(&mds_st, a.ds_scratch, tqp, tkp, a.B * a.H, tqp, 128) ||
      !make_map3(&mds_ld, a.ds_scratch, tqp, tkp, a.B * a.H, tqp, 64))
    return cudaErrorInvalidValue;
  {
    int smem = KvfLayout<DK>::bytes(a.Tq, a.dbias_delta != nullptr);
    cudaError_t e = cudaFuncSetAttribute(attn_bwd_kvf_tc_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    dim3 grid((a.Tk + 127) / 128, a.H, a.B);
    e = launch_pdl(attn_bwd_kvf_tc_kernel<DK>, grid, dim3(kKvfThreads), smem, st, mq, mdo, mk, mv, mds_st, mdk_out, mdv_out, p);
    if (e != cudaSuccess) return e;
  }
  {
    int smem = DqsLayout<DK>::kTotal;
    cudaError_t e = cudaFuncSetAttribute(attn_bwd_dq_ds_tc_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    p.out0 = a.dQ; p.ld0 = a.lddq;
    dim3 grid((a.Tq + 127) / 128, a.H, a.B);
    return launch_pdl(attn_bwd_dq_ds_tc_kernel<DK>, grid, dim3(192), smem, st, mds_ld, mk64, p);
  }
}

template <int DK>
cudaError_t bwd_launch(const AttnArgs& a, int* status, cudaStream_t st) {
  int I = a.H * DK;
  const int64_t dthreads = (int64_t)a.B * a.Tq * (I / 8);
  cudaError_t e = launch_pdl(attn_delta_tc_kernel<DK>, dim3((unsigned)((dthreads + 255) / 256)), dim3(256), 0, st,
                             (const bf16*)a.O, a.ldo, (const float*)a.O32, a.ldo32, (const bf16*)a.dO, a.lddo, a.delta, a.B, a.H,
                             a.Tq);
  if (e != cudaSuccess) return e;
  if (attn_tc_onepass_supported(a)) return bwd_fused_launch<DK>(a, status, st);
  TcParams p = base_params(a, status);
  {
    CUtensorMap mq, mdo, mk, mv;
    if (!make_map3(&mq, a.Q, I, a.Tq, a.B, a.ldq, 128) || !make_map3(&mdo, a.dO, I, a.Tq, a.B, a.lddo, 128) ||
        !make_map3(&mk, a.K, I, a.Tk, a.B, a.ldk, 64) || !make_map3(&mv, a.V, I, a.Tk, a.B, a.ldv, 64))
      return cudaErrorInvalidValue;
    int smem = DqLayout<DK>::bytes(a.Tk);
    e = cudaFuncSetAttribute(attn_bwd_dq_tc_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    p.out0 = a.dQ; p.ld0 = a.lddq;
    dim3 grid((a.Tq + 127) / 128, a.H, a.B);
    attn_bwd_dq_tc_kernel<DK><<<grid, 256, smem, st>>>(mq, mdo, mk, mv, p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  {
    CUtensorMap mq, mdo, mk, mv;
    if (!make_map3(&mq, a.Q, I, a.Tq, a.B, a.ldq, 64) || !make_map3(&mdo, a.dO, I, a.Tq, a.B, a.lddo, 64) ||
        !make_map3(&mk, a.K, I, a.Tk, a.B, a.ldk, 128) || !make_map3(&mv, a.V, I, a.Tk, a.B, a.ldv, 128))
      return cudaErrorInvalidValue;
    int smem = DkvLayout<DK>::bytes(a.Tq);
    e = cudaFuncSetAttribute(attn_bwd_dkv_tc_kernel<DK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    p.out0 = a.dK; p.ld0 = a.lddk; p.out1 = a.dV; p.ld1 = a.lddv;
    dim3 grid((a.Tk + 127) / 128, a.H, a.B);
    attn_bwd_dkv_tc_kernel<DK><<<grid, 256, smem, st>>>(mq, mdo, mk, mv, p);
    e = cudaGetLastError();
  }
  return e;
}

}  // namespace

int64_t attn_tc_ds_scratch_bytes(int B, int H, int Tq, int Tk) {
  int64_t tqp = (Tq + 63) / 64 * 64, tkp = (Tk + 127) / 128 * 128;
  return (int64_t)B * H * tqp * tkp * 2;
}

bool attn_tc_onepass_supported(const AttnArgs& a) {
  if ((a.dk != 64 && a.dk != 128) || !a.ds_scratch || ((uintptr_t)a.ds_scratch & 127) != 0 ||
      a.ds_bytes < attn_tc_ds_scratch_bytes(a.B, a.H, a.Tq, a.Tk))
    return false;
  const bool db = a.dbias_delta != nullptr;
  return (a.dk == 64 ? KvfLayout<64>::bytes(a.Tq, db) : KvfLayout<128>::bytes(a.Tq, db)) <= 227 * 1024;
}

bool attn_tc_supported(const AttnArgs& a) {
  if (a.dk != 64 && a.dk != 128) return false;
  if (a.Tq < 1 || a.Tk < 1 || a.Tq > 8192 || a.Tk > 8192) return false;
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (!al16(a.Q) || !al16(a.K) || !al16(a.V) || !al16(a.O)) return false;
  if (a.ldq % 8 || a.ldk % 8 || a.ldv % 8 || a.ldo % 8) return false;
  if (a.O32 && (!al16(a.O32) || a.ldo32 % 4)) return false;
  if (a.causal && a.Tq != a.Tk) return false;
  // every kernel's shared-memory footprint (tiles + distance-indexed windows) must fit one CTA
  const int kSmemMax = 227 * 1024;
  int need = a.dk == 64 ? max(FwdLayout<64>::bytes(a.Tk), max(DqLayout<64>::bytes(a.Tk), DkvLayout<64>::bytes(a.Tq)))
                        : max(FwdLayout<128>::bytes(a.Tk), max(DqLayout<128>::bytes(a.Tk), DkvLayout<128>::bytes(a.Tq)));
  if (need > kSmemMax) return false;
  return tc::get_encode() != nullptr;
}

cudaError_t attn_fwd_tc(const AttnArgs& a, int* d_status, cudaStream_t st) {
  if (a.B == 0) return cudaSuccess;
  return a.dk == 64 ? fwd_launch<64>(a, d_status, st) : fwd_launch<128>(a, d_status, st);
}

cudaError_t attn_bwd_tc(const AttnArgs& a, int* d_status, cudaStream_t st) {
  if (a.B == 0) return cudaSuccess;
  auto al16 = [](const void* p) { return ((uintptr_t)p & 15) == 0; };
  if (!al16(a.dO) || !al16(a.dQ) || !al16(a.dK) || !al16(a.dV) || a.lddo % 8 || a.lddq % 8 || a.lddk % 8 ||
      a.lddv % 8)
    return cudaErrorInvalidValue;
  return a.dk == 64 ? bwd_launch<64>(a, d_status, st) : bwd_launch<128>(a, d_status, st);
}
