// Fused scaled-dot-product attention on tcgen05 (Section VII "MHA": two batch matmuls with the softmax and
// the binary ops between them fused after the first one; the two matmul loop nests merged).
//
// Persistent CTAs (one per SM, 384 threads) walk over work units (batch, head, 128-query tile):
//   warp 0      TMA producer: Q tile, all K rows and all V rows of the unit into one of two shared-memory
//               slots (128B / 64B swizzle), one unit ahead of the math (no multicast)
//   warp 1      MMA issuer (one thread): S = Q K^T in 128-key blocks into tensor memory, O = P V in 128-key
//               blocks as soon as each P block is ready; the next unit's S blocks are issued as soon as the
//               softmax warps release the corresponding TMEM columns
//   warps 2-3   per-unit preparation: u8 -> s8 flip of Q (int8 path), mask row scaled by log2(e)
//   warps 4-11  softmax: two threads per query row (TMEM lane), each owning 64 of every 128 key columns.
//               Pass A: scale + mask, running row max, exp2 and running row sum (int8: the exponentials
//               are written back to tensor memory); the two threads of a row combine their statistics;
//               Pass B: normalise, quantise to u8 (int8) or cast to bf16, write P to shared memory as the
//               K-major A operand of the second MMA.  V is consumed from its [key][d] layout as an
//               MN-major B operand, so nothing is transposed in memory.
// The whole score row of a query stays in tensor memory (S <= 384 columns + 64 for O), which makes the
// exact two-pass softmax possible that quantised probabilities need (the row sum must be final before
// any probability is rounded).
//
// int8 zero points: Q (u8, zero point 128) is flipped to s8 in shared memory: (u8 ^ 0x80) as s8 = u8 - 128.
// K stays as stored: sum_d q'_d (k_d - z) = sum_d q'_d k_d - z sum_d q'_d differs from the wanted score
// by a per-row constant, which softmax cancels.  V stays u8 and its zero point is removed from the
// accumulator with the row sum of P:  sum_j P_j (V_j - z) = sum_j P_j V_j - z sum_j P_j.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int SDPA_D = 64;
constexpr int SDPA_BLOCK_Q = 128;
constexpr int SDPA_THREADS = 384;
constexpr int SDPA_SOFTMAX_WARPS = 8;
constexpr float LOG2E = 1.4426950408889634f;

template <bool INT8>
struct SdpaSmem {
  static constexpr int ESZ = INT8 ? 1 : 2;
  static constexpr int ROW_BYTES = SDPA_D * ESZ;               // 64 (SW64) or 128 (SW128)
  __host__ __device__ static constexpr int q_bytes() { return SDPA_BLOCK_Q * ROW_BYTES; }
  __host__ __device__ static constexpr int kv_bytes(int S) { return S * ROW_BYTES; }
  // P: per 128-key block, 128 rows x (128 keys * ESZ) bytes = 16 KB (int8) or 32 KB (bf16)
  __host__ __device__ static constexpr int p_bytes(int S) { return (S / 128) * SDPA_BLOCK_Q * 128 * ESZ; }
  __host__ __device__ static constexpr int slot_bytes(int S) { return q_bytes() + 2 * kv_bytes(S); }
  __host__ __device__ static constexpr int total(int S, int slots) {
    return slots * slot_bytes(S) + p_bytes(S) + slots * S * 4 /*mask*/ + 4 * 128 * 4 /*row statistics*/ + 256;
  }
};

static int sdpa_slots(int S, int is_int8, size_t smem_limit) {
  for (int slots = 2; slots >= 1; --slots) {
    const size_t need = 1024 + (is_int8 ? SdpaSmem<true>::total(S, slots) : SdpaSmem<false>::total(S, slots));
    if (need <= smem_limit) return slots;
  }
  return 0;
}

size_t sdpa_tc_smem_bytes(int S, int is_int8) {
  const int slots = sdpa_slots(S, is_int8, 227 * 1024);
  if (!slots) return static_cast<size_t>(1) << 30;
  return 1024 + (is_int8 ? SdpaSmem<true>::total(S, slots) : SdpaSmem<false>::total(S, slots));
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <bool INT8>
__global__ void __launch_bounds__(SDPA_THREADS, 1)
sdpa_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const SdpaParams p, const int slots) {
  using L = SdpaSmem<INT8>;
  constexpr int ROW_BYTES = L::ROW_BYTES;
  constexpr uint32_t SWZ = INT8 ? SWZ_64B : SWZ_128B;
  constexpr uint32_t SBO = 8 * ROW_BYTES;                       // 8-row group stride: 512 or 1024 bytes
  constexpr int P_BLOCK_BYTES = SDPA_BLOCK_Q * 128 * L::ESZ;    // one 128-key block of P
  constexpr uint32_t TMEM_COLS = 512;

  const int S = p.S;
  const int NB = S / 128;                                       // key blocks
  const int O_COL = S;                                          // TMEM column of the output accumulator
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sSlots = smem;
  uint8_t* sP = sSlots + slots * L::slot_bytes(S);
  float* sMask = reinterpret_cast<float*>(sP + L::p_bytes(S));  // [slots][S]
  float* sStat = sMask + slots * S;                             // [4][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sStat + 4 * 128);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 20);
  const uint32_t b0 = smem_u32(bars);
  const uint32_t bar_kv_full = b0, bar_kv_empty = b0 + 16, bar_kv_ready = b0 + 32;   // [2] each
  const uint32_t bar_s_full = b0 + 48, bar_s_free = b0 + 72, bar_p_full = b0 + 96;   // [3] each
  const uint32_t bar_o_full = b0 + 120, bar_o_free = b0 + 128, bar_xchg = b0 + 136;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q_tiles = S / SDPA_BLOCK_Q;
  const int num_units = p.B * p.H * q_tiles;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_kv_full + 8 * i, 1);
      mbar_init(bar_kv_empty + 8 * i, 1);
      mbar_init(bar_kv_ready + 8 * i, 2);
    }
    for (int i = 0; i < 3; ++i) {
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_s_free + 8 * i, SDPA_SOFTMAX_WARPS);
      mbar_init(bar_p_full + 8 * i, SDPA_SOFTMAX_WARPS);
    }
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, SDPA_SOFTMAX_WARPS);
    mbar_init(bar_xchg, SDPA_SOFTMAX_WARPS);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  bool failed = false;
  auto slot_q = [&](int s) { return sSlots + s * L::slot_bytes(S); };
  auto slot_k = [&](int s) { return slot_q(s) + L::q_bytes(); };
  auto slot_v = [&](int s) { return slot_k(s) + L::kv_bytes(S); };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units; unit += gridDim.x, ++n) {
        const int s = n % slots;
        const uint32_t par = (n / slots) & 1;
        if (!mbar_wait(bar_kv_empty + 8 * s, par ^ 1)) {
          report(p.status, DEV_TIMEOUT_PRODUCER);
          failed = true;
          break;
        }
        const int bh = unit / q_tiles, qt = unit % q_tiles;
        mbar_arrive_expect_tx(bar_kv_full + 8 * s, static_cast<uint32_t>(L::slot_bytes(S)));
        tma_load_2d(smem_u32(slot_q(s)), &tmQ, 0, bh * S + qt * SDPA_BLOCK_Q, bar_kv_full + 8 * s);
        for (int j = 0; j < NB; ++j) {
          tma_load_2d(smem_u32(slot_k(s)) + j * 128 * ROW_BYTES, &tmK, 0, bh * S + j * 128, bar_kv_full + 8 * s);
          tma_load_2d(smem_u32(slot_v(s)) + j * 128 * ROW_BYTES, &tmV, 0, bh * S + j * 128, bar_kv_full + 8 * s);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = INT8 ? make_idesc(ACC_S32, FMT_S8, p.k_signed ? FMT_S8 : FMT_U8, 128, 128)
                                   : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, 128);
      const uint32_t idesc2 = INT8 ? make_idesc(ACC_S32, FMT_U8, p.v_signed ? FMT_S8 : FMT_U8, 128, SDPA_D, 0, 1)
                                   : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, SDPA_D, 0, 1);
      constexpr int K1_STEPS = ROW_BYTES / 32;                  // 32 bytes of the head dimension per MMA
      constexpr int K2_STEPS = 128 / (INT8 ? 32 : 16);          // MMAs per 128-key block of P.V
      auto mma1 = [&](int s, int b) {                           // S[:, 128b .. 128b+127] = Q K_b^T
        const uint64_t a_desc = make_smem_desc(smem_u32(slot_q(s)), 16, SBO, SWZ);
        const uint64_t b_desc = make_smem_desc(smem_u32(slot_k(s)) + b * 128 * ROW_BYTES, 16, SBO, SWZ);
#pragma unroll
        for (int k = 0; k < K1_STEPS; ++k)
          umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + b * 128, a_desc + 2 * k, b_desc + 2 * k, idesc1, k != 0);
        umma_commit(bar_s_full + 8 * b);
      };
      auto mma2 = [&](int s, int b) {                           // O += P_b V_b
#pragma unroll
        for (int ks = 0; ks < K2_STEPS; ++ks) {
          // A: P block, K-major, 128B swizzle: 4 MMA steps of 32 bytes per 128-byte span, spans 16 KB apart
          const uint64_t a_desc = make_smem_desc(smem_u32(sP) + b * P_BLOCK_BYTES + (ks >> 2) * (SDPA_BLOCK_Q * 128) +
                                                     (ks & 3) * 32, 16, 1024, SWZ_128B);
          // B: V as stored [key][d] = MN-major: one key per ROW_BYTES, 8-key groups SBO apart
          const int key0 = b * 128 + ks * (128 / K2_STEPS);
          const uint64_t b_desc = make_smem_desc(smem_u32(slot_v(s)) + key0 * ROW_BYTES, SBO, SBO, SWZ);
          umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + O_COL, a_desc, b_desc, idesc2, (b | ks) != 0);
        }
      };
      const bool interleave = slots == 2;
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        const int s = n % slots;
        const bool has_next = unit + static_cast<int>(gridDim.x) < num_units;
        const int sn = (n + 1) % slots;
        if (n == 0) {
          if (!mbar_wait(bar_kv_ready + 8 * s, 0) || !mbar_wait(bar_kv_full + 8 * s, 0)) { failed = true; break; }
          tc_fence_after();
          for (int b = 0; b < NB; ++b) mma1(s, b);
        }
        bool next_ready = false;
        for (int b = 0; b < NB && !failed; ++b) {
          if (!mbar_wait(bar_p_full + 8 * b, n & 1)) { failed = true; break; }
          if (b == 0 && !mbar_wait(bar_o_free, (n & 1) ^ 1)) { failed = true; break; }
          tc_fence_after();
          mma2(s, b);
          if (b == NB - 1) {
            umma_commit(bar_o_full);
            umma_commit(bar_kv_empty + 8 * s);
          }
          if (has_next && interleave) {
            if (!next_ready) {
              if (!mbar_wait(bar_kv_ready + 8 * sn, ((n + 1) / slots) & 1) ||
                  !mbar_wait(bar_kv_full + 8 * sn, ((n + 1) / slots) & 1)) { failed = true; break; }
              next_ready = true;
            }
            if (!mbar_wait(bar_s_free + 8 * b, n & 1)) { failed = true; break; }
            tc_fence_after();
            mma1(sn, b);
          }
        }
        if (!failed && has_next && !interleave) {
          if (!mbar_wait(bar_kv_ready + 8 * sn, ((n + 1) / slots) & 1) ||
              !mbar_wait(bar_kv_full + 8 * sn, ((n + 1) / slots) & 1)) { failed = true; break; }
          for (int b = 0; b < NB && !failed; ++b) {
            if (!mbar_wait(bar_s_free + 8 * b, n & 1)) { failed = true; break; }
            tc_fence_after();
            mma1(sn, b);
          }
        }
      }
      if (failed) report(p.status, DEV_TIMEOUT_MMA);
    }
  } else if (warp < 4) {
    // ------------------------------------------------------------------ per-unit preparation
    const int t = tid - 64;                                     // 0..63
    int n = 0;
    for (int unit = blockIdx.x; unit < num_units; unit += gridDim.x, ++n) {
      const int s = n % slots;
      const int b = (unit / q_tiles) / p.H;
      float* mk = sMask + s * S;
      // the mask slot is free once the unit that used it two steps ago has been fully consumed, which
      // the producer's own wait on kv_empty guarantees before kv_full can complete for this unit
      if (!mbar_wait(bar_kv_full + 8 * s, (n / slots) & 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        failed = true;
        break;
      }
      for (int j = t; j < S; j += 64) mk[j] = p.mask ? __ldg(p.mask + static_cast<int64_t>(b) * S + j) * LOG2E : 0.0f;
      if (INT8 && !p.q_signed) {
        uint4* q4 = reinterpret_cast<uint4*>(slot_q(s));
        for (int i = t; i < L::q_bytes() / 16; i += 64) {
          uint4 v = q4[i];
          v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
          q4[i] = v;
        }
        fence_proxy_async_smem();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_kv_ready + 8 * s);
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    const int sw = warp - 4;                                    // 0..7
    const int q = warp & 3;                                     // TMEM lane quarter
    const int h = sw >> 2;                                      // which 64 of every 128 key columns
    const int r = q * 32 + lane;                                // query row within the tile = TMEM lane
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const float c2 = (INT8 ? __fmul_rn(p.dq1, p.scalar) : p.scalar) * LOG2E;
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    uint32_t xphase = 0;
    float* stA = sStat + h * 128;                               // my statistics
    float* stB = sStat + (h ^ 1) * 128;                         // my partner's
    float* stA2 = sStat + 256 + h * 128;
    float* stB2 = sStat + 256 + (h ^ 1) * 128;

    auto xchg_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_xchg);
      const bool ok = mbar_wait(bar_xchg, xphase);
      xphase ^= 1;
      return ok;
    };
    // epilogue of unit (bh, qt): my 32 of the 64 output columns
    auto epilogue = [&](int unit, uint32_t par, float stat_total) -> bool {
      if (!mbar_wait(bar_o_full, par)) return false;
      tc_fence_after();
      uint32_t v[32];
      tmem_ld32(t_row + O_COL + h * 32, v);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_o_free);
      const int bh = unit / q_tiles, qt = unit % q_tiles;
      const int64_t grow = static_cast<int64_t>(bh) * S + qt * SDPA_BLOCK_Q + r;
      if constexpr (INT8) {
        const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
        const int corr = p.zp_v * __float_as_int(stat_total);   // zero point of V times the row sum of P
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          uint32_t word = 0;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int acc = static_cast<int>(v[4 * i + k]) - corr;
            const float t = __fmul_rn(__int2float_rn(acc), p.dq2);
            word |= static_cast<uint32_t>(quantize_value(t, p.inv_o, p.zp_o, lo, hi) & 0xFF) << (8 * k);
          }
          w[i] = word;
        }
        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.O) + grow * SDPA_D + h * 32);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else {
        const float rl = 1.0f / stat_total;                     // deferred normalisation by the row sum
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[2 * i]) * rl, __uint_as_float(v[2 * i + 1]) * rl);
          w[i] = *reinterpret_cast<uint32_t*>(&hh);
        }
        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.O) + grow * SDPA_D + h * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
      }
      return true;
    };

    int n = 0;
    int prev_unit = -1;
    float prev_stat = 0.f;                                      // row sum of P (int8: integer bits) of the previous unit
    for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
      const int s = n % slots;
      const float* mk = sMask + s * S;
      const uint32_t par = n & 1;
      if (!mbar_wait(bar_kv_ready + 8 * s, (n / slots) & 1)) { failed = true; break; }

      // ---------------- pass A
      float m = -INFINITY, l = 0.f;
      float mc[6];                                              // running max after each of my chunks (int8)
#pragma unroll
      for (int i = 0; i < 6; ++i) mc[i] = 0.f;
      for (int b = 0; b < NB && !failed; ++b) {
        if (!mbar_wait(bar_s_full + 8 * b, par)) { failed = true; break; }
        tc_fence_after();
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int col = b * 128 + h * 64 + cc * 32;
          uint32_t v[32];
          tmem_ld32(t_row + col, v);
          tmem_wait_ld();
          float x[32];
          float cmax = -INFINITY;
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float a = INT8 ? __int2float_rn(static_cast<int>(v[i])) : __uint_as_float(v[i]);
            x[i] = fmaf(a, c2, mk[col + i]);
            cmax = fmaxf(cmax, x[i]);
          }
          if constexpr (INT8) {
            const float m_new = fmaxf(m, cmax);
            float sum = 0.f;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const float e = ex2(x[i] - m_new);
              sum += e;
              v[i] = __float_as_uint(e);
            }
            l = l * ex2(m - m_new) + sum;
            m = m_new;
            if (b * 2 + cc == 0) mc[0] = m; else if (b * 2 + cc == 1) mc[1] = m; else if (b * 2 + cc == 2) mc[2] = m;
            else if (b * 2 + cc == 3) mc[3] = m; else if (b * 2 + cc == 4) mc[4] = m; else mc[5] = m;
            tmem_st32(t_row + col, v);
          } else {
            m = fmaxf(m, cmax);
          }
        }
      }
      if (failed) break;
      if constexpr (INT8) tmem_wait_st();
      stA[r] = m;
      if constexpr (INT8) stA2[r] = l;
      if (!xchg_sync()) { failed = true; break; }
      float scale;                                              // int8: inv_p / row sum
      float M;
      {
        const float m_p = stB[r];
        M = fmaxf(m, m_p);
        if constexpr (INT8) {
          const float l_p = stB2[r];
          const float Lsum = l * ex2(m - M) + l_p * ex2(m_p - M);
          scale = p.inv_p / Lsum;
        } else {
          scale = 1.f;
        }
      }
      // both threads of every row have read the statistics before they are overwritten below
      if (!xchg_sync()) { failed = true; break; }

      // ---------------- epilogue of the previous unit (its second MMA has had a whole pass to finish)
      if (prev_unit >= 0) {
        if (!epilogue(prev_unit, (n - 1) & 1, prev_stat)) { failed = true; break; }
      }

      // ---------------- pass B
      int psum = 0;
      float lsum = 0.f;
      for (int b = 0; b < NB; ++b) {
#pragma unroll
        for (int cc = 0; cc < 2; ++cc) {
          const int col = b * 128 + h * 64 + cc * 32;
          uint32_t v[32];
          tmem_ld32(t_row + col, v);
          tmem_wait_ld();
          if constexpr (INT8) {
            const int ci = b * 2 + cc;
            const float mcv = ci == 0 ? mc[0] : ci == 1 ? mc[1] : ci == 2 ? mc[2] : ci == 3 ? mc[3] : ci == 4 ? mc[4] : mc[5];
            const float f = ex2(mcv - M) * scale;
            uint32_t w[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int q0 = __float2int_rn(__uint_as_float(v[4 * i + 0]) * f);
              const int q1 = __float2int_rn(__uint_as_float(v[4 * i + 1]) * f);
              const int q2 = __float2int_rn(__uint_as_float(v[4 * i + 2]) * f);
              const int q3 = __float2int_rn(__uint_as_float(v[4 * i + 3]) * f);
              // p <= 1 and inv_p <= 255, so the codes are already in [0, 255]; min() guards rounding noise
              w[i] = min(q0, 255) | (min(q1, 255) << 8) | (min(q2, 255) << 16) | (min(q3, 255) << 24);
              psum = static_cast<int>(__dp4a(w[i], 0x01010101u, static_cast<unsigned>(psum)));
            }
            uint8_t* blk = sP + b * P_BLOCK_BYTES + row_off;
            const int c0 = h * 4 + cc * 2;                      // 16-byte chunk index inside the 128-byte row
            *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float e0 = ex2(fmaf(__uint_as_float(v[2 * i]), c2, mk[col + 2 * i]) - M);
              const float e1 = ex2(fmaf(__uint_as_float(v[2 * i + 1]), c2, mk[col + 2 * i + 1]) - M);
              __nv_bfloat162 hh = __floats2bfloat162_rn(e0, e1);
              // the row sum is taken over the rounded values the second MMA will actually use
              lsum += __low2float(hh) + __high2float(hh);
              w[i] = *reinterpret_cast<uint32_t*>(&hh);
            }
            // bf16: 64 keys = one 128-byte row of sub-tile (2b + h); this chunk covers 16-byte chunks 4cc..4cc+3
            uint8_t* blk = sP + b * P_BLOCK_BYTES + h * (SDPA_BLOCK_Q * 128) + row_off;
#pragma unroll
            for (int i = 0; i < 4; ++i)
              *reinterpret_cast<uint4*>(blk + (((cc * 4 + i) ^ (r & 7)) * 16)) =
                  make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_p_full + 8 * b);
          mbar_arrive(bar_s_free + 8 * b);
        }
      }
      // combine the two halves' row sums
      stA[r] = INT8 ? __int_as_float(psum) : lsum;
      if (!xchg_sync()) { failed = true; break; }
      if constexpr (INT8) prev_stat = __int_as_float(psum + __float_as_int(stB[r]));
      else prev_stat = lsum + stB[r];
      if (!xchg_sync()) { failed = true; break; }
      prev_unit = unit;
    }
    if (!failed && prev_unit >= 0) {
      if (!epilogue(prev_unit, (n - 1) & 1, prev_stat)) failed = true;
    }
    if (failed) report(p.status, DEV_TIMEOUT_EPILOGUE);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (failed) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

cudaError_t launch_sdpa_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                           int num_sms, cudaStream_t s) {
  const int slots = sdpa_slots(p.S, p.is_int8, 227 * 1024);
  if (!slots) return cudaErrorInvalidValue;
  const size_t smem = sdpa_tc_smem_bytes(p.S, p.is_int8);
  const int units = p.B * p.H * (p.S / SDPA_BLOCK_Q);
  const int grid = units < num_sms ? units : num_sms;
  cudaError_t e;
  if (p.is_int8) {
    e = cudaFuncSetAttribute(sdpa_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    sdpa_tc_kernel<true><<<grid, SDPA_THREADS, smem, s>>>(tmQ, tmK, tmV, p, slots);
  } else {
    e = cudaFuncSetAttribute(sdpa_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    sdpa_tc_kernel<false><<<grid, SDPA_THREADS, smem, s>>>(tmQ, tmK, tmV, p, slots);
  }
  return cudaGetLastError();
}

}  // namespace gc
