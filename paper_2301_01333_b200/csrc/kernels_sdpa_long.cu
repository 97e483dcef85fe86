// Fused scaled-dot-product attention on tcgen05 for rows longer than tensor memory can hold (more than 512 keys), head
// dimension 64, 96 or 128, bf16 or 8-bit (Section VII "MHA": two batch matmuls with the softmax and the binary ops
// between them fused after the first one).
//
// A score row of more than 512 keys no longer fits next to the output accumulator, and quantised probabilities need
// the FINAL row sum before any of them is rounded, so the softmax is blockwise with the scores computed twice:
//   pass 1   per 128-key block: S_b = Q K_b^T into one of two score buffers in tensor memory; the softmax warps fold
//            the block into a running row maximum and a running row sum (the sum rescaled whenever the maximum grows:
//            the online softmax recurrence), and release the buffer.  Nothing is written.
//   pass 2   per block again: S_b = Q K_b^T recomputed, p = 2^(x - max) with the final maximum, normalised and
//            rounded to a u8 code with the final sum (8-bit) or cast to bf16 with the division by the sum deferred to
//            the epilogue (bf16), P_b through a shared-memory ring, O += P_b V_b.
// The tensor core is idle most of the time in this subgraph, so the second Q K^T costs little; the exponentials are
// evaluated twice, which is the price of exact probabilities without the row resident.
//
// Persistent CTAs (one per SM, 704 threads) walk over work units (batch, head, 128-query tile):
//   warp 0      TMA producer: Q tile, then the K and V blocks in the order the MMA issuer consumes them, through one
//               ring of 128-key blocks (3-D tensor maps: rows past the end of a head's sequence arrive as zeros)
//   warp 1      MMA issuer (one thread)
//   warps 2-5   per-unit preparation (mask row times log2(e) with minus infinity past the sequence end, u8 -> s8
//               flip of Q) and the epilogue of the previous unit
//   warps 6-21  softmax, four threads per query row, 32 of every 128 key columns each
// Operand layouts, zero points and the 1.5 * 2^23 conversions follow the streaming kernel (kernels_sdpa_wide.cu).
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

namespace {

constexpr int G_BLOCK_Q = 128;
constexpr int G_THREADS = 704;
constexpr int G_SOFTMAX_WARPS = 16;
constexpr int G_MAX_STAGES = 8;
constexpr int G_NP = 2;                         // P ring entries
constexpr float G_LOG2E = 1.4426950408889634f;
constexpr float G_MAGIC_F = 12582912.0f;        // 1.5 * 2^23
constexpr int G_MAGIC_I = 0x4B400000;           // its bit pattern
constexpr uint32_t G_O_COL = 256;               // two score buffers of 128 columns, then the output accumulator

template <bool INT8, int D>
struct LongLayout {
  static constexpr int ESZ = INT8 ? 1 : 2;
  static constexpr int ROWB = (D * ESZ <= 64) ? 64 : 128;             // bytes per shared-memory row
  static constexpr int NSUB = (D * ESZ + ROWB - 1) / ROWB;            // sub-tiles across the head dimension
  static constexpr int SUB_ELEMS = ROWB / ESZ;
  static constexpr int SUB_BYTES = 128 * ROWB;
  static constexpr int TILE_BYTES = NSUB * SUB_BYTES;                 // Q tile, or one 128-key block of K or V
  static constexpr int P_BYTES = G_BLOCK_Q * 128 * ESZ;               // one 128-key block of P
  static constexpr uint32_t SWZ = ROWB == 64 ? SWZ_64B : SWZ_128B;
  static constexpr uint32_t SBO = 8 * ROWB;
  static constexpr int K1_STEPS = D * ESZ / 32;
  static constexpr int K1_PER_SUB = ROWB / 32;
  static constexpr int K2_STEPS = 128 / (INT8 ? 32 : 16);
  static constexpr int FIXED_BYTES = 32 * 128 * 4 /*row statistics*/ + 512 /*barriers, TMEM address*/;
};

struct LongCfg {
  int stages;
  size_t smem;
};

template <bool INT8, int D>
LongCfg long_cfg_t(int S) {
  using L = LongLayout<INT8, D>;
  const long s_pad = (S + 127) / 128 * 128;
  const long fixed = 1024 + L::TILE_BYTES + G_NP * L::P_BYTES + 2 * s_pad * 4 + L::FIXED_BYTES;
  long st = (227 * 1024 - fixed) / L::TILE_BYTES;
  if (st > G_MAX_STAGES) st = G_MAX_STAGES;
  if (st < 3) return {0, 0};
  return {static_cast<int>(st), static_cast<size_t>(fixed + st * L::TILE_BYTES)};
}

LongCfg long_cfg(int S, int D, int is_int8) {
  if (S < 1 || S > 16384) return {0, 0};
  if (is_int8) {
    if (D == 64) return long_cfg_t<true, 64>(S);
    if (D == 96) return long_cfg_t<true, 96>(S);
    if (D == 128) return long_cfg_t<true, 128>(S);
  } else {
    if (D == 64) return long_cfg_t<false, 64>(S);
    if (D == 96) return long_cfg_t<false, 96>(S);
    if (D == 128) return long_cfg_t<false, 128>(S);
  }
  return {0, 0};
}

__device__ __forceinline__ float g_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// exact (float)a for |a| < 2^22 without a conversion instruction
__device__ __forceinline__ float g_int_to_float(int a) { return __int_as_float(a + G_MAGIC_I) - G_MAGIC_F; }

template <bool INT8, int D>
__global__ void __launch_bounds__(G_THREADS, 1)
sdpa_long_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const SdpaParams p, const int stages) {
  using L = LongLayout<INT8, D>;
  constexpr uint32_t TMEM_COLS = 512;
  const int s_real = p.S;
  const int NB = (s_real + 127) / 128;                          // key blocks
  const int S = NB * 128;
  const int q_tiles = NB;
  const int num_units = p.B * p.H * q_tiles;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sKV = sQ + L::TILE_BYTES;                            // [stages] blocks of K or V
  uint8_t* sPall = sKV + stages * L::TILE_BYTES;                // [G_NP] blocks of P
  float* sMask = reinterpret_cast<float*>(sPall + G_NP * L::P_BYTES);   // [2 unit parities][S]
  float* sStat = sMask + 2 * S;                                 // [2 unit parities][16 slots][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sStat + 32 * 128);
  const uint32_t b0 = smem_u32(bars);
  const uint32_t bar_q_full = b0, bar_q_empty = b0 + 8, bar_q_ready = b0 + 16;
  const uint32_t bar_o_full = b0 + 24, bar_o_free = b0 + 32, bar_xchg = b0 + 40;
  const uint32_t bar_st_ready = b0 + 48, bar_st_free = b0 + 64;                      // [2] each
  const uint32_t bar_s_full = b0 + 80, bar_s_free = b0 + 96;                         // [2] each
  const uint32_t bar_p_full = b0 + 112, bar_p_free = b0 + 128;                       // [2] each
  const uint32_t bar_kv_full = b0 + 144, bar_kv_empty = b0 + 144 + 8 * G_MAX_STAGES; // [8] each -> ends at 272
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 36);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_empty, 1);
    mbar_init(bar_q_ready, 4);
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, 4);
    mbar_init(bar_xchg, G_SOFTMAX_WARPS);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_st_ready + 8 * i, G_SOFTMAX_WARPS);
      mbar_init(bar_st_free + 8 * i, 4);
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_s_free + 8 * i, G_SOFTMAX_WARPS);
      mbar_init(bar_p_full + 8 * i, G_SOFTMAX_WARPS);
      mbar_init(bar_p_free + 8 * i, 1);
    }
    for (int i = 0; i < G_MAX_STAGES; ++i) {
      mbar_init(bar_kv_full + 8 * i, 1);
      mbar_init(bar_kv_empty + 8 * i, 1);
    }
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

  // programmatic dependent launch: nothing touches global memory before the preceding kernel has completed
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t ring = 0;                                        // blocks loaded so far: stage = ring % stages
      auto load_block = [&](const CUtensorMap* tm, int bh, int b) -> bool {
        const uint32_t st = ring % static_cast<uint32_t>(stages), use = ring / static_cast<uint32_t>(stages);
        ++ring;
        if (!mbar_wait(bar_kv_empty + 8 * st, (use & 1) ^ 1)) return false;
        mbar_arrive_expect_tx(bar_kv_full + 8 * st, static_cast<uint32_t>(L::TILE_BYTES));
        for (int j = 0; j < L::NSUB; ++j)
          tma_load_3d(smem_u32(sKV) + st * L::TILE_BYTES + j * L::SUB_BYTES, tm, j * L::SUB_ELEMS, b * 128, bh, bar_kv_full + 8 * st);
        return true;
      };
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        const int bh = unit / q_tiles, qt = unit % q_tiles;
        if (!mbar_wait(bar_q_empty, (n & 1) ^ 1)) { failed = true; break; }
        mbar_arrive_expect_tx(bar_q_full, static_cast<uint32_t>(L::TILE_BYTES));
        for (int j = 0; j < L::NSUB; ++j)
          tma_load_3d(smem_u32(sQ) + j * L::SUB_BYTES, &tmQ, j * L::SUB_ELEMS, qt * G_BLOCK_Q, bh, bar_q_full);
        // pass 1: every K block; pass 2 in the issuer's order: K_0, then K_{b+1} ahead of V_b
        for (int b = 0; b < NB && !failed; ++b) failed = !load_block(&tmK, bh, b);
        if (!failed) failed = !load_block(&tmK, bh, 0);
        for (int b = 0; b < NB && !failed; ++b) {
          if (b + 1 < NB) failed = !load_block(&tmK, bh, b + 1);
          if (!failed) failed = !load_block(&tmV, bh, b);
        }
      }
      if (failed) report(p.status, DEV_TIMEOUT_PRODUCER);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = INT8 ? make_idesc(ACC_S32, FMT_S8, p.k_signed ? FMT_S8 : FMT_U8, 128, 128)
                                   : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, 128);
      uint32_t idesc2[L::NSUB];
#pragma unroll
      for (int j = 0; j < L::NSUB; ++j) {
        const int nj = (D - j * L::SUB_ELEMS) < L::SUB_ELEMS ? (D - j * L::SUB_ELEMS) : L::SUB_ELEMS;
        idesc2[j] = INT8 ? make_idesc(ACC_S32, FMT_U8, p.v_signed ? FMT_S8 : FMT_U8, 128, nj, 0, 1)
                         : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, nj, 0, 1);
      }
      uint32_t ring = 0, sk = 0, pj = 0;                        // blocks consumed, score blocks issued, P blocks consumed
      // S = Q K^T for the next block of the ring into the next score buffer
      auto mma1 = [&]() -> bool {
        const uint32_t st = ring % static_cast<uint32_t>(stages), use = ring / static_cast<uint32_t>(stages);
        ++ring;
        const uint32_t buf = sk & 1, suse = sk >> 1;
        ++sk;
        if (!mbar_wait(bar_kv_full + 8 * st, use & 1) || !mbar_wait(bar_s_free + 8 * buf, (suse & 1) ^ 1)) return false;
        tc_fence_after();
        const uint32_t kb = smem_u32(sKV) + st * L::TILE_BYTES;
#pragma unroll
        for (int k = 0; k < L::K1_STEPS; ++k) {
          const uint32_t off = (k / L::K1_PER_SUB) * L::SUB_BYTES + (k % L::K1_PER_SUB) * 32;
          umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + buf * 128, make_smem_desc(smem_u32(sQ) + off, 16, L::SBO, L::SWZ),
                                              make_smem_desc(kb + off, 16, L::SBO, L::SWZ), idesc1, k != 0);
        }
        umma_commit(bar_s_full + 8 * buf);
        umma_commit(bar_kv_empty + 8 * st);
        return true;
      };
      // O += P V for the next P block and the next block of the ring
      auto mma2 = [&](bool first) -> bool {
        const uint32_t pe = pj % G_NP, puse = pj / G_NP;
        ++pj;
        const uint32_t st = ring % static_cast<uint32_t>(stages), use = ring / static_cast<uint32_t>(stages);
        ++ring;
        if (!mbar_wait(bar_p_full + 8 * pe, puse & 1) || !mbar_wait(bar_kv_full + 8 * st, use & 1)) return false;
        tc_fence_after();
        const uint32_t sP = smem_u32(sPall) + pe * L::P_BYTES;
        const uint32_t vb = smem_u32(sKV) + st * L::TILE_BYTES;
#pragma unroll
        for (int ks = 0; ks < L::K2_STEPS; ++ks) {
          const uint64_t a_desc = make_smem_desc(sP + (ks >> 2) * (G_BLOCK_Q * 128) + (ks & 3) * 32, 16, 1024, SWZ_128B);
          const int key0 = ks * (128 / L::K2_STEPS);
#pragma unroll
          for (int j = 0; j < L::NSUB; ++j) {
            const uint64_t b_desc = make_smem_desc(vb + j * L::SUB_BYTES + key0 * L::ROWB, L::SBO, L::SBO, L::SWZ);
            umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + G_O_COL + j * L::SUB_ELEMS, a_desc, b_desc, idesc2[j], !(first && ks == 0));
          }
        }
        umma_commit(bar_kv_empty + 8 * st);
        umma_commit(bar_p_free + 8 * pe);
        return true;
      };
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        if (!mbar_wait(bar_q_ready, n & 1)) { failed = true; break; }
        for (int b = 0; b < NB && !failed; ++b) failed = !mma1();          // pass 1
        if (!failed) failed = !mma1();                                    // pass 2: block 0
        for (int b = 0; b < NB && !failed; ++b) {
          if (b + 1 < NB) failed = !mma1();
          else umma_commit(bar_q_empty);                                  // every Q K^T of this unit has been issued
          if (failed) break;
          if (b == 0 && !mbar_wait(bar_o_free, (n & 1) ^ 1)) { failed = true; break; }
          failed = !mma2(b == 0);
        }
        if (!failed) umma_commit(bar_o_full);
      }
      if (failed) report(p.status, DEV_TIMEOUT_MMA);
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ auxiliary warps
    const int t = tid - 64;                                     // 0..127
    const int q = warp & 3;                                     // TMEM lane quarter this warp may access
    const int r = q * 32 + lane;                                // query row within the tile
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    constexpr int OUT_ROW_BYTES = D * L::ESZ;

    auto epilogue = [&](int unit, int n0) -> bool {
      const int par = n0 & 1;
      if (!mbar_wait(bar_st_ready + 8 * par, (n0 >> 1) & 1)) return false;
      // the row sum of the exponentials (bf16: the deferred normalisation) and of the codes (8-bit: zero point of V)
      const float* st = sStat + par * 16 * 128 + r;             // slots: m[4], l[4], code sums[4], row sum
      const float total = st[12 * 128];
      int code_sum = 0;
      if constexpr (INT8) {
#pragma unroll
        for (int o = 0; o < 4; ++o) code_sum += __float_as_int(st[(8 + o) * 128]);
      }
      if (!mbar_wait(bar_o_full, n0 & 1)) return false;
      tc_fence_after();
      const int bh = unit / q_tiles, qt = unit % q_tiles;
      const bool row_ok = qt * G_BLOCK_Q + r < s_real;           // query rows past the sequence end are not stored
      const int64_t grow = static_cast<int64_t>(bh) * s_real + qt * G_BLOCK_Q + r;
      uint8_t* dst = static_cast<uint8_t*>(p.O) + grow * OUT_ROW_BYTES;
      const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
      const int corr = INT8 ? p.zp_v * code_sum : 0;            // zero point of V times the row sum of P
      const float u_lo = static_cast<float>(lo - p.zp_o), u_hi = static_cast<float>(hi - p.zp_o);
      const int kadd = p.zp_o - G_MAGIC_I;
      const float rl = INT8 ? 0.f : 1.0f / total;
      uint32_t v[32];
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        tmem_ld32(t_lane + G_O_COL + c * 32, v);
        tmem_wait_ld();
        if (c == D / 32 - 1) {                                  // O has been read completely
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar_o_free);
            mbar_arrive(bar_st_free + 8 * par);
          }
        }
        if constexpr (INT8) {
          uint32_t w[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            uint32_t y[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int acc = static_cast<int>(v[4 * i + k]) - corr;
              const float tt = __fmul_rn(__int2float_rn(acc), p.dq2);
              const float u = fminf(fmaxf(__fmul_rn(tt, p.inv_o), u_lo), u_hi);
              y[k] = static_cast<uint32_t>(__float_as_int(u + G_MAGIC_F) + kadd);
            }
            w[i] = __byte_perm(__byte_perm(y[0], y[1], 0x0040), __byte_perm(y[2], y[3], 0x0040), 0x5410);
          }
          if (row_ok) {
            uint4* d4 = reinterpret_cast<uint4*>(dst + c * 32);
            d4[0] = make_uint4(w[0], w[1], w[2], w[3]);
            d4[1] = make_uint4(w[4], w[5], w[6], w[7]);
          }
        } else {
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[2 * i]) * rl, __uint_as_float(v[2 * i + 1]) * rl);
            w[i] = *reinterpret_cast<uint32_t*>(&hh);
          }
          if (row_ok) {
            uint4* d4 = reinterpret_cast<uint4*>(dst + c * 64);
#pragma unroll
            for (int i = 0; i < 4; ++i) d4[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          }
        }
      }
      return true;
    };

    int n = 0;
    int prev_unit = -1;
    for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
      const int b = (unit / q_tiles) / p.H;
      float* mk = sMask + (n & 1) * S;
      // the softmax warps are done with the mask row of unit n-2 before unit n's Q can land (its load waits for
      // every Q K^T of unit n-1, which needs their releases)
      if (!mbar_wait(bar_q_full, n & 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        failed = true;
        break;
      }
      for (int j = t; j < S; j += 128)
        mk[j] = j >= s_real ? -INFINITY : (p.mask ? __ldg(p.mask + static_cast<int64_t>(b) * s_real + j) * G_LOG2E : 0.0f);
      if (INT8 && !p.q_signed) {
        uint4* q4 = reinterpret_cast<uint4*>(sQ);
        for (int i = t; i < L::TILE_BYTES / 16; i += 128) {
          uint4 v = q4[i];
          v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
          q4[i] = v;
        }
        fence_proxy_async_smem();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_q_ready);
      if (prev_unit >= 0 && !epilogue(prev_unit, n - 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        failed = true;
        break;
      }
      prev_unit = unit;
    }
    if (!failed && prev_unit >= 0 && !epilogue(prev_unit, n - 1)) {
      report(p.status, DEV_TIMEOUT_OTHER);
      failed = true;
    }
  } else {
    // ------------------------------------------------------------------ softmax warps
    // Four threads share a query row (TMEM lane): warp w covers lane quarter (w % 4) and, of every 128-key block,
    // the 32 columns [32 g, 32 g + 32) with g = (w - 6) / 4.
    const int sw = warp - 6;                                    // 0..15
    const int q = warp & 3;                                     // TMEM lane quarter
    const int g = sw >> 2;                                      // which 32 of every 128 key columns
    const int r = q * 32 + lane;                                // query row within the tile = TMEM lane
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + g * 32;
    const float c2 = (INT8 ? __fmul_rn(p.dq1, p.scalar) : p.scalar) * G_LOG2E;
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    uint32_t sk = 0, pj = 0, xphase = 0;                         // score blocks and P blocks so far; exchange phase

    // scores of my chunk of the next score block, scaled and masked (log2 units); releases the score buffer
    auto next_scores = [&](float (&x)[32], const float* mk) -> bool {
      const uint32_t buf = sk & 1, suse = sk >> 1;
      ++sk;
      if (!mbar_wait(bar_s_full + 8 * buf, suse & 1)) return false;
      tc_fence_after();
      uint32_t v[32];
      tmem_ld32(t_row + buf * 128, v);
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_s_free + 8 * buf);         // my columns are in registers
      const float4* mk4 = reinterpret_cast<const float4*>(mk);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 mv = mk4[i];
        const float mm[4] = {mv.x, mv.y, mv.z, mv.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float a = INT8 ? g_int_to_float(static_cast<int>(v[4 * i + j])) : __uint_as_float(v[4 * i + j]);
          x[4 * i + j] = fmaf(a, c2, mm[j]);
        }
      }
      return true;
    };

    int n = 0;
    for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
      const float* mk = sMask + (n & 1) * S + g * 32;
      const int par = n & 1;
      float* st = sStat + par * 16 * 128 + r;                   // [16 slots][128]: m[4], l[4], code sums[4], row sum
      if (!mbar_wait(bar_q_ready, n & 1)) { failed = true; break; }

      // ---------------- pass 1: running row maximum and row sum (online softmax recurrence)
      float m = -INFINITY, l = 0.f;
      float x[32];
      for (int b = 0; b < NB; ++b) {
        if (!next_scores(x, mk + b * 128)) { failed = true; break; }
        float cm[4] = {x[0], x[1], x[2], x[3]};
#pragma unroll
        for (int i = 4; i < 32; i += 4) {
#pragma unroll
          for (int j = 0; j < 4; ++j) cm[j] = fmaxf(cm[j], x[i + j]);
        }
        const float m_new = fmaxf(m, fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3])));
        const float ms = m_new == -INFINITY ? 0.f : m_new;      // a chunk of masked-out keys only: everything is zero
        float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < 32; i += 4) {
#pragma unroll
          for (int j = 0; j < 4; ++j) sm[j] += g_ex2(x[i + j] - ms);
        }
        l = l * g_ex2(m - ms) + ((sm[0] + sm[1]) + (sm[2] + sm[3]));
        m = m_new;
      }
      if (failed) break;
      st[(0 + g) * 128] = m;
      st[(4 + g) * 128] = l;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_xchg);
      if (!mbar_wait(bar_xchg, xphase)) { failed = true; break; }
      xphase ^= 1;
      // every thread of a row combines the four parts in the same order, so all four get identical values
      float M = -INFINITY;
#pragma unroll
      for (int o = 0; o < 4; ++o) M = fmaxf(M, st[o * 128]);
      const float Ms = M == -INFINITY ? 0.f : M;
      float Lsum = 0.f;
#pragma unroll
      for (int o = 0; o < 4; ++o) Lsum += st[(4 + o) * 128] * g_ex2(st[o * 128] - Ms);
      const float scale = INT8 ? p.inv_p / Lsum : 1.f;

      // ---------------- pass 2: the scores again, final maximum and sum: normalise, round, write P into the ring
      int psum = 0;
      for (int b = 0; b < NB; ++b) {
        if (!next_scores(x, mk + b * 128)) { failed = true; break; }
        const uint32_t pe = pj % G_NP, puse = pj / G_NP;
        ++pj;
        uint8_t* sP = sPall + pe * L::P_BYTES;
        if constexpr (INT8) {
          uint32_t w[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            // rne(e * scale) lands in the low mantissa bits of (e * scale + 1.5 * 2^23); codes are within [0, 255]
            uint32_t y[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) y[j] = __float_as_uint(fmaf(g_ex2(x[4 * i + j] - Ms), scale, G_MAGIC_F));
            w[i] = __byte_perm(__byte_perm(y[0], y[1], 0x0040), __byte_perm(y[2], y[3], 0x0040), 0x5410);
            psum = static_cast<int>(__dp4a(w[i], 0x01010101u, static_cast<unsigned>(psum)));
          }
          if (!mbar_wait(bar_p_free + 8 * pe, (puse & 1) ^ 1)) { failed = true; break; }
          uint8_t* blk = sP + row_off;
          const int c0 = g * 2;                                 // 16-byte chunk index inside the 128-byte row
          *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
        } else {
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(g_ex2(x[2 * i] - Ms), g_ex2(x[2 * i + 1] - Ms));
            w[i] = *reinterpret_cast<uint32_t*>(&h);
          }
          if (!mbar_wait(bar_p_free + 8 * pe, (puse & 1) ^ 1)) { failed = true; break; }
          // bf16: a 128-key block is two 64-key sub-tiles (128-byte rows); my 32 keys are 4 chunks of 16 bytes
          uint8_t* blk = sP + (g >> 1) * (G_BLOCK_Q * 128) + row_off;
          const int c0 = (g & 1) * 4;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(blk + (((c0 + i) ^ (r & 7)) * 16)) =
                make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_p_full + 8 * pe);
      }
      if (failed) break;
      // the row sum (bf16: the division deferred to the epilogue) and my part of the sum of the codes go to the
      // auxiliary warps; the slot is free once they have read the values of the unit that used it two units ago
      if (!mbar_wait(bar_st_free + 8 * par, ((n >> 1) & 1) ^ 1)) { failed = true; break; }
      st[(8 + g) * 128] = __int_as_float(psum);
      if (g == 0) st[12 * 128] = Lsum;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_st_ready + 8 * par);
    }
    if (failed) report(p.status, DEV_TIMEOUT_EPILOGUE);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (failed) {                                                 // let copies in flight land before the block exits
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

template <bool INT8, int D>
cudaError_t launch_long_t(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                          int num_sms, cudaStream_t s) {
  const LongCfg cfg = long_cfg_t<INT8, D>(p.S);
  if (!cfg.smem) return cudaErrorInvalidValue;
  auto kern = sdpa_long_kernel<INT8, D>;
  const int units = p.B * p.H * ((p.S + G_BLOCK_Q - 1) / G_BLOCK_Q);
  const int grid = units < num_sms ? units : num_sms;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), cfg.smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(G_THREADS);
  lc.dynamicSmemBytes = cfg.smem;
  lc.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kern, tmQ, tmK, tmV, p, cfg.stages);
}

}  // namespace

size_t sdpa_long_smem_bytes(int S, int D, int is_int8) { return long_cfg(S, D, is_int8).smem; }

cudaError_t launch_sdpa_long(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                             int num_sms, cudaStream_t s) {
  if (p.is_int8) {
    if (p.D == 64) return launch_long_t<true, 64>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 96) return launch_long_t<true, 96>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 128) return launch_long_t<true, 128>(tmQ, tmK, tmV, p, num_sms, s);
  } else {
    if (p.D == 64) return launch_long_t<false, 64>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 96) return launch_long_t<false, 96>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 128) return launch_long_t<false, 128>(tmQ, tmK, tmV, p, num_sms, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace gc
