// Fused scaled-dot-product attention on tcgen05 for the wider shapes of the evaluation (Section VII, Table I):
// head dimension 64, 96 or 128 and up to 512 keys, bf16 or 8-bit.  Same computation and the same two-pass
// softmax over a score row held in tensor memory as the D = 64 kernel, but K and V are streamed through a ring
// of 128-key blocks instead of being resident per work unit, P goes through a ring of 128-key blocks, and the
// output accumulator takes over the columns of the first score block when the row alone fills tensor memory
// (512 keys).  That is what lets 128-wide heads and 512-key rows fit in 227 KB of shared memory.
//
// Persistent CTAs (one per SM, 704 threads) walk over work units (batch, head, 128-query tile):
//   warp 0      TMA producer: Q tile and 128-key blocks of K and V into the ring, in the order the MMA issuer
//               consumes them (no multicast)
//   warp 1      MMA issuer (one thread): S_b = Q K_b^T per block, O += P_b V_b per block; unless O shares
//               columns with the scores, the next unit's S_b is issued right after this unit's P_b V_b, as
//               soon as the softmax warps have released block b
//   warps 2-5   per-unit preparation (mask row times log2(e), chunk flags, u8 -> s8 flip of Q) and the epilogue
//               of the previous unit (O out of tensor memory, normalise or requantise, vector stores)
//   warps 6-21  softmax, four threads per query row, 32 of every 128 key columns each (two passes)
//
// Shared-memory operand layout: rows of 128 bytes under the 128-byte swizzle (64 bytes / 64-byte swizzle when
// the whole head fits in 64 bytes).  A head wider than one row is split into sub-tiles of 64 bf16 elements;
// a head that does not fill its last row (D = 96) is loaded with a box that reaches past the tensor's edge,
// which TMA fills with zeros.  Q and K are K-major operands; V is consumed as stored ([key][d], MN-major).
//
// Zero points, the conversions by the 1.5 * 2^23 bias trick and the skipping of fully masked 32-key chunks
// follow the D = 64 kernel.
//
// Sequence lengths that are not a multiple of 128 run as the next multiple: Q, K and V are addressed through 3-D
// tensor maps [batch x head][key][d], so rows past the end of a head's sequence arrive as zeros; the keys past the end
// carry a mask term of minus infinity (their exponentials, hence their codes, are exactly zero) and the query rows
// past the end are computed but not stored.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

namespace {

constexpr int W_BLOCK_Q = 128;
constexpr int W_THREADS = 704;
constexpr int W_SOFTMAX_WARPS = 16;
constexpr int W_MAX_STAGES = 16;
constexpr float W_LOG2E = 1.4426950408889634f;
constexpr float W_MAGIC_F = 12582912.0f;        // 1.5 * 2^23
constexpr int W_MAGIC_I = 0x4B400000;           // its bit pattern

template <bool INT8, int D>
struct WideLayout {
  static constexpr int ESZ = INT8 ? 1 : 2;
  static constexpr int ROWB = (D * ESZ <= 64) ? 64 : 128;             // bytes per shared-memory row
  static constexpr int NSUB = (D * ESZ + ROWB - 1) / ROWB;            // sub-tiles across the head dimension
  static constexpr int SUB_ELEMS = ROWB / ESZ;                        // elements per sub-tile row
  static constexpr int SUB_BYTES = 128 * ROWB;                        // one sub-tile of 128 rows
  static constexpr int TILE_BYTES = NSUB * SUB_BYTES;                 // Q tile, or one 128-key block of K or V
  static constexpr int P_BYTES = W_BLOCK_Q * 128 * ESZ;               // one 128-key block of P
  static constexpr uint32_t SWZ = ROWB == 64 ? SWZ_64B : SWZ_128B;
  static constexpr uint32_t SBO = 8 * ROWB;
  static constexpr int K1_STEPS = D * ESZ / 32;                       // 32 bytes of the head dimension per MMA
  static constexpr int K1_PER_SUB = ROWB / 32;
  static constexpr int K2_STEPS = 128 / (INT8 ? 32 : 16);             // MMAs (per sub-tile) per 128-key block of P.V
  static constexpr int FIXED_BYTES = 24 * 128 * 4 /*row statistics*/ + 768 /*barriers, TMEM address, chunk flags*/;
  __host__ __device__ static constexpr int fixed(int S) { return TILE_BYTES + 2 * S * 4 + FIXED_BYTES; }
};

struct WideCfg {
  int np;         // P ring entries (128-key blocks)
  int stages;     // K/V ring entries (128-key blocks)
  size_t smem;    // dynamic shared memory to request; 0 = the shape does not fit
};

template <bool INT8, int D>
constexpr WideCfg wide_cfg_t(int S) {
  using L = WideLayout<INT8, D>;
  const int NB = S / 128;
  const long limit = 227 * 1024;
  const long avail = limit - 1024 - L::fixed(S);
  const int np_min = NB < 2 ? NB : 2;
  for (int np = NB; np >= np_min; --np) {
    long st = (avail - static_cast<long>(np) * L::P_BYTES) / L::TILE_BYTES;
    if (st > 2 * NB + 2) st = 2 * NB + 2;
    if (st > W_MAX_STAGES) st = W_MAX_STAGES;
    const long want = 2 * NB < 3 ? 2 * NB : 3;
    if (st >= want || (np == np_min && st >= 2))
      return {np, static_cast<int>(st),
              static_cast<size_t>(1024 + L::fixed(S) + static_cast<long>(np) * L::P_BYTES + st * L::TILE_BYTES)};
  }
  return {0, 0, 0};
}

WideCfg wide_cfg(int S, int D, int is_int8) {
  if (S < 1 || S > 512) return {0, 0, 0};
  S = (S + 127) / 128 * 128;                                    // runs as the next multiple of 128 keys
  if (is_int8) {
    if (D == 64) return wide_cfg_t<true, 64>(S);
    if (D == 96) return wide_cfg_t<true, 96>(S);
    if (D == 128) return wide_cfg_t<true, 128>(S);
  } else {
    if (D == 64) return wide_cfg_t<false, 64>(S);
    if (D == 96) return wide_cfg_t<false, 96>(S);
    if (D == 128) return wide_cfg_t<false, 128>(S);
  }
  return {0, 0, 0};
}

__device__ __forceinline__ float w_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// exact (float)a for |a| < 2^22 without a conversion instruction
__device__ __forceinline__ float w_int_to_float(int a) { return __int_as_float(a + W_MAGIC_I) - W_MAGIC_F; }

// NB_CT, NP_CT, ST_CT: key blocks and ring sizes as compile-time constants (the launcher instantiates every
// sequence length the kernel takes); with them the per-block loops unroll and the ring bookkeeping folds away.
template <bool INT8, int D, int NB_CT, int NP_CT, int ST_CT>
__global__ void __launch_bounds__(W_THREADS, 1)
sdpa_wide_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const SdpaParams p) {
  using L = WideLayout<INT8, D>;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr int S = NB_CT * 128;
  constexpr int NB = NB_CT;
  constexpr int np = NP_CT;
  constexpr int stages = ST_CT;
  const bool alias = S + D > 512;                               // O takes over the columns of score block 0
  const uint32_t o_col = alias ? 0u : static_cast<uint32_t>(S);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sKV = sQ + L::TILE_BYTES;                            // [stages] blocks of K or V
  uint8_t* sPall = sKV + stages * L::TILE_BYTES;                // [np] blocks of P
  float* sMask = reinterpret_cast<float*>(sPall + np * L::P_BYTES);   // [2][S]
  float* sStat = sMask + 2 * S;                                 // [3 kinds][2 parities][4 groups][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sStat + 24 * 128);
  const uint32_t b0 = smem_u32(bars);
  const uint32_t bar_q_full = b0, bar_q_empty = b0 + 8, bar_q_ready = b0 + 16;
  const uint32_t bar_o_full = b0 + 24, bar_o_free = b0 + 32;
  const uint32_t bar_st_ready = b0 + 48, bar_st_free = b0 + 64;                      // [2] each
  const uint32_t bar_s_full = b0 + 80, bar_s_free = b0 + 112, bar_p_full = b0 + 144, bar_p_free = b0 + 176;   // [4] each
  const uint32_t bar_kv_full = b0 + 208, bar_kv_empty = b0 + 208 + 8 * W_MAX_STAGES;   // [16] each -> ends at 464
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 60);                      // byte 480
  // per mask buffer and 32-key chunk: 1 = every key masked out, 2 = has an unmasked key, 0 = neither
  uint32_t* sChunk = tmem_slot + 4;                                                  // [2][16], bytes 496..624
  // per mask buffer and group of 32 columns (g): bits 0-7 = key blocks up to the last one whose chunk g is not fully
  // masked, bit 8 = the group has a chunk with an unmasked key
  uint32_t* sTail = sChunk + 32;                                                     // [2][4], bytes 624..656
  const uint32_t bar_xchg = smem_u32(sTail + 8);                                     // bytes 656..664: row statistics exchange

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q_tiles = S / W_BLOCK_Q;
  const int num_units = p.B * p.H * q_tiles;
  const int s_real = p.S;                                       // S is its next multiple of 128

  if (tid == 0) {
    mbar_init(bar_q_full, 1);
    mbar_init(bar_q_empty, 1);
    mbar_init(bar_q_ready, 4);
    mbar_init(bar_o_full, 1);
    mbar_init(bar_o_free, 4);
    mbar_init(bar_xchg, W_SOFTMAX_WARPS);
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_st_ready + 8 * i, W_SOFTMAX_WARPS);
      mbar_init(bar_st_free + 8 * i, 4);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_s_free + 8 * i, W_SOFTMAX_WARPS);
      mbar_init(bar_p_full + 8 * i, W_SOFTMAX_WARPS);
      mbar_init(bar_p_free + 8 * i, 1);
    }
    for (int i = 0; i < W_MAX_STAGES; ++i) {
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

  // Programmatic dependent launch: the set-up above may overlap the tail of the preceding kernel on the stream.
  // While waiting for it, the first unit's operands are pulled into L2 (a prefetch has no destination the kernel
  // could read too early, and L2 stays coherent with whatever the preceding kernel still writes); nothing else
  // touches global memory before that kernel has completed (the wait is a no-op for an ordinary launch).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0 && static_cast<int>(blockIdx.x) < p.B * p.H * (S / W_BLOCK_Q)) {
    const int unit = blockIdx.x, qt0 = S / W_BLOCK_Q;
    const int bh0 = unit / qt0;
    for (int j = 0; j < L::NSUB; ++j) tma_prefetch_3d(&tmQ, j * L::SUB_ELEMS, (unit % qt0) * W_BLOCK_Q, bh0);
    for (int b = 0; b < NB; ++b)
      for (int j = 0; j < L::NSUB; ++j) {
        tma_prefetch_3d(&tmK, j * L::SUB_ELEMS, b * 128, bh0);
        tma_prefetch_3d(&tmV, j * L::SUB_ELEMS, b * 128, bh0);
      }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int n = 0;
      uint32_t ring_st = 0, ring_use = 0;                        // ring position: stage and how often the ring has wrapped
      auto ring_next = [&]() {
        if (++ring_st == static_cast<uint32_t>(stages)) {
          ring_st = 0;
          ++ring_use;
        }
      };
      auto load_q = [&](int u, int nn) -> bool {                 // Q tile of unit u, this CTA's nn-th unit
        if (!mbar_wait(bar_q_empty, (nn & 1) ^ 1)) return false;
        mbar_arrive_expect_tx(bar_q_full, static_cast<uint32_t>(L::TILE_BYTES));
        for (int j = 0; j < L::NSUB; ++j)
          tma_load_3d(smem_u32(sQ) + j * L::SUB_BYTES, &tmQ, j * L::SUB_ELEMS, (u % q_tiles) * W_BLOCK_Q, u / q_tiles,
                      bar_q_full);
        return true;
      };
      auto load_block = [&](const CUtensorMap* tm, int u, int b) -> bool {   // one 128-key block into the next stage
        const uint32_t st = ring_st, use = ring_use;
        ring_next();
        if (!mbar_wait(bar_kv_empty + 8 * st, (use & 1) ^ 1)) return false;
        mbar_arrive_expect_tx(bar_kv_full + 8 * st, static_cast<uint32_t>(L::TILE_BYTES));
        for (int j = 0; j < L::NSUB; ++j)
          tma_load_3d(smem_u32(sKV) + st * L::TILE_BYTES + j * L::SUB_BYTES, tm, j * L::SUB_ELEMS, b * 128, u / q_tiles,
                      bar_kv_full + 8 * st);
        return true;
      };
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        // Blocks go into the ring in the order the MMA issuer consumes them: the next unit's K block b right before
        // this unit's V block b.  When O shares the columns of score block 0, that block's K comes last: its
        // Q.K^T has to wait for the previous unit's output to be read, the others need not.
        const int next = unit + static_cast<int>(gridDim.x);
        const bool ahead = next < num_units;
        const int b_first = alias ? 1 : 0;
        if (n == 0) {
          failed = !load_q(unit, 0);
          for (int i = 0; i < NB && !failed; ++i) failed = !load_block(&tmK, unit, (b_first + i) % NB);
        }
        if (ahead && !failed) failed = !load_q(next, n + 1);
        for (int b = 0; b < NB && !failed; ++b) {
          if (ahead && b >= b_first) failed = !load_block(&tmK, next, b);
          if (!failed) failed = !load_block(&tmV, unit, b);
        }
        if (ahead && alias && !failed) failed = !load_block(&tmK, next, 0);
      }
      if (failed) report(p.status, DEV_TIMEOUT_PRODUCER);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc1 = INT8 ? make_idesc(ACC_S32, FMT_S8, p.k_signed ? FMT_S8 : FMT_U8, 128, 128)
                                   : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, 128);
      // P.V: one MMA per sub-tile of V; its N is the part of the head dimension that sub-tile holds
      uint32_t idesc2[L::NSUB];
#pragma unroll
      for (int j = 0; j < L::NSUB; ++j) {
        const int nj = (D - j * L::SUB_ELEMS) < L::SUB_ELEMS ? (D - j * L::SUB_ELEMS) : L::SUB_ELEMS;
        idesc2[j] = INT8 ? make_idesc(ACC_S32, FMT_U8, p.v_signed ? FMT_S8 : FMT_U8, 128, nj, 0, 1)
                         : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, nj, 0, 1);
      }
      int n = 0;
      uint32_t ring_st = 0, ring_use = 0, pe = 0;                // K/V ring position; P ring entry of the next block
      auto ring_next = [&]() {
        if (++ring_st == static_cast<uint32_t>(stages)) {
          ring_st = 0;
          ++ring_use;
        }
      };
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        const uint32_t upar = n & 1;
        const bool ahead = unit + static_cast<int>(gridDim.x) < num_units;
        const int b_first = alias ? 1 : 0;                      // first / last score block of a unit in issue order
        const int b_last = alias ? 0 : NB - 1;
        // S_b = Q K_b^T for this CTA's nn-th unit (block b of the ring's next stage)
        auto mma1 = [&](int nn, int b) -> bool {
          const uint32_t st = ring_st, use = ring_use, par = nn & 1;
          ring_next();
          if (b == b_first && !mbar_wait(bar_q_ready, par)) return false;
          if (!mbar_wait(bar_kv_full + 8 * st, use & 1) || !mbar_wait(bar_s_free + 8 * b, par ^ 1)) return false;
          if (alias && b == 0 && !mbar_wait(bar_o_free, par ^ 1)) return false;
          tc_fence_after();
          const uint32_t kb = smem_u32(sKV) + st * L::TILE_BYTES;
#pragma unroll
          for (int k = 0; k < L::K1_STEPS; ++k) {
            const uint32_t off = (k / L::K1_PER_SUB) * L::SUB_BYTES + (k % L::K1_PER_SUB) * 32;
            umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + b * 128, make_smem_desc(smem_u32(sQ) + off, 16, L::SBO, L::SWZ),
                                                make_smem_desc(kb + off, 16, L::SBO, L::SWZ), idesc1, k != 0);
          }
          umma_commit(bar_s_full + 8 * b);
          umma_commit(bar_kv_empty + 8 * st);
          if (b == b_last) umma_commit(bar_q_empty);
          return true;
        };
        if (n == 0)
          for (int i = 0; i < NB && !failed; ++i) failed = !mma1(0, (b_first + i) % NB);
        if (failed) break;
        // O += P_b V_b
        for (int b = 0; b < NB; ++b) {
          if (!mbar_wait(bar_p_full + 8 * b, upar)) { failed = true; break; }
          // the next unit's scores for this block first: the softmax warps will wait for them, nobody waits for
          // this O yet, and the tensor pipe runs the MMAs in issue order
          if (ahead && b >= b_first && !mma1(n + 1, b)) { failed = true; break; }
          const uint32_t st = ring_st, use = ring_use;
          ring_next();
          if (!mbar_wait(bar_kv_full + 8 * st, use & 1)) { failed = true; break; }
          if (!alias && b == 0 && !mbar_wait(bar_o_free, upar ^ 1)) { failed = true; break; }
          tc_fence_after();
          const uint32_t sP = smem_u32(sPall) + pe * L::P_BYTES;
          const uint32_t vb = smem_u32(sKV) + st * L::TILE_BYTES;
#pragma unroll
          for (int ks = 0; ks < L::K2_STEPS; ++ks) {
            // A: P block, K-major, 128B swizzle: 4 MMA steps of 32 bytes per 128-byte span, spans 16 KB apart
            const uint64_t a_desc = make_smem_desc(sP + (ks >> 2) * (W_BLOCK_Q * 128) + (ks & 3) * 32, 16, 1024, SWZ_128B);
            const int key0 = ks * (128 / L::K2_STEPS);
#pragma unroll
            for (int j = 0; j < L::NSUB; ++j) {
              // B: V as stored [key][d] = MN-major: one key per row, 8-key groups SBO apart
              const uint64_t b_desc = make_smem_desc(vb + j * L::SUB_BYTES + key0 * L::ROWB, L::SBO, L::SBO, L::SWZ);
              umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + o_col + j * L::SUB_ELEMS, a_desc, b_desc, idesc2[j], (b | ks) != 0);
            }
          }
          umma_commit(bar_kv_empty + 8 * st);
          umma_commit(bar_p_free + 8 * pe);
          if (++pe == static_cast<uint32_t>(np)) pe = 0;
          if (b == NB - 1) umma_commit(bar_o_full);
        }
        // score block 0 of the next unit overwrites this unit's O: issued once the epilogue has read it
        if (!failed && ahead && alias && !mma1(n + 1, 0)) failed = true;
      }
      if (failed) report(p.status, DEV_TIMEOUT_MMA);
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ auxiliary warps
    // Per unit: (1) preparation once Q has landed: mask row scaled by log2(e), chunk flags, u8 -> s8 flip of Q;
    // (2) epilogue of the previous unit: O out of tensor memory in 32-column pieces, finished with the row
    // statistics the softmax warps left in shared memory, written with 16-byte vector stores.
    const int t = tid - 64;                                     // 0..127
    const int q = warp & 3;                                     // TMEM lane quarter this warp may access
    const int r = q * 32 + lane;                                // query row within the tile
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    constexpr int OUT_ROW_BYTES = D * L::ESZ;
    auto stat2 = [&](int par, int grp) { return sStat + ((2 * 2 + par) * 4 + grp) * 128 + r; };

    auto epilogue = [&](int unit, int n0) -> bool {
      const int par = n0 & 1;
      if (!mbar_wait(bar_st_ready + 8 * par, (n0 >> 1) & 1)) return false;
      float total;
      if constexpr (INT8) {
        int ti = 0;
#pragma unroll
        for (int o = 0; o < 4; ++o) ti += __float_as_int(*stat2(par, o));
        total = __int_as_float(ti);
      } else {
        total = 0.f;
#pragma unroll
        for (int o = 0; o < 4; ++o) total += *stat2(par, o);
      }
      if (!mbar_wait(bar_o_full, n0 & 1)) return false;
      tc_fence_after();
      const int bh = unit / q_tiles, qt = unit % q_tiles;
      const bool row_ok = qt * W_BLOCK_Q + r < s_real;           // query rows past the sequence end are not stored
      const int64_t grow = static_cast<int64_t>(bh) * s_real + qt * W_BLOCK_Q + r;
      uint8_t* dst = static_cast<uint8_t*>(p.O) + grow * OUT_ROW_BYTES;
      const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
      const int corr = INT8 ? p.zp_v * __float_as_int(total) : 0;   // zero point of V times the row sum of P
      const float u_lo = static_cast<float>(lo - p.zp_o), u_hi = static_cast<float>(hi - p.zp_o);
      const int kadd = p.zp_o - W_MAGIC_I;
      const float rl = INT8 ? 0.f : 1.0f / total;               // bf16: deferred normalisation by the row sum
      uint32_t v[32];
#pragma unroll 1
      for (int c = 0; c < D / 32; ++c) {
        tmem_ld32(t_lane + o_col + c * 32, v);
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
              // saturate(rne(u) + zp) = rne(clamp(u, lo - zp, hi - zp)) + zp, rounded with the bias trick
              const float u = fminf(fmaxf(__fmul_rn(tt, p.inv_o), u_lo), u_hi);
              y[k] = static_cast<uint32_t>(__float_as_int(u + W_MAGIC_F) + kadd);
            }
            w[i] = __byte_perm(__byte_perm(y[0], y[1], 0x0040), __byte_perm(y[2], y[3], 0x0040), 0x5410);
          }
          uint4* d4 = reinterpret_cast<uint4*>(dst + c * 32);
          if (row_ok) {
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
          uint4* d4 = reinterpret_cast<uint4*>(dst + c * 64);
          if (row_ok) {
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
      // Q(n) lands only after every Q K^T of unit n-1 has completed, which needed the softmax warps to be done
      // with unit n-2: the mask buffer and chunk flags of that unit are free
      // the mask values are fetched before the wait so that their latency hides behind the unit's loads
      float mreg[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = t + 128 * i;
        mreg[i] = j >= s_real ? -INFINITY : (p.mask ? __ldg(p.mask + static_cast<int64_t>(b) * s_real + j) * W_LOG2E : 0.0f);
      }
      if (!mbar_wait(bar_q_full, n & 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        failed = true;
        break;
      }
      uint32_t tail = 0;                                        // see sTail: this warp covers group (warp - 2) of every block
#pragma unroll
      for (int i = 0; i < 4; ++i) {                             // a warp covers one aligned 32-key chunk per step
        const int j = t + 128 * i;
        if (j >= S) break;
        const float mv = mreg[i];
        mk[j] = mv;
        if constexpr (INT8) {
          const bool all_masked = __all_sync(0xffffffffu, p.skip_thr > 0.f && mv <= -p.skip_thr);
          const bool any_valid = __any_sync(0xffffffffu, mv >= -1.0f);
          // bit 2: all 32 keys of the chunk carry the same mask value, so the largest score is the largest accumulator
          const bool uniform = __all_sync(0xffffffffu, __float_as_uint(mv) == __shfl_sync(0xffffffffu, __float_as_uint(mv), 0));
          if (lane == 0) sChunk[(n & 1) * 16 + (j >> 5)] = (all_masked ? 1u : (any_valid ? 2u : 0u)) | (uniform ? 4u : 0u);
          if (!all_masked) tail = (tail & 0x100u) | static_cast<uint32_t>(i + 1);
          if (any_valid && !all_masked) tail |= 0x100u;
        }
      }
      if (INT8 && lane == 0) sTail[(n & 1) * 4 + (warp - 2)] = tail;
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
    // Four threads share a query row (TMEM lane): warp w covers lane quarter (w % 4) and, of every 128-key
    // block, the 32 columns [32 g, 32 g + 32) with g = (w - 6) / 4.
    const int sw = warp - 6;                                    // 0..15
    const int q = warp & 3;                                     // TMEM lane quarter
    const int g = sw >> 2;                                      // which 32 of every 128 key columns
    const int r = q * 32 + lane;                                // query row within the tile = TMEM lane
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const float c2 = (INT8 ? __fmul_rn(p.dq1, p.scalar) : p.scalar) * W_LOG2E;
    const float neg_c0 = -__fmul_rn(W_MAGIC_F, c2);              // cancels the bias of the int -> float trick inside an FMA
    const float rho = fmaf(W_MAGIC_F, c2, neg_c0);               // ... up to this rounding residue, a launch-wide constant
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    uint32_t xphase = 0;
    uint32_t p_entry = 0, p_use = 0;                              // P ring: entry of the next block, wraps so far
    auto stat = [&](int kind, int par, int grp) { return sStat + ((kind * 2 + par) * 4 + grp) * 128 + r; };
    auto xchg_sync = [&]() -> bool {
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_xchg);
      const bool ok = mbar_wait(bar_xchg, xphase);
      xphase ^= 1;
      return ok;
    };

    int n = 0;
    for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
      const float* mk = sMask + (n & 1) * S;
      const uint32_t upar = n & 1;
      if (!mbar_wait(bar_q_ready, upar)) { failed = true; break; }
      int nbp = NB;                                             // my chunks of key blocks nbp .. NB-1 are skipped
      if constexpr (INT8) {
        const uint4 tl = *reinterpret_cast<const uint4*>(sTail + (n & 1) * 4);   // prepared with the mask row
        const bool any_valid = ((tl.x | tl.y | tl.z | tl.w) & 0x100u) != 0;
        const uint32_t mine = g == 0 ? tl.x : (g == 1 ? tl.y : (g == 2 ? tl.z : tl.w));
        if (any_valid) nbp = static_cast<int>(mine & 0xFFu);
      }

      // ---------------- pass A: scale + mask, running row max [int8: exp2 and running sum, written back]
      float m = -INFINITY, l = 0.f;
      float mc[4] = {0.f, 0.f, 0.f, 0.f};                       // running max after each block (int8)
      uint32_t v[32];
      for (int i = 0; i < nbp; ++i) {
        // when O shares columns with score block 0, that block's Q.K^T is the last one issued: take it last
        const int b = alias ? (i + 1 < nbp ? i + 1 : 0) : i;
        const int col = b * 128 + g * 32;
        if (!mbar_wait(bar_s_full + 8 * b, upar)) { failed = true; break; }
        tc_fence_after();
        if constexpr (INT8) tmem_wait_st();                     // v[] may still feed the previous block's store
        tmem_ld32(t_row + col, v);
        tmem_wait_ld();
        if (INT8 && D <= 64 && (sChunk[(n & 1) * 16 + b * 4 + g] & 4u)) {
          // Uniform mask over my 32 keys: the largest score belongs to the largest accumulator (integer compares);
          // with it as the reference each exponential is 2^((a - a_max) c2), the integer difference going through
          // the 1.5 * 2^23 bias trick in one add (|a - a_max| < 2^22 for heads up to 64 wide) and the FMA's addend
          // cancelling the bias; its rounding residue is the same factor for every score of the launch.
          int vm[4] = {static_cast<int>(v[0]), static_cast<int>(v[1]), static_cast<int>(v[2]), static_cast<int>(v[3])};
#pragma unroll
          for (int ii = 4; ii < 32; ii += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) vm[j] = max(vm[j], static_cast<int>(v[ii + j]));
          }
          const int vmax = max(max(vm[0], vm[1]), max(vm[2], vm[3]));
          const float tmax = fmaf(__int2float_rn(vmax), c2, mk[col]);
          const float m_new = fmaxf(m, tmax);
          const int kadd = W_MAGIC_I - vmax;
          float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int ii = 0; ii < 32; ii += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float e = w_ex2(fmaf(__int_as_float(static_cast<int>(v[ii + j]) + kadd), c2, neg_c0));
              v[ii + j] = __float_as_uint(e);
              sm[j] += e;
            }
          }
          l = l * w_ex2(m - m_new) + ((sm[0] + sm[1]) + (sm[2] + sm[3])) * w_ex2(tmax - m_new);
          m = m_new;
          if (b == 0) mc[0] = tmax; else if (b == 1) mc[1] = tmax; else if (b == 2) mc[2] = tmax; else mc[3] = tmax;
          tmem_st32(t_row + col, v);
          continue;
        }
        const float4* mk4 = reinterpret_cast<const float4*>(mk + col);
        float cm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 mv = mk4[i];
          const float mm[4] = {mv.x, mv.y, mv.z, mv.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float a = INT8 ? w_int_to_float(static_cast<int>(v[4 * i + j])) : __uint_as_float(v[4 * i + j]);
            const float xv = fmaf(a, c2, mm[j]);
            v[4 * i + j] = __float_as_uint(xv);
            cm[j] = fmaxf(cm[j], xv);
          }
        }
        const float cmax = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
        if constexpr (INT8) {
          const float m_new = fmaxf(m, cmax);
          const float m_sub = D <= 64 ? m_new - rho : m_new;      // same constant factor 2^rho as the fast path above
          float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float e = w_ex2(__uint_as_float(v[i + j]) - m_sub);
              v[i + j] = __float_as_uint(e);
              sm[j] += e;
            }
          }
          l = l * w_ex2(m - m_new) + ((sm[0] + sm[1]) + (sm[2] + sm[3]));
          m = m_new;
          if (b == 0) mc[0] = m; else if (b == 1) mc[1] = m; else if (b == 2) mc[2] = m; else mc[3] = m;
          tmem_st32(t_row + col, v);
        } else {
          m = fmaxf(m, cmax);
        }
      }
      if (failed) break;
      if constexpr (INT8) tmem_wait_st();
      *stat(0, upar, g) = m;
      if constexpr (INT8) *stat(1, upar, g) = l;
      if (!xchg_sync()) { failed = true; break; }
      // every thread of a row combines the four parts in the same order, so all four get identical values
      float M = -INFINITY;
#pragma unroll
      for (int o = 0; o < 4; ++o) M = fmaxf(M, *stat(0, upar, o));
      float scale = 1.f;                                        // int8: inv_p / row sum
      if constexpr (INT8) {
        float Lsum = 0.f;
#pragma unroll
        for (int o = 0; o < 4; ++o) Lsum += *stat(1, upar, o) * w_ex2(*stat(0, upar, o) - M);
        scale = p.inv_p / Lsum;
      }

      // ---------------- pass B: normalise, round, write P into the ring
      int psum = 0;
      float lsum = 0.f;
      for (int b = 0; b < nbp; ++b) {
        const int col = b * 128 + g * 32;
        const uint32_t pe = p_entry, puse = p_use;
        if (++p_entry == static_cast<uint32_t>(np)) {
          p_entry = 0;
          ++p_use;
        }
        uint8_t* sP = sPall + pe * L::P_BYTES;
        if constexpr (INT8) {
          uint32_t w[8];
          {
            tmem_ld32(t_row + col, v);
            tmem_wait_ld();
            const float f = w_ex2((b == 0 ? mc[0] : b == 1 ? mc[1] : b == 2 ? mc[2] : mc[3]) - M) * scale;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              // rne(e * f) lands in the low mantissa bits of (e * f + 1.5 * 2^23); codes are within [0, 255]
              const uint32_t y0 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 0]), f, W_MAGIC_F));
              const uint32_t y1 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 1]), f, W_MAGIC_F));
              const uint32_t y2 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 2]), f, W_MAGIC_F));
              const uint32_t y3 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 3]), f, W_MAGIC_F));
              w[i] = __byte_perm(__byte_perm(y0, y1, 0x0040), __byte_perm(y2, y3, 0x0040), 0x5410);
              psum = static_cast<int>(__dp4a(w[i], 0x01010101u, static_cast<unsigned>(psum)));
            }
          }
          if (!mbar_wait(bar_p_free + 8 * pe, (puse & 1) ^ 1)) { failed = true; break; }
          uint8_t* blk = sP + row_off;
          const int c0 = g * 2;                                 // 16-byte chunk index inside the 128-byte row
          *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
          if (p.P_out) {                                          // optional output: the codes the second MMA consumes
            const int64_t grow = static_cast<int64_t>(unit / q_tiles) * S + (unit % q_tiles) * W_BLOCK_Q + r;
            uint4* po = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.P_out) + grow * S + col);
            po[0] = make_uint4(w[0], w[1], w[2], w[3]);
            po[1] = make_uint4(w[4], w[5], w[6], w[7]);
          }
        } else {
          if (NB > 1) {                                         // with one key block the scores are still in v[]
            tmem_ld32(t_row + col, v);
            tmem_wait_ld();
            const float4* mk4 = reinterpret_cast<const float4*>(mk + col);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float4 mv = mk4[i];
              v[4 * i + 0] = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 0]), c2, mv.x));
              v[4 * i + 1] = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 1]), c2, mv.y));
              v[4 * i + 2] = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 2]), c2, mv.z));
              v[4 * i + 3] = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 3]), c2, mv.w));
            }
          }
          uint32_t w[16];
          float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float e0 = w_ex2(__uint_as_float(v[4 * i + 0]) - M);
            const float e1 = w_ex2(__uint_as_float(v[4 * i + 1]) - M);
            const float e2 = w_ex2(__uint_as_float(v[4 * i + 2]) - M);
            const float e3 = w_ex2(__uint_as_float(v[4 * i + 3]) - M);
            ls[0] += e0; ls[1] += e1; ls[2] += e2; ls[3] += e3;
            __nv_bfloat162 h0 = __floats2bfloat162_rn(e0, e1), h1 = __floats2bfloat162_rn(e2, e3);
            w[2 * i] = *reinterpret_cast<uint32_t*>(&h0);
            w[2 * i + 1] = *reinterpret_cast<uint32_t*>(&h1);
          }
          lsum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
          if (!mbar_wait(bar_p_free + 8 * pe, (puse & 1) ^ 1)) { failed = true; break; }
          // bf16: a 128-key block is two 64-key sub-tiles (128-byte rows); my 32 keys are 4 chunks of 16 bytes
          uint8_t* blk = sP + (g >> 1) * (W_BLOCK_Q * 128) + row_off;
          const int c0 = (g & 1) * 4;
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(blk + (((c0 + i) ^ (r & 7)) * 16)) =
                make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
        // this block of P is complete and its score columns have been read for the last time
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(bar_p_full + 8 * b);
          mbar_arrive(bar_s_free + 8 * b);
        }
      }
      if (failed) break;
      if constexpr (INT8) {
        for (int b = nbp; b < NB; ++b) {                        // skipped chunks: their codes are zero
          const int col = b * 128 + g * 32;
          const uint32_t pe = p_entry, puse = p_use;
          if (++p_entry == static_cast<uint32_t>(np)) {
            p_entry = 0;
            ++p_use;
          }
          if (!mbar_wait(bar_p_free + 8 * pe, (puse & 1) ^ 1)) { failed = true; break; }
          uint8_t* blk = sPall + pe * L::P_BYTES + row_off;
          const int c0 = g * 2;
          *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
          if (p.P_out) {
            const int64_t grow = static_cast<int64_t>(unit / q_tiles) * S + (unit % q_tiles) * W_BLOCK_Q + r;
            uint4* po = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.P_out) + grow * S + col);
            po[0] = make_uint4(0u, 0u, 0u, 0u);
            po[1] = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar_p_full + 8 * b);
            mbar_arrive(bar_s_free + 8 * b);
          }
        }
        if (failed) break;
      }
      // my part of the row sum goes to the auxiliary warps, which finish and store the output; the slot is
      // free once they have read the sums of the unit that used it two units ago
      if (!mbar_wait(bar_st_free + 8 * upar, ((n >> 1) & 1) ^ 1)) { failed = true; break; }
      *stat(2, upar, g) = INT8 ? __int_as_float(psum) : lsum;
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_st_ready + 8 * upar);
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

template <bool INT8, int D, int NB>
cudaError_t launch_wide_nb(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                           int num_sms, cudaStream_t s) {
  constexpr WideCfg cfg = wide_cfg_t<INT8, D>(NB * 128);
  if constexpr (cfg.smem == 0) {
    return cudaErrorInvalidValue;
  } else {
    auto kern = sdpa_wide_kernel<INT8, D, NB, cfg.np, cfg.stages>;
    const int units = p.B * p.H * ((p.S + W_BLOCK_Q - 1) / W_BLOCK_Q);
    const int grid = units < num_sms ? units : num_sms;
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), cfg.smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid);
    lc.blockDim = dim3(W_THREADS);
    lc.dynamicSmemBytes = cfg.smem;
    lc.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kern, tmQ, tmK, tmV, p);
  }
}

template <bool INT8, int D>
cudaError_t launch_wide_t(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                          int num_sms, cudaStream_t s) {
  switch ((p.S + 127) / 128) {
    case 1: return launch_wide_nb<INT8, D, 1>(tmQ, tmK, tmV, p, num_sms, s);
    case 2: return launch_wide_nb<INT8, D, 2>(tmQ, tmK, tmV, p, num_sms, s);
    case 3: return launch_wide_nb<INT8, D, 3>(tmQ, tmK, tmV, p, num_sms, s);
    case 4: return launch_wide_nb<INT8, D, 4>(tmQ, tmK, tmV, p, num_sms, s);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

size_t sdpa_wide_smem_bytes(int S, int D, int is_int8) { return wide_cfg(S, D, is_int8).smem; }

void sdpa_wide_box(int D, int is_int8, int* box_elems, int* swizzle_bytes) {
  const int esz = is_int8 ? 1 : 2;
  const int rowb = D * esz <= 64 ? 64 : 128;
  *box_elems = rowb / esz;
  *swizzle_bytes = rowb;
}

cudaError_t launch_sdpa_wide(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                             int num_sms, cudaStream_t s) {
  if (p.is_int8) {
    if (p.D == 64) return launch_wide_t<true, 64>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 96) return launch_wide_t<true, 96>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 128) return launch_wide_t<true, 128>(tmQ, tmK, tmV, p, num_sms, s);
  } else {
    if (p.D == 64) return launch_wide_t<false, 64>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 96) return launch_wide_t<false, 96>(tmQ, tmK, tmV, p, num_sms, s);
    if (p.D == 128) return launch_wide_t<false, 128>(tmQ, tmK, tmV, p, num_sms, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace gc
