// Fused scaled-dot-product attention on tcgen05 (Section VII "MHA": two batch matmuls with the softmax and
// the binary ops between them fused after the first one; the two matmul loop nests merged).
//
// Persistent CTAs (one per SM, 704 threads) walk over work units (batch, head, 128-query tile):
//   warp 0      TMA producer: Q tile, all K rows and all V rows of the unit into one of two shared-memory
//               slots (128B / 64B swizzle), one unit ahead of the math (no multicast)
//   warp 1      MMA issuer (one thread): S = Q K^T in 128-key blocks into tensor memory, O = P V in 128-key
//               blocks as soon as each P block is ready.  When two score buffers fit in tensor memory
//               (S = 128) the next unit's S is issued a whole unit early; otherwise its blocks are issued as
//               soon as the softmax warps release the corresponding TMEM columns
//   warps 2-5   per-unit preparation (u8 -> s8 flip of Q on the int8 path, mask row scaled by log2(e)) and the
//               epilogue of the previous unit: O out of tensor memory, deferred normalisation (bf16) or
//               dequantize/requantize (int8), swizzled staging, one TMA store per 32 rows
//   warps 6-21  softmax: four threads per query row (TMEM lane), each owning 32 of every 128 key columns.
//               Pass A: scale + mask, running row max, exp2 and running row sum (int8: the exponentials
//               are written back to tensor memory); the four threads of a row combine their statistics;
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
//
// Integer <-> float conversions in the inner loops use the 1.5 * 2^23 bias trick on the FMA/ALU pipes
// (exact for |x| < 2^22) because the conversion instructions share the special-function unit with exp2,
// which is the busiest pipe of this kernel.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int SDPA_D = 64;
constexpr int SDPA_BLOCK_Q = 128;
constexpr int SDPA_THREADS = 704;
constexpr int SDPA_SOFTMAX_WARPS = 16;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float MAGIC_F = 12582912.0f;          // 1.5 * 2^23
constexpr int MAGIC_I = 0x4B400000;             // its bit pattern

template <bool INT8>
struct SdpaSmem {
  static constexpr int ESZ = INT8 ? 1 : 2;
  static constexpr int ROW_BYTES = SDPA_D * ESZ;               // 64 (SW64) or 128 (SW128)
  static constexpr int OUT_STAGING_BYTES = 4 * 4096;           // per auxiliary warp: 32 rows x <= 128 bytes
  __host__ __device__ static constexpr int q_bytes() { return SDPA_BLOCK_Q * ROW_BYTES; }
  __host__ __device__ static constexpr int kv_bytes(int S) { return S * ROW_BYTES; }
  // P: per 128-key block, 128 rows x (128 keys * ESZ) bytes = 16 KB (int8) or 32 KB (bf16)
  __host__ __device__ static constexpr int p_bytes(int S) { return (S / 128) * SDPA_BLOCK_Q * 128 * ESZ; }
  __host__ __device__ static constexpr int slot_bytes(int S) { return q_bytes() + 2 * kv_bytes(S); }
  __host__ __device__ static constexpr int total(int S, int slots, int nsb, int stage_out) {
    return slots * slot_bytes(S) + nsb * p_bytes(S) + (stage_out ? OUT_STAGING_BYTES : 0) + slots * S * 4 /*mask*/ +
           24 * 128 * 4 /*row statistics*/ + 448 /*barriers, TMEM address, chunk flags*/;
  }
};

struct SdpaCfg {
  int slots;      // shared-memory slots for (Q, K, V): 2 = next unit prefetched
  int nsb;        // score/output buffers in tensor memory and P buffers in shared memory
  int stage_out;  // 1: outputs staged in shared memory and written with TMA stores; 0: plain vector stores
  size_t smem;
};

static SdpaCfg sdpa_cfg(int S, int is_int8) {
  const size_t limit = 227 * 1024;
  const int tries[4][3] = {{2, 2, 1}, {2, 1, 1}, {1, 1, 1}, {1, 1, 0}};
  for (auto& t : tries) {
    if (t[1] == 2 && 2 * (S + SDPA_D) > 512) continue;
    const size_t need = 1024 + (is_int8 ? SdpaSmem<true>::total(S, t[0], t[1], t[2]) : SdpaSmem<false>::total(S, t[0], t[1], t[2]));
    if (need <= limit) return {t[0], t[1], t[2], need};
  }
  return {0, 0, 0, static_cast<size_t>(1) << 30};
}

size_t sdpa_tc_smem_bytes(int S, int is_int8) { return sdpa_cfg(S, is_int8).smem; }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// exact (float)a for |a| < 2^22 without a conversion instruction
__device__ __forceinline__ float int_to_float_magic(int a) { return __int_as_float(a + MAGIC_I) - MAGIC_F; }
// exact (float)a for |a| < 2^24: high and low parts converted separately, recombined with one exact FMA
__device__ __forceinline__ float int_to_float_magic24(int a) {
  const float hi = int_to_float_magic(a >> 11), lo = int_to_float_magic(a & 0x7FF);
  return fmaf(hi, 2048.0f, lo);
}
// saturate(rne(u) + zp) with the rounding done by the bias trick
__device__ __forceinline__ int quantize_magic(float u, int zp, int lo, int hi) {
  u = fminf(fmaxf(u, -1024.0f), 1024.0f);
  const int r = __float_as_int(u + MAGIC_F) - MAGIC_I;
  return min(max(r + zp, lo), hi);
}

// MAXFREE: the planner has bounded every score (see SdpaParams::max_free); a separate instantiation keeps the
// general int8 kernel's code as it is.
// S_CT / CFG: sequence length and buffer configuration (100 slots + 10 score buffers + staged outputs) as
// compile-time constants; S_CT = 0: both at run time.  With them the per-block loops unroll and the buffer
// bookkeeping folds away: 112 -> 98 µs on the 384-key int8 benchmark shape, 11.8 -> 10.5 µs on the 128-key bf16 one.
template <bool INT8, bool MAXFREE = false, int S_CT = 0, int CFG = 0>
__global__ void __launch_bounds__(SDPA_THREADS, 1)
sdpa_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, const SdpaParams p,
               const int slots_rt, const int nsb_rt, const int stage_out_rt) {
  const int slots = S_CT ? CFG / 100 : slots_rt;
  const int nsb = S_CT ? (CFG / 10) % 10 : nsb_rt;
  const int stage_out = S_CT ? CFG % 10 : stage_out_rt;
  using L = SdpaSmem<INT8>;
  constexpr int ROW_BYTES = L::ROW_BYTES;
  constexpr uint32_t SWZ = INT8 ? SWZ_64B : SWZ_128B;
  constexpr uint32_t SBO = 8 * ROW_BYTES;                       // 8-row group stride: 512 or 1024 bytes
  constexpr int P_BLOCK_BYTES = SDPA_BLOCK_Q * 128 * L::ESZ;    // one 128-key block of P
  constexpr uint32_t TMEM_COLS = 512;

  const int S = S_CT ? S_CT : p.S;
  const int NB = S / 128;                                       // key blocks
  const int BUF_COLS = S + SDPA_D;                              // TMEM columns per (S, O) buffer
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sSlots = smem;
  uint8_t* sPall = sSlots + slots * L::slot_bytes(S);
  uint8_t* sOut = sPall + nsb * L::p_bytes(S);                            // output staging, 4 KB per auxiliary warp
  float* sMask = reinterpret_cast<float*>(sOut + (stage_out ? L::OUT_STAGING_BYTES : 0));   // [slots][S]
  float* sStat = sMask + slots * S;                                       // [3 kinds][2 parities][4 groups][128]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sStat + 24 * 128);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 26);
  // per slot and 32-key chunk: 1 = every key of the chunk is masked out, 2 = the chunk has an unmasked key, 0 = neither
  uint32_t* sChunk = tmem_slot + 4;                                       // [2 slots][16]
  // per slot and group of 32 columns (g): bits 0-7 = key blocks up to the last one whose chunk g is not fully masked,
  // bit 8 = the group has a chunk with an unmasked key
  uint32_t* sTail = sChunk + 32;                                          // [2 slots][4]
  const uint32_t bar_xchg = smem_u32(sTail + 8);                          // the softmax warps exchange row statistics
  const uint32_t b0 = smem_u32(bars);
  const uint32_t bar_kv_full = b0, bar_kv_empty = b0 + 16, bar_kv_ready = b0 + 32;   // [2] each
  const uint32_t bar_s_full = b0 + 48, bar_s_free = b0 + 72, bar_p_full = b0 + 96;   // [3] each
  const uint32_t bar_o_full = b0 + 120, bar_o_free = b0 + 136;                       // [2], [2]
  const uint32_t bar_st_ready = b0 + 160, bar_st_free = b0 + 176;                    // [2], [2]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q_tiles = S / SDPA_BLOCK_Q;
  const int num_units = p.B * p.H * q_tiles;

  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(bar_kv_full + 8 * i, 1);
      mbar_init(bar_kv_empty + 8 * i, 1);
      mbar_init(bar_kv_ready + 8 * i, 4);
      mbar_init(bar_o_full + 8 * i, 1);
      mbar_init(bar_o_free + 8 * i, 4);
      mbar_init(bar_st_ready + 8 * i, SDPA_SOFTMAX_WARPS);
      mbar_init(bar_st_free + 8 * i, 4);
    }
    for (int i = 0; i < 3; ++i) {
      mbar_init(bar_s_full + 8 * i, 1);
      mbar_init(bar_s_free + 8 * i, SDPA_SOFTMAX_WARPS);
      mbar_init(bar_p_full + 8 * i, SDPA_SOFTMAX_WARPS);
    }
    mbar_init(bar_xchg, SDPA_SOFTMAX_WARPS);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
    tma_prefetch_desc(&tmO);
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
  // While waiting for it, the first units' operands are pulled into L2 (a prefetch has no destination the kernel
  // could read too early, and L2 stays coherent with whatever the preceding kernel still writes); nothing else
  // touches global memory before that kernel has completed (the wait is a no-op for an ordinary launch).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    const int q_tiles0 = S / SDPA_BLOCK_Q;
    int unit = blockIdx.x;
    for (int n0 = 0; n0 < slots && unit < p.B * p.H * q_tiles0; ++n0, unit += gridDim.x) {
      const int bh = unit / q_tiles0, qt = unit % q_tiles0;
      tma_prefetch_2d(&tmQ, 0, bh * S + qt * SDPA_BLOCK_Q);
      for (int j = 0; j < NB; ++j) {
        tma_prefetch_2d(&tmK, 0, bh * S + j * 128);
        tma_prefetch_2d(&tmV, 0, bh * S + j * 128);
      }
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  bool failed = false;
  auto slot_q = [&](int s) { return sSlots + s * L::slot_bytes(S); };
  auto slot_k = [&](int s) { return slot_q(s) + L::q_bytes(); };
  auto slot_v = [&](int s) { return slot_k(s) + L::kv_bytes(S); };
  // Unit n of this CTA uses score/output buffer buf(n); it is that buffer's cnt(n)-th use.  With one
  // buffer the per-key-block barriers are indexed by block, with two (one block per unit) by buffer.
  auto slot_of = [&](int n) { return slots == 2 ? (n & 1) : 0; };   // slots is 1 or 2: no division needed
  auto use_of = [&](int n) { return slots == 2 ? (n >> 1) : n; };
  auto buf_of = [&](int n) { return nsb == 2 ? (n & 1) : 0; };
  auto cnt_of = [&](int n) { return nsb == 2 ? (n >> 1) : n; };
  auto bx = [&](int buf, int b) { return nsb == 2 ? buf : b; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units; unit += gridDim.x, ++n) {
        const int s = slot_of(n);
        const uint32_t par = use_of(n) & 1;
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
      // S[:, 128b .. 128b+127] = Q K_b^T for unit n1 (waits until the softmax warps have released the columns)
      auto mma1 = [&](int n1, int b) -> bool {
        const int s = slot_of(n1), buf = buf_of(n1);
        if (!mbar_wait(bar_s_free + 8 * bx(buf, b), (cnt_of(n1) & 1) ^ 1)) return false;
        tc_fence_after();
        const uint64_t a_desc = make_smem_desc(smem_u32(slot_q(s)), 16, SBO, SWZ);
        const uint64_t b_desc = make_smem_desc(smem_u32(slot_k(s)) + b * 128 * ROW_BYTES, 16, SBO, SWZ);
#pragma unroll
        for (int k = 0; k < K1_STEPS; ++k)
          umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + buf * BUF_COLS + b * 128, a_desc + 2 * k, b_desc + 2 * k, idesc1,
                                              k != 0);
        umma_commit(bar_s_full + 8 * bx(buf, b));
        return true;
      };
      auto mma2 = [&](int n0, int b) {                          // O += P_b V_b for unit n0
        const int s = slot_of(n0), buf = buf_of(n0);
        const uint32_t sP = smem_u32(sPall) + buf * L::p_bytes(S);
#pragma unroll
        for (int ks = 0; ks < K2_STEPS; ++ks) {
          // A: P block, K-major, 128B swizzle: 4 MMA steps of 32 bytes per 128-byte span, spans 16 KB apart
          const uint64_t a_desc =
              make_smem_desc(sP + b * P_BLOCK_BYTES + (ks >> 2) * (SDPA_BLOCK_Q * 128) + (ks & 3) * 32, 16, 1024, SWZ_128B);
          // B: V as stored [key][d] = MN-major: one key per ROW_BYTES, 8-key groups SBO apart
          const int key0 = b * 128 + ks * (128 / K2_STEPS);
          const uint64_t b_desc = make_smem_desc(smem_u32(slot_v(s)) + key0 * ROW_BYTES, SBO, SBO, SWZ);
          umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + buf * BUF_COLS + S, a_desc, b_desc, idesc2, (b | ks) != 0);
        }
      };
      auto wait_inputs = [&](int n1) -> bool {
        const int s = slot_of(n1);
        const uint32_t par = use_of(n1) & 1;
        return mbar_wait(bar_kv_ready + 8 * s, par) && mbar_wait(bar_kv_full + 8 * s, par);
      };
      int n = 0;
      for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
        const int s = slot_of(n), buf = buf_of(n);
        const uint32_t fpar = cnt_of(n) & 1;
        const bool has_next = unit + static_cast<int>(gridDim.x) < num_units;
        if (n == 0) {
          if (!wait_inputs(0)) { failed = true; break; }
          for (int b = 0; b < NB && !failed; ++b) failed = !mma1(0, b);
          if (failed) break;
        }
        bool next_issued = false;
        if (has_next && nsb == 2) {                             // the other score buffer: a whole unit early
          if (!wait_inputs(n + 1)) { failed = true; break; }
          for (int b = 0; b < NB && !failed; ++b) failed = !mma1(n + 1, b);
          if (failed) break;
          next_issued = true;
        }
        bool next_ready = false;
        for (int b = 0; b < NB && !failed; ++b) {
          if (!mbar_wait(bar_p_full + 8 * bx(buf, b), fpar)) { failed = true; break; }
          if (b == 0 && !mbar_wait(bar_o_free + 8 * buf, fpar ^ 1)) { failed = true; break; }
          tc_fence_after();
          // Same buffer: the next unit's scores block by block as the columns free up - and BEFORE this unit's
          // P.V for the block: the softmax warps will wait for those scores, nobody waits for this O yet, and
          // the tensor pipe runs the MMAs in issue order.
          if (has_next && !next_issued && slots == 2) {
            if (!next_ready) {
              if (!wait_inputs(n + 1)) { failed = true; break; }
              next_ready = true;
            }
            if (!mma1(n + 1, b)) { failed = true; break; }
          }
          mma2(n, b);
          if (b == NB - 1) {
            umma_commit(bar_o_full + 8 * buf);
            umma_commit(bar_kv_empty + 8 * s);
          }
        }
        if (!failed && has_next && !next_issued && slots == 1) {
          if (!wait_inputs(n + 1)) { failed = true; break; }
          for (int b = 0; b < NB && !failed; ++b) failed = !mma1(n + 1, b);
        }
      }
      if (failed) report(p.status, DEV_TIMEOUT_MMA);
    }
  } else if (warp < 6) {
    // ------------------------------------------------------------------ auxiliary warps
    // Per unit: (1) preparation of the inputs that have just landed - mask row scaled by log2(e), u8 -> s8
    // flip of Q on the int8 path; (2) epilogue of the previous unit - read O from tensor memory once its
    // second MMA has completed, finish it with the row statistics the softmax warps left in shared memory,
    // stage it and hand it to a TMA store.  This keeps the whole epilogue off the softmax warps' critical path.
    const int t = tid - 64;                                     // 0..127
    const int aw = warp - 2;                                    // staging buffer index
    const int q = warp & 3;                                     // TMEM lane quarter this warp may access
    const int r = q * 32 + lane;                                // query row within the tile
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    constexpr int OUT_ROW_BYTES = SDPA_D * L::ESZ;              // 64 (int8) or 128 (bf16)
    uint8_t* my_out = sOut + aw * 4096;
    auto stat2 = [&](int par, int grp) { return sStat + ((2 * 2 + par) * 4 + grp) * 128 + r; };

    auto epilogue = [&](int unit, int n0) -> bool {
      const int buf = buf_of(n0), par = n0 & 1;
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
      if (!mbar_wait(bar_o_full + 8 * buf, cnt_of(n0) & 1)) return false;
      tc_fence_after();
      uint32_t v[64];
      {
        uint32_t (&v0)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[0]);
        uint32_t (&v1)[32] = *reinterpret_cast<uint32_t(*)[32]>(&v[32]);
        tmem_ld32(t_lane + buf * BUF_COLS + S, v0);
        tmem_ld32(t_lane + buf * BUF_COLS + S + 32, v1);
      }
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(bar_o_free + 8 * buf);
        mbar_arrive(bar_st_free + 8 * par);
        if (stage_out) tma_store_wait_read<0>();                // the previous store has read the staging buffer
      }
      __syncwarp();
      const int bh = unit / q_tiles, qt = unit % q_tiles;
      const int64_t grow = static_cast<int64_t>(bh) * S + qt * SDPA_BLOCK_Q + r;
      uint8_t* dst_direct = static_cast<uint8_t*>(p.O) + grow * OUT_ROW_BYTES;
      if constexpr (INT8) {
        const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
        const int corr = p.zp_v * __float_as_int(total);       // zero point of V times the row sum of P
        // saturate(rne(u) + zp) = rne(clamp(u, lo - zp, hi - zp)) + zp: clamp in float, round with the bias
        // trick, and fold "- bias bits + zp" into one integer add; the code is the low byte of the result
        const float u_lo = static_cast<float>(lo - p.zp_o), u_hi = static_cast<float>(hi - p.zp_o);
        const int kadd = p.zp_o - MAGIC_I;
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          uint32_t y[4];
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int acc = static_cast<int>(v[4 * i + k]) - corr;
            const float tt = __fmul_rn(__int2float_rn(acc), p.dq2);
            const float u = fminf(fmaxf(__fmul_rn(tt, p.inv_o), u_lo), u_hi);
            y[k] = static_cast<uint32_t>(__float_as_int(u + MAGIC_F) + kadd);
          }
          w[i] = __byte_perm(__byte_perm(y[0], y[1], 0x0040), __byte_perm(y[2], y[3], 0x0040), 0x5410);
        }
        // 64-byte rows, 64B swizzle: 16-byte chunk c of row r goes to chunk c ^ ((r >> 1) & 3)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint8_t* dst = stage_out ? my_out + lane * OUT_ROW_BYTES + ((c ^ ((lane >> 1) & 3)) * 16) : dst_direct + c * 16;
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
        }
      } else {
        const float rl = 1.0f / total;                         // deferred normalisation by the row sum
        uint32_t w[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[2 * i]) * rl, __uint_as_float(v[2 * i + 1]) * rl);
          w[i] = *reinterpret_cast<uint32_t*>(&hh);
        }
        // 128-byte rows, 128B swizzle: chunk c of row r goes to chunk c ^ (r & 7)
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          uint8_t* dst = stage_out ? my_out + lane * OUT_ROW_BYTES + ((c ^ (lane & 7)) * 16) : dst_direct + c * 16;
          *reinterpret_cast<uint4*>(dst) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
        }
      }
      if (stage_out) {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmO, 0, bh * S + qt * SDPA_BLOCK_Q + q * 32, smem_u32(my_out));
          tma_store_commit();
        }
      }
      return true;
    };

    int n = 0;
    int prev_unit = -1;
    for (int unit = blockIdx.x; unit < num_units && !failed; unit += gridDim.x, ++n) {
      const int s = slot_of(n);
      const int b = (unit / q_tiles) / p.H;
      float* mk = sMask + s * S;
      // the mask slot is free once the unit that used this slot before has been fully consumed, which
      // the producer's own wait on kv_empty guarantees before kv_full can complete for this unit
      // the mask values are fetched before the wait so that their latency hides behind the unit's loads
      float mreg[3];
#pragma unroll
      for (int i = 0; i < 3; ++i) {
        const int j = t + 128 * i;
        mreg[i] = (p.mask && j < S) ? __ldg(p.mask + static_cast<int64_t>(b) * S + j) * LOG2E : 0.0f;
      }
      if (!mbar_wait(bar_kv_full + 8 * s, use_of(n) & 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        failed = true;
        break;
      }
      uint32_t tail = 0;                                        // see sTail: this warp covers group (warp - 2) of every block
#pragma unroll
      for (int i = 0; i < 3; ++i) {                             // a warp covers one aligned 32-key chunk per step
        const int j = t + 128 * i;
        if (j >= S) break;
        const float mv = mreg[i];
        mk[j] = mv;
        if constexpr (INT8) {
          const bool all_masked = __all_sync(0xffffffffu, p.skip_thr > 0.f && mv <= -p.skip_thr);
          const bool any_valid = __any_sync(0xffffffffu, mv >= -1.0f);
          // bit 2: all 32 keys of the chunk carry the same mask value, so the largest score is the largest accumulator
          const bool uniform = __all_sync(0xffffffffu, __float_as_uint(mv) == __shfl_sync(0xffffffffu, __float_as_uint(mv), 0));
          if (lane == 0) sChunk[s * 16 + (j >> 5)] = (all_masked ? 1u : (any_valid ? 2u : 0u)) | (uniform ? 4u : 0u);
          if (!all_masked) tail = (tail & 0x100u) | static_cast<uint32_t>(i + 1);
          if (any_valid && !all_masked) tail |= 0x100u;
        }
      }
      if (INT8 && lane == 0) sTail[s * 4 + (warp - 2)] = tail;
      if (INT8 && !p.q_signed) {
        uint4* q4 = reinterpret_cast<uint4*>(slot_q(s));
        for (int i = t; i < L::q_bytes() / 16; i += 128) {
          uint4 v = q4[i];
          v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
          q4[i] = v;
        }
        fence_proxy_async_smem();
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_kv_ready + 8 * s);
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
    if (lane == 0) tma_store_wait_read<0>();   // (reads of the staging buffers, not completion: the stores complete with the kernel)
  } else {
    // ------------------------------------------------------------------ softmax warps
    // Four threads share a query row (TMEM lane): warp w covers lane quarter (w % 4) and, of every 128-key
    // block, the 32 columns [32 g, 32 g + 32) with g = (w - 6) / 4.  Four warps per scheduler keep the
    // TMEM / barrier / exp latencies of one warp hidden behind the others.
    const int sw = warp - 6;                                    // 0..15
    const int q = warp & 3;                                     // TMEM lane quarter
    const int g = sw >> 2;                                      // which 32 of every 128 key columns
    const int r = q * 32 + lane;                                // query row within the tile = TMEM lane
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const float c2 = (INT8 ? __fmul_rn(p.dq1, p.scalar) : p.scalar) * LOG2E;
    const float neg_c0 = -__fmul_rn(MAGIC_F, c2);                // cancels the bias of the int -> float trick inside an FMA
    const float rho = fmaf(MAGIC_F, c2, neg_c0);                 // ... up to this rounding residue, a launch-wide constant
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    uint32_t xphase = 0;
    // statistics shared between the four threads of a row and the auxiliary warps: [kind][unit parity][group][row]
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
      const int s = slot_of(n), buf = buf_of(n);
      const float* mk = sMask + s * S;
      const uint32_t fpar = cnt_of(n) & 1;
      const int upar = n & 1;
      const uint32_t t_row = t_lane + buf * BUF_COLS;
      uint8_t* sP = sPall + buf * L::p_bytes(S);
      if (!mbar_wait(bar_kv_ready + 8 * s, use_of(n) & 1)) { failed = true; break; }
      // Mask-aware skipping (int8): with at least one unmasked key in the row, a chunk whose keys are all
      // masked has exponentials that underflow to exactly zero, so neither pass needs to touch it: its codes are
      // zero.  Only the trailing run of such chunks is left out (a padding mask is a valid-length prefix), which
      // keeps the two passes free of per-chunk branches: they simply run over fewer blocks.
      int nbp = NB;                                             // my chunks of key blocks nbp .. NB-1 are skipped
      if constexpr (INT8) {
        const uint4 tl = *reinterpret_cast<const uint4*>(sTail + s * 4);   // prepared with the mask row
        const bool any_valid = ((tl.x | tl.y | tl.z | tl.w) & 0x100u) != 0;
        const uint32_t mine = g == 0 ? tl.x : (g == 1 ? tl.y : (g == 2 ? tl.z : tl.w));
        if (any_valid) nbp = static_cast<int>(mine & 0xFFu);
      }

      // ---------------- pass A: one 32-column chunk per key block, transformed in place
      // (accumulator -> scaled, masked score [-> exponential, stored back to tensor memory on the int8 path])
      float m = -INFINITY, l = 0.f;
      float mc[3] = {0.f, 0.f, 0.f};                            // int8: the exponent the stored exponentials of block b refer to
      uint32_t v[32];
      // The four warps of a scheduler (same lane quarter, g = 0..3) would otherwise walk through pass A in step: all
      // loading and searching the maximum while the exponential unit idles, then all queueing for it.  A small stagger
      // lets the exponentials of one overlap the loads of the next (96.97 -> 95.15 µs on the 384-key benchmark shape).
      if (INT8 && S_CT == 384 && g > 0) __nanosleep(120 * g);
      for (int b = 0; b < nbp; ++b) {
        const int col = b * 128 + g * 32;
        if (!mbar_wait(bar_s_full + 8 * bx(buf, b), fpar)) { failed = true; break; }
        tc_fence_after();
        if constexpr (INT8) tmem_wait_st();                     // v[] may still feed the previous block's store
        tmem_ld32(t_row + col, v);
        tmem_wait_ld();
        if constexpr (INT8 && MAXFREE) {
          // "Fast softmax" (Section VII): the planner has shown that no exponential and no row sum can leave fp32's
          // range (8-bit operands, small scales, no mask), so the scores go through exp2 as they are.  The common
          // factor 2^rho of the bias trick's rounding residue drops out of the softmax as on the path below.
          float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float e = ex2(fmaf(__int_as_float(static_cast<int>(v[i + j]) + MAGIC_I), c2, neg_c0));
              v[i + j] = __float_as_uint(e);
              sm[j] += e;
            }
          }
          l += (sm[0] + sm[1]) + (sm[2] + sm[3]);
          m = 0.f;                                               // every stored exponential refers to exponent 0
          tmem_st32(t_row + col, v);
          continue;
        }
        if (INT8 && (sChunk[s * 16 + b * 4 + g] & 4u)) {
          // Uniform mask over my 32 keys (the usual case: unmasked, or padding): the largest score belongs to the
          // largest accumulator, found with integer compares.  With it as the reference, each exponential is
          // 2^((a - a_max) c2): the integer difference goes through the 1.5 * 2^23 bias trick in ONE add
          // (|a - a_max| < 2^22 for 64-wide heads), the FMA's addend cancels the bias (its rounding residue is the
          // same factor for every score of the launch and drops out of the softmax), and no per-score
          // max or subtraction is left.
          int vm[4] = {static_cast<int>(v[0]), static_cast<int>(v[1]), static_cast<int>(v[2]), static_cast<int>(v[3])};
#pragma unroll
          for (int i = 4; i < 32; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) vm[j] = max(vm[j], static_cast<int>(v[i + j]));
          }
          const int vmax = max(max(vm[0], vm[1]), max(vm[2], vm[3]));
          // (the conversion by the bias trick, not by an instruction of the unit the exponentials queue for)
          const float tmax = fmaf(int_to_float_magic(vmax), c2, mk[col]);   // largest scaled, masked score of the chunk
          const float m_new = fmaxf(m, tmax);
          const int kadd = MAGIC_I - vmax;
          float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float e = ex2(fmaf(__int_as_float(static_cast<int>(v[i + j]) + kadd), c2, neg_c0));
              v[i + j] = __float_as_uint(e);
              sm[j] += e;
            }
          }
          l = l * ex2(m - m_new) + ((sm[0] + sm[1]) + (sm[2] + sm[3])) * ex2(tmax - m_new);
          m = m_new;
          if (b == 0) mc[0] = tmax; else if (b == 1) mc[1] = tmax; else mc[2] = tmax;
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
            const float a = INT8 ? int_to_float_magic(static_cast<int>(v[4 * i + j])) : __uint_as_float(v[4 * i + j]);
            const float xv = fmaf(a, c2, mm[j]);
            v[4 * i + j] = __float_as_uint(xv);
            cm[j] = fmaxf(cm[j], xv);
          }
        }
        const float cmax = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
        if constexpr (INT8) {
          const float m_new = fmaxf(m, cmax);
          const float m_sub = m_new - rho;                       // same constant factor 2^rho as the fast path above
          float sm[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float e = ex2(__uint_as_float(v[i + j]) - m_sub);
              v[i + j] = __float_as_uint(e);
              sm[j] += e;
            }
          }
          l = l * ex2(m - m_new) + ((sm[0] + sm[1]) + (sm[2] + sm[3]));
          m = m_new;
          if (b == 0) mc[0] = m; else if (b == 1) mc[1] = m; else mc[2] = m;
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
        for (int o = 0; o < 4; ++o) Lsum += *stat(1, upar, o) * ex2(*stat(0, upar, o) - M);
        scale = p.inv_p / Lsum;
      }

      // ---------------- pass B: normalise, round, write P
      int psum = 0;
      float lsum = 0.f;
      for (int b = 0; b < nbp; ++b) {
        const int col = b * 128 + g * 32;
        if constexpr (INT8) {
          uint32_t w[8];
          tmem_ld32(t_row + col, v);
          tmem_wait_ld();
          const float f = ex2((b == 0 ? mc[0] : b == 1 ? mc[1] : mc[2]) - M) * scale;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            // rne(e * f) lands in the low mantissa bits of (e * f + 1.5 * 2^23); codes are within [0, 255]
            // because p <= 1 and inv_p <= 255
            const uint32_t y0 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 0]), f, MAGIC_F));
            const uint32_t y1 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 1]), f, MAGIC_F));
            const uint32_t y2 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 2]), f, MAGIC_F));
            const uint32_t y3 = __float_as_uint(fmaf(__uint_as_float(v[4 * i + 3]), f, MAGIC_F));
            w[i] = __byte_perm(__byte_perm(y0, y1, 0x0040), __byte_perm(y2, y3, 0x0040), 0x5410);
            psum = static_cast<int>(__dp4a(w[i], 0x01010101u, static_cast<unsigned>(psum)));
          }
          uint8_t* blk = sP + b * P_BLOCK_BYTES + row_off;
          const int c0 = g * 2;                                 // 16-byte chunk index inside the 128-byte row
          *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
          if (S_CT == 0 && p.P_out) {                             // optional output (run-time variant only): the codes the second MMA consumes
            const int64_t grow = static_cast<int64_t>(unit / q_tiles) * S + (unit % q_tiles) * SDPA_BLOCK_Q + r;
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
            const float e0 = ex2(__uint_as_float(v[4 * i + 0]) - M);
            const float e1 = ex2(__uint_as_float(v[4 * i + 1]) - M);
            const float e2 = ex2(__uint_as_float(v[4 * i + 2]) - M);
            const float e3 = ex2(__uint_as_float(v[4 * i + 3]) - M);
            ls[0] += e0; ls[1] += e1; ls[2] += e2; ls[3] += e3;
            __nv_bfloat162 h0 = __floats2bfloat162_rn(e0, e1), h1 = __floats2bfloat162_rn(e2, e3);
            w[2 * i] = *reinterpret_cast<uint32_t*>(&h0);
            w[2 * i + 1] = *reinterpret_cast<uint32_t*>(&h1);
          }
          lsum += (ls[0] + ls[1]) + (ls[2] + ls[3]);
          // bf16: a 128-key block is two 64-key sub-tiles (128-byte rows); my 32 keys are 4 chunks of 16 bytes
          uint8_t* blk = sP + b * P_BLOCK_BYTES + (g >> 1) * (SDPA_BLOCK_Q * 128) + row_off;
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
          mbar_arrive(bar_p_full + 8 * bx(buf, b));
          mbar_arrive(bar_s_free + 8 * bx(buf, b));
        }
      }
      if constexpr (INT8) {
        for (int b = nbp; b < NB; ++b) {                        // skipped chunks: their codes are zero
          const int col = b * 128 + g * 32;
          uint8_t* blk = sP + b * P_BLOCK_BYTES + row_off;
          const int c0 = g * 2;
          *reinterpret_cast<uint4*>(blk + (((c0 + 0) ^ (r & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
          *reinterpret_cast<uint4*>(blk + (((c0 + 1) ^ (r & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
          if (S_CT == 0 && p.P_out) {
            const int64_t grow = static_cast<int64_t>(unit / q_tiles) * S + (unit % q_tiles) * SDPA_BLOCK_Q + r;
            uint4* po = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.P_out) + grow * S + col);
            po[0] = make_uint4(0u, 0u, 0u, 0u);
            po[1] = make_uint4(0u, 0u, 0u, 0u);
          }
          fence_proxy_async_smem();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(bar_p_full + 8 * bx(buf, b));
            mbar_arrive(bar_s_free + 8 * bx(buf, b));
          }
        }
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
  if (failed) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

cudaError_t launch_sdpa_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmO,
                           const SdpaParams& p, int num_sms, cudaStream_t s) {
  const SdpaCfg cfg = sdpa_cfg(p.S, p.is_int8);
  if (!cfg.slots) return cudaErrorInvalidValue;
  const int units = p.B * p.H * (p.S / SDPA_BLOCK_Q);
  const int grid = units < num_sms ? units : num_sms;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(SDPA_THREADS);
  lc.dynamicSmemBytes = cfg.smem;
  lc.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  const int code = cfg.slots * 100 + cfg.nsb * 10 + cfg.stage_out;
  auto go = [&](auto kern) -> cudaError_t {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), cfg.smem);
    if (e != cudaSuccess) return e;
    return cudaLaunchKernelEx(&lc, kern, tmQ, tmK, tmV, tmO, p, cfg.slots, cfg.nsb, cfg.stage_out);
  };
  // the shapes the resident-K/V kernel takes, each with the configuration sdpa_cfg gives it: compile-time variants
#define GC_SDPA_CASE(I8, MF, S_, C_) \
  if (static_cast<bool>(p.is_int8) == I8 && static_cast<bool>(p.max_free) == MF && p.S == S_ && code == C_ && !p.P_out) \
    return go(sdpa_tc_kernel<I8, MF, S_, C_>);
  GC_SDPA_CASE(true, false, 128, 221)
  GC_SDPA_CASE(true, false, 256, 211)
  GC_SDPA_CASE(true, false, 384, 211)
  GC_SDPA_CASE(true, true, 128, 221)
  GC_SDPA_CASE(true, true, 256, 211)
  GC_SDPA_CASE(true, true, 384, 211)
  GC_SDPA_CASE(false, false, 128, 221)
  GC_SDPA_CASE(false, false, 256, 111)
  GC_SDPA_CASE(false, false, 384, 110)
#undef GC_SDPA_CASE
  if (p.is_int8 && p.max_free) return go(sdpa_tc_kernel<true, true>);
  if (p.is_int8) return go(sdpa_tc_kernel<true>);
  return go(sdpa_tc_kernel<false>);
}

}  // namespace gc
