// Fused scaled-dot-product attention on tcgen05 (Section VII "MHA": two batch matmuls with the softmax and
// the binary ops between them fused after the first one; the two matmul loop nests merged).
//
// One CTA (128 threads) handles one (batch, head, 128-query tile):
//   TMA: Q tile, all K rows, all V rows of the head -> swizzled shared memory (no multicast)
//   MMA 1: S = Q K^T, 128 x S accumulator kept whole in tensor memory (S <= 384 columns)
//   softmax: thread r owns query row r (TMEM lane r): scale + additive mask, row max, exp, row sum,
//            normalise - all in registers; bf16 path casts P to bf16, int8 path quantises P to u8
//   P goes to shared memory as the K-major A operand of MMA 2; V is consumed straight from its
//   [key][d] layout as an MN-major B operand, so nothing is transposed in memory
//   MMA 2: O = P V into 64 more TMEM columns; epilogue casts (bf16) or dequantizes/requantizes (int8).
// int8: Q and K have zero point 128; (u8 ^ 0x80) reinterpreted as s8 equals u8 - 128, so both are
// flipped in shared memory once and fed to an s8 x s8 MMA (exact s32).  V stays u8 and its zero point is
// removed from the accumulator with the row sum of P:  sum_j P_j (V_j - z) = sum_j P_j V_j - z sum_j P_j.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int SDPA_D = 64;
constexpr int SDPA_BLOCK_Q = 128;
constexpr float LOG2E = 1.4426950408889634f;

template <bool INT8>
struct SdpaSmem {
  static constexpr int ESZ = INT8 ? 1 : 2;
  static constexpr int ROW_BYTES = SDPA_D * ESZ;               // 64 (SW64) or 128 (SW128)
  static constexpr int P_BLOCK_KEYS = INT8 ? 128 : 64;         // keys per 128-byte span of P
  __host__ __device__ static constexpr int q_bytes() { return SDPA_BLOCK_Q * ROW_BYTES; }
  __host__ __device__ static constexpr int kv_bytes(int S) { return S * ROW_BYTES; }
  __host__ __device__ static constexpr int p_bytes(int S) { return (S / P_BLOCK_KEYS) * SDPA_BLOCK_Q * 128; }
  __host__ __device__ static constexpr int total(int S) {
    return q_bytes() + 2 * kv_bytes(S) + p_bytes(S) + S * 4 + 64;
  }
};

size_t sdpa_tc_smem_bytes(int S, int is_int8) {
  return 1024 + (is_int8 ? SdpaSmem<true>::total(S) : SdpaSmem<false>::total(S));
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

template <bool INT8>
__global__ void __launch_bounds__(128)
sdpa_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const SdpaParams p) {
  using L = SdpaSmem<INT8>;
  constexpr int ROW_BYTES = L::ROW_BYTES;
  constexpr uint32_t SWZ = INT8 ? SWZ_64B : SWZ_128B;
  constexpr uint32_t SBO = 8 * ROW_BYTES;                       // 8-row group stride: 512 or 1024 bytes

  const int S = p.S;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + L::q_bytes();
  uint8_t* sV = sK + L::kv_bytes(S);
  uint8_t* sP = sV + L::kv_bytes(S);
  float* sMask = reinterpret_cast<float*>(sP + L::p_bytes(S));
  uint64_t* bars = reinterpret_cast<uint64_t*>(sMask + S);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2);
  const uint32_t bar_load = smem_u32(bars), bar_mma = bar_load + 8;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int q_tiles = S / SDPA_BLOCK_Q;
  const int bh = blockIdx.x / q_tiles, qt = blockIdx.x % q_tiles;
  const int b = bh / p.H;
  const uint32_t tmem_cols = (S + SDPA_D) <= 256 ? 256u : 512u;

  if (tid == 0) {
    mbar_init(bar_load, 1);
    mbar_init(bar_mma, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 0) {
    tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (tid == 0) {
    mbar_arrive_expect_tx(bar_load, static_cast<uint32_t>(L::q_bytes() + 2 * L::kv_bytes(S)));
    tma_load_2d(smem_u32(sQ), &tmQ, 0, bh * S + qt * SDPA_BLOCK_Q, bar_load);
    for (int j = 0; j < S / 128; ++j) {
      tma_load_2d(smem_u32(sK) + j * 128 * ROW_BYTES, &tmK, 0, bh * S + j * 128, bar_load);
      tma_load_2d(smem_u32(sV) + j * 128 * ROW_BYTES, &tmV, 0, bh * S + j * 128, bar_load);
    }
  }
  for (int j = tid; j < S; j += 128) sMask[j] = p.mask ? p.mask[static_cast<int64_t>(b) * S + j] * LOG2E : 0.0f;

  bool ok = mbar_wait(bar_load, 0);
  if (!ok) report(p.status, DEV_TIMEOUT_PRODUCER);

  if (INT8 && ok) {
    // u8 with zero point 128 -> s8: flip the top bit of every byte (swizzling only permutes 16-byte chunks)
    if (!p.q_signed) {
      uint4* q4 = reinterpret_cast<uint4*>(sQ);
      for (int i = tid; i < L::q_bytes() / 16; i += 128) {
        uint4 v = q4[i];
        v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
        q4[i] = v;
      }
    }
    if (!p.k_signed) {
      uint4* k4 = reinterpret_cast<uint4*>(sK);
      for (int i = tid; i < L::kv_bytes(S) / 16; i += 128) {
        uint4 v = k4[i];
        v.x ^= 0x80808080u; v.y ^= 0x80808080u; v.z ^= 0x80808080u; v.w ^= 0x80808080u;
        k4[i] = v;
      }
    }
    fence_proxy_async_smem();
  }
  __syncthreads();

  // ---------------------------------------------------------------- MMA 1: S = Q K^T
  if (tid == 0 && ok) {
    tc_fence_after();
    constexpr int KSTEPS = ROW_BYTES / 32;                      // 4 (bf16) or 2 (int8) steps of 32 bytes
    for (int n0 = 0; n0 < S; n0 += 256) {
      const int nc = min(256, S - n0);
      const uint32_t idesc = INT8 ? make_idesc(ACC_S32, FMT_S8, FMT_S8, 128, nc)
                                  : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, nc);
      const uint64_t a_desc = make_smem_desc(smem_u32(sQ), 16, SBO, SWZ);
      const uint64_t b_desc = make_smem_desc(smem_u32(sK) + n0 * ROW_BYTES, 16, SBO, SWZ);
#pragma unroll
      for (int k = 0; k < KSTEPS; ++k)
        umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + n0, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0 ? 1u : 0u);
    }
    umma_commit(bar_mma);
  }
  if (ok) {
    ok = mbar_wait(bar_mma, 0);
    if (!ok) report(p.status, DEV_TIMEOUT_MMA);
  }
  tc_fence_after();

  // ---------------------------------------------------------------- softmax (thread = query row)
  const int r = tid;                                            // row within the tile = TMEM lane
  const uint32_t t_row = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
  const float c2 = (INT8 ? __fmul_rn(p.dq1, p.scalar) : p.scalar) * LOG2E;
  int p_rowsum = 0;
  if (ok) {
    float m = -INFINITY;
    for (int c = 0; c < S / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(t_row + c * 32, v);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float a = INT8 ? __int2float_rn(static_cast<int>(v[i])) : __uint_as_float(v[i]);
        m = fmaxf(m, fmaf(a, c2, sMask[c * 32 + i]));
      }
    }
    float l = 0.f;
    for (int c = 0; c < S / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(t_row + c * 32, v);
      tmem_wait_ld();
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float a = INT8 ? __int2float_rn(static_cast<int>(v[i])) : __uint_as_float(v[i]);
        l += ex2(fmaf(a, c2, sMask[c * 32 + i]) - m);
      }
    }
    const float rl = 1.0f / l;
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    for (int c = 0; c < S / 32; ++c) {
      uint32_t v[32];
      tmem_ld32(t_row + c * 32, v);
      tmem_wait_ld();
      float pr[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const float a = INT8 ? __int2float_rn(static_cast<int>(v[i])) : __uint_as_float(v[i]);
        pr[i] = ex2(fmaf(a, c2, sMask[c * 32 + i]) - m) * rl;
      }
      const int j0 = c * 32;
      if constexpr (INT8) {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int q0 = quantize_value(pr[4 * i + 0], p.inv_p, 0, 0, 255);
          const int q1 = quantize_value(pr[4 * i + 1], p.inv_p, 0, 0, 255);
          const int q2 = quantize_value(pr[4 * i + 2], p.inv_p, 0, 0, 255);
          const int q3 = quantize_value(pr[4 * i + 3], p.inv_p, 0, 0, 255);
          p_rowsum += q0 + q1 + q2 + q3;
          w[i] = q0 | (q1 << 8) | (q2 << 16) | (q3 << 24);
        }
        uint8_t* blk = sP + (j0 / 128) * (SDPA_BLOCK_Q * 128) + row_off;
        const int ci = (j0 % 128) / 16;
        *reinterpret_cast<uint4*>(blk + (((ci + 0) ^ (r & 7)) * 16)) = make_uint4(w[0], w[1], w[2], w[3]);
        *reinterpret_cast<uint4*>(blk + (((ci + 1) ^ (r & 7)) * 16)) = make_uint4(w[4], w[5], w[6], w[7]);
      } else {
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          __nv_bfloat162 h = __floats2bfloat162_rn(pr[2 * i], pr[2 * i + 1]);
          w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        uint8_t* blk = sP + (j0 / 64) * (SDPA_BLOCK_Q * 128) + row_off;
        const int ci = (j0 % 64) / 8;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4*>(blk + (((ci + i) ^ (r & 7)) * 16)) =
              make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
      }
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();

  // ---------------------------------------------------------------- MMA 2: O = P V
  if (tid == 0 && ok) {
    tc_fence_after();
    const uint32_t idesc = INT8 ? make_idesc(ACC_S32, FMT_U8, p.v_signed ? FMT_S8 : FMT_U8, 128, SDPA_D, 0, 1)
                                : make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, SDPA_D, 0, 1);
    constexpr int KEYS_PER_STEP = INT8 ? 32 : 16;
    const int steps = S / KEYS_PER_STEP;
    for (int ks = 0; ks < steps; ++ks) {
      // A: P, K-major, 128B swizzle: 4 steps of 32 bytes per 128-byte span, spans 16 KB apart
      const uint64_t a_desc =
          make_smem_desc(smem_u32(sP) + (ks >> 2) * (SDPA_BLOCK_Q * 128) + (ks & 3) * 32, 16, 1024, SWZ_128B);
      // B: V as stored [key][d] = MN-major: one key row per ROW_BYTES, 8-key groups SBO apart
      const uint64_t b_desc = make_smem_desc(smem_u32(sV) + ks * KEYS_PER_STEP * ROW_BYTES, SBO, SBO, SWZ);
      umma_ss<INT8 ? KIND_I8 : KIND_BF16>(tmem_base + S, a_desc, b_desc, idesc, ks != 0 ? 1u : 0u);
    }
    umma_commit(bar_mma);
  }
  if (ok) {
    ok = mbar_wait(bar_mma, 1);
    if (!ok) report(p.status, DEV_TIMEOUT_MMA);
  }
  tc_fence_after();

  // ---------------------------------------------------------------- epilogue
  if (ok) {
    const int64_t grow = static_cast<int64_t>(bh) * S + qt * SDPA_BLOCK_Q + r;
#pragma unroll 1
    for (int c = 0; c < 2; ++c) {
      uint32_t v[32];
      tmem_ld32(t_row + S + c * 32, v);
      tmem_wait_ld();
      if constexpr (INT8) {
        const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
        const int corr = p.zp_v * p_rowsum;
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
        uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(p.O) + grow * SDPA_D + c * 32);
        dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
        dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
      } else {
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
          w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        uint4* dst = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.O) + grow * SDPA_D + c * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) dst[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
  if (!ok) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

cudaError_t launch_sdpa_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                           cudaStream_t s) {
  const size_t smem = sdpa_tc_smem_bytes(p.S, p.is_int8);
  const int grid = p.B * p.H * (p.S / SDPA_BLOCK_Q);
  cudaError_t e;
  if (p.is_int8) {
    e = cudaFuncSetAttribute(sdpa_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    sdpa_tc_kernel<true><<<grid, 128, smem, s>>>(tmQ, tmK, tmV, p);
  } else {
    e = cudaFuncSetAttribute(sdpa_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    sdpa_tc_kernel<false><<<grid, 128, smem, s>>>(tmQ, tmK, tmV, p);
  }
  return cudaGetLastError();
}

}  // namespace gc
