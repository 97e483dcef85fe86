// tcgen05 GEMM with a fused epilogue:  D[M,N] = A[M,K] * Wt[N,K]^T  ->  dequantize / bias / activation /
// requantize  ->  store.  One kernel serves every layer of the MLP chains (Sections III-V: the Tunable op
// with its post-ops fused at the innermost anchor).
//
// Structure (one persistent CTA per SM, 192 threads):
//   warp 0     TMA producer: 128-byte-swizzled [128 x 128B] A tiles and [BLOCK_N x 128B] Wt tiles into a
//              STAGES-deep shared-memory ring, completion on "full" mbarriers
//   warp 1     MMA issuer: one thread issues tcgen05.mma (kind::i8 / f16 / tf32) into one of two TMEM
//              accumulators; tcgen05.commit releases ring slots ("empty") and publishes accumulators
//   warps 2-5  epilogue: tcgen05.ld the accumulator (lane = row), apply the post-ops, store; then hand
//              the accumulator back, so the epilogue of tile i overlaps the main loop of tile i+1
// K tails and M/N tails are zero-filled by TMA; every mbarrier wait is bounded (ptx.cuh).
#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int GEMM_BLOCK_M = 128;
constexpr int GEMM_TILE_K_BYTES = 128;   // one swizzle span: 128 i8 / 64 bf16 / 32 tf32 elements
constexpr int GEMM_THREADS = 192;

__host__ __device__ constexpr int gemm_stages(int block_n) {
  return block_n >= 256 ? 4 : (block_n >= 128 ? 6 : 8);
}
__host__ __device__ constexpr int gemm_stage_bytes(int block_n) {
  return GEMM_BLOCK_M * GEMM_TILE_K_BYTES + block_n * GEMM_TILE_K_BYTES;
}

bool gemm_tc_supported_block_n(int bn) { return bn == 16 || bn == 32 || bn == 64 || bn == 128 || bn == 256; }
size_t gemm_tc_smem_bytes(int bn) {
  return static_cast<size_t>(gemm_stages(bn)) * gemm_stage_bytes(bn) + 1024 /*alignment slack*/ + 256 /*barriers*/;
}

template <int KIND, int BLOCK_N, bool A_SIGNED>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const GemmTcParams p) {
  constexpr int STAGES = gemm_stages(BLOCK_N);
  constexpr int STAGE_BYTES = gemm_stage_bytes(BLOCK_N);
  constexpr int A_BYTES = GEMM_BLOCK_M * GEMM_TILE_K_BYTES;
  constexpr int TMEM_COLS = 2 * BLOCK_N < 32 ? 32 : 2 * BLOCK_N;
  constexpr int K_ELEMS = KIND == KIND_I8 ? 128 : (KIND == KIND_BF16 ? 64 : 32);   // per 128-byte span
  constexpr uint32_t IDESC =
      KIND == KIND_I8   ? make_idesc(ACC_S32, A_SIGNED ? FMT_S8 : FMT_U8, FMT_S8, GEMM_BLOCK_M, BLOCK_N)
      : KIND == KIND_BF16 ? make_idesc(ACC_F32, FMT_BF16, FMT_BF16, GEMM_BLOCK_M, BLOCK_N)
                          : make_idesc(ACC_F32, FMT_TF32, FMT_TF32, GEMM_BLOCK_M, BLOCK_N);

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_u32(bars);                       // [STAGES]
  const uint32_t bar_empty = bar_full + 8 * STAGES;               // [STAGES]
  const uint32_t bar_tfull = bar_empty + 8 * STAGES;              // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                     // [2]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 4);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Programmatic dependent launch: the set-up above may overlap the previous layer's tail; from here on
  // this layer reads what the previous one wrote, so wait for it (no-op for an ordinary launch).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  const int num_tiles = p.m_tiles * p.n_tiles;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x) {
        const int m_blk = tile / p.n_tiles, n_blk = tile % p.n_tiles;
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1)) {
            report(p.status, DEV_TIMEOUT_PRODUCER);
            failed = true;
            break;
          }
          const uint32_t sA = smem_base + stage * STAGE_BYTES, sB = sA + A_BYTES;
          mbar_arrive_expect_tx(bar_full + 8 * stage, STAGE_BYTES);
          tma_load_2d(sA, &tmA, kb * K_ELEMS, m_blk * GEMM_BLOCK_M, bar_full + 8 * stage);
          tma_load_2d(sB, &tmB, kb * K_ELEMS, n_blk * BLOCK_N, bar_full + 8 * stage);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      for (int tile = blockIdx.x; tile < num_tiles && !failed; tile += gridDim.x) {
        if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1)) {
          report(p.status, DEV_TIMEOUT_MMA);
          failed = true;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * BLOCK_N;
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase)) {
            report(p.status, DEV_TIMEOUT_MMA);
            failed = true;
            break;
          }
          tc_fence_after();
          const uint32_t sA = smem_base + stage * STAGE_BYTES, sB = sA + A_BYTES;
          // K-major, 128B swizzle: 8-row groups are 1024 bytes apart; 32 bytes per MMA step along K.
          const uint64_t a_desc = make_smem_desc(sA, 16, 1024, SWZ_128B);
          const uint64_t b_desc = make_smem_desc(sB, 16, 1024, SWZ_128B);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss<KIND>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, IDESC, (kb | k) != 0 ? 1u : 0u);
          umma_commit(bar_empty + 8 * stage);
          if (++stage == STAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
        if (failed) break;
        umma_commit(bar_tfull + 8 * acc);
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int q = warp & 3;   // TMEM lane quarter this warp may access
    int acc = 0;
    uint32_t acc_phase = 0;
    const int out_elem = (p.epi.acc_is_int && !p.epi.has_dq) ? 4
                         : (p.epi.out_dtype == GC_F32 ? 4 : (p.epi.out_dtype == GC_BF16 ? 2 : 1));
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m_blk = tile / p.n_tiles, n_blk = tile % p.n_tiles;
      if (!mbar_wait(bar_tfull + 8 * acc, acc_phase)) {
        report(p.status, DEV_TIMEOUT_EPILOGUE);
        failed = true;
        break;
      }
      tc_fence_after();
      const int row = m_blk * GEMM_BLOCK_M + q * 32 + lane;
      char* dst_row = static_cast<char*>(p.out) + static_cast<int64_t>(row) * p.out_pitch * out_elem;
      const uint32_t t_row = tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
      if constexpr (BLOCK_N >= 32) {
#pragma unroll 1
        for (int c = 0; c < BLOCK_N / 32; ++c) {
          uint32_t r[32];
          tmem_ld32(t_row + c * 32, r);
          tmem_wait_ld();
          const int n0 = n_blk * BLOCK_N + c * 32;
          if (row < p.M) {
            if (n0 < p.N) epi_store16(r, dst_row, n0, p.epi);
            if (n0 + 16 < p.N) epi_store16(r + 16, dst_row, n0 + 16, p.epi);
          }
        }
      } else {
        uint32_t r[16];
        tmem_ld16(t_row, r);
        tmem_wait_ld();
        const int n0 = n_blk * BLOCK_N;
        if (row < p.M && n0 < p.N) epi_store16(r, dst_row, n0, p.epi);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (failed) {
    // an expired wait may leave bulk copies in flight: give them time to land before the CTA retires
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

template <int KIND, int BLOCK_N, bool A_SIGNED>
static cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmTcParams& p, int grid, bool pdl,
                              cudaStream_t s) {
  const size_t smem = gemm_tc_smem_bytes(BLOCK_N);
  auto kern = gemm_tc_kernel<KIND, BLOCK_N, A_SIGNED>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(GEMM_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = pdl ? 1 : 0;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, p);
}

template <int KIND, bool A_SIGNED>
static cudaError_t launch_bn(int bn, const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmTcParams& p, int grid,
                             bool pdl, cudaStream_t s) {
  switch (bn) {
    case 16: return launch_one<KIND, 16, A_SIGNED>(tmA, tmB, p, grid, pdl, s);
    case 32: return launch_one<KIND, 32, A_SIGNED>(tmA, tmB, p, grid, pdl, s);
    case 64: return launch_one<KIND, 64, A_SIGNED>(tmA, tmB, p, grid, pdl, s);
    case 128: return launch_one<KIND, 128, A_SIGNED>(tmA, tmB, p, grid, pdl, s);
    case 256: return launch_one<KIND, 256, A_SIGNED>(tmA, tmB, p, grid, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gemm_tc(int kind, int block_n, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB,
                           const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  if (kind == KIND_I8)
    return a_signed ? launch_bn<KIND_I8, true>(block_n, tmA, tmB, p, grid, pdl, s)
                    : launch_bn<KIND_I8, false>(block_n, tmA, tmB, p, grid, pdl, s);
  if (kind == KIND_BF16) return launch_bn<KIND_BF16, false>(block_n, tmA, tmB, p, grid, pdl, s);
  if (kind == KIND_TF32) return launch_bn<KIND_TF32, false>(block_n, tmA, tmB, p, grid, pdl, s);
  return cudaErrorInvalidValue;
}

}  // namespace gc
