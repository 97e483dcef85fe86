// tcgen05 GEMM with a fused epilogue:  D[M,N] = A[M,K] * Wt[N,K]^T  ->  dequantize / bias / activation /
// requantize  ->  store.  One kernel serves every layer of the MLP chains (Sections III-V: the Tunable op
// with its post-ops fused at the innermost anchor).
//
// Structure (one persistent CTA per SM, 320 threads):
//   warp 0     TMA producer: 128-byte-swizzled [128 x 128B] A tiles and [BLOCK_N x 128B] Wt tiles into a
//              STAGES-deep shared-memory ring, completion on "full" mbarriers
//   warp 1     MMA issuer: one thread issues tcgen05.mma (kind::i8 / f16 / tf32) into one of two TMEM
//              accumulators; tcgen05.commit releases ring slots ("empty") and publishes accumulators
//   warps 2-9  epilogue: two warps per TMEM lane quarter, each taking alternate 128-byte-wide column
//              groups: tcgen05.ld (lane = row), post-ops in registers, swizzled staging in shared memory,
//              one TMA store per [32 rows x 128 B] box; then the accumulator is handed back, so the
//              epilogue of tile i overlaps the main loop of tile i+1
// K tails and M/N tails are zero-filled by TMA loads and clipped by TMA stores; every mbarrier wait is
// bounded (ptx.cuh).  Narrow tiles whose rows are shorter than 128 bytes are stored with plain vector
// stores instead of TMA.
#include <cuda_bf16.h>

#include "gemm_epilogue.cuh"

namespace gc {

constexpr int GEMM_BLOCK_M = 128;
constexpr int GEMM_TILE_K_BYTES = 128;   // one swizzle span: 128 i8 / 64 bf16 / 32 tf32 elements
constexpr int GEMM_EPI_WARPS = 8;
constexpr int GEMM_THREADS = 64 + 32 * GEMM_EPI_WARPS;
constexpr int GEMM_STAGING_BYTES = GEMM_EPI_WARPS * 4096;

__host__ __device__ constexpr int gemm_stage_bytes(int block_n) {
  return GEMM_BLOCK_M * GEMM_TILE_K_BYTES + block_n * GEMM_TILE_K_BYTES;
}
__host__ __device__ constexpr int gemm_stages(int block_n) {
  return block_n >= 256 ? 4 : (block_n >= 128 ? 5 : 8);
}

bool gemm_tc_supported_block_n(int bn) { return bn == 32 || bn == 64 || bn == 128 || bn == 256; }
size_t gemm_tc_smem_bytes(int bn) {
  return static_cast<size_t>(gemm_stages(bn)) * gemm_stage_bytes(bn) + GEMM_STAGING_BYTES + 1024 /*alignment slack*/ +
         256 /*barriers*/;
}
int gemm_tc_store_box_cols(int block_n, int out_elem_bytes) {
  return (block_n * out_elem_bytes) % 128 == 0 ? 128 / out_elem_bytes : 0;
}

template <int KIND, int BLOCK_N, int OUT>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmD, const GemmTcParams p) {
  constexpr int STAGES = gemm_stages(BLOCK_N);
  constexpr int STAGE_BYTES = gemm_stage_bytes(BLOCK_N);
  constexpr int A_BYTES = GEMM_BLOCK_M * GEMM_TILE_K_BYTES;
  constexpr int TMEM_COLS = 2 * BLOCK_N < 32 ? 32 : 2 * BLOCK_N;
  constexpr int K_ELEMS = KIND == KIND_I8 ? 128 : (KIND == KIND_BF16 ? 64 : 32);   // per 128-byte span
  constexpr int OUT_BYTES = out_bytes(OUT);
  constexpr bool TMA_STORE = (BLOCK_N * OUT_BYTES) % 128 == 0;
  constexpr int BOX_COLS = 128 / OUT_BYTES;                     // columns per 128-byte staging row
  constexpr int NUM_BOXES = TMA_STORE ? BLOCK_N / BOX_COLS : 0;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + GEMM_STAGING_BYTES);
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
      mbar_init(bar_tempty + 8 * a, GEMM_EPI_WARPS);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (TMA_STORE) tma_prefetch_desc(&tmD);
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
            umma_ss<KIND>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, p.idesc, (kb | k) != 0 ? 1u : 0u);
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
    const int ew = warp - 2;          // 0..7
    const int q = warp & 3;           // TMEM lane quarter this warp may access
    const int half = ew >> 2;         // which alternate column groups this warp takes
    int acc = 0;
    uint32_t acc_phase = 0;
    uint8_t* my_stage = staging + ew * 4096;
    const uint32_t my_stage_u32 = smem_u32(my_stage);
    const uint32_t row_off = (lane >> 3) * 1024 + (lane & 7) * 128;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m_blk = tile / p.n_tiles, n_blk = tile % p.n_tiles;
      if (!mbar_wait(bar_tfull + 8 * acc, acc_phase)) {
        report(p.status, DEV_TIMEOUT_EPILOGUE);
        failed = true;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + acc * BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
      if constexpr (TMA_STORE) {
        for (int box = half; box < NUM_BOXES; box += 2) {
          // the previous store out of this warp's staging buffer must have read it completely
          if (lane == 0) tma_store_wait_read<0>();
          __syncwarp();
#pragma unroll 1
          for (int sub = 0; sub < BOX_COLS / 32; ++sub) {
            uint32_t r[32];
            tmem_ld32(t_row + box * BOX_COLS + sub * 32, r);
            tmem_wait_ld();
            constexpr int NW = 32 * OUT_BYTES / 4;              // packed words for 32 columns
            uint32_t w[NW];
            epi_chunk32<KIND, OUT>(r, w, n_blk * BLOCK_N + box * BOX_COLS + sub * 32, p.N, p.epi);
            const int c0 = sub * (NW / 4);                      // first 16-byte chunk of this sub-block
#pragma unroll
            for (int i = 0; i < NW / 4; ++i)
              *reinterpret_cast<uint4*>(my_stage + row_off + (((c0 + i) ^ (lane & 7)) * 16)) =
                  make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmD, n_blk * BLOCK_N + box * BOX_COLS, m_blk * GEMM_BLOCK_M + q * 32, my_stage_u32);
            tma_store_commit();
          }
        }
      } else {
        // rows shorter than 128 bytes: 16-column groups stored straight from registers
        const int row = m_blk * GEMM_BLOCK_M + q * 32 + lane;
        char* dst_row = static_cast<char*>(p.out) + static_cast<int64_t>(row) * p.out_pitch * OUT_BYTES;
        for (int c = half; c < BLOCK_N / 32; c += 2) {
          uint32_t r[32];
          tmem_ld32(t_row + c * 32, r);
          tmem_wait_ld();
          const int n0 = n_blk * BLOCK_N + c * 32;
          if (row < p.M) {
            if (n0 < p.N) epi_store16(r, dst_row, n0, p.epi);
            if (n0 + 16 < p.N) epi_store16(r + 16, dst_row, n0 + 16, p.epi);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_tempty + 8 * acc);
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (TMA_STORE && lane == 0) tma_store_wait_read<0>();   // (reads of the staging buffers, not completion: the stores complete with the kernel)
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

template <int KIND, int BLOCK_N, int OUT>
static cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                              const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  const size_t smem = gemm_tc_smem_bytes(BLOCK_N);
  auto kern = gemm_tc_kernel<KIND, BLOCK_N, OUT>;
  static bool attr_set[64] = {};     // per instantiation and device
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
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
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmD, p);
}

template <int KIND, int OUT>
static cudaError_t launch_bn(int bn, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                             const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  switch (bn) {
    case 32: return launch_one<KIND, 32, OUT>(tmA, tmB, tmD, p, grid, pdl, s);
    case 64: return launch_one<KIND, 64, OUT>(tmA, tmB, tmD, p, grid, pdl, s);
    case 128: return launch_one<KIND, 128, OUT>(tmA, tmB, tmD, p, grid, pdl, s);
    case 256: return launch_one<KIND, 256, OUT>(tmA, tmB, tmD, p, grid, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

template <int KIND>
static cudaError_t launch_out(int out, int bn, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                              const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  switch (out) {
    case OUT_F32: return launch_bn<KIND, OUT_F32>(bn, tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_BF16: return launch_bn<KIND, OUT_BF16>(bn, tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_Q8: return launch_bn<KIND, OUT_Q8>(bn, tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_RAW32:
      if constexpr (KIND == KIND_I8) return launch_bn<KIND, OUT_RAW32>(bn, tmA, tmB, tmD, p, grid, pdl, s);
      return launch_bn<KIND, OUT_F32>(bn, tmA, tmB, tmD, p, grid, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gemm_tc(int kind, int block_n, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB,
                           const CUtensorMap& tmD, const GemmTcParams& p_in, int grid, bool pdl, cudaStream_t s) {
  GemmTcParams p = p_in;
  const Epilogue& e = p.epi;
  const int out = (e.acc_is_int && !e.has_dq) ? OUT_RAW32
                  : e.out_dtype == GC_F32    ? OUT_F32
                  : e.out_dtype == GC_BF16   ? OUT_BF16
                                             : OUT_Q8;
  if (kind == KIND_I8) {
    p.idesc = make_idesc(ACC_S32, a_signed ? FMT_S8 : FMT_U8, FMT_S8, GEMM_BLOCK_M, block_n);
    return launch_out<KIND_I8>(out, block_n, tmA, tmB, tmD, p, grid, pdl, s);
  }
  if (kind == KIND_BF16) {
    p.idesc = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, GEMM_BLOCK_M, block_n);
    return launch_out<KIND_BF16>(out, block_n, tmA, tmB, tmD, p, grid, pdl, s);
  }
  if (kind == KIND_TF32) {
    p.idesc = make_idesc(ACC_F32, FMT_TF32, FMT_TF32, GEMM_BLOCK_M, block_n);
    return launch_out<KIND_TF32>(out, block_n, tmA, tmB, tmD, p, grid, pdl, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace gc
