// tcgen05 GEMM on CTA pairs (cta_group::2) with the same fused epilogue as kernels_gemm_tc.cu, for large
// problems:  D[M,N] = A[M,K] * Wt[N,K]^T  ->  post-ops  ->  store.
//
// A cluster of two CTAs (two SMs) owns a 256 x 256 output tile.  Each CTA loads its own 128 rows of A and its
// own 128 of the tile's 256 Wt rows per k-block (32 KB instead of the 48 KB a lone CTA needs for a 128 x 256
// tile, which is what lifts the operand-fetch bound of the one-CTA kernel), the leader CTA issues one
// tcgen05.mma.cta_group::2 (M = 256, N = 256) that reads both CTAs' shared memory, and each CTA ends up with
// its own 128 x 256 accumulator in its own tensor memory, which its own epilogue warps drain.
//
// Barrier protocol (every wait bounded, see ptx.cuh):
//   full[s]    in the leader; both CTAs' TMA loads count their bytes on it (plain loads, no multicast)
//   empty[s]   in each CTA; the leader's tcgen05.commit signals both (commit multicast is a signal, not a load)
//   tfull[a]   in each CTA; commit-signalled by the leader when a tile's accumulator is complete
//   tempty[a]  in the leader; the epilogue warps of both CTAs arrive on it (peer: remote arrive)
// Cluster-wide barriers bracket the kernel so that neither CTA touches the other's barriers before they are
// initialised nor retires while its peer can still read its shared memory.
#include "gemm_epilogue.cuh"

namespace gc {

constexpr int G2_BLOCK_M = 128;          // rows per CTA (256 per pair)
constexpr int G2_BLOCK_N = 256;
constexpr int G2_B_ROWS = 128;           // Wt rows each CTA loads
constexpr int G2_STAGES = 5;
constexpr int G2_STAGE_BYTES = (G2_BLOCK_M + G2_B_ROWS) * 128;
constexpr int G2_EPI_WARPS = 8;
constexpr int G2_THREADS = 64 + 32 * G2_EPI_WARPS;
constexpr int G2_STAGING_BYTES = G2_EPI_WARPS * 4096;       // one [32 rows x 128 B] box per epilogue warp
constexpr int G2_BIAS_BYTES = G2_EPI_WARPS * G2_BLOCK_N * 4;  // per epilogue warp: the tile's 256 bias values
constexpr int G2_TMEM_COLS = 512;

size_t gemm_tc2_smem_bytes() {
  return static_cast<size_t>(G2_STAGES) * G2_STAGE_BYTES + G2_STAGING_BYTES + G2_BIAS_BYTES + 1024 + 256;
}

template <int KIND, int OUT>
__global__ void __launch_bounds__(G2_THREADS, 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmD, const GemmTcParams p) {
  constexpr int A_BYTES = G2_BLOCK_M * 128;
  constexpr int K_ELEMS = KIND == KIND_I8 ? 128 : (KIND == KIND_BF16 ? 64 : 32);
  constexpr int OUT_BYTES = out_bytes(OUT);
  constexpr int BOX_COLS = 128 / OUT_BYTES;
  constexpr int NUM_BOXES = G2_BLOCK_N / BOX_COLS;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + G2_STAGES * G2_STAGE_BYTES;
  float* bias_smem = reinterpret_cast<float*>(staging + G2_STAGING_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + G2_STAGING_BYTES + G2_BIAS_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * G2_STAGES + 4);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_u32(bars);                       // [STAGES]  (used in the leader)
  const uint32_t bar_empty = bar_full + 8 * G2_STAGES;            // [STAGES]
  const uint32_t bar_tfull = bar_empty + 8 * G2_STAGES;           // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                     // [2]       (used in the leader)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < G2_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 2 * G2_EPI_WARPS);
    }
    fence_mbar_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    tma_prefetch_desc(&tmD);
  }
  if (warp == 1) {
    tmem_alloc2(smem_u32(tmem_slot), G2_TMEM_COLS);
    tmem_relinquish2();
  }
  tc_fence_before();
  cluster_sync_all();                                             // both CTAs' barriers exist from here on
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // pair tiles: m_pairs x n_tiles; this CTA handles 128-row block 2 * m_pair + rank
  const int m_pairs = (p.m_tiles + 1) / 2;
  const int num_tiles = m_pairs * p.n_tiles;
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t leader_full = leader ? bar_full : mapa_shared(bar_full, 0);
      for (int tile = cluster_id; tile < num_tiles && !failed; tile += num_clusters) {
        const int m_blk = (tile / p.n_tiles) * 2 + static_cast<int>(rank), n_blk = tile % p.n_tiles;
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1)) {
            report(p.status, DEV_TIMEOUT_PRODUCER);
            failed = true;
            break;
          }
          const uint32_t sA = smem_base + stage * G2_STAGE_BYTES, sB = sA + A_BYTES;
          if (leader) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * G2_STAGE_BYTES);   // both CTAs' bytes
          tma_load_2d_pair(sA, &tmA, kb * K_ELEMS, m_blk * G2_BLOCK_M, leader_full + 8 * stage);
          tma_load_2d_pair(sB, &tmB, kb * K_ELEMS, n_blk * G2_BLOCK_N + static_cast<int>(rank) * G2_B_ROWS,
                           leader_full + 8 * stage);
          if (++stage == G2_STAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (leader && lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      for (int tile = cluster_id; tile < num_tiles && !failed; tile += num_clusters) {
        if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1)) {
          report(p.status, DEV_TIMEOUT_MMA);
          failed = true;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * G2_BLOCK_N;
        for (int kb = 0; kb < p.num_k_blocks; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase)) {
            report(p.status, DEV_TIMEOUT_MMA);
            failed = true;
            break;
          }
          tc_fence_after();
          const uint32_t sA = smem_base + stage * G2_STAGE_BYTES, sB = sA + A_BYTES;
          const uint64_t a_desc = make_smem_desc(sA, 16, 1024, SWZ_128B);
          const uint64_t b_desc = make_smem_desc(sB, 16, 1024, SWZ_128B);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss2<KIND>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, p.idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit2(bar_empty + 8 * stage, 3);                // frees the stage in both CTAs
          if (++stage == G2_STAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
        if (failed) break;
        umma_commit2(bar_tfull + 8 * acc, 3);                    // accumulators of both CTAs are complete
        acc ^= 1;
        if (acc == 0) acc_phase ^= 1;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint8_t* my_stage = staging + ew * 4096;
    const uint32_t my_stage_u32 = smem_u32(my_stage);
    float* my_bias = bias_smem + ew * G2_BLOCK_N;
    const uint32_t row_off = (lane >> 3) * 1024 + (lane & 7) * 128;
    const uint32_t leader_tempty = leader ? bar_tempty : mapa_shared(bar_tempty, 0);
    for (int tile = cluster_id; tile < num_tiles; tile += num_clusters) {
      const int m_blk = (tile / p.n_tiles) * 2 + static_cast<int>(rank), n_blk = tile % p.n_tiles;
      // Copy this tile's bias slice into shared memory while the accumulator is still being produced: a
      // global load in the per-chunk loop would put its full latency on the critical path of every chunk.
      Epilogue epi = p.epi;
      if (p.epi.bias) {
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const int c = n_blk * G2_BLOCK_N + (lane + 32 * i) * 4;
          const float4 v = c < p.N ? __ldg(reinterpret_cast<const float4*>(p.epi.bias + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
          reinterpret_cast<float4*>(my_bias)[lane + 32 * i] = v;
        }
        __syncwarp();
        epi.bias = my_bias - n_blk * G2_BLOCK_N;                   // indexed by absolute column below
      }
      if (!mbar_wait(bar_tfull + 8 * acc, acc_phase)) {
        report(p.status, DEV_TIMEOUT_EPILOGUE);
        failed = true;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + acc * G2_BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
      for (int box = half; box < NUM_BOXES; box += 2) {
        // the previous store out of this warp's staging buffer must have read it completely
        if (lane == 0) tma_store_wait_read<0>();
        __syncwarp();
#pragma unroll 1
        for (int sub = 0; sub < BOX_COLS / 32; ++sub) {
          uint32_t r[32];
          tmem_ld32(t_row + box * BOX_COLS + sub * 32, r);
          tmem_wait_ld();
          constexpr int NW = 32 * OUT_BYTES / 4;
          uint32_t w[NW];
          epi_chunk32<KIND, OUT>(r, w, n_blk * G2_BLOCK_N + box * BOX_COLS + sub * 32, p.N, epi);
          const int c0 = sub * (NW / 4);
#pragma unroll
          for (int i = 0; i < NW / 4; ++i)
            *reinterpret_cast<uint4*>(my_stage + row_off + (((c0 + i) ^ (lane & 7)) * 16)) =
                make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(&tmD, n_blk * G2_BLOCK_N + box * BOX_COLS, m_blk * G2_BLOCK_M + q * 32, my_stage_u32);
          tma_store_commit();
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (leader) mbar_arrive(bar_tempty + 8 * acc);
        else mbar_arrive_cluster(leader_tempty + 8 * acc);
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) tma_store_wait_all<0>();
  }

  // ---------------------------------------------------------------------- teardown
  tc_fence_before();
  cluster_sync_all();                                             // the peer no longer reads this CTA's smem
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, G2_TMEM_COLS);
  }
  if (failed) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

template <int KIND, int OUT>
static cudaError_t launch_one2(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                               const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  const size_t smem = gemm_tc2_smem_bytes();
  auto kern = gemm_tc2_kernel<KIND, OUT>;
  static bool attr_set[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(G2_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmD, p);
}

template <int KIND>
static cudaError_t launch_out2(int out, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                               const GemmTcParams& p, int grid, bool pdl, cudaStream_t s) {
  switch (out) {
    case OUT_F32: return launch_one2<KIND, OUT_F32>(tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_BF16: return launch_one2<KIND, OUT_BF16>(tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_Q8: return launch_one2<KIND, OUT_Q8>(tmA, tmB, tmD, p, grid, pdl, s);
    case OUT_RAW32:
      if constexpr (KIND == KIND_I8) return launch_one2<KIND, OUT_RAW32>(tmA, tmB, tmD, p, grid, pdl, s);
      return launch_one2<KIND, OUT_F32>(tmA, tmB, tmD, p, grid, pdl, s);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_gemm_tc2(int kind, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB,
                            const CUtensorMap& tmD, const GemmTcParams& p_in, int grid, bool pdl, cudaStream_t s) {
  GemmTcParams p = p_in;
  const Epilogue& e = p.epi;
  const int out = (e.acc_is_int && !e.has_dq) ? OUT_RAW32
                  : e.out_dtype == GC_F32    ? OUT_F32
                  : e.out_dtype == GC_BF16   ? OUT_BF16
                                             : OUT_Q8;
  if (kind == KIND_I8) {
    p.idesc = make_idesc(ACC_S32, a_signed ? FMT_S8 : FMT_U8, FMT_S8, 256, G2_BLOCK_N);
    return launch_out2<KIND_I8>(out, tmA, tmB, tmD, p, grid, pdl, s);
  }
  if (kind == KIND_BF16) {
    p.idesc = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 256, G2_BLOCK_N);
    return launch_out2<KIND_BF16>(out, tmA, tmB, tmD, p, grid, pdl, s);
  }
  if (kind == KIND_TF32) {
    p.idesc = make_idesc(ACC_F32, FMT_TF32, FMT_TF32, 256, G2_BLOCK_N);
    return launch_out2<KIND_TF32>(out, tmA, tmB, tmD, p, grid, pdl, s);
  }
  return cudaErrorInvalidValue;
}

}  // namespace gc
