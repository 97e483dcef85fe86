// tcgen05 GEMM on CTA pairs (cta_group::2) with the fused epilogue of kernels_gemm_tc.cu, for large problems:
//   D[M,N] = A[M,K] * Wt[N,K]^T  ->  post-ops  ->  store,
// for one layer or for two consecutive layers in ONE persistent launch.
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
//
// Two layers in one launch (the bf16 FFN: matmul + bias + GELU, matmul + bias) are the analogue of the paper's
// coarse-grain fusion for the large-batch case (Section V: consecutive fused ops merged so that the intermediate
// stays in cache and the per-op synchronisation disappears).  What one launch buys over two:
//   * no second ramp (set-up, first loads) and no tail in between (the last tiles' epilogues of the first matmul
//     overlap the first main loops of the second);
//   * a tile schedule over BOTH matmuls, built by the host: each cluster walks its own list of tiles;
//   * the hidden tensor is read back soon after it was written, while it is still in L2.
// Dependency: a tile of the second matmul reads 256 rows of the hidden tensor, which the n_tiles tiles of that
// row block of the first matmul write (TMA stores of 2 CTAs x 8 epilogue warps each).  Every epilogue warp, once its
// stores of a first-matmul tile have COMPLETED, adds one to that tile's counter in global memory (one releasing
// reduction: a release costs 1300-2000 clocks here, so there is exactly one per warp and tile, and for all tiles
// but the last first-matmul tile of a list it is deferred by one tile so that the wait for the stores is free).
// The producer warp of a second-matmul tile reads the counters of the row block's tiles (acquiring, one per lane)
// before it issues the loads of its A operand; for the tiles that are not complete yet it polls (bounded) right
// before the group of k-blocks that covers that tile's 256 hidden columns, so the tile runs right behind its
// producers.  The counters only grow; the value they reach in this launch follows from an epoch word kept on the
// device.  The schedule puts
// every first-matmul tile before every second-matmul tile in each cluster's list and all clusters are resident
// (one CTA per SM), so the waits cannot deadlock.  Without a schedule (one layer) the clusters take the tiles
// round robin.
#include <type_traits>

#include "gemm_epilogue.cuh"

namespace gc {

namespace {

constexpr int F2_BLOCK_M = 128;          // rows per CTA (256 per pair)
constexpr int F2_BLOCK_N = 256;
constexpr int F2_B_ROWS = 128;           // Wt rows each CTA loads
constexpr int F2_STAGES = 5;
constexpr int F2_STAGE_BYTES = (F2_BLOCK_M + F2_B_ROWS) * 128;
constexpr int F2_EPI_WARPS = 8;
constexpr int F2_THREADS = 64 + 32 * F2_EPI_WARPS + 32;   // producer, MMA issuer, epilogue warps, announcer
constexpr int F2_STAGING_BYTES = F2_EPI_WARPS * 4096;
constexpr int F2_BIAS_BYTES = F2_EPI_WARPS * F2_BLOCK_N * 4;
constexpr int F2_TMEM_COLS = 512;

size_t fused_smem_bytes() {
  return static_cast<size_t>(F2_STAGES) * F2_STAGE_BYTES + F2_STAGING_BYTES + F2_BIAS_BYTES + 1024 + 256;
}

__device__ __forceinline__ unsigned long long f2_ld_acquire(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

template <int KIND, int OUT>
__global__ void __launch_bounds__(F2_THREADS, 1) gemm_tc2_kernel(const __grid_constant__ GemmPairParams p) {
  constexpr int A_BYTES = F2_BLOCK_M * 128;
  constexpr int K_ELEMS = KIND == KIND_I8 ? 128 : (KIND == KIND_BF16 ? 64 : 32);
  constexpr int K_PER_TILE = F2_BLOCK_N / K_ELEMS;                // k-blocks of a second layer per first-layer tile
  constexpr int OUT_BYTES = out_bytes(OUT);
  constexpr int BOX_COLS = 128 / OUT_BYTES;
  constexpr int NUM_BOXES = F2_BLOCK_N / BOX_COLS;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* staging = smem + F2_STAGES * F2_STAGE_BYTES;
  float* bias_smem = reinterpret_cast<float*>(staging + F2_STAGING_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(staging + F2_STAGING_BYTES + F2_BIAS_BYTES);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * F2_STAGES + 6);
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_full = smem_u32(bars);                       // [STAGES]  (used in the leader)
  const uint32_t bar_empty = bar_full + 8 * F2_STAGES;            // [STAGES]
  const uint32_t bar_tfull = bar_empty + 8 * F2_STAGES;           // [2]
  const uint32_t bar_tempty = bar_tfull + 16;                     // [2]       (used in the leader)
  const uint32_t bar_ann = bar_tempty + 16;                       // [2]  stores of a first-layer tile completed (per CTA)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < F2_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_tfull + 8 * a, 1);
      mbar_init(bar_tempty + 8 * a, 2 * F2_EPI_WARPS);
      mbar_init(bar_ann + 8 * a, F2_EPI_WARPS);
    }
    fence_mbar_init();
    for (int i = 0; i < 6; ++i) tma_prefetch_desc(&p.tm[i]);
  }
  if (warp == 1) {
    tmem_alloc2(smem_u32(tmem_slot), F2_TMEM_COLS);
    tmem_relinquish2();
  }
  tc_fence_before();
  cluster_sync_all();                                             // both CTAs' barriers exist from here on
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");

  // this cluster's tile list: entries (layer << 24) | tile, terminated by a negative entry; without a list the
  // clusters take the tiles of the (single) layer round robin
  const int cluster_id = blockIdx.x >> 1, num_clusters = gridDim.x >> 1;
  const int* sched = p.sched ? p.sched + static_cast<int64_t>(cluster_id) * p.sched_pitch : nullptr;
  const int list_len = p.sched ? p.sched_pitch : (p.implicit_tiles + num_clusters - 1) / num_clusters;
  auto entry = [&](int i) -> int {
    if (sched) return __ldg(sched + i);
    const int t = cluster_id + i * num_clusters;
    return t < p.implicit_tiles ? t : -1;
  };
  // tile number -> (256-row block, 256-column tile).  Scheduled launches number the tiles row block by row block.
  // Without a schedule, row blocks are taken in groups of p.raster_rows and a group is walked column by column, so
  // that the clusters working at the same time share a few row blocks of A and a few column tiles of the weights
  // (both stay in L2) instead of sweeping the whole weight matrix once per round.
  auto decode = [&](int tile, int n_tiles, int& m_pair, int& n_blk) {
    if (sched || p.raster_rows <= 1) {
      m_pair = tile / n_tiles;
      n_blk = tile % n_tiles;
      return;
    }
    const int per_group = p.raster_rows * n_tiles;
    const int g = tile / per_group, r = tile - g * per_group;
    const int rows = min(p.raster_rows, p.m_pairs - g * p.raster_rows);   // the last group may be shorter
    n_blk = r / rows;
    m_pair = g * p.raster_rows + r - n_blk * rows;
  };
  bool failed = false;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    // Lane 0 issues the loads; the whole warp walks the tile list so that, for a second-layer tile, 32 lanes can read
    // the counters of the row block's first-layer tiles in one round trip.
    int stage = 0;
    uint32_t phase = 0;
    const uint32_t leader_full = leader ? bar_full : mapa_shared(bar_full, 0);
    // the value a tile's counter reaches in this launch: completed launches are counted on the device;
    // 2 = one announcement by each of the two CTAs
    const unsigned long long tile_target = p.ready ? (f2_ld_acquire(p.ready) + 1ULL) * 2ULL : 0ULL;
    for (int i = 0; i < list_len; ++i) {
      const int e = entry(i);
      if (e < 0) break;
      const int l = e >> 24, tile = e & 0xFFFFFF;
      const int n_tiles = p.L[l].n_tiles, nkb = p.L[l].num_k_blocks;
      int m_pair, n_blk;
      decode(tile, n_tiles, m_pair, n_blk);
      const int m_blk = m_pair * 2 + static_cast<int>(rank);
      // The 256 hidden rows a second-layer tile reads are written by the first-layer tiles of its row block, 256
      // hidden columns (K_PER_TILE k-blocks) each.  known: bit j set = tile j's stores have completed.
      uint32_t known = 0xFFFFFFFFu;
      const unsigned long long* tile_ready = nullptr;
      if (l == 1) {
        tile_ready = p.ready + 2 + static_cast<int64_t>(m_pair) * p.L[0].n_tiles;
        const bool ok = lane >= p.L[0].n_tiles || f2_ld_acquire(tile_ready + lane) >= tile_target;
        known = __ballot_sync(0xFFFFFFFFu, ok);
      }
      if (lane == 0) {
        if (l == 1) asm volatile("fence.proxy.async.global;" ::: "memory");   // acquire (generic) before the TMA loads (async proxy)
        const CUtensorMap* tmA = &p.tm[3 * l];
        const CUtensorMap* tmB = &p.tm[3 * l + 1];
        for (int kb = 0; kb < nkb; ++kb) {
          if (l == 1 && kb % K_PER_TILE == 0) {
            const int j = kb / K_PER_TILE;
            if (j < p.L[0].n_tiles && (j >= 32 || !((known >> j) & 1u))) {
              const uint64_t t0 = globaltimer_ns();
              uint32_t spins = 0;
              while (f2_ld_acquire(tile_ready + j) < tile_target) {
                if ((++spins & 255u) == 0 && globaltimer_ns() - t0 > 2000000000ull) {
                  report(p.status, DEV_TIMEOUT_PRODUCER);
                  failed = true;
                  break;
                }
              }
              if (failed) break;
              asm volatile("fence.proxy.async.global;" ::: "memory");
            }
          }
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1)) {
            report(p.status, DEV_TIMEOUT_PRODUCER);
            failed = true;
            break;
          }
          const uint32_t sA = smem_base + stage * F2_STAGE_BYTES, sB = sA + A_BYTES;
          if (leader) mbar_arrive_expect_tx(bar_full + 8 * stage, 2 * F2_STAGE_BYTES);   // both CTAs' bytes
          tma_load_2d_pair(sA, tmA, kb * K_ELEMS, m_blk * F2_BLOCK_M, leader_full + 8 * stage);
          tma_load_2d_pair(sB, tmB, kb * K_ELEMS, n_blk * F2_BLOCK_N + static_cast<int>(rank) * F2_B_ROWS,
                           leader_full + 8 * stage);
          if (++stage == F2_STAGES) {
            stage = 0;
            phase ^= 1;
          }
        }
      }
      failed = __shfl_sync(0xFFFFFFFFu, failed ? 1 : 0, 0) != 0;
      if (failed) break;
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (leader && lane == 0) {
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      for (int i = 0; i < list_len && !failed; ++i) {
        const int e = entry(i);
        if (e < 0) break;
        const int l = e >> 24;
        const int nkb = p.L[l].num_k_blocks;
        const uint32_t idesc = p.L[l].idesc;
        if (!mbar_wait(bar_tempty + 8 * acc, acc_phase ^ 1)) {
          report(p.status, DEV_TIMEOUT_MMA);
          failed = true;
          break;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * F2_BLOCK_N;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase)) {
            report(p.status, DEV_TIMEOUT_MMA);
            failed = true;
            break;
          }
          tc_fence_after();
          const uint32_t sA = smem_base + stage * F2_STAGE_BYTES, sB = sA + A_BYTES;
          const uint64_t a_desc = make_smem_desc(sA, 16, 1024, SWZ_128B);
          const uint64_t b_desc = make_smem_desc(sB, 16, 1024, SWZ_128B);
#pragma unroll
          for (int k = 0; k < 4; ++k)
            umma_ss2<KIND>(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit2(bar_empty + 8 * stage, 3);                // frees the stage in both CTAs
          if (++stage == F2_STAGES) {
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
  } else if (warp < 2 + F2_EPI_WARPS) {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int ew = warp - 2;
    const int q = warp & 3;
    const int half = ew >> 2;
    int acc = 0;
    uint32_t acc_phase = 0;
    uint8_t* my_stage = staging + ew * 4096;
    const uint32_t my_stage_u32 = smem_u32(my_stage);
    float* my_bias = bias_smem + ew * F2_BLOCK_N;
    const uint32_t row_off = (lane >> 3) * 1024 + (lane & 7) * 128;
    const uint32_t leader_tempty = leader ? bar_tempty : mapa_shared(bar_tempty, 0);
    // A first-layer tile is announced to the other clusters once the stores of all 8 epilogue warps have COMPLETED.
    // Each warp tells the announcer warp (an mbarrier arrival, cheap) when its own stores of the tile have; the
    // announcer then performs the one releasing reduction per CTA and tile (a release at GPU scope costs
    // 1300-2000 clocks here: far too much for the path of every epilogue warp).  Waiting for the stores right after
    // a tile would put their latency on that path too, so a tile that is followed by another first-layer tile is
    // reported at the end of that next tile, when all but the newest BOXES_PER_WARP bulk groups have long completed.
    // The last first-layer tile of the list is reported at once: what follows it may wait for other clusters.
    // Two barriers alternate: a warp is never two first-layer tiles ahead of another one at this point.
    constexpr int BOXES_PER_WARP = NUM_BOXES / 2;
    bool pending = false;
    int n_first = 0;                                               // first-layer tiles reported so far
    auto report_stores = [&]() {
      asm volatile("fence.proxy.async.global;" ::: "memory");
      mbar_arrive(bar_ann + 8 * (n_first & 1));
      ++n_first;
    };
    for (int i = 0; i < list_len; ++i) {
      const int e = entry(i);
      if (e < 0) break;
      const int l = e >> 24, tile = e & 0xFFFFFF;
      const int n_tiles = p.L[l].n_tiles, N = p.L[l].N;
      int m_pair, n_blk;
      decode(tile, n_tiles, m_pair, n_blk);
      const int m_blk = m_pair * 2 + static_cast<int>(rank);
      const CUtensorMap* tmD = &p.tm[3 * l + 2];
      // Copy this tile's bias slice into shared memory while the accumulator is still being produced: a
      // global load in the per-chunk loop would put its full latency on the critical path of every chunk.
      Epilogue epi = p.L[l].epi;
      if (epi.bias) {
        __syncwarp();
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int c = n_blk * F2_BLOCK_N + (lane + 32 * j) * 4;
          const float4 v = c < N ? __ldg(reinterpret_cast<const float4*>(epi.bias + c)) : make_float4(0.f, 0.f, 0.f, 0.f);
          reinterpret_cast<float4*>(my_bias)[lane + 32 * j] = v;
        }
        __syncwarp();
        epi.bias = my_bias - n_blk * F2_BLOCK_N;                   // indexed by absolute column below
      }
      if (!mbar_wait_prompt(bar_tfull + 8 * acc, acc_phase)) {
        report(p.status, DEV_TIMEOUT_EPILOGUE);
        failed = true;
        break;
      }
      tc_fence_after();
      const uint32_t t_row = tmem_base + acc * F2_BLOCK_N + (static_cast<uint32_t>(q * 32) << 16);
      for (int box = half; box < NUM_BOXES; box += 2) {
#pragma unroll 1
        for (int sub = 0; sub < BOX_COLS / 32; ++sub) {
          uint32_t r[32];
          tmem_ld32(t_row + box * BOX_COLS + sub * 32, r);
          tmem_wait_ld();
          constexpr int NW = 32 * OUT_BYTES / 4;
          uint32_t w[NW];
          epi_chunk32<KIND, OUT>(r, w, n_blk * F2_BLOCK_N + box * BOX_COLS + sub * 32, N, epi);
          if (sub == 0) {
            // the previous store out of this warp's staging buffer must have read it completely (checked only
            // now, with the first chunk's values already in registers)
            if (lane == 0) tma_store_wait_read<0>();
            __syncwarp();
          }
          const int c0 = sub * (NW / 4);
#pragma unroll
          for (int j = 0; j < NW / 4; ++j)
            *reinterpret_cast<uint4*>(my_stage + row_off + (((c0 + j) ^ (lane & 7)) * 16)) =
                make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_2d(tmD, n_blk * F2_BLOCK_N + box * BOX_COLS, m_blk * F2_BLOCK_M + q * 32, my_stage_u32);
          tma_store_commit();
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (pending) {
          tma_store_wait_all<BOXES_PER_WARP>();                   // everything but this tile's own stores
          report_stores();
          pending = false;
        }
        if (leader) mbar_arrive(bar_tempty + 8 * acc);
        else mbar_arrive_cluster_nomem(leader_tempty + 8 * acc);
        if (l == 0 && p.ready) {
          // my part of the hidden row block is in memory once my stores have completed (not merely been read)
          const int e2 = i + 1 < list_len ? entry(i + 1) : -1;
          if (e2 >= 0 && (e2 >> 24) == 0) {
            pending = true;
          } else {
            tma_store_wait_all<0>();
            report_stores();
          }
        }
      }
      acc ^= 1;
      if (acc == 0) acc_phase ^= 1;
    }
    if (lane == 0) tma_store_wait_read<0>();   // (reads of the staging buffers, not completion: the stores complete with the kernel)
  } else if (p.ready && lane == 0) {
    // ------------------------------------------------------------------ announcer (both CTAs)
    int n_first = 0;
    for (int i = 0; i < list_len; ++i) {
      const int e = entry(i);
      if (e < 0) break;
      if ((e >> 24) != 0) continue;
      if (!mbar_wait(bar_ann + 8 * (n_first & 1), (n_first >> 1) & 1)) {
        report(p.status, DEV_TIMEOUT_OTHER);
        break;
      }
      ++n_first;
      asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p.ready + 2 + (e & 0xFFFFFF)), "l"(1ULL) : "memory");
    }
  }

  // ---------------------------------------------------------------------- teardown
  __syncwarp();                                                   // single-lane roles: reconverge before the aligned barrier
  tc_fence_before();
  cluster_sync_all();                                             // the peer no longer reads this CTA's smem
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc2(tmem_base, F2_TMEM_COLS);
  }
  // the last CTA to get here closes the launch (see GemmPairParams::ready)
  if (p.ready && threadIdx.x == 0) {
    const unsigned long long prev = atomicAdd(p.ready + 1, 1ULL);
    if (prev + 1 == gridDim.x) {
      atomicExch(p.ready + 1, 0ULL);
      __threadfence();
      atomicAdd(p.ready, 1ULL);
    }
  }
  if (failed) {
    const uint64_t t0 = globaltimer_ns();
    while (globaltimer_ns() - t0 < 200000ull) {
    }
  }
}

template <int KIND, int OUT>
cudaError_t launch_fused_t(const GemmPairParams& p, int grid, bool pdl, cudaStream_t s) {
  const size_t smem = fused_smem_bytes();
  auto kern = gemm_tc2_kernel<KIND, OUT>;
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(kern), smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(F2_THREADS);
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
  return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace

size_t gemm_tc2_smem_bytes() { return fused_smem_bytes(); }

int gemm_tc2_max_clusters(int kind, int out_dtype) {
  const void* kern = nullptr;
  if (kind == KIND_BF16 && out_dtype == GC_BF16) kern = reinterpret_cast<const void*>(gemm_tc2_kernel<KIND_BF16, OUT_BF16>);
  else if (kind == KIND_I8 && (out_dtype == GC_U8 || out_dtype == GC_S8)) kern = reinterpret_cast<const void*>(gemm_tc2_kernel<KIND_I8, OUT_Q8>);
  else if (kind == KIND_TF32 && out_dtype == GC_F32) kern = reinterpret_cast<const void*>(gemm_tc2_kernel<KIND_TF32, OUT_F32>);
  if (!kern) return 0;
  const size_t smem = fused_smem_bytes();
  if (ensure_dynamic_smem(kern, smem) != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2);
  cfg.blockDim = dim3(F2_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) return 0;
  return n;
}

// kind: 0 = i8, 1 = bf16, 2 = tf32; both layers share the MMA kind and the output element type.
cudaError_t launch_gemm_tc2_fused(int kind, int a_signed, const GemmPairParams& p_in, int grid, cudaStream_t s) {
  GemmPairParams p = p_in;
  const int out_dtype = p.L[0].epi.out_dtype;
  for (int l = 0; l < 2; ++l) {
    p.L[l].idesc = kind == KIND_I8     ? make_idesc(ACC_S32, (l == 0 ? a_signed : (out_dtype == GC_S8)) ? FMT_S8 : FMT_U8, FMT_S8, 256, F2_BLOCK_N)
                   : kind == KIND_BF16 ? make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 256, F2_BLOCK_N)
                                       : make_idesc(ACC_F32, FMT_TF32, FMT_TF32, 256, F2_BLOCK_N);
  }
  if (kind == KIND_BF16 && out_dtype == GC_BF16) return launch_fused_t<KIND_BF16, OUT_BF16>(p, grid, true, s);
  if (kind == KIND_I8 && (out_dtype == GC_U8 || out_dtype == GC_S8)) return launch_fused_t<KIND_I8, OUT_Q8>(p, grid, true, s);
  if (kind == KIND_TF32 && out_dtype == GC_F32) return launch_fused_t<KIND_TF32, OUT_F32>(p, grid, true, s);
  return cudaErrorInvalidValue;
}

// One layer: the clusters take its tiles round robin (no schedule table, no counters).
cudaError_t launch_gemm_tc2(int kind, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB,
                            const CUtensorMap& tmD, const GemmTcParams& g, int grid, bool pdl, cudaStream_t s) {
  GemmPairParams p = {};
  p.L[0].N = g.N;
  p.L[0].num_k_blocks = g.num_k_blocks;
  p.L[0].n_tiles = g.n_tiles;
  p.L[0].epi = g.epi;
  p.implicit_tiles = ((g.m_tiles + 1) / 2) * g.n_tiles;
  p.m_pairs = (g.m_tiles + 1) / 2;
  p.raster_rows = 8;
  p.status = g.status;
  p.tm[0] = tmA;
  p.tm[1] = tmB;
  p.tm[2] = tmD;
  p.tm[3] = tmA;                                                  // unused; valid descriptors for the prefetch
  p.tm[4] = tmB;
  p.tm[5] = tmD;
  p.L[0].idesc = kind == KIND_I8     ? make_idesc(ACC_S32, a_signed ? FMT_S8 : FMT_U8, FMT_S8, 256, F2_BLOCK_N)
                 : kind == KIND_BF16 ? make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 256, F2_BLOCK_N)
                                     : make_idesc(ACC_F32, FMT_TF32, FMT_TF32, 256, F2_BLOCK_N);
  const Epilogue& e = g.epi;
  const int out = (e.acc_is_int && !e.has_dq) ? OUT_RAW32
                  : e.out_dtype == GC_F32    ? OUT_F32
                  : e.out_dtype == GC_BF16   ? OUT_BF16
                                             : OUT_Q8;
  auto dispatch = [&](auto kind_tag) -> cudaError_t {
    constexpr int K = decltype(kind_tag)::value;
    switch (out) {
      case OUT_F32: return launch_fused_t<K, OUT_F32>(p, grid, pdl, s);
      case OUT_BF16: return launch_fused_t<K, OUT_BF16>(p, grid, pdl, s);
      case OUT_Q8: return launch_fused_t<K, OUT_Q8>(p, grid, pdl, s);
      default:
        if constexpr (K == KIND_I8) return launch_fused_t<K, OUT_RAW32>(p, grid, pdl, s);
        return launch_fused_t<K, OUT_F32>(p, grid, pdl, s);
    }
  };
  if (kind == KIND_I8) return dispatch(std::integral_constant<int, KIND_I8>());
  if (kind == KIND_BF16) return dispatch(std::integral_constant<int, KIND_BF16>());
  if (kind == KIND_TF32) return dispatch(std::integral_constant<int, KIND_TF32>());
  return cudaErrorInvalidValue;
}

}  // namespace gc
