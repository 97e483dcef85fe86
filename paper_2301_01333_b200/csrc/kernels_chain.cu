// One persistent kernel for a whole small-batch MLP chain (the analogue of the paper's coarse-grain fusion,
// Section V: the outer loops of consecutive fused ops merged so that activations stay in the fastest cache
// and the per-op synchronisation overhead disappears; Section VII: 2.0x on the int8 MLP-1).
//
// Shape of the problem: M <= 512 rows (up to four independent 128-row MMA tiles), L layers with N_l output columns.  CTA c owns
// output columns [32 c, 32 c + 32) of every tensor-core layer that has that many columns:
//   * at kernel start it TMA-loads its 32-row slice of EVERY layer's prepacked weight into shared memory
//     (HBM latency is paid once, not once per layer);
//   * per layer it fetches the layer's A operand (the previous activation, L2-resident) with as many
//     k-blocks in flight as shared memory allows - normally all of them, so the L2 latency is paid once per
//     layer -, issues tcgen05.mma into a 32-column TMEM accumulator, applies the post-ops and stores its
//     32 columns of the next activation.  A stage holds only round_up(M, 8) rows; the MMA still reads 128
//     rows, the surplus rows come from whatever follows in shared memory and only feed accumulator rows
//     that are never stored (rows of a matmul are independent);
//   * the reduction axis of every layer is split over the KS CTAs of a thread-block cluster (KS = 1, 2 or 4): each
//     CTA loads, holds and multiplies only its share of the k-blocks, which divides the serial chain of MMAs
//     (about 120 clocks each however narrow the tile) and the A-operand traffic per CTA by KS.  The partial
//     accumulators meet in distributed shared memory: every CTA of the cluster finishes 128 / KS rows, so warp q
//     sends its 32 rows to the CTA that owns them and signals that CTA's mbarrier; the owner adds the KS partials
//     in a fixed order (exact for s32, deterministic for fp32), applies the post-ops and stores;
//   * a grid-wide barrier (epoch-counted atomic in global memory, bounded spin) separates the layers;
//   * layers the tensor-core path does not take (N not a multiple of 16) run on CUDA cores inside the same kernel,
//     one warp per output - except the one-column last layer of an 8-bit chain (the 256 -> 1 tail of a recommender's
//     top MLP), which is folded into the finishing step of the layer before it: the finishing threads add their part
//     of the dot product per row with a global atomic instead of storing the row, and whoever counts a row last
//     applies the last layer's post-ops; that takes a grid barrier and a layer out of the chain;
//   * an input whose row pitch TMA cannot address (the graph-entry reorder, Section V: pre-op fusion "only at the
//     entry point of the graph") is read with plain loads by the four epilogue warps, which are idle at that point,
//     realigned in registers and written straight into the swizzled A-operand stages of the first layer.
// At most one CTA per SM, and the host checks that all clusters of the grid can be resident together.
// The code between the waits runs once per launch in warps that are alone on their schedulers, where a branch costs
// about 30 clocks and an integer division a hundred: hence the shifts by log2(KS), the selects instead of per-part
// and per-chunk tests, and the finishing step spread over all 128 epilogue threads.
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int CH_THREADS = 192;          // warp 0 producer, warp 1 MMA, warps 2-5 epilogue
constexpr int CH_MAX_STAGES = 32;
constexpr int CH_BLOCK_N = 32;
// One 32-column accumulator.  Dealing the four k-steps of a k-block onto four independent accumulators was tried and
// kept for a while: it takes the MMAs from about 130 to about 118 clocks each, but the epilogue then reads four times
// the tensor memory and adds it up, which costs a lone warp more than the MMAs gain (config 2: 21.06 us with four
// accumulators, 20.42 us with one).
constexpr int CH_NACC = 1;
constexpr int CH_RED_BYTES = 128 * 32 * 4;   // partial-sum exchange buffer: 128 rows x 32 columns x 4 bytes

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}

// Grid-wide barrier: every CTA adds one to a counter that only grows; the caller passes the value the
// counter reaches when all CTAs of this launch have arrived at this barrier.  Bounded: gives up after 2 s.
// `on_release` runs in thread 0 as soon as the barrier opens, before the CTA's other threads are released: the
// place to issue the loads that only waited for the other CTAs' stores.
template <typename F>
__device__ __forceinline__ bool grid_barrier(unsigned long long* ctr, unsigned long long target, F on_release) {
  __syncthreads();
  int ok = 1;
  if (threadIdx.x == 0) {
    // generic-proxy stores of this CTA (made CTA-visible by the barrier above) must be visible to the other CTAs'
    // TMA loads: proxy fence on the global space, then a releasing reduction (no return value to wait for)
    asm volatile("fence.proxy.async.global;" ::: "memory");
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(ctr), "l"(1ULL) : "memory");
    uint64_t t0 = 0;
    uint32_t i = 0;
    while (ld_acquire_u64(ctr) < target) {
      if ((++i & 1023u) == 0) {
        const uint64_t t = globaltimer_ns();
        if (t0 == 0) t0 = t;
        else if (t - t0 > 2000000000ull) {
          ok = 0;
          break;
        }
      }
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");
    if (ok) on_release();
  }
  return __syncthreads_and(ok) != 0;
}

__device__ __forceinline__ float ch_load_f(const void* p, int64_t i, int dtype) {
  if (dtype == GC_F32) return static_cast<const float*>(p)[i];
  return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[i]);
}
__device__ __forceinline__ int ch_load_i(const void* p, int64_t i, int dtype) {
  if (dtype == GC_U8) return static_cast<const uint8_t*>(p)[i];
  return static_cast<const int8_t*>(p)[i];
}

// One finishing thread: add the KS partial sums of NC consecutive columns of one row (column group `cgrp` of the 32
// the CTA owns) and store them with the post-ops applied.  All four possible parts are loaded (what lies behind the
// buffer for KS < 4 is shared memory of this CTA) and a select drops the surplus ones: no branch per part - a lone
// warp pays about 30 clocks for each.  Fixed order: exact for s32, deterministic for fp32.
template <int KIND, int NC>
__device__ __forceinline__ void chain_finish(const uint8_t* sRed, int rows_per, int KS, int frow, int cgrp, void* dst_row,
                                             int fcol, const Epilogue& epi, const EpiColsT<NC>& fk) {
  uint32_t a[NC];
#pragma unroll
  for (int i = 0; i < NC; ++i) a[i] = 0u;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const uint8_t* src = sRed + (s * rows_per + frow) * 128;
    const bool use = s < KS;
#pragma unroll
    for (int c = 0; c < NC / 4; ++c) {
      const uint4 v = *reinterpret_cast<const uint4*>(src + (((cgrp * (NC / 4) + c) ^ (frow & 7)) << 4));
      if constexpr (KIND == KIND_I8) {
        a[4 * c] += use ? v.x : 0u; a[4 * c + 1] += use ? v.y : 0u;
        a[4 * c + 2] += use ? v.z : 0u; a[4 * c + 3] += use ? v.w : 0u;
      } else {
        a[4 * c] = __float_as_uint(__uint_as_float(a[4 * c]) + (use ? __uint_as_float(v.x) : 0.f));
        a[4 * c + 1] = __float_as_uint(__uint_as_float(a[4 * c + 1]) + (use ? __uint_as_float(v.y) : 0.f));
        a[4 * c + 2] = __float_as_uint(__uint_as_float(a[4 * c + 2]) + (use ? __uint_as_float(v.z) : 0.f));
        a[4 * c + 3] = __float_as_uint(__uint_as_float(a[4 * c + 3]) + (use ? __uint_as_float(v.w) : 0.f));
      }
    }
  }
  epi_store_cols<NC>(a, dst_row, fcol, epi, fk);
}

// The same for the layer before a folded one-column last layer: the NC finished values are quantised as they would
// have been stored, and what leaves is their part of the last layer's dot product, sum (code - zero point) x weight.
template <int KIND, int NC>
__device__ __forceinline__ int chain_finish_dot(const uint8_t* sRed, int rows_per, int KS, int frow, int cgrp, const Epilogue& epi,
                                                const EpiColsT<NC>& fk, const int (&wt)[NC], int a_zp) {
  uint32_t a[NC];
#pragma unroll
  for (int i = 0; i < NC; ++i) a[i] = 0u;
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const uint8_t* src = sRed + (s * rows_per + frow) * 128;
    const bool use = s < KS;
#pragma unroll
    for (int c = 0; c < NC / 4; ++c) {
      const uint4 v = *reinterpret_cast<const uint4*>(src + (((cgrp * (NC / 4) + c) ^ (frow & 7)) << 4));
      a[4 * c] += use ? v.x : 0u; a[4 * c + 1] += use ? v.y : 0u;
      a[4 * c + 2] += use ? v.z : 0u; a[4 * c + 3] += use ? v.w : 0u;
    }
  }
  float t[NC];
  epi_values<NC>(a, t, epi, fk);
  const int lo = epi.out_dtype == GC_U8 ? 0 : -128, hi = epi.out_dtype == GC_U8 ? 255 : 127;
  int d = 0;
#pragma unroll
  for (int i = 0; i < NC; ++i) d += (quantize_value(t[i], epi.inv, epi.zp, lo, hi) - a_zp) * wt[i];
  return d;
}

template <int KIND>
__global__ void __launch_bounds__(CH_THREADS, 1) mlp_chain_kernel(const __grid_constant__ ChainParams p) {
  constexpr int K_ELEMS = KIND == KIND_I8 ? 128 : (KIND == KIND_BF16 ? 64 : 32);
  constexpr int ESZ = KIND == KIND_I8 ? 1 : (KIND == KIND_BF16 ? 2 : 4);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int CH_STAGES = p.a_stages;
  const int CH_A_STAGE_BYTES = p.a_stage_bytes;
  const int KS = p.ks;                                            // CTAs per cluster = parts of the reduction axis
  // (1, 2 or 4: shifts and masks instead of divisions, which cost a lone thread a hundred clocks each on the way from
  // one layer to the next)
  const int KS_SH = __ffs(KS) - 1;
  uint8_t* sA = smem;                                             // a_stages x a_stage_bytes
  // the weight slices (padded to at least 16 KB) follow the ring, so the 128-row MMA reads of the last stages
  // stay inside this CTA's shared memory
  uint8_t* sW = sA + ((CH_STAGES * CH_A_STAGE_BYTES + 1023) & ~1023);
  // partial sums from the cluster: [KS sources][128 / KS rows][32 columns] s32 / fp32, 16-byte chunks XOR-swizzled
  uint8_t* sRed = sW + (p.w_smem_bytes < 16384u ? 16384u : p.w_smem_bytes);
  uint8_t* sSend = sRed + CH_RED_BYTES;                           // my own partial sums, staged for the bulk copies
  // (neither buffer exists when the reduction axis is not split)
  uint64_t* bars = reinterpret_cast<uint64_t*>(sRed + (KS > 1 ? 2 * CH_RED_BYTES : 0));
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * CH_MAX_STAGES + 3 + CHAIN_MAX_LAYERS);
  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * CH_MAX_STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * CH_MAX_STAGES;       // [1]
  const uint32_t bar_red = bar_tfull + 8;                         // [1] partials of the cluster have arrived
  const uint32_t bar_a0 = bar_red + 8;                            // [1] first layer's A operand written by the epilogue warps
  const uint32_t bar_wfull = bar_a0 + 8;                          // [CHAIN_MAX_LAYERS]
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int ksr = KS > 1 ? static_cast<int>(cluster_ctarank()) : 0;   // my part of the reduction axis
  // CTA index -> (row tile, 32-column slice, part of the reduction axis): batches above 128 rows are cut into row
  // tiles that run as independent CTAs (rows of a matmul are independent); only the grid barrier joins them
  const int cta = static_cast<int>(blockIdx.x >> KS_SH) % p.slices;   // my 32-column slice
  const int row0 = static_cast<int>(blockIdx.x >> KS_SH) / p.slices * 128;   // first row of my row tile

  if (threadIdx.x == 0) {
    for (int s = 0; s < CH_STAGES; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_a0, 4);                                         // one arrival per epilogue warp
    mbar_init(bar_red, 1);                                        // armed per layer with the bytes the cluster will send
    for (int l = 0; l < CHAIN_MAX_LAYERS; ++l) mbar_init(bar_wfull + 8 * l, 1);
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), CH_NACC * CH_BLOCK_N);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // nobody may signal a barrier of another CTA before that CTA has initialised it
  if (KS > 1) cluster_sync_all();

  // Programmatic dependent launch: everything above may overlap the tail of the preceding kernel on the stream.
  // The prepacked weights are constants; unless this very call has just enqueued their prepack, their loads may
  // start before the preceding kernel has finished, too.  Everything else waits for it.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!p.early_weights) asm volatile("griddepcontrol.wait;" ::: "memory");

  // my k-blocks of layer L: [kb_lo, kb_hi)
  auto kb_lo = [&](const ChainLayer& L) { return (ksr * L.nkb) >> KS_SH; };
  auto kb_hi = [&](const ChainLayer& L) { return ((ksr + 1) * L.nkb) >> KS_SH; };

  // every layer's weight slice starts moving now (constants: they do not depend on earlier layers)
  if (warp == 0 && lane == 0) {
    for (int l = 0; l < p.n_layers; ++l) {
      const ChainLayer& L = p.L[l];
      if (L.active_ctas == 0 || cta >= L.active_ctas) continue;
      const int lo = kb_lo(L), hi = kb_hi(L);
      if (hi == lo) continue;
      mbar_arrive_expect_tx(bar_wfull + 8 * l, static_cast<uint32_t>(hi - lo) * (CH_BLOCK_N * 128));
      for (int kb = lo; kb < hi; ++kb)
        tma_load_2d(smem_u32(sW) + L.w_smem_off + (kb - lo) * (CH_BLOCK_N * 128), p.tmaps + L.b_tm, kb * K_ELEMS,
                    cta * CH_BLOCK_N, bar_wfull + 8 * l);
    }
  }

  if (p.early_weights) asm volatile("griddepcontrol.wait;" ::: "memory");

  // the per-column constants this CTA's epilogues will need: start them on their way from DRAM now
  if (warp >= 2 && threadIdx.x - 64 < p.n_layers) {
    const ChainLayer& L = p.L[threadIdx.x - 64];
    const int col = cta * CH_BLOCK_N;
    if (L.active_ctas > 0 && cta < L.active_ctas) {
      if (L.epi.bias) asm volatile("prefetch.global.L2 [%0];" ::"l"(L.epi.bias + col));
      if (L.epi.dqv) asm volatile("prefetch.global.L2 [%0];" ::"l"(L.epi.dqv + col));
      if (L.epi.comp) asm volatile("prefetch.global.L2 [%0];" ::"l"(L.epi.comp + col));
    }
  }

  bool failed = false;
  // Counter value before this launch (only thread 0 uses it).  Every completed launch has added
  // (n_barriers + 1) * gridDim.x: one per CTA and barrier, plus one per CTA on the way out.  CTAs that are ahead of
  // this one may already have arrived at the first barrier, but fewer than gridDim.x of them (this CTA has not), so
  // rounding the value down to a multiple of the per-launch total recovers the start value.  Deriving it on the
  // device instead of passing it as a launch parameter is what lets a captured launch be replayed.
  unsigned long long bar_count = 0;
  if (threadIdx.x == 0) {
    const unsigned long long per_launch = static_cast<unsigned long long>(p.n_barriers + 1) * gridDim.x;
    bar_count = ld_acquire_u64(p.barrier) / per_launch * per_launch;
  }
  int stage = 0;                 // ring position, shared by construction between producer and MMA thread
  uint32_t phase = 0;
  uint32_t tphase = 0;           // parity of the accumulator-ready barrier (one completion per active layer)
  bool a_issued = false;         // thread 0: the A loads of the coming layer went out from inside the barrier

  // Thread 0 (the TMA producer) issues my k-blocks of layer l's A operand.  a_stages >= my k-blocks (planner): a
  // stage is never reused within a layer, and between layers the accumulator-ready commit plus the grid barrier
  // guarantee that every MMA has read its stage.
  auto issue_a_loads = [&](int l) {
    const ChainLayer& L = p.L[l];
    if (L.active_ctas == 0 || cta >= L.active_ctas || (l == 0 && p.pack_rows > 0)) return;
    const int lo = kb_lo(L), hi = kb_hi(L);
    for (int kb = lo; kb < hi; ++kb) {
      mbar_arrive_expect_tx(bar_full + 8 * stage, CH_A_STAGE_BYTES);
      tma_load_2d(smem_u32(sA) + stage * CH_A_STAGE_BYTES, p.tmaps + L.a_tm, kb * K_ELEMS, row0, bar_full + 8 * stage);
      if (++stage == CH_STAGES) {
        stage = 0;
        phase ^= 1;
      }
    }
    a_issued = true;
  };
  // Grid barrier before layer l_next: its A operand is what the other CTAs have just stored, so thread 0 sends the
  // loads the moment the barrier opens (its proxy fence after the acquire orders those stores before the loads).
  auto next_barrier = [&](int l_next) {
    bar_count += gridDim.x;
    if (!grid_barrier(p.barrier, bar_count, [&]() { issue_a_loads(l_next); })) {
      failed = true;
      report(p.status, DEV_TIMEOUT_OTHER);
    }
  };
  const int rows_per = 128 >> KS_SH; // rows of the tile this CTA finishes
  const int n_run = p.fold_tail ? p.n_layers - 1 : p.n_layers;   // layers that run as layers
  for (int l = 0; l < n_run && !failed; ++l) {
    // A by-value copy: fields read through a reference into the parameter space are re-fetched around every
    // store (possible aliasing) at a few hundred clocks each, which made a 16-element epilogue cost thousands.
    const ChainLayer L = p.L[l];
    if (L.active_ctas > 0) {
      if (cta < L.active_ctas) {
        const int lo = kb_lo(L), my_nkb = kb_hi(L) - lo;
        // first layer fed by plain loads (graph-entry reorder): its blocks use stages 0 .. my_nkb-1 outside the ring
        const bool manual_a = l == 0 && p.pack_rows > 0;
        if (warp == 0) {
          if (lane == 0) {
            if (!a_issued) issue_a_loads(l);                     // first layer: no barrier preceded it
            a_issued = false;
          }
        } else if (warp == 1) {
          if (lane == 0) {
            if (my_nkb == 0) {
              mbar_arrive(bar_tfull);                             // nothing to multiply: my partial sums are zero
            } else {
              bool ok = mbar_wait(bar_wfull + 8 * l, 0);
              if (manual_a) ok = ok && mbar_wait(bar_a0, 0);
              const uint32_t idesc = L.idesc;
              const uint64_t a_desc0 = make_smem_desc(smem_u32(sA), 16, 1024, SWZ_128B);
              uint64_t b_desc = make_smem_desc(smem_u32(sW) + L.w_smem_off, 16, 1024, SWZ_128B);
              const uint32_t a_step = static_cast<uint32_t>(CH_A_STAGE_BYTES) >> 4;   // descriptor address units of 16 bytes
              for (int i = 0; i < my_nkb && ok; ++i, b_desc += (CH_BLOCK_N * 128) >> 4) {
                if (!manual_a) ok = mbar_wait(bar_full + 8 * stage, phase);
                if (!ok) break;
                tc_fence_after();
                const uint64_t a_desc = a_desc0 + static_cast<uint64_t>(manual_a ? i : stage) * a_step;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_ss<KIND>(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, (i | k) != 0);
                if (!manual_a && ++stage == CH_STAGES) {
                  stage = 0;
                  phase ^= 1;
                }
              }
              if (ok) umma_commit(bar_tfull);
              else report(p.status, DEV_TIMEOUT_MMA);
            }
          }
        } else {
          const int q = warp & 3;
          if (manual_a) {
            // Row r of my k-blocks (thread per row), realigned in registers and stored where TMA would have put it.
            const int r = q * 32 + lane;
            const int a_rows = CH_A_STAGE_BYTES / 128;
            const int kbytes = row0 + r < L.M ? L.K * ESZ : 0;  // valid bytes of my row (none beyond the matrix)
            const uint8_t* src_row = static_cast<const uint8_t*>(p.pack_src) + static_cast<int64_t>(row0 + r) * p.pack_src_pitch;
            if (r < a_rows) {
              for (int i = 0; i < my_nkb; ++i) {
                const int off = (lo + i) * 128;                  // byte offset of the k-block inside the row
                pack_row_kblock(src_row + off, min(max(kbytes - off, 0), 128), sA + i * CH_A_STAGE_BYTES, r);
              }
            }
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_a0);
          }
          // expect the partial sums of the whole cluster for my rows of the tile (senders may be ahead of this)
          if (KS > 1 && threadIdx.x == 64) mbar_arrive_expect_tx(bar_red, CH_RED_BYTES);
          // the per-column constants of the outputs this thread will finish: fetched now, used after the waits
          // With four parts every CTA finishes 32 rows: four threads per row, 8 columns each, so that all 128 epilogue
          // threads share the work; with two parts (64 rows) two threads per row, 16 columns each.
          const int ft = threadIdx.x - 64;
          const bool fine = KS == 4;
          const int frow = fine ? ft >> 2 : ft >> 1, cgrp = fine ? ft & 3 : ft & 1;
          const int fcol = cta * CH_BLOCK_N + (fine ? 8 : 16) * cgrp;
          const bool finisher = KS > 1 && frow < rows_per && fcol < L.N;
          EpiColsT<16> fk16;
          EpiColsT<8> fk8;
          if (finisher) {
            if (fine) epi_load_cols<8>(fk8, fcol, L.epi);
            else epi_load_cols<16>(fk16, fcol, L.epi);
          }
          // the layer before a folded last layer: my columns' weights of that layer (s8, one output column)
          const bool fold = KIND == KIND_I8 && p.fold_tail && l == n_run - 1;
          int wt16[16];
          if (fold && finisher) {
            const int8_t* wp = static_cast<const int8_t*>(p.L[n_run].wt_ptr) + fcol;
#pragma unroll
            for (int i = 0; i < 16; ++i) wt16[i] = (fine && i >= 8) ? 0 : static_cast<int>(wp[i]);
          }
          if (KS == 1 && L.epi.bias && lane < 2 && cta * CH_BLOCK_N + 16 * lane < L.N)
            asm volatile("prefetch.global.L1 [%0];" ::"l"(L.epi.bias + cta * CH_BLOCK_N + 16 * lane));
          if (mbar_wait(bar_tfull, tphase)) {
            tc_fence_after();
            uint32_t r[32];
            if (my_nkb > 0) {
              const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
              tmem_ld32(t_row, r);
              tmem_wait_ld();
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) r[i] = 0u;
            }
            tc_fence_before();
            const int n0 = cta * CH_BLOCK_N;
            if (KS == 1) {
              const int row = row0 + q * 32 + lane;
              if (row < L.M) {
                char* dst_row = static_cast<char*>(L.out) + static_cast<int64_t>(row) * L.out_pitch * L.out_elem;
                if (n0 < L.N) epi_store16(r, dst_row, n0, L.epi);
                if (n0 + 16 < L.N) epi_store16(r + 16, dst_row, n0 + 16, L.epi);
              }
            } else {
              // my warp's 32 rows belong to CTA `dest` of the cluster: 128 bytes per row into its buffer
              const int row = q * 32 + lane;
              const int dest = row >> (7 - KS_SH), lrow = row & (rows_per - 1);
              // stage the row locally (16-byte chunks XOR-swizzled by the row), then one bulk copy per warp: its 32
              // rows are contiguous here and in the owner's buffer
              uint8_t* my = sSend + row * 128;
#pragma unroll
              for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(my + ((c ^ (row & 7)) << 4)) = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
              fence_proxy_async_smem();
              __syncwarp();
              if (lane == 0)
                bulk_copy_to_cluster(mapa_shared(smem_u32(sRed) + static_cast<uint32_t>((ksr * rows_per + lrow) * 128), dest),
                                     smem_u32(sSend) + static_cast<uint32_t>(row * 128), 32 * 128, mapa_shared(bar_red, dest));
              // finish my rows of the tile
              if (__all_sync(0xffffffffu, mbar_wait_cluster(bar_red, tphase) ? 1 : 0)) {   // (warp-uniform: shuffles follow)
                const int grow = row0 + ksr * rows_per + frow;
                if (!fold) {
                  if (finisher && grow < L.M) {
                    char* dst_row = static_cast<char*>(L.out) + static_cast<int64_t>(grow) * L.out_pitch * L.out_elem;
                    if (fine) chain_finish<KIND, 8>(sRed, rows_per, KS, frow, cgrp, dst_row, fcol, L.epi, fk8);
                    else chain_finish<KIND, 16>(sRed, rows_per, KS, frow, cgrp, dst_row, fcol, L.epi, fk16);
                  }
                } else if constexpr (KIND == KIND_I8) {
                  // Folded last layer: the row is not stored.  The 2 or 4 threads of a row (neighbouring lanes) add
                  // up their parts of the dot product; the first of them adds the CTA's part to the row's sum in
                  // global memory and counts the row; whoever counts last takes the sum (leaving zero behind for the
                  // next launch), applies the last layer's post-ops and stores the one output of the row.
                  const ChainLayer& T = p.L[n_run];
                  int d = 0;
                  if (finisher && grow < L.M) {
                    if (fine) {
                      int w8[8];
#pragma unroll
                      for (int i = 0; i < 8; ++i) w8[i] = wt16[i];
                      d = chain_finish_dot<KIND, 8>(sRed, rows_per, KS, frow, cgrp, L.epi, fk8, w8, T.a_zp);
                    } else {
                      d = chain_finish_dot<KIND, 16>(sRed, rows_per, KS, frow, cgrp, L.epi, fk16, wt16, T.a_zp);
                    }
                  }
                  d += __shfl_xor_sync(0xffffffffu, d, 1);
                  if (fine) d += __shfl_xor_sync(0xffffffffu, d, 2);
                  if (cgrp == 0 && frow < rows_per && grow < L.M) {
                    asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p.tail_acc + grow), "r"(d) : "memory");
                    unsigned int seen;
                    asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(seen) : "l"(p.tail_cnt + grow), "r"(1u) : "memory");
                    if (seen == static_cast<unsigned int>(L.active_ctas) - 1u) {
                      const int sum = atomicExch(p.tail_acc + grow, 0);
                      p.tail_cnt[grow] = 0u;
                      char* dst_row = static_cast<char*>(T.out) + static_cast<int64_t>(grow) * T.out_pitch * T.out_elem;
                      epi_store1(static_cast<uint32_t>(sum), dst_row, 0, T.epi);
                    }
                  }
                }
              } else {
                report(p.status, DEV_TIMEOUT_EPILOGUE);
              }
            }
          } else {
            report(p.status, DEV_TIMEOUT_EPILOGUE);
          }
        }
        // the ring position advances identically in the threads that did not walk it
        if (!manual_a && !(warp <= 1 && lane == 0)) {
          const int pos = stage + my_nkb;
          phase ^= (pos / CH_STAGES) & 1;
          stage = pos % CH_STAGES;
        }
        tphase ^= 1;
      }
    } else {
      // CUDA-core layer: one warp per output element, lanes stride the reduction axis
      const int64_t outputs = static_cast<int64_t>(L.M) * L.N;
      for (int64_t o = static_cast<int64_t>(blockIdx.x) * (CH_THREADS / 32) + warp; o < outputs;
           o += static_cast<int64_t>(gridDim.x) * (CH_THREADS / 32)) {
        const int m = static_cast<int>(o / L.N), n = static_cast<int>(o % L.N);
        const char* A = static_cast<const char*>(L.a_ptr) + static_cast<int64_t>(m) * L.a_pitch * ESZ;
        const char* Wt = static_cast<const char*>(L.wt_ptr) + static_cast<int64_t>(n) * L.w_pitch * ESZ;
        uint32_t raw;
        if (L.epi.acc_is_int) {
          int acc = 0;
          for (int k = lane; k < L.K; k += 32) acc += (ch_load_i(A, k, L.a_dtype) - L.a_zp) * ch_load_i(Wt, k, L.w_dtype);
#pragma unroll
          for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
          raw = static_cast<uint32_t>(acc);
        } else {
          float acc = 0.f;
          for (int k = lane; k < L.K; k += 32) acc = fmaf(ch_load_f(A, k, L.a_dtype), ch_load_f(Wt, k, L.w_dtype), acc);
#pragma unroll
          for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
          raw = __float_as_uint(acc);
        }
        if (lane == 0) {
          char* row = static_cast<char*>(L.out) + static_cast<int64_t>(m) * L.out_pitch * L.out_elem;
          epi_store1(raw, row, n, L.epi);
        }
      }
    }
    if (l + 1 < n_run) next_barrier(l + 1);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, CH_NACC * CH_BLOCK_N);
  }
  // one more count per CTA on the way out (nobody waits for it): it keeps the counter a multiple of the per-launch
  // total between launches, which the start-value computation above relies on.  Relaxed: the next launch reads the
  // counter only after this one has completed, and a release here would hold the CTA back for over a thousand clocks.
  if (threadIdx.x == 0) asm volatile("red.relaxed.gpu.global.add.u64 [%0], %1;" ::"l"(p.barrier), "l"(1ULL) : "memory");
  // no CTA leaves while another one of its cluster may still write into its shared memory or read a copy out of it
  // (every CTA has seen all copies addressed to it complete before it arrives here; nothing else is ordered)
  if (KS > 1) cluster_sync_all_relaxed();
}

size_t mlp_chain_smem_bytes(size_t w_smem_bytes, int a_stages, int a_stage_bytes, int ks) {
  return ((static_cast<size_t>(a_stages) * a_stage_bytes + 1023) & ~size_t(1023)) +
         (w_smem_bytes < 16384 ? size_t(16384) : w_smem_bytes) + (ks > 1 ? 2 * CH_RED_BYTES : 0) + 1024 + 1024;
}

cudaError_t launch_mlp_chain(int kind, const ChainParams& p, int grid, cudaStream_t s) {
  const size_t smem = mlp_chain_smem_bytes(p.w_smem_bytes, p.a_stages, p.a_stage_bytes, p.ks);
  void* kern = kind == KIND_I8 ? reinterpret_cast<void*>(mlp_chain_kernel<KIND_I8>)
               : kind == KIND_BF16 ? reinterpret_cast<void*>(mlp_chain_kernel<KIND_BF16>)
                                   : reinterpret_cast<void*>(mlp_chain_kernel<KIND_TF32>);
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(CH_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  // No cooperative-launch attribute: it costs tens of microseconds per launch, more than the whole chain.
  // The grid is at most one CTA per SM, so its CTAs become resident together whenever the SMs are free; if
  // they are not, the waiting CTAs only wait for unrelated work to finish, and every spin is bounded anyway.
  // Programmatic dependent launch: the set-up may overlap the tail of whatever precedes on the stream; the
  // kernel waits for that work to complete before its first global access.
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = static_cast<unsigned>(p.ks);
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = p.ks > 1 ? 2 : 1;
  void* args[] = {const_cast<ChainParams*>(&p)};
  return cudaLaunchKernelExC(&cfg, kern, args);
}

int mlp_chain_max_clusters(int kind, int ks, size_t smem) {
  void* kern = kind == KIND_I8 ? reinterpret_cast<void*>(mlp_chain_kernel<KIND_I8>)
               : kind == KIND_BF16 ? reinterpret_cast<void*>(mlp_chain_kernel<KIND_BF16>)
                                   : reinterpret_cast<void*>(mlp_chain_kernel<KIND_TF32>);
  if (ensure_dynamic_smem(kern, smem) != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(ks));
  cfg.blockDim = dim3(CH_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(ks);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) return 0;
  return n;
}

}  // namespace gc
