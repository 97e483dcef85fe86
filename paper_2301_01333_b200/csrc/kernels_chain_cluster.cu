// A whole small fp32 MLP chain inside ONE thread-block cluster (the analogue of the paper's coarse-grain fusion,
// Section V: activations stay in the fastest memory from layer to layer and the synchronisation between the fused
// ops shrinks to what the data dependence itself needs).
//
// The chain kernel in kernels_chain.cu spreads every layer over the whole GPU and hands activations over through the
// L2 behind a grid-wide barrier.  For the smallest chains (a few dozen rows, layers of a few hundred columns) that
// hand-over is most of the time.  Here the C CTAs of one cluster (8 or 16) hold the weights of every layer in shared
// memory, and an activation goes from the CTA that finished it straight into the A-operand stages of the CTAs that
// multiply it next, by bulk copies through distributed shared memory that report to the receiver's mbarrier:
//   * layer l has slices_l = N_l / 32 column slices and splits its reduction axis into ks_l parts
//     (slices_l * ks_l <= C); CTA r works on slice r / ks_l, part r % ks_l, and is idle in layers with fewer parts;
//   * per layer a CTA waits for its k-blocks of the A operand (first layer: TMA from global memory, or rows packed
//     by the epilogue warps when TMA cannot address the row pitch; later layers: the bulk copies of the finishing
//     CTAs), issues tcgen05.mma (tf32, M = 64, N = 32, four 8-deep k-steps per k-block, one accumulator), and its
//     epilogue warps read the accumulator;
//   * with ks_l > 1 the partial sums meet as in the grid-wide kernel: every CTA of a group finishes rows_per rows and
//     receives those rows of the others' partial sums; they are added in a fixed order;
//   * a finished row of 32 fp32 values IS a 128-byte row of a k-block of the next layer's A operand (k-block = my
//     slice index): it is written in the swizzled operand layout into a local buffer and copied to every CTA of the
//     next layer whose part of the reduction axis contains that k-block; the last layer stores to global memory.
//   * a first layer with a short reduction axis (at most two k-blocks) is not distributed at all: every CTA of the
//     second layer multiplies the input by the first-layer weight columns that make up its own part of the second
//     layer's reduction axis (up to 256 of them) and writes the result, bias and activation applied, straight into
//     its own A-operand stages - redundant arithmetic across the column slices, no exchange.  That product is taken
//     transposed (weight rows on the M side, 128 per MMA; batch rows on the N side), so that every one of the 128
//     epilogue threads owns an accumulator row.
// The code between the waits runs once per launch in warps that are alone on their schedulers: every branch costs such
// a warp about 30 clocks and every integer division a hundred, so the epilogues use selects, shifts and tests per
// group of rows instead, loops with run-time trip counts stay rolled, and waits and rare activations are out of line.
// A-operand stages alternate between two regions by layer parity, and so do the staging buffers; every buffer is
// reused two layers later, by which time the data dependence chain guarantees that all copies out of it and all MMAs
// reading it have completed (a CTA can only reach layer l + 2 after every CTA has finished layer l).
// All waits are bounded; a CTA that gives up records a code, skips the remaining layers and still joins the final
// cluster barrier.
#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

constexpr int CC_THREADS = 192;          // warp 0 producer, warp 1 MMA, warps 2-5 epilogue
constexpr int CC_BLOCK_N = 32;
constexpr int CC_NACC = 1;               // one accumulator: four did not overlap the MMAs and cost the epilogue three more loads
constexpr int CC_K_ELEMS = 32;           // fp32 elements per 128-byte k-block
constexpr int CC_RED_BYTES = 128 * 128;  // partial sums received: at most 128 rows of 128 bytes
constexpr int CC_T0_COL = 128;                     // tensor-memory column of the recomputed first layer's accumulator
constexpr int CC_T0_MAX = 256;                     // its widest form (first-layer columns per CTA)
constexpr int CC_T0_STRIDE = 64;                   // columns between its 128-row blocks (at most 64 batch rows)

// AND of a flag over the 128 threads of the four epilogue warps (named barrier 1): after a bounded wait every one of
// them takes the same branch, so the named barriers that follow are reached by all or by none.
__device__ __forceinline__ bool cc_epi_all(bool ok) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.and.pred q, 1, 128, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(ok ? 1u : 0u)
      : "memory");
  return r != 0;
}

// Bounded waits out of line: this kernel's code runs once per launch, so every inlined copy of a polling loop is
// instruction-cache misses on the way to the code that matters.
static __device__ __noinline__ bool cc_wait(uint32_t bar, uint32_t parity) { return mbar_wait_prompt(bar, parity); }
static __device__ __noinline__ bool cc_wait_cluster(uint32_t bar, uint32_t parity) { return mbar_wait_cluster<100u>(bar, parity); }

// One lane of the warp polls, the others wait for it at the warp barrier of the shuffle: 128 polling threads keep the
// shared-memory pipeline busy that the working warp needs.
template <typename F>
__device__ __forceinline__ bool cc_lane0_wait(int lane, F wait) {
  int ok = 1;
  if (lane == 0) ok = wait() ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

__global__ void __launch_bounds__(CC_THREADS, 1) mlp_cluster_kernel(const __grid_constant__ ChainParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int STAGE = p.a_stage_bytes;                              // bytes per A-operand stage (rows x 128)
  const int REGION = p.a_stages * STAGE;                          // one of the two A-operand regions
  uint8_t* sA = smem;                                             // 2 regions
  // the weight slices (padded to at least 16 KB) follow, so the 64-row MMA reads of the last stages (a stage may hold
  // fewer rows) stay inside this CTA's shared memory
  uint8_t* sW = sA + ((2 * REGION + 1023) & ~1023);
  uint8_t* sRed = sW + (p.w_smem_bytes < 16384u ? 16384u : p.w_smem_bytes);   // partial sums from my group
  uint8_t* sSend = sRed + CC_RED_BYTES;                           // 2 x STAGE: my partial sums, staged for the copies
  uint8_t* sOut = sSend + 2 * STAGE;                              // 2 x STAGE: rows I finished, in operand layout
  uint64_t* bars = reinterpret_cast<uint64_t*>(sOut + 2 * STAGE);
  const uint32_t bar_w = smem_u32(bars);                          // [CHAIN_MAX_LAYERS] weight slice of layer l has landed
  const uint32_t bar_a = bar_w + 8 * CHAIN_MAX_LAYERS;            // [CHAIN_MAX_LAYERS] my k-blocks of layer l's A operand
  const uint32_t bar_tfull = bar_a + 8 * CHAIN_MAX_LAYERS;        // accumulators ready
  const uint32_t bar_red = bar_tfull + 8;                         // partial sums of my group have arrived
  const uint32_t bar_a0 = bar_red + 8;                            // first layer's A operand packed by the epilogue warps
  const uint32_t bar_a1 = bar_a0 + 8;                             // second layer's A operand written by the epilogue warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * CHAIN_MAX_LAYERS + 4);
  float* sBias0 = reinterpret_cast<float*>(bars + 2 * CHAIN_MAX_LAYERS + 6);   // [CC_T0_MAX] first-layer bias of my columns
  float* sBias = sBias0 + CC_T0_MAX;                              // [CHAIN_MAX_LAYERS][32] bias of my slice of every layer
  const bool recompute = p.recompute_first != 0;
  const int tmem_cols = recompute ? 256 : 32;                     // (128 + two blocks of CC_T0_STRIDE columns)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_ctarank());

  // my role in layer l
  // (ks_l is 1, 2 or 4: shifts and masks, not divisions - they sit between the layers of a latency chain)
  auto ks_sh = [](const ChainLayer& L) { return __ffs(L.ks_l) - 1; };
  auto active = [&](const ChainLayer& L) { return rank < ((L.N >> 5) << ks_sh(L)); };
  auto kb_lo = [&](const ChainLayer& L, int part) { return (part * L.nkb) >> ks_sh(L); };
  auto part_of = [&](const ChainLayer& L) { return rank & (L.ks_l - 1); };
  auto slice_of = [&](const ChainLayer& L) { return rank >> ks_sh(L); };
  const bool manual_a = p.pack_rows > 0;

  if (threadIdx.x == 0) {
#pragma unroll 1
    for (int l = 0; l < CHAIN_MAX_LAYERS; ++l) {
      mbar_init(bar_w + 8 * l, 1);
      mbar_init(bar_a + 8 * l, 1);
    }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_red, 1);
    mbar_init(bar_a0, 4);                                         // one arrival per epilogue warp
    mbar_init(bar_a1, 4);
    fence_mbar_init();
    // the bytes the finishing CTAs of layer l - 1 will copy into my stages of layer l: armed before anybody can send
#pragma unroll 1
    for (int l = recompute ? 2 : 1; l < p.n_layers; ++l) {
      const ChainLayer& L = p.L[l];
      if (!active(L)) continue;
      const int part = part_of(L);
      const int my_nkb = kb_lo(L, part + 1) - kb_lo(L, part);
      const ChainLayer& P = p.L[l - 1];
      mbar_arrive_expect_tx(bar_a + 8 * l, static_cast<uint32_t>(my_nkb * P.ks_l * P.rows_per * 128));
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // nobody may signal a barrier of another CTA before that CTA has initialised and armed it
  cluster_sync_all();

  // Programmatic dependent launch: everything above may overlap the tail of the preceding kernel on the stream.  The
  // prepacked weights are constants; unless this very call has just enqueued their prepack, their loads may start
  // before the preceding kernel has finished, too.  Everything else waits for it.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (!p.early_weights) asm volatile("griddepcontrol.wait;" ::: "memory");
  if (warp == 0 && lane == 0) {
    if (recompute && active(p.L[1])) {
      // the first-layer weight rows (= output columns) that form my part of the second layer's reduction axis
      const ChainLayer& L0 = p.L[0];
      const ChainLayer& L1 = p.L[1];
      const int part = part_of(L1);
      const int lo1 = kb_lo(L1, part), n1 = kb_lo(L1, part + 1) - lo1;
      mbar_arrive_expect_tx(bar_w, static_cast<uint32_t>(L0.nkb * n1) * (CC_BLOCK_N * 128));
#pragma unroll 1
      for (int kb = 0; kb < L0.nkb; ++kb)
#pragma unroll 1
        for (int j = 0; j < n1; ++j)
          tma_load_2d(smem_u32(sW) + L0.w_smem_off + (kb * n1 + j) * (CC_BLOCK_N * 128), p.tmaps + L0.b_tm, kb * CC_K_ELEMS,
                      (lo1 + j) * CC_BLOCK_N, bar_w);
    }
#pragma unroll 1
    for (int l = recompute ? 1 : 0; l < p.n_layers; ++l) {
      const ChainLayer& L = p.L[l];
      if (!active(L)) continue;
      const int slice = slice_of(L), part = part_of(L);
      const int lo = kb_lo(L, part), hi = kb_lo(L, part + 1);
      if (hi == lo) continue;
      mbar_arrive_expect_tx(bar_w + 8 * l, static_cast<uint32_t>(hi - lo) * (CC_BLOCK_N * 128));
#pragma unroll 1
      for (int kb = lo; kb < hi; ++kb)
        tma_load_2d(smem_u32(sW) + L.w_smem_off + (kb - lo) * (CC_BLOCK_N * 128), p.tmaps + L.b_tm, kb * CC_K_ELEMS,
                    slice * CC_BLOCK_N, bar_w + 8 * l);
    }
  }
  // The per-column constants my epilogues will need are constants like the weights: start them on their way now (the
  // recomputed first layer's bias into shared memory, the others into the L2).
  if (warp >= 2) {
#pragma unroll 1
    for (int i = threadIdx.x - 64; i < p.n_layers * CC_BLOCK_N; i += 128) {
      const ChainLayer& L = p.L[i >> 5];
      if ((recompute && i < CC_BLOCK_N) || !active(L)) continue;
      sBias[i] = L.epi.bias ? __ldg(L.epi.bias + slice_of(L) * CC_BLOCK_N + (i & 31)) : 0.f;
    }
  }
  if (recompute && warp >= 2 && active(p.L[1])) {
    const ChainLayer& L1 = p.L[1];
    const int part = part_of(L1);
    const int lo1 = kb_lo(L1, part), ncol = (kb_lo(L1, part + 1) - lo1) * CC_BLOCK_N;
#pragma unroll 1
    for (int i = threadIdx.x - 64; i < ncol; i += 128) sBias0[i] = p.L[0].epi.bias ? __ldg(p.L[0].epi.bias + lo1 * CC_BLOCK_N + i) : 0.f;
  }
  if (p.early_weights) asm volatile("griddepcontrol.wait;" ::: "memory");

  bool failed = false;
  uint32_t tphase = 0;           // parity of the accumulator-ready barrier (one completion per layer I am active in)
  uint32_t rphase = 0;           // parity of the partial-sum barrier (one completion per such layer with ks_l > 1)

#pragma unroll 1
  for (int l = 0; l < p.n_layers && !failed; ++l) {
    // (a by-value copy: fields read through a reference into the parameter space are re-fetched around every store)
    const ChainLayer L = p.L[l];
    // a recomputed first layer is the business of the CTAs of the second layer, each with the whole reduction axis
    const bool rc0 = recompute && l == 0;
    if (!active(rc0 ? p.L[1] : L)) continue;
    const int KS = rc0 ? 1 : L.ks_l, rows_per = L.rows_per;
    const int slice = rc0 ? rank : slice_of(L), part = rc0 ? 0 : part_of(L);
    const int lo = rc0 ? 0 : kb_lo(L, part), my_nkb = rc0 ? L.nkb : kb_lo(L, part + 1) - lo;
    // (recomputed first layer: the k-blocks of the second layer that are mine, i.e. 32-column groups to produce)
    const int n1 = rc0 ? kb_lo(p.L[1], part_of(p.L[1]) + 1) - kb_lo(p.L[1], part_of(p.L[1])) : 0;
    const int nb0 = min(64, (L.M + 15) / 16 * 16);               // batch rows as the N of the transposed first layer
    const bool last = l + 1 == p.n_layers;
    uint8_t* region = sA + (l & 1) * REGION;
    uint8_t* send = sSend + (l & 1) * STAGE;
    uint8_t* outb = sOut + (l & 1) * STAGE;

    if (warp == 0) {
      if (lane == 0 && l == 0 && !manual_a && my_nkb > 0) {
        const uint32_t box_bytes = static_cast<uint32_t>((L.M < 128 ? (L.M + 7) / 8 * 8 : 128) * 128);
        mbar_arrive_expect_tx(bar_a, static_cast<uint32_t>(my_nkb) * box_bytes);
#pragma unroll 1
        for (int i = 0; i < my_nkb; ++i)
          tma_load_2d(smem_u32(region) + i * STAGE, p.tmaps + L.a_tm, (lo + i) * CC_K_ELEMS, 0, bar_a);
      }
    } else if (warp == 1) {
      if (lane == 0) {
        if (my_nkb == 0) {
          mbar_arrive(bar_tfull);                                 // nothing to multiply: my partial sums are zero
        } else {
          bool ok = cc_wait(bar_w + 8 * l, 0);
          if (ok) ok = (l == 0 && manual_a) ? cc_wait(bar_a0, 0)
                       : (l == 1 && recompute) ? cc_wait(bar_a1, 0) : cc_wait_cluster(bar_a + 8 * l, 0);
          if (ok && rc0) {
            tc_fence_after();
            const uint32_t x0 = smem_u32(region), w0 = smem_u32(sW) + L.w_smem_off;
            // The product is taken transposed: the weight rows (= my 32 n1 first-layer columns, 128 per MMA) are the
            // M side, the batch rows the N side, so that all 128 epilogue threads own an accumulator row (a column
            // of the activation) instead of the 32 that would own a batch row.  M = 128, N = batch rows rounded up
            // to 16 (N field: bits 17..22 in units of 8; M field: bits 24..28 in units of 16).
            const uint32_t idesc = (L.idesc & ~((0x1Fu << 24) | (0x3Fu << 17))) | ((128u >> 4) << 24) |
                                   ((static_cast<uint32_t>(nb0) >> 3) << 17);
#pragma unroll 1
            for (int m = 0; m * 128 < n1 * CC_BLOCK_N; ++m) {
#pragma unroll 1
              for (int i = 0; i < my_nkb; ++i) {
#pragma unroll
                for (int k = 0; k < 4; ++k)
                  umma_ss<KIND_TF32>(tmem_base + CC_T0_COL + m * CC_T0_STRIDE,
                                     make_smem_desc(w0 + i * n1 * (CC_BLOCK_N * 128) + m * (128 * 128) + 32 * k, 16, 1024, SWZ_128B),
                                     make_smem_desc(x0 + i * STAGE + 32 * k, 16, 1024, SWZ_128B), idesc, (i | k) != 0);
              }
            }
            umma_commit(bar_tfull);
          } else if (ok) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(region), b0 = smem_u32(sW) + L.w_smem_off;
            // at most 64 rows are ever finished: M = 64 (the M field of the descriptor is bits 24..28, in units of 16)
            const uint32_t idesc = (L.idesc & ~(0x1Fu << 24)) | ((64u >> 4) << 24);
#pragma unroll 1
            for (int i = 0; i < my_nkb; ++i) {
#pragma unroll
              for (int k = 0; k < 4; ++k)   // (each descriptor is built from its address, not stepped as an integer)
                umma_ss<KIND_TF32>(tmem_base, make_smem_desc(a0 + i * STAGE + 32 * k, 16, 1024, SWZ_128B),
                                   make_smem_desc(b0 + i * (CC_BLOCK_N * 128) + 32 * k, 16, 1024, SWZ_128B), idesc, (i | k) != 0);
            }
            umma_commit(bar_tfull);
          } else {
            report(p.status, DEV_TIMEOUT_MMA);
            failed = true;
          }
        }
      }
    } else {
      const int q = warp & 3;
      const int et = threadIdx.x - 64;                            // 0..127
      if (l == 0 && manual_a) {
        // Row r of my k-blocks (thread per row), zero beyond the row's K bytes and beyond row M, stored where TMA would
        // have put them (128-byte rows, 8-row groups of 1024 bytes, chunk index XOR row mod 8).
        const int r = et;
        const int a_rows = STAGE / 128;
        const int64_t kbytes = static_cast<int64_t>(L.K) * 4;
        const uint8_t* src_row = static_cast<const uint8_t*>(p.pack_src) + static_cast<int64_t>(r) * p.pack_src_pitch;
        const bool words_ok = ((reinterpret_cast<uintptr_t>(p.pack_src) | static_cast<uintptr_t>(p.pack_src_pitch)) & 3) == 0;
        if (r < a_rows && words_ok) {
          // rows of whole 32-bit words (every fp32 input): 32 independent predicated loads per k-block and not one
          // branch (a lone warp pays about 30 clocks for each)
          const uint32_t* src_w = reinterpret_cast<const uint32_t*>(src_row);
          const int kmax = r < L.M ? L.K : 0;
#pragma unroll 1
          for (int i = 0; i < my_nkb; ++i) {
            uint8_t* dst = region + i * STAGE + (r >> 3) * 1024 + (r & 7) * 128;
            const int k0 = (lo + i) * CC_K_ELEMS;
            uint32_t w[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) w[j] = (k0 + j < kmax) ? __ldg(src_w + k0 + j) : 0u;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              *reinterpret_cast<uint4*>(dst + ((c ^ (r & 7)) << 4)) = make_uint4(w[4 * c], w[4 * c + 1], w[4 * c + 2], w[4 * c + 3]);
          }
        } else if (r < a_rows) {
          const int kb_bytes = r < L.M ? static_cast<int>(kbytes) : 0;
#pragma unroll 1
          for (int i = 0; i < my_nkb; ++i) {
            const int off = (lo + i) * 128;
            pack_row_kblock(src_row + off, min(max(kb_bytes - off, 0), 128), region + i * STAGE, r);
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_a0);
      }
      if (rc0) {
        // Recomputed first layer, computed transposed: accumulator row = one of my 32 n1 first-layer columns (warp q of
        // block m owns columns 128 m + 32 q .. + 32, i.e. k-block 4 m + q of the second layer's A operand),
        // accumulator column = batch row.  Bias and activation applied, the 32 lanes of a warp write one swizzled
        // 128-byte operand row per batch row.
        const int act = L.epi.act;
        const bool relu = act == ACT_RELU, other_act = act != ACT_NONE && !relu;
        uint8_t* region1 = sA + REGION;
        const int rows_st = min(STAGE / 128, nb0);               // batch rows that exist in a stage
        const bool ok = cc_epi_all(cc_lane0_wait(lane, [&]() { return cc_wait(bar_tfull, tphase); }));   // (also orders the writes of sBias0 before its reads)
        if (ok) {
          tc_fence_after();
#pragma unroll 1
          for (int m = 0; m * 128 < n1 * CC_BLOCK_N; ++m) {
            const int j = m * 4 + q;                              // my k-block of the second layer
            if (j >= n1) break;                                   // (warp-uniform)
            const float bias = sBias0[j * CC_BLOCK_N + lane];
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + CC_T0_COL + m * CC_T0_STRIDE;
            uint8_t* st = region1 + j * STAGE + (lane & 3) * 4;
#pragma unroll 1
            for (int h = 0; h * 32 < rows_st; ++h) {
              uint32_t r[32];
              tmem_ld32(t_row + h * 32, r);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) {                      // (no branch per element: see the finishing step below)
                const float t = __fadd_rn(__uint_as_float(r[i]), bias);
                r[i] = __float_as_uint(relu ? fmaxf(t, 0.f) : t);
              }
              if (other_act) {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(apply_act_cold(__uint_as_float(r[i]), act));
              }
              // row brow, 16-byte chunk (lane / 4) XOR (brow mod 8), word lane mod 4.  The rows of a stage come in groups
              // of 8: one test per group, not one per row (a predicated store becomes a branch, and a lone warp pays
              // about 30 clocks for each).
#pragma unroll
              for (int g8 = 0; g8 < 4; ++g8) {
                if (h * 32 + g8 * 8 < rows_st) {
#pragma unroll
                  for (int i = 0; i < 8; ++i)
                    *reinterpret_cast<float*>(st + (h * 4 + g8) * 1024 + i * 128 + (((lane >> 2) ^ i) << 4)) =
                        __uint_as_float(r[g8 * 8 + i]);
                }
              }
            }
          }
          tc_fence_before();
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_a1);
        } else {
          report(p.status, DEV_TIMEOUT_EPILOGUE);
          failed = true;
        }
        tphase ^= 1;
        continue;
      }
      const int rows_all = KS * rows_per;                         // rows of the tile that are finished at all
      // expect my rows of the partial sums of the whole group (senders cannot be ahead of this by a whole layer)
      if (KS > 1 && et == 0) mbar_arrive_expect_tx(bar_red, static_cast<uint32_t>(rows_all * 128));
      // The M = 64 accumulator keeps tile row i in tensor-memory lane 32 (i / 16) + i % 16: warp q reads rows
      // 16 q .. 16 q + 15 with its lanes 0 .. 15.
      const int row = q * 16 + lane;                              // my accumulator row (lanes 0..15)
      const bool has_row = lane < 16 && row < rows_all;
      // split layers: thread et finishes row et / 2 of my rows, columns 16 (et % 2) .. + 16 of my slice;
      // unsplit layers: the thread that read a row finishes all 32 columns of it
      const int frow = KS > 1 ? (et >> 1) : row, half = et & 1;
      const bool finisher = KS > 1 ? frow < rows_per : has_row;
      const int ncol4 = KS > 1 ? 4 : 8;                           // float4 groups this thread finishes
      const int fcol = slice * CC_BLOCK_N + (KS > 1 ? 16 * half : 0);
      // (the bias of my slice sits in shared memory since the start of the kernel; the named barrier below orders it)
      const float4* bias4 = reinterpret_cast<const float4*>(sBias + l * CC_BLOCK_N + (KS > 1 ? 16 * half : 0));
      const int act = L.epi.act;
      bool ok = cc_epi_all(cc_lane0_wait(lane, [&]() { return cc_wait(bar_tfull, tphase); }));
      float4 acc4[8];
      if (ok) {
        tc_fence_after();
        uint32_t r[32];
        if (my_nkb > 0 && q * 16 < rows_all) {
          const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
          tmem_ld32(t_row, r);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i) r[i] = 0u;
        }
        tc_fence_before();
        if (KS > 1) {
          // my accumulator row goes to the staging buffer (16-byte chunks XOR-swizzled by the row) and from there to
          // the CTA of my group that finishes it
          if (has_row) {
            uint8_t* my = send + row * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              *reinterpret_cast<uint4*>(my + ((c ^ (row & 7)) << 4)) = make_uint4(r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
          }
          fence_proxy_async_smem();
          __syncwarp();
          if (lane < KS) {                                        // lane d serves the CTA that finishes rows [d rows_per, + rows_per)
            const int base = rank - part, d = lane;               // (base: first CTA of my group)
            const int ra = max(d * rows_per, q * 16), rb = min((d + 1) * rows_per, q * 16 + 16);
            if (ra < rb)
              bulk_copy_to_cluster(mapa_shared(smem_u32(sRed) + static_cast<uint32_t>((part * rows_per + ra - d * rows_per) * 128), base + d),
                                   smem_u32(send) + static_cast<uint32_t>(ra * 128), static_cast<uint32_t>((rb - ra) * 128),
                                   mapa_shared(bar_red, base + d));
          }
          ok = cc_epi_all(cc_lane0_wait(lane, [&]() { return cc_wait_cluster(bar_red, rphase); }));
          if (ok && finisher) {
#pragma unroll
            for (int c = 0; c < 8; ++c) acc4[c] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int s = 0; s < 4; ++s) {                         // fixed order: deterministic; parts beyond KS add zero
              // (all four loads are issued - the rows exist in the buffer - and a select drops the surplus ones: no
              // branch per part)
              const uint8_t* src = sRed + (s * rows_per + frow) * 128;
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                float4 v = *reinterpret_cast<const float4*>(src + (((half * 4 + c) ^ (frow & 7)) << 4));
                const bool use = s < KS;
                acc4[c].x += use ? v.x : 0.f; acc4[c].y += use ? v.y : 0.f; acc4[c].z += use ? v.z : 0.f; acc4[c].w += use ? v.w : 0.f;
              }
            }
          }
        } else {
#pragma unroll
          for (int c = 0; c < 8; ++c)
            acc4[c] = make_float4(__uint_as_float(r[4 * c]), __uint_as_float(r[4 * c + 1]), __uint_as_float(r[4 * c + 2]),
                                  __uint_as_float(r[4 * c + 3]));
        }
      }
      if (ok) {
        if (finisher) {
          // bias and activation (fp32 chains only: this kernel takes no other).  No branch per element: a lone warp
          // pays dozens of clocks for every one, so ReLU / none is a select, and anything else one pass of its own
          // behind a single branch.
          const bool relu = act == ACT_RELU;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            float4 t = acc4[c];
            t.x = __fadd_rn(t.x, bias4[c & (ncol4 - 1)].x); t.y = __fadd_rn(t.y, bias4[c & (ncol4 - 1)].y);
            t.z = __fadd_rn(t.z, bias4[c & (ncol4 - 1)].z); t.w = __fadd_rn(t.w, bias4[c & (ncol4 - 1)].w);
            t.x = relu ? fmaxf(t.x, 0.f) : t.x; t.y = relu ? fmaxf(t.y, 0.f) : t.y;
            t.z = relu ? fmaxf(t.z, 0.f) : t.z; t.w = relu ? fmaxf(t.w, 0.f) : t.w;
            acc4[c] = t;
          }
          if (act != ACT_NONE && !relu) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              acc4[c].x = apply_act_cold(acc4[c].x, act); acc4[c].y = apply_act_cold(acc4[c].y, act);
              acc4[c].z = apply_act_cold(acc4[c].z, act); acc4[c].w = apply_act_cold(acc4[c].w, act);
            }
          }
          const int grow = part * rows_per + frow;                // row of the tile
          if (last) {
            if (grow < L.M) {
              float4* d = reinterpret_cast<float4*>(static_cast<float*>(L.out) + static_cast<int64_t>(grow) * L.out_pitch + fcol);
#pragma unroll
              for (int c = 0; c < 8; ++c)
                if (c < ncol4) d[c] = acc4[c];
            }
          } else {
            uint8_t* my = outb + frow * 128;
            const int c0 = KS > 1 ? half * 4 : 0;
#pragma unroll
            for (int c = 0; c < 8; ++c)
              if (c < ncol4) *reinterpret_cast<float4*>(my + (((c0 + c) ^ (frow & 7)) << 4)) = acc4[c];
          }
        }
        if (!last) {
          // my finished rows are rows [part rows_per, + rows_per) of k-block `slice` of the next layer's A operand:
          // one copy to every CTA of that layer whose part of the reduction axis contains the k-block (each copy
          // issued by a thread of its own)
          fence_proxy_async_smem();
          asm volatile("bar.sync 1, 128;" ::: "memory");
          const ChainLayer& Nx = p.L[l + 1];
          const int nslices = Nx.N / CC_BLOCK_N;
          if (et < nslices) {
            int np = 0;
            while (np + 1 < Nx.ks_l && kb_lo(Nx, np + 1) <= slice) ++np;                 // the part that holds k-block `slice`
            const int st = slice - kb_lo(Nx, np);                                        // its stage there
            const uint32_t dst = smem_u32(sA) + static_cast<uint32_t>(((l + 1) & 1) * REGION + st * STAGE + part * rows_per * 128);
            const int rc = et * Nx.ks_l + np;
            bulk_copy_to_cluster(mapa_shared(dst, rc), smem_u32(outb), static_cast<uint32_t>(rows_per * 128),
                                 mapa_shared(bar_a + 8 * (l + 1), rc));
          }
        }
      } else {
        report(p.status, DEV_TIMEOUT_EPILOGUE);
        failed = true;
      }
      if (KS > 1) rphase ^= 1;
    }
    tphase ^= 1;
    if (warp == 1) failed = __shfl_sync(0xffffffffu, failed ? 1 : 0, 0) != 0;
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, tmem_cols);
  }
  // no CTA leaves while another one of its cluster may still write into its shared memory or read a copy out of it
  // (every CTA has seen all copies addressed to it complete before it arrives here; nothing else is ordered)
  cluster_sync_all_relaxed();
}

size_t mlp_cluster_smem_bytes(size_t w_smem_bytes, int a_stages, int a_stage_bytes) {
  // (the last two terms: barriers and the two bias tables; slack for the 1024-byte alignment of the base)
  return ((2 * static_cast<size_t>(a_stages) * a_stage_bytes + 1023) & ~size_t(1023)) +
         (w_smem_bytes < 16384 ? size_t(16384) : w_smem_bytes) + CC_RED_BYTES + 4 * static_cast<size_t>(a_stage_bytes) + 3072 + 1024;
}

static cudaError_t cluster_kernel_ready(size_t smem) {
  static bool nonportable_set = false;
  const void* kern = reinterpret_cast<const void*>(mlp_cluster_kernel);
  cudaError_t e = ensure_dynamic_smem(kern, smem);
  if (e != cudaSuccess) return e;
  if (!nonportable_set) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    nonportable_set = true;
  }
  return cudaSuccess;
}

cudaError_t launch_mlp_cluster(const ChainParams& p, int cluster, cudaStream_t s) {
  const size_t smem = mlp_cluster_smem_bytes(p.w_smem_bytes, p.a_stages, p.a_stage_bytes);
  cudaError_t e = cluster_kernel_ready(smem);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cluster));
  cfg.blockDim = dim3(CC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  void* args[] = {const_cast<ChainParams*>(&p)};
  return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(mlp_cluster_kernel), args);
}

int mlp_cluster_max_clusters(int cluster, size_t smem) {
  if (cluster_kernel_ready(smem) != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(cluster));
  cfg.blockDim = dim3(CC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(cluster);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, reinterpret_cast<const void*>(mlp_cluster_kernel), &cfg) != cudaSuccess) return 0;
  return n;
}

}  // namespace gc
