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
//     CTAs), issues tcgen05.mma (tf32, M = 64, N = 32; the four 8-deep k-steps of a k-block go to four independent
//     accumulators), and its epilogue warps read the accumulators;
//   * with ks_l > 1 the partial sums meet as in the grid-wide kernel: every CTA of a group finishes rows_per rows and
//     receives those rows of the others' partial sums; they are added in a fixed order;
//   * a finished row of 32 fp32 values IS a 128-byte row of a k-block of the next layer's A operand (k-block = my
//     slice index): it is written in the swizzled operand layout into a local buffer and copied to every CTA of the
//     next layer whose part of the reduction axis contains that k-block; the last layer stores to global memory.
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
constexpr int CC_NACC = 4;
constexpr int CC_K_ELEMS = 32;           // fp32 elements per 128-byte k-block
constexpr int CC_RED_BYTES = 128 * 128;  // partial sums received: at most 128 rows of 128 bytes

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
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * CHAIN_MAX_LAYERS + 3);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_ctarank());

  // my role in layer l
  auto active = [&](const ChainLayer& L) { return rank < (L.N / CC_BLOCK_N) * L.ks_l; };
  auto kb_lo = [&](const ChainLayer& L, int part) { return part * L.nkb / L.ks_l; };
  const bool manual_a = p.pack_rows > 0;

  if (threadIdx.x == 0) {
    for (int l = 0; l < CHAIN_MAX_LAYERS; ++l) {
      mbar_init(bar_w + 8 * l, 1);
      mbar_init(bar_a + 8 * l, 1);
    }
    mbar_init(bar_tfull, 1);
    mbar_init(bar_red, 1);
    mbar_init(bar_a0, 4);                                         // one arrival per epilogue warp
    fence_mbar_init();
    // the bytes the finishing CTAs of layer l - 1 will copy into my stages of layer l: armed before anybody can send
    for (int l = 1; l < p.n_layers; ++l) {
      const ChainLayer& L = p.L[l];
      if (!active(L)) continue;
      const int part = rank % L.ks_l;
      const int my_nkb = kb_lo(L, part + 1) - kb_lo(L, part);
      const ChainLayer& P = p.L[l - 1];
      mbar_arrive_expect_tx(bar_a + 8 * l, static_cast<uint32_t>(my_nkb * P.ks_l * P.rows_per * 128));
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), CC_NACC * CC_BLOCK_N);
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
    for (int l = 0; l < p.n_layers; ++l) {
      const ChainLayer& L = p.L[l];
      if (!active(L)) continue;
      const int slice = rank / L.ks_l, part = rank % L.ks_l;
      const int lo = kb_lo(L, part), hi = kb_lo(L, part + 1);
      if (hi == lo) continue;
      mbar_arrive_expect_tx(bar_w + 8 * l, static_cast<uint32_t>(hi - lo) * (CC_BLOCK_N * 128));
      for (int kb = lo; kb < hi; ++kb)
        tma_load_2d(smem_u32(sW) + L.w_smem_off + (kb - lo) * (CC_BLOCK_N * 128), p.tmaps + L.b_tm, kb * CC_K_ELEMS,
                    slice * CC_BLOCK_N, bar_w + 8 * l);
    }
  }
  if (p.early_weights) asm volatile("griddepcontrol.wait;" ::: "memory");

  // the per-column constants my epilogues will need: start them on their way from DRAM now
  if (warp >= 2 && threadIdx.x - 64 < p.n_layers) {
    const ChainLayer& L = p.L[threadIdx.x - 64];
    if (active(L) && L.epi.bias) asm volatile("prefetch.global.L2 [%0];" ::"l"(L.epi.bias + (rank / L.ks_l) * CC_BLOCK_N));
  }

  bool failed = false;
  uint32_t tphase = 0;           // parity of the accumulator-ready barrier (one completion per layer I am active in)
  uint32_t rphase = 0;           // parity of the partial-sum barrier (one completion per such layer with ks_l > 1)

  for (int l = 0; l < p.n_layers && !failed; ++l) {
    // (a by-value copy: fields read through a reference into the parameter space are re-fetched around every store)
    const ChainLayer L = p.L[l];
    if (!active(L)) continue;
    const int KS = L.ks_l, rows_per = L.rows_per;
    const int slice = rank / KS, part = rank % KS;
    const int lo = kb_lo(L, part), my_nkb = kb_lo(L, part + 1) - lo;
    const bool last = l + 1 == p.n_layers;
    uint8_t* region = sA + (l & 1) * REGION;
    uint8_t* send = sSend + (l & 1) * STAGE;
    uint8_t* outb = sOut + (l & 1) * STAGE;

    if (warp == 0) {
      if (lane == 0 && l == 0 && !manual_a && my_nkb > 0) {
        const uint32_t box_bytes = static_cast<uint32_t>((L.M < 128 ? (L.M + 7) / 8 * 8 : 128) * 128);
        mbar_arrive_expect_tx(bar_a, static_cast<uint32_t>(my_nkb) * box_bytes);
        for (int i = 0; i < my_nkb; ++i)
          tma_load_2d(smem_u32(region) + i * STAGE, p.tmaps + L.a_tm, (lo + i) * CC_K_ELEMS, 0, bar_a);
      }
    } else if (warp == 1) {
      if (lane == 0) {
        if (my_nkb == 0) {
          mbar_arrive(bar_tfull);                                 // nothing to multiply: my partial sums are zero
        } else {
          bool ok = mbar_wait(bar_w + 8 * l, 0);
          if (ok) ok = (l == 0 && manual_a) ? mbar_wait(bar_a0, 0) : mbar_wait_cluster(bar_a + 8 * l, 0);
          if (ok) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(region), b0 = smem_u32(sW) + L.w_smem_off;
            // at most 64 rows are ever finished: M = 64 (the M field of the descriptor is bits 24..28, in units of 16)
            const uint32_t idesc = (L.idesc & ~(0x1Fu << 24)) | ((64u >> 4) << 24);
            for (int i = 0; i < my_nkb; ++i) {
#pragma unroll
              for (int k = 0; k < 4; ++k)   // (each descriptor is built from its address, not stepped as an integer)
                umma_ss<KIND_TF32>(tmem_base + k * CC_BLOCK_N, make_smem_desc(a0 + i * STAGE + 32 * k, 16, 1024, SWZ_128B),
                                   make_smem_desc(b0 + i * (CC_BLOCK_N * 128) + 32 * k, 16, 1024, SWZ_128B), idesc, i != 0);
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
        // Row r of my k-blocks (thread per row): 16-byte chunks assembled from aligned 32-bit words of the
        // (arbitrarily aligned) source row with funnel shifts, zero beyond the row's K bytes and beyond row M, stored
        // where TMA would have put them (128-byte rows, 8-row groups of 1024 bytes, chunk index XOR row mod 8).
        const int r = et;
        const int a_rows = STAGE / 128;
        const int64_t kbytes = static_cast<int64_t>(L.K) * 4;
        const uint8_t* src_row = static_cast<const uint8_t*>(p.pack_src) + static_cast<int64_t>(r) * p.pack_src_pitch;
        if (r < a_rows) {
          for (int i = 0; i < my_nkb; ++i) {
            uint8_t* dst = region + i * STAGE + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const int64_t off = static_cast<int64_t>(lo + i) * 128 + c * 16;
              int64_t nv = kbytes - off;
              nv = r < L.M ? (nv > 16 ? 16 : nv) : 0;
              uint32_t o[4] = {0u, 0u, 0u, 0u};
              if (nv > 0) {
                const uintptr_t a = reinterpret_cast<uintptr_t>(src_row + off);
                const uint32_t sh = static_cast<uint32_t>(a & 3);
                const uint32_t* aw = reinterpret_cast<const uint32_t*>(a - sh);
                uint32_t w[5];
#pragma unroll
                for (int j = 0; j < 5; ++j) w[j] = (4 * j - static_cast<int>(sh) < nv) ? __ldg(aw + j) : 0u;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                  const uint32_t v = __funnelshift_r(w[j], w[j + 1], sh * 8);
                  const int64_t left = nv - 4 * j;
                  o[j] = left >= 4 ? v : (left <= 0 ? 0u : (v & ((1u << (8 * static_cast<int>(left))) - 1u)));
                }
              }
              *reinterpret_cast<uint4*>(dst + ((c ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
            }
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_a0);
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
      float4 bias4[8];
      if (finisher && L.epi.bias) {
        const float4* bp = reinterpret_cast<const float4*>(L.epi.bias + fcol);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          if (i < ncol4) bias4[i] = __ldg(bp + i);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) bias4[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
      const int act = L.epi.act;
      bool ok = cc_epi_all(mbar_wait(bar_tfull, tphase));
      float4 acc4[8];
      if (ok) {
        tc_fence_after();
        uint32_t r[32];
        if (my_nkb > 0 && q * 16 < rows_all) {
          uint32_t r1[32], r2[32], r3[32];
          const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
          tmem_ld32(t_row, r);
          tmem_ld32(t_row + CC_BLOCK_N, r1);
          tmem_ld32(t_row + 2 * CC_BLOCK_N, r2);
          tmem_ld32(t_row + 3 * CC_BLOCK_N, r3);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i)
            r[i] = __float_as_uint((__uint_as_float(r[i]) + __uint_as_float(r1[i])) +
                                   (__uint_as_float(r2[i]) + __uint_as_float(r3[i])));
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
          if (lane == 0) {
            const int base = rank - part;                         // first CTA of my group
            for (int d = 0; d < KS; ++d) {                        // rows [d rows_per, (d + 1) rows_per) belong to part d
              const int ra = max(d * rows_per, q * 16), rb = min((d + 1) * rows_per, q * 16 + 16);
              if (ra >= rb) continue;
              bulk_copy_to_cluster(mapa_shared(smem_u32(sRed) + static_cast<uint32_t>((part * rows_per + ra - d * rows_per) * 128), base + d),
                                   smem_u32(send) + static_cast<uint32_t>(ra * 128), static_cast<uint32_t>((rb - ra) * 128),
                                   mapa_shared(bar_red, base + d));
            }
          }
          ok = cc_epi_all(mbar_wait_cluster(bar_red, rphase));
          if (ok && finisher) {
#pragma unroll
            for (int c = 0; c < 4; ++c) acc4[c] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int s = 0; s < KS; ++s) {                        // fixed order: deterministic
              const uint8_t* src = sRed + (s * rows_per + frow) * 128;
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                const float4 v = *reinterpret_cast<const float4*>(src + (((half * 4 + c) ^ (frow & 7)) << 4));
                acc4[c].x += v.x; acc4[c].y += v.y; acc4[c].z += v.z; acc4[c].w += v.w;
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
          // bias and activation (fp32 chains only: this kernel takes no other)
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            if (c < ncol4) {
              float4 t = acc4[c];
              t.x = __fadd_rn(t.x, bias4[c].x); t.y = __fadd_rn(t.y, bias4[c].y);
              t.z = __fadd_rn(t.z, bias4[c].z); t.w = __fadd_rn(t.w, bias4[c].w);
              if (act == ACT_RELU) {
                t.x = fmaxf(t.x, 0.f); t.y = fmaxf(t.y, 0.f); t.z = fmaxf(t.z, 0.f); t.w = fmaxf(t.w, 0.f);
              } else if (act != ACT_NONE) {
                t.x = apply_act(t.x, act); t.y = apply_act(t.y, act); t.z = apply_act(t.z, act); t.w = apply_act(t.w, act);
              }
              acc4[c] = t;
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
            while (np + 1 < Nx.ks_l && (np + 1) * Nx.nkb / Nx.ks_l <= slice) ++np;     // the part that holds k-block `slice`
            const int st = slice - np * Nx.nkb / Nx.ks_l;                                // its stage there
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
    tmem_dealloc(tmem_base, CC_NACC * CC_BLOCK_N);
  }
  // no CTA leaves while another one of its cluster may still write into its shared memory or read a copy out of it
  // (every CTA has seen all copies addressed to it complete before it arrives here; nothing else is ordered)
  cluster_sync_all_relaxed();
}

size_t mlp_cluster_smem_bytes(size_t w_smem_bytes, int a_stages, int a_stage_bytes) {
  return ((2 * static_cast<size_t>(a_stages) * a_stage_bytes + 1023) & ~size_t(1023)) +
         (w_smem_bytes < 16384 ? size_t(16384) : w_smem_bytes) + CC_RED_BYTES + 4 * static_cast<size_t>(a_stage_bytes) + 1024 + 1024;
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
