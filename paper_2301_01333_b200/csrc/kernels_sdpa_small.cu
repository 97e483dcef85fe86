// The bf16 attention block (Section VII, "MHA": Q.K^T, scale, additive mask, softmax, .V as one fused op) for
// 128-key heads of width 64, one (batch, head) unit per CTA and several CTAs per SM.
//
// A unit of this shape is a chain of fixed latencies (operands from DRAM, two short MMAs, 128 exponentials per row
// between them), and a single persistent CTA per SM walks those chains one after the other.  Here the CTA is made
// small enough that four of them share an SM - 50 KB of shared memory, 128 tensor-memory columns, 160 threads - and
// the hardware interleaves their chains: while one unit waits for its operands or its MMA, the exponentials of
// another keep the special-function unit busy.  The whole batch of the evaluation's shape (384 units) is resident at
// once on 148 SMs, so there is neither a unit loop nor a tail wave.
//   warp 0      one thread: TMA loads of Q, K, V; S = Q.K^T into tensor-memory columns 0..127; later O = P.V into
//               columns 0..63, which the softmax warps have finished reading by then
//   warps 1..4  one query row per thread (tensor-memory lane): row maximum in a first sweep over the 128 scores,
//               exponentials, row sum and the bf16 probabilities in a second one; P goes to shared memory as the
//               K-major A operand of the second MMA, over Q and K, which nobody reads any more; the output row is
//               scaled by 1 / row sum when it leaves tensor memory (the normalisation of the softmax, deferred) and
//               stored straight to global memory, 128 contiguous bytes per thread
// Every wait is bounded; a wait that gives up records a code in the status word and the CTA leaves in order.
#include <cuda_bf16.h>

#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

namespace {
constexpr int SM_THREADS = 160;
constexpr int SM_S = 128, SM_D = 64;
constexpr int SM_TILE = 128 * 128;                              // one operand tile: 128 rows of 128 bytes
constexpr int SM_SMEM = 3 * SM_TILE + 1024 + 1024;              // Q, K, V; mask and barriers; alignment slack
constexpr float SM_LOG2E = 1.4426950408889634f;

__device__ __forceinline__ float sm_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
}  // namespace

__global__ void __launch_bounds__(SM_THREADS, 3)
sdpa_small_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SdpaParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;                                           // later the first 64 keys of P
  uint8_t* sK = smem + SM_TILE;                                 // later the second 64 keys of P
  uint8_t* sV = smem + 2 * SM_TILE;
  float* sMask = reinterpret_cast<float*>(smem + 3 * SM_TILE);  // mask row times log2(e)
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 3 * SM_TILE + 512);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
  const uint32_t bar_qk = smem_u32(bars), bar_v = bar_qk + 8, bar_s = bar_qk + 16, bar_p = bar_qk + 24, bar_o = bar_qk + 32;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int bh = blockIdx.x;                                    // my unit: (batch, head)

  if (threadIdx.x == 0) {
    mbar_init(bar_qk, 1);
    mbar_init(bar_v, 1);
    mbar_init(bar_s, 1);
    mbar_init(bar_p, 4);                                        // one arrival per softmax warp
    mbar_init(bar_o, 1);
    fence_mbar_init();
    tma_prefetch_desc(&tmQ);
    tma_prefetch_desc(&tmK);
    tma_prefetch_desc(&tmV);
  }
  if (warp == 0) {
    __syncwarp();
    tmem_alloc(smem_u32(tmem_slot), 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Everything above may overlap the tail of the preceding kernel on the stream, and so may the trip of my operands
  // from DRAM into the L2: a prefetch consumes nothing, and whatever that kernel still writes goes through the same L2.
  // Its results are read from the wait on.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (threadIdx.x == 0) {
    tma_prefetch_2d(&tmQ, 0, bh * SM_S);
    tma_prefetch_2d(&tmK, 0, bh * SM_S);
    tma_prefetch_2d(&tmV, 0, bh * SM_S);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");

  bool failed = false;
  if (warp == 0) {
    if (lane == 0) {
      mbar_arrive_expect_tx(bar_qk, 2 * SM_TILE);
      tma_load_2d(smem_u32(sQ), &tmQ, 0, bh * SM_S, bar_qk);
      tma_load_2d(smem_u32(sK), &tmK, 0, bh * SM_S, bar_qk);
      mbar_arrive_expect_tx(bar_v, SM_TILE);
      tma_load_2d(smem_u32(sV), &tmV, 0, bh * SM_S, bar_v);
      const uint32_t idesc1 = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, 128);
      const uint32_t idesc2 = make_idesc(ACC_F32, FMT_BF16, FMT_BF16, 128, SM_D, 0, 1);
      if (mbar_wait(bar_qk, 0)) {
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < 4; ++k)                             // 16 of the 64 head-dimension elements per MMA
          umma_ss<KIND_BF16>(tmem_base, make_smem_desc(smem_u32(sQ) + 32 * k, 16, 1024, SWZ_128B),
                             make_smem_desc(smem_u32(sK) + 32 * k, 16, 1024, SWZ_128B), idesc1, k != 0);
        umma_commit(bar_s);
        if (mbar_wait(bar_p, 0) && mbar_wait(bar_v, 0)) {
          tc_fence_after();
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)                        // 16 keys per MMA
            // A: P, K-major, two 64-key tiles of 128-byte rows.  B: V as stored, [key][d] = MN-major: one key per
            // 128-byte row, 8-key groups 1024 bytes apart
            umma_ss<KIND_BF16>(tmem_base, make_smem_desc(smem_u32(sQ) + (ks >> 2) * SM_TILE + (ks & 3) * 32, 16, 1024, SWZ_128B),
                               make_smem_desc(smem_u32(sV) + ks * 16 * 128, 1024, 1024, SWZ_128B), idesc2, ks != 0);
          umma_commit(bar_o);
        } else {
          failed = true;
        }
      } else {
        failed = true;
      }
      if (failed) report(p.status, DEV_TIMEOUT_MMA);
    }
  } else {
    const int q = warp & 3;                                     // the tensor-memory lane quarter this warp may access
    const int r = q * 32 + lane;                                // my query row
    const int t = static_cast<int>(threadIdx.x) - 32;           // 0..127
    const int b = bh / p.H;
    sMask[t] = p.mask ? __ldg(p.mask + static_cast<int64_t>(b) * SM_S + t) * SM_LOG2E : 0.0f;
    asm volatile("bar.sync 1, 128;" ::: "memory");              // the four softmax warps only
    const float c2 = p.scalar * SM_LOG2E;
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const uint32_t row_off = (r >> 3) * 1024 + (r & 7) * 128;
    if (__all_sync(0xffffffffu, mbar_wait(bar_s, 0) ? 1 : 0)) {
      tc_fence_after();
      uint32_t v[32];
      // first sweep: the row maximum of the scaled, masked scores
      float cm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        tmem_ld32(t_row + 32 * c, v);
        tmem_wait_ld();
        const float4* mk4 = reinterpret_cast<const float4*>(sMask + 32 * c);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 mv = mk4[i];
          cm[0] = fmaxf(cm[0], fmaf(__uint_as_float(v[4 * i + 0]), c2, mv.x));
          cm[1] = fmaxf(cm[1], fmaf(__uint_as_float(v[4 * i + 1]), c2, mv.y));
          cm[2] = fmaxf(cm[2], fmaf(__uint_as_float(v[4 * i + 2]), c2, mv.z));
          cm[3] = fmaxf(cm[3], fmaf(__uint_as_float(v[4 * i + 3]), c2, mv.w));
        }
      }
      const float m = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
      const float ms = m == -INFINITY ? 0.0f : m;               // a row without an unmasked key: all exponentials are zero
      // second sweep: exponentials, their sum, bf16 probabilities into the A operand of the second MMA
      float ls[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        tmem_ld32(t_row + 32 * c, v);
        tmem_wait_ld();
        const float4* mk4 = reinterpret_cast<const float4*>(sMask + 32 * c);
        uint32_t w[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float4 mv = mk4[i];
          const float e0 = sm_ex2(fmaf(__uint_as_float(v[4 * i + 0]), c2, mv.x) - ms);
          const float e1 = sm_ex2(fmaf(__uint_as_float(v[4 * i + 1]), c2, mv.y) - ms);
          const float e2 = sm_ex2(fmaf(__uint_as_float(v[4 * i + 2]), c2, mv.z) - ms);
          const float e3 = sm_ex2(fmaf(__uint_as_float(v[4 * i + 3]), c2, mv.w) - ms);
          ls[0] += e0; ls[1] += e1; ls[2] += e2; ls[3] += e3;
          __nv_bfloat162 h0 = __floats2bfloat162_rn(e0, e1), h1 = __floats2bfloat162_rn(e2, e3);
          w[2 * i] = *reinterpret_cast<uint32_t*>(&h0);
          w[2 * i + 1] = *reinterpret_cast<uint32_t*>(&h1);
        }
        // my 32 keys of this sweep step: four 16-byte chunks of the (c / 2)-th 64-key tile
        uint8_t* blk = sQ + (c >> 1) * SM_TILE + row_off;
        const int c0 = (c & 1) * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4*>(blk + (((c0 + i) ^ (r & 7)) * 16)) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
      }
      const float lsum = (ls[0] + ls[1]) + (ls[2] + ls[3]);
      // P is complete and the score columns have been read for the last time
      fence_proxy_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_p);
      if (__all_sync(0xffffffffu, mbar_wait(bar_o, 0) ? 1 : 0)) {
        tc_fence_after();
        const float rl = 1.0f / lsum;                           // the softmax's division, deferred to the output
        uint8_t* dst = static_cast<uint8_t*>(p.O) + (static_cast<int64_t>(bh) * SM_S + r) * (SM_D * 2);
#pragma unroll 1
        for (int hcol = 0; hcol < 2; ++hcol) {
          tmem_ld32(t_row + 32 * hcol, v);
          tmem_wait_ld();
          uint32_t w[16];
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[2 * i]) * rl, __uint_as_float(v[2 * i + 1]) * rl);
            w[i] = *reinterpret_cast<uint32_t*>(&hh);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<uint4*>(dst + hcol * 64 + i * 16) = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
        }
      } else {
        failed = true;
      }
    } else {
      failed = true;
    }
    if (failed) report(p.status, DEV_TIMEOUT_EPILOGUE);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 128);
  }
}

bool sdpa_small_supported(int S, int D, int is_int8) { return !is_int8 && S == SM_S && D == SM_D; }

cudaError_t launch_sdpa_small(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                              cudaStream_t s) {
  cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(sdpa_small_kernel), SM_SMEM);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t lc = {};
  lc.gridDim = dim3(static_cast<unsigned>(p.B * p.H));
  lc.blockDim = dim3(SM_THREADS);
  lc.dynamicSmemBytes = SM_SMEM;
  lc.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, sdpa_small_kernel, tmQ, tmK, tmV, p);
}

}  // namespace gc
