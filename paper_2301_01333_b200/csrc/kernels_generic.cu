// Shape-generic CUDA-core kernels: the constant-weight prepack (Section V), the graph-entry reorder of
// inputs whose row pitch TMA cannot address (the pre-op reorder of Section IV / V), and reference-shaped
// GEMM / attention kernels for shapes the tcgen05 kernels do not take (GEMV tails, ragged sizes).
#include <cuda_bf16.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <utility>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

// ------------------------------------------------------------------------------------------------
// pack_rows: dst[r][0..dst_pitch) = src[r][0..src_pitch) followed by zeros.  Byte granular.
// ------------------------------------------------------------------------------------------------
__global__ void pack_rows_kernel(const uint8_t* __restrict__ src, uint8_t* __restrict__ dst, int rows,
                                 int64_t src_pitch, int64_t dst_pitch) {
  const int64_t words_per_row = dst_pitch / 4;   // dst_pitch is a multiple of 16
  const int64_t total = static_cast<int64_t>(rows) * words_per_row;
  for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
       i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t r = i / words_per_row, c = (i % words_per_row) * 4;
    const uint8_t* s = src + r * src_pitch;
    uint32_t w = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b)
      if (c + b < src_pitch) w |= static_cast<uint32_t>(s[c + b]) << (8 * b);
    *reinterpret_cast<uint32_t*>(dst + r * dst_pitch + c) = w;
  }
}

cudaError_t launch_pack_rows(const void* src, void* dst, int rows, int64_t src_pitch_bytes, int64_t dst_pitch_bytes,
                             cudaStream_t s) {
  const int64_t total = static_cast<int64_t>(rows) * (dst_pitch_bytes / 4);
  const int block = 256;
  const int grid = static_cast<int>(std::min<int64_t>((total + block - 1) / block, 148 * 8));
  pack_rows_kernel<<<std::max(grid, 1), block, 0, s>>>(static_cast<const uint8_t*>(src), static_cast<uint8_t*>(dst), rows,
                                                   src_pitch_bytes, dst_pitch_bytes);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// prepack_weight: Wt[n][k] = W[k][n] (or W[n][k]), k < K; zeros for K <= k < Kp.
// Tiled 32x32 transpose through shared memory so both sides are coalesced.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float round_to_tf32(float x) {
  uint32_t u;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(u) : "f"(x));
  return __uint_as_float(u);
}

template <typename T, bool TF32>
__global__ void prepack_weight_kernel(const T* __restrict__ W, T* __restrict__ Wt, int K, int N, int Kp,
                                      int transposed) {
  __shared__ T tile[32][33];
  const int k0 = blockIdx.x * 32, n0 = blockIdx.y * 32;
  const int tx = threadIdx.x, ty = threadIdx.y;   // 32 x 8
  for (int j = ty; j < 32; j += 8) {
    T v = T(0);
    if (!transposed) {
      const int k = k0 + j, n = n0 + tx;          // read W[k][n], n fastest
      if (k < K && n < N) v = W[static_cast<int64_t>(k) * N + n];
      tile[j][tx] = v;                            // tile[k][n]
    } else {
      const int n = n0 + j, k = k0 + tx;          // read W[n][k], k fastest
      if (k < K && n < N) v = W[static_cast<int64_t>(n) * K + k];
      tile[tx][j] = v;                            // tile[k][n]
    }
  }
  __syncthreads();
  for (int j = ty; j < 32; j += 8) {
    const int n = n0 + j, k = k0 + tx;            // write Wt[n][k], k fastest
    if (n < N && k < Kp) {
      T v = tile[tx][j];
      if constexpr (TF32) v = round_to_tf32(v);
      Wt[static_cast<int64_t>(n) * Kp + k] = v;
    }
  }
}

cudaError_t launch_prepack_weight(const void* W, void* Wt, int K, int N, int Kp, int transposed, int dtype,
                                  cudaStream_t s) {
  dim3 block(32, 8), grid((Kp + 31) / 32, (N + 31) / 32);
  if (dtype == GC_F32)
    prepack_weight_kernel<float, true><<<grid, block, 0, s>>>(static_cast<const float*>(W), static_cast<float*>(Wt), K, N,
                                                             Kp, transposed);
  else if (dtype == GC_BF16)
    prepack_weight_kernel<uint16_t, false><<<grid, block, 0, s>>>(static_cast<const uint16_t*>(W),
                                                                 static_cast<uint16_t*>(Wt), K, N, Kp, transposed);
  else
    prepack_weight_kernel<uint8_t, false><<<grid, block, 0, s>>>(static_cast<const uint8_t*>(W),
                                                                static_cast<uint8_t*>(Wt), K, N, Kp, transposed);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Self-test of the bounded-wait error path: a wait on a barrier that nobody arrives on, limited in time.
// ------------------------------------------------------------------------------------------------
__global__ void bounded_wait_selftest_kernel(uint32_t* status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  const uint32_t b = smem_u32(&bar);
  if (threadIdx.x == 0) {
    mbar_init(b, 1);
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const uint64_t t0 = globaltimer_ns();
    bool done = false;
    while (!done && globaltimer_ns() - t0 < limit_ns) done = mbar_try_wait(b, 0, 1000u);
    if (!done) report(status, DEV_TIMEOUT_OTHER);
  }
}

cudaError_t launch_bounded_wait_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t s) {
  bounded_wait_selftest_kernel<<<1, 32, 0, s>>>(status, limit_ns);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Compensated weight (Section V, constant weight preprocessing; Section VII "compensated weight"):
// sum_k (a_k - a_z) w_kn = sum_k a_k w_kn - a_z colsum(W)_n.  The second term depends on constants only and is
// formed once from the prepacked s8 weight Wt[N][Kp]; one warp per output column.
// ------------------------------------------------------------------------------------------------
__global__ void weight_compensation_kernel(const int8_t* __restrict__ Wt, int N, int Kp, int a_zp, int* __restrict__ comp) {
  const int lane = threadIdx.x & 31;
  const int n = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  if (n >= N) return;
  const int8_t* row = Wt + static_cast<int64_t>(n) * Kp;
  int acc = 0;
  for (int k = lane; k < Kp; k += 32) acc += row[k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) comp[n] = a_zp * acc;
}

cudaError_t launch_weight_compensation(const void* Wt, int N, int Kp, int a_zp, int* comp, cudaStream_t s) {
  const int threads = 256, blocks = (N * 32 + threads - 1) / threads;
  weight_compensation_kernel<<<blocks, threads, 0, s>>>(static_cast<const int8_t*>(Wt), N, Kp, a_zp, comp);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// gemm_simt: one warp per output element, lanes stride the reduction axis, fixed-order shuffle tree.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float load_as_float(const void* p, int64_t i, int dtype) {
  if (dtype == GC_F32) return static_cast<const float*>(p)[i];
  return __bfloat162float(static_cast<const __nv_bfloat16*>(p)[i]);
}
__device__ __forceinline__ int load_as_int(const void* p, int64_t i, int dtype) {
  if (dtype == GC_U8) return static_cast<const uint8_t*>(p)[i];
  if (dtype == GC_S8) return static_cast<const int8_t*>(p)[i];
  return static_cast<const int*>(p)[i];
}
__device__ __forceinline__ int dtype_size(int dtype) {
  return dtype == GC_F32 || dtype == GC_S32 ? 4 : (dtype == GC_BF16 ? 2 : 1);
}

__global__ void gemm_simt_kernel(const GemmSimtParams p) {
  const int lane = threadIdx.x & 31;
  const int64_t warp = (blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x) >> 5;
  const int64_t per_batch = static_cast<int64_t>(p.M) * p.N;
  if (warp >= per_batch * p.batch) return;
  const int b = static_cast<int>(warp / per_batch);
  const int m = static_cast<int>((warp % per_batch) / p.N), n = static_cast<int>(warp % p.N);
  const char* A = static_cast<const char*>(p.A) + (b * p.a_batch_stride + m * p.a_pitch) * dtype_size(p.a_dtype);
  const char* Wt = static_cast<const char*>(p.Wt) + (b * p.w_batch_stride + n * p.w_pitch) * dtype_size(p.w_dtype);
  uint32_t raw;
  if (p.epi.acc_is_int) {
    int acc = 0;
    for (int k = lane; k < p.K; k += 32)
      acc += (load_as_int(A, k, p.a_dtype) - p.a_zp) * (load_as_int(Wt, k, p.w_dtype) - p.w_zp);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    raw = static_cast<uint32_t>(acc);
  } else {
    float acc = 0.f;
    for (int k = lane; k < p.K; k += 32) acc = fmaf(load_as_float(A, k, p.a_dtype), load_as_float(Wt, k, p.w_dtype), acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    raw = __float_as_uint(acc);
  }
  if (lane == 0) {
    const int osz = (p.epi.acc_is_int && !p.epi.has_dq) ? 4 : dtype_size(p.epi.out_dtype);
    char* row = static_cast<char*>(p.out) + (b * p.out_batch_stride + m * p.out_pitch) * osz;
    epi_store1(raw, row, n, p.epi);
  }
}

cudaError_t ensure_dynamic_smem(const void* kern, size_t smem) {
  static std::mutex mu;
  static std::map<std::pair<const void*, int>, size_t> done;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> lock(mu);
  size_t& have = done[std::make_pair(kern, dev)];
  if (have >= smem && have != 0) return cudaSuccess;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e == cudaSuccess) have = smem;
  return e;
}

cudaError_t launch_gemm_simt(const GemmSimtParams& p, cudaStream_t s) {
  const int64_t warps = static_cast<int64_t>(p.M) * p.N * p.batch;
  const int block = 256;
  const int64_t grid = (warps * 32 + block - 1) / block;
  if (grid > 0x7FFFFFFFLL) return cudaErrorInvalidValue;          // one warp per output element: beyond the x-dimension limit
  gemm_simt_kernel<<<static_cast<unsigned>(std::max<int64_t>(grid, 1)), block, 0, s>>>(p);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// sdpa_simt: one warp per query row; scores live in shared memory.
// ------------------------------------------------------------------------------------------------
constexpr int SDPA_SIMT_WARPS = 4;

__global__ void sdpa_simt_kernel(const SdpaParams p) {
  extern __shared__ float sdpa_smem[];
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  float* x = sdpa_smem + static_cast<size_t>(w) * p.S;
  const int64_t row = blockIdx.x * static_cast<int64_t>(SDPA_SIMT_WARPS) + w;
  const int64_t rows = static_cast<int64_t>(p.B) * p.H * p.S;
  if (row >= rows) return;
  const int64_t bh = row / p.S;
  const int b = static_cast<int>(bh / p.H);
  const int64_t base = bh * p.S * p.D;
  const int S = p.S, D = p.D;
  const int esz = p.is_int8 ? 1 : 2;
  const char* Q = static_cast<const char*>(p.Q) + row * D * esz;
  const char* K = static_cast<const char*>(p.K) + base * esz;
  const char* V = static_cast<const char*>(p.V) + base * esz;
  const int qdt = p.is_int8 ? (p.q_signed ? GC_S8 : GC_U8) : GC_BF16;
  const int kdt = p.is_int8 ? (p.k_signed ? GC_S8 : GC_U8) : GC_BF16;
  const int vdt = p.is_int8 ? (p.v_signed ? GC_S8 : GC_U8) : GC_BF16;

  float mx = -INFINITY;
  for (int j = lane; j < S; j += 32) {
    float t;
    if (p.is_int8) {
      int acc = 0;
      for (int d = 0; d < D; ++d)
        acc += (load_as_int(Q, d, qdt) - p.zp_q) * (load_as_int(K, static_cast<int64_t>(j) * D + d, kdt) - p.zp_k);
      t = __fmul_rn(__int2float_rn(acc), p.dq1);
      t = __fmul_rn(t, p.scalar);
    } else {
      float acc = 0.f;
      for (int d = 0; d < D; ++d)
        acc = fmaf(load_as_float(Q, d, qdt), load_as_float(K, static_cast<int64_t>(j) * D + d, kdt), acc);
      t = __fmul_rn(acc, p.scalar);
    }
    if (p.mask) t = __fadd_rn(t, p.mask[static_cast<int64_t>(b) * S + j]);
    x[j] = t;
    mx = fmaxf(mx, t);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  float sum = 0.f;
  for (int j = lane; j < S; j += 32) {
    const float e = expf(x[j] - mx);
    x[j] = e;
    sum += e;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  const float rl = 1.0f / sum;
  for (int j = lane; j < S; j += 32) {
    const float pj = x[j] * rl;
    if (p.p_is_quant) {
      const int code = quantize_value(pj, p.inv_p, p.zp_p, 0, 255);
      if (p.P_out) static_cast<uint8_t*>(p.P_out)[row * S + j] = static_cast<uint8_t>(code);
      x[j] = static_cast<float>(code - p.zp_p);
    } else {
      const __nv_bfloat16 pb = __float2bfloat16_rn(pj);
      if (p.P_out) static_cast<__nv_bfloat16*>(p.P_out)[row * S + j] = pb;
      x[j] = __bfloat162float(pb);
    }
  }
  __syncwarp();
  for (int d = lane; d < D; d += 32) {
    if (p.is_int8) {
      int acc = 0;
      for (int j = 0; j < S; ++j)
        acc += static_cast<int>(x[j]) * (load_as_int(V, static_cast<int64_t>(j) * D + d, vdt) - p.zp_v);
      float t = __fmul_rn(__int2float_rn(acc), p.dq2);
      const int lo = p.out_dtype == GC_U8 ? 0 : -128, hi = p.out_dtype == GC_U8 ? 255 : 127;
      static_cast<uint8_t*>(p.O)[row * D + d] = static_cast<uint8_t>(quantize_value(t, p.inv_o, p.zp_o, lo, hi));
    } else {
      float acc = 0.f;
      for (int j = 0; j < S; ++j) acc = fmaf(x[j], load_as_float(V, static_cast<int64_t>(j) * D + d, vdt), acc);
      static_cast<__nv_bfloat16*>(p.O)[row * D + d] = __float2bfloat16_rn(acc);
    }
  }
}

cudaError_t launch_sdpa_simt(const SdpaParams& p, cudaStream_t s) {
  const int64_t rows = static_cast<int64_t>(p.B) * p.H * p.S;
  const size_t smem = static_cast<size_t>(SDPA_SIMT_WARPS) * p.S * sizeof(float);
  if (smem > 48 * 1024) {
    cudaError_t e = ensure_dynamic_smem(reinterpret_cast<const void*>(sdpa_simt_kernel), smem);
    if (e != cudaSuccess) return e;
  }
  const int64_t grid = (rows + SDPA_SIMT_WARPS - 1) / SDPA_SIMT_WARPS;
  sdpa_simt_kernel<<<static_cast<unsigned>(grid), SDPA_SIMT_WARPS * 32, smem, s>>>(p);
  return cudaGetLastError();
}

}  // namespace gc
