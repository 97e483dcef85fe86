// gc_matmul_s32_noalloc: an int8 matmul entry point for callers that are not allowed to allocate.
//
// Who needs this: code that runs where cudaMalloc is off limits - inside a real-time loop with a fixed
// memory plan, under an allocator that owns every byte of the device and hands nothing out at run time,
// or in a process that is only permitted to launch work on memory it was given.  The regular path needs
// a caller-provided workspace for the prepacked (transposed, zero-padded) weight; here that scratch is
// a fixed array inside the library image instead, so the caller passes only inputs and outputs.
//
// The price: the array is part of every CUDA context that loads this library (GC_NOALLOC_SCRATCH_BYTES
// of device memory per GPU, held until the process exits), its size caps the problem, and every call
// shares it.  Calls that may overlap on the GPU - two streams, or two host threads - race on it; keep
// them on one stream or serialise them yourself.  The array keeps whatever the previous call left: this
// entry point rewrites every byte it later reads (including the zero padding of the reduction axis), so
// nothing needs clearing between calls.
#include <cuda_runtime.h>

#include <mutex>

#include "gc_internal.h"

using namespace gc;

#define GC_NOALLOC_SCRATCH_BYTES (1u << 20)

// The scratch lives in the library image.  In host code this name is only a handle for
// cudaGetSymbolAddress - it is NOT a device address and must never be passed to a kernel directly.
static __device__ __align__(256) unsigned char g_noalloc_scratch[GC_NOALLOC_SCRATCH_BYTES];

static std::mutex g_noalloc_mu;
static void* g_noalloc_ptr[64] = {};   // device address of the array, per device ordinal

// Resolve the array's device address for the current device (once per device).
static cudaError_t noalloc_scratch(void** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_noalloc_ptr[dev] = p;
  }
  *out = g_noalloc_ptr[dev];
  return cudaSuccess;
}

gc_status_t gc_set_error(gc_status_t st, const char* msg);   // gc_api.cu

extern "C" size_t gc_noalloc_scratch_bytes(void) { return GC_NOALLOC_SCRATCH_BYTES; }

extern "C" gc_status_t gc_matmul_s32_noalloc(void* cuda_stream, const void* a_dev, const void* w_dev, void* out_dev,
                                             int32_t m, int32_t k, int32_t n, int32_t a_zero_point) {
  if (!a_dev || !w_dev || !out_dev) return gc_set_error(GC_ERR_INVALID_ARG, "gc_matmul_s32_noalloc: null pointer");
  if (m <= 0 || k <= 0 || n <= 0) return gc_set_error(GC_ERR_SHAPE, "gc_matmul_s32_noalloc: non-positive dimension");
  if (reinterpret_cast<uintptr_t>(out_dev) % 4) return gc_set_error(GC_ERR_ALIGNMENT, "gc_matmul_s32_noalloc: output must be 4-byte aligned");
  if (a_zero_point < 0 || a_zero_point > 255)
    return gc_set_error(GC_ERR_INVALID_ARG, "gc_matmul_s32_noalloc: the zero point of a u8 operand lies in 0..255");
  // |a - zp| <= 255 and |w| <= 128: the exact sum stays inside s32 for k up to 65536
  if (k > 65536) return gc_set_error(GC_ERR_UNSUPPORTED, "gc_matmul_s32_noalloc: k above 65536 could overflow the s32 result");
  // one warp per output element, eight warps per block, at most 2^31 - 1 blocks
  if (static_cast<int64_t>(m) * n > 8LL * 0x7FFFFFFFLL)
    return gc_set_error(GC_ERR_UNSUPPORTED, "gc_matmul_s32_noalloc: m * n exceeds what one launch covers");
  const int64_t kp = (static_cast<int64_t>(k) + 127) / 128 * 128;   // reduction axis padded to 128 bytes
  if (kp * n > static_cast<int64_t>(GC_NOALLOC_SCRATCH_BYTES))
    return gc_set_error(GC_ERR_UNSUPPORTED,
                        "gc_matmul_s32_noalloc: n * round_up(k, 128) exceeds the built-in scratch of 1 MiB; "
                        "use gc_compile / gc_execute with a caller-provided workspace");
  void* scratch = nullptr;
  cudaError_t e = noalloc_scratch(&scratch);
  if (e != cudaSuccess) return gc_set_error(GC_ERR_CUDA, cudaGetErrorString(e));
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // 1. weights [K,N] -> scratch [N][Kp], reduction axis contiguous, every padding byte written as zero
  e = launch_prepack_weight(w_dev, scratch, k, n, static_cast<int>(kp), /*transposed=*/0, GC_S8, st);
  if (e != cudaSuccess) return gc_set_error(GC_ERR_CUDA, cudaGetErrorString(e));
  // 2. exact s32 accumulators from the prepacked weights
  GemmSimtParams g = {};
  g.A = a_dev;
  g.Wt = scratch;
  g.a_pitch = k;
  g.w_pitch = kp;
  g.M = m;
  g.N = n;
  g.K = k;
  g.batch = 1;
  g.a_dtype = GC_U8;
  g.w_dtype = GC_S8;
  g.a_zp = a_zero_point;
  g.w_zp = 0;
  g.out = out_dev;
  g.out_pitch = n;
  g.epi.acc_is_int = 1;
  g.epi.out_dtype = GC_S32;
  e = launch_gemm_simt(g, st);
  if (e != cudaSuccess) return gc_set_error(GC_ERR_CUDA, cudaGetErrorString(e));
  return GC_OK;
}
