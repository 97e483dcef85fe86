// Epilogue building blocks shared by the tcgen05 GEMM kernels: post-op evaluation on 32 accumulator words of
// one row (compile-time accumulator kind and activation) and packing into the output element type.
#pragma once
#include <cuda_bf16.h>

#include "epilogue.cuh"
#include "gc_internal.h"
#include "ptx.cuh"

namespace gc {

enum OutKind { OUT_F32 = 0, OUT_BF16 = 1, OUT_Q8 = 2, OUT_RAW32 = 3 };
__host__ __device__ constexpr int out_bytes(int ok) { return ok == OUT_BF16 ? 2 : (ok == OUT_Q8 ? 1 : 4); }

// 32 accumulator words of one row -> 32 post-op values (fp32), columns n0 .. n0+31
template <int KIND, int ACT>
__device__ __forceinline__ void epi_values32(const uint32_t (&raw)[32], float (&t)[32], int n0, int n_end,
                                             const Epilogue& e) {
  float b[32];
  if (e.bias) {
    const float4* bp = reinterpret_cast<const float4*>(e.bias + n0);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      // columns at or beyond n_end belong to a clipped tile tail: never read the bias there.  The pointer
      // may address global memory or a shared-memory copy of the tile's bias slice (generic load).
      const float4 v = n0 + 4 * i < n_end ? bp[i] : make_float4(0.f, 0.f, 0.f, 0.f);
      b[4 * i] = v.x; b[4 * i + 1] = v.y; b[4 * i + 2] = v.z; b[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 32; ++i) b[i] = 0.f;
  }
  // integer path: optional per-column compensation and per-column scales (global memory, a multiple of 16
  // columns is always allocated so whole vectors inside [n0, n_end rounded up to 16) are readable)
  int c[32];
  float dq[32];
  if constexpr (KIND == KIND_I8) {
    if (e.comp) {
      const int4* cp = reinterpret_cast<const int4*>(e.comp + n0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int4 v = n0 + 4 * i < n_end ? __ldg(cp + i) : make_int4(0, 0, 0, 0);
        c[4 * i] = v.x; c[4 * i + 1] = v.y; c[4 * i + 2] = v.z; c[4 * i + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) c[i] = 0;
    }
    if (e.dqv) {
      const float4* dp = reinterpret_cast<const float4*>(e.dqv + n0);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float4 v = n0 + 4 * i < n_end ? __ldg(dp + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        dq[4 * i] = v.x; dq[4 * i + 1] = v.y; dq[4 * i + 2] = v.z; dq[4 * i + 3] = v.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) dq[i] = e.dq;
    }
  }
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float x;
    if constexpr (KIND == KIND_I8) {
      x = __fmul_rn(__int2float_rn(static_cast<int>(raw[i]) - c[i]), dq[i]);
      x = e.bias ? __fadd_rn(x, b[i]) : x;                      // separately rounded on the integer path
    } else {
      x = __uint_as_float(raw[i]) + b[i];
    }
    if constexpr (ACT == ACT_RELU) {
      x = fmaxf(x, 0.f);
    } else if constexpr (ACT == ACT_GELU_TANH) {
      // 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3))) = h + h tanh(x (c0 + c1 x^2)), h = x/2
      const float x2 = x * x;
      const float u = x * fmaf(x2, 0.7978845608028654f * 0.044715f, 0.7978845608028654f);
      const float h = 0.5f * x;
      x = fmaf(h, tanh_approx(u), h);
    } else if constexpr (ACT == ACT_SIGMOID) {
      x = 1.0f / (1.0f + expf(-x));
    }
    t[i] = x;
  }
}

// post-op values -> packed output words (NW = 32 * out_bytes / 4)
template <int OUT>
__device__ __forceinline__ void epi_pack32(const float (&t)[32], uint32_t* w, const Epilogue& e) {
  if constexpr (OUT == OUT_F32) {
#pragma unroll
    for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(t[i]);
  } else if constexpr (OUT == OUT_BF16) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(t[2 * i], t[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
  } else {
    const int lo = e.out_dtype == GC_U8 ? 0 : -128, hi = e.out_dtype == GC_U8 ? 255 : 127;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t word = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k)
        word |= static_cast<uint32_t>(quantize_value(t[4 * i + k], e.inv, e.zp, lo, hi) & 0xFF) << (8 * k);
      w[i] = word;
    }
  }
}

template <int KIND, int OUT>
__device__ __forceinline__ void epi_chunk32(const uint32_t (&raw)[32], uint32_t* w, int n0, int n_end,
                                            const Epilogue& e) {
  if constexpr (OUT == OUT_RAW32) {
    if (KIND == KIND_I8 && e.comp) {
#pragma unroll
      for (int i = 0; i < 32; ++i) w[i] = raw[i] - static_cast<uint32_t>(n0 + i < n_end ? __ldg(e.comp + n0 + i) : 0);
    } else {
#pragma unroll
      for (int i = 0; i < 32; ++i) w[i] = raw[i];
    }
  } else {
    float t[32];
    switch (e.act) {
      case ACT_RELU: epi_values32<KIND, ACT_RELU>(raw, t, n0, n_end, e); break;
      case ACT_GELU_TANH: epi_values32<KIND, ACT_GELU_TANH>(raw, t, n0, n_end, e); break;
      case ACT_SIGMOID: epi_values32<KIND, ACT_SIGMOID>(raw, t, n0, n_end, e); break;
      default: epi_values32<KIND, ACT_NONE>(raw, t, n0, n_end, e); break;
    }
    epi_pack32<OUT>(t, w, e);
  }
}

}  // namespace gc
