// Per-element post-op evaluation shared by the GEMM kernels (tcgen05 and CUDA-core variants).
#pragma once
#include <cuda_bf16.h>

#include "gc_internal.h"

namespace gc {

__device__ __forceinline__ float tanh_approx(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float apply_act(float t, int act) {
  switch (act) {
    case ACT_RELU:
      return fmaxf(t, 0.0f);
    case ACT_GELU_TANH: {
      // 0.5 x (1 + tanh(sqrt(2/pi) (x + 0.044715 x^3)))
      const float u = 0.7978845608028654f * (t + 0.044715f * t * t * t);
      return 0.5f * t * (1.0f + tanh_approx(u));
    }
    case ACT_SIGMOID:
      return 1.0f / (1.0f + expf(-t));
    default:
      return t;
  }
}

// The same out of line: for kernels whose code runs once per launch (the small-batch chain kernels), where every
// inlined copy of the exponential / tanh sequences is instruction-cache misses and nothing else.
static __device__ __noinline__ float apply_act_cold(float t, int act) { return apply_act(t, act); }

// Value after dequantize / bias / activation.  `raw` holds the accumulator bits (s32 or f32).
__device__ __forceinline__ float epi_value(uint32_t raw, int n, const Epilogue& e) {
  float t;
  if (e.acc_is_int) {
    t = __int2float_rn(static_cast<int>(raw) - (e.comp ? __ldg(e.comp + n) : 0));
    t = __fmul_rn(t, e.dqv ? __ldg(e.dqv + n) : e.dq);
  } else {
    t = __uint_as_float(raw);
  }
  if (e.bias) t = __fadd_rn(t, __ldg(e.bias + n));
  return apply_act(t, e.act);
}

// saturate(rne(t * inv) + zp) to u8 / s8
__device__ __forceinline__ int quantize_value(float t, float inv, int zp, int lo, int hi) {
  int r = __float2int_rn(__fmul_rn(t, inv));      // cvt.rni.s32.f32 saturates
  r = min(max(r, -(1 << 24)), 1 << 24);           // keep r + zp free of overflow
  return min(max(r + zp, lo), hi);
}

// Per-column constants of NC (8 or 16) consecutive output columns (bias, dequantisation scale, zero-point
// compensation).  Loading them is separated from using them so that a kernel can issue the loads before it waits for
// its accumulators.
template <int NC>
struct EpiColsT {
  float b[NC];
  float dq[NC];
  int c[NC];
};
using EpiCols16 = EpiColsT<16>;

template <int NC>
__device__ __forceinline__ void epi_load_cols(EpiColsT<NC>& k, int n0, const Epilogue& e) {
  if (e.comp) {
    const int4* cp = reinterpret_cast<const int4*>(e.comp + n0);
#pragma unroll
    for (int i = 0; i < NC / 4; ++i) {
      const int4 v = __ldg(cp + i);
      k.c[4 * i] = v.x; k.c[4 * i + 1] = v.y; k.c[4 * i + 2] = v.z; k.c[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < NC; ++i) k.c[i] = 0;
  }
  if (e.bias) {
    const float4* bp = reinterpret_cast<const float4*>(e.bias + n0);
#pragma unroll
    for (int i = 0; i < NC / 4; ++i) {
      const float4 v = __ldg(bp + i);
      k.b[4 * i] = v.x; k.b[4 * i + 1] = v.y; k.b[4 * i + 2] = v.z; k.b[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < NC; ++i) k.b[i] = 0.f;
  }
  if (e.dqv) {
    const float4* dp = reinterpret_cast<const float4*>(e.dqv + n0);
#pragma unroll
    for (int i = 0; i < NC / 4; ++i) {
      const float4 v = __ldg(dp + i);
      k.dq[4 * i] = v.x; k.dq[4 * i + 1] = v.y; k.dq[4 * i + 2] = v.z; k.dq[4 * i + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < NC; ++i) k.dq[i] = e.dq;
  }
}
__device__ __forceinline__ void epi_load_cols16(EpiCols16& k, int n0, const Epilogue& e) { epi_load_cols<16>(k, n0, e); }

// The NC values after dequantisation, bias and activation (fp32, before any conversion to the output type).
template <int NC>
__device__ __forceinline__ void epi_values(const uint32_t* raw, float (&t)[NC], const Epilogue& e, const EpiColsT<NC>& k) {
  const bool has_bias = e.bias != nullptr, acc_int = e.acc_is_int != 0;
  const int act = e.act;
#pragma unroll
  for (int i = 0; i < NC; ++i) {
    float x = acc_int ? __fmul_rn(__int2float_rn(static_cast<int>(raw[i]) - k.c[i]), k.dq[i]) : __uint_as_float(raw[i]);
    x = has_bias ? __fadd_rn(x, k.b[i]) : x;      // separately rounded: exact on the integer path
    t[i] = x;
  }
  if (act == ACT_RELU) {
#pragma unroll
    for (int i = 0; i < NC; ++i) t[i] = fmaxf(t[i], 0.0f);
  } else if (act != ACT_NONE) {
#pragma unroll
    for (int i = 0; i < NC; ++i) t[i] = apply_act(t[i], act);
  }
}
__device__ __forceinline__ void epi_values16(const uint32_t* raw, float (&t)[16], const Epilogue& e, const EpiCols16& k) {
  epi_values<16>(raw, t, e, k);
}

// Store NC consecutive outputs of one row (columns n0..n0+NC-1) from NC raw accumulator words.
// `dst_row` points at column 0 of the row; n0 is a multiple of NC and the row pitch keeps the alignment of
// (dst_row + n0) that the vector stores need (NC output elements) for every supported dtype.
template <int NC>
__device__ __forceinline__ void epi_store_cols(const uint32_t* raw, void* dst_row, int n0, const Epilogue& e,
                                               const EpiColsT<NC>& k) {
  if (e.acc_is_int && !e.has_dq) {   // raw s32 accumulators (zero-point compensation is exact in s32)
    int4* d = reinterpret_cast<int4*>(static_cast<int*>(dst_row) + n0);
#pragma unroll
    for (int i = 0; i < NC / 4; ++i)
      d[i] = make_int4(static_cast<int>(raw[4 * i]) - k.c[4 * i], static_cast<int>(raw[4 * i + 1]) - k.c[4 * i + 1],
                       static_cast<int>(raw[4 * i + 2]) - k.c[4 * i + 2], static_cast<int>(raw[4 * i + 3]) - k.c[4 * i + 3]);
    return;
  }
  float t[NC];
  epi_values<NC>(raw, t, e, k);
  if (e.out_dtype == GC_F32) {
    float4* d = reinterpret_cast<float4*>(static_cast<float*>(dst_row) + n0);
#pragma unroll
    for (int i = 0; i < NC / 4; ++i) d[i] = make_float4(t[4 * i], t[4 * i + 1], t[4 * i + 2], t[4 * i + 3]);
  } else if (e.out_dtype == GC_BF16) {
    uint32_t w[NC / 2];
#pragma unroll
    for (int i = 0; i < NC / 2; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(t[2 * i], t[2 * i + 1]);
      w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    uint4* d = reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(dst_row) + n0);
#pragma unroll
    for (int i = 0; i < NC / 8; ++i) d[i] = make_uint4(w[4 * i], w[4 * i + 1], w[4 * i + 2], w[4 * i + 3]);
  } else {
    const int lo = e.out_dtype == GC_U8 ? 0 : -128, hi = e.out_dtype == GC_U8 ? 255 : 127;
    uint32_t w[NC / 4];
#pragma unroll
    for (int i = 0; i < NC / 4; ++i) {
      uint32_t b0 = quantize_value(t[4 * i + 0], e.inv, e.zp, lo, hi) & 0xFF;
      uint32_t b1 = quantize_value(t[4 * i + 1], e.inv, e.zp, lo, hi) & 0xFF;
      uint32_t b2 = quantize_value(t[4 * i + 2], e.inv, e.zp, lo, hi) & 0xFF;
      uint32_t b3 = quantize_value(t[4 * i + 3], e.inv, e.zp, lo, hi) & 0xFF;
      w[i] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
    }
    if constexpr (NC == 16)
      *reinterpret_cast<uint4*>(static_cast<uint8_t*>(dst_row) + n0) = make_uint4(w[0], w[1], w[2], w[3]);
    else
      *reinterpret_cast<uint2*>(static_cast<uint8_t*>(dst_row) + n0) = make_uint2(w[0], w[1]);
  }
}
__device__ __forceinline__ void epi_store16_cols(const uint32_t* raw, void* dst_row, int n0, const Epilogue& e,
                                                 const EpiCols16& k) {
  epi_store_cols<16>(raw, dst_row, n0, e, k);
}

__device__ __forceinline__ void epi_store16(const uint32_t* raw, void* dst_row, int n0, const Epilogue& e) {
  EpiCols16 k;
  epi_load_cols16(k, n0, e);
  epi_store16_cols(raw, dst_row, n0, e, k);
}

// Scalar store of one output (generic kernels).
__device__ __forceinline__ void epi_store1(uint32_t raw, void* dst_row, int n, const Epilogue& e) {
  if (e.acc_is_int && !e.has_dq) {
    static_cast<int*>(dst_row)[n] = static_cast<int>(raw);
    return;
  }
  const float t = epi_value(raw, n, e);
  if (e.out_dtype == GC_F32) {
    static_cast<float*>(dst_row)[n] = t;
  } else if (e.out_dtype == GC_BF16) {
    static_cast<__nv_bfloat16*>(dst_row)[n] = __float2bfloat16_rn(t);
  } else if (e.out_dtype == GC_U8) {
    static_cast<uint8_t*>(dst_row)[n] = static_cast<uint8_t>(quantize_value(t, e.inv, e.zp, 0, 255));
  } else {
    static_cast<int8_t*>(dst_row)[n] = static_cast<int8_t>(quantize_value(t, e.inv, e.zp, -128, 127));
  }
}

// ---- the graph-entry reorder as a pre-op (Section V: fused "only at the entry point of the graph") ----
// One 128-byte k-block of one input row, read from an arbitrarily aligned source with aligned 32-bit loads and
// written where TMA would have put it: row r of a 128B-swizzled K-major tile (8-row groups of 1024 bytes, 16-byte chunk
// index XOR row mod 8).  `src` points at the k-block's first byte in the row, `nv` (0..128) is the number of valid
// bytes from there (0 for rows beyond the matrix); the rest is zero filled.  Straight-line code: 33 predicated loads
// that are independent of one another (one memory round trip), 32 funnel shifts, masks by selects - no branch, no
// 64-bit arithmetic (the code runs once per launch in a warp that is alone on its scheduler, where a branch costs
// about 30 clocks).
__device__ __forceinline__ void pack_row_kblock(const uint8_t* src, int nv, uint8_t* dst_tile, int r) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(src);
  const int sh = static_cast<int>(a & 3);
  const uint32_t* aw = reinterpret_cast<const uint32_t*>(a - sh);
  uint32_t w[33];
#pragma unroll
  for (int u = 0; u < 33; ++u)   // word u holds k-block bytes [4u - sh, 4u - sh + 4): load it only if one of them is valid
    w[u] = (nv > 0 && 4 * u - sh < nv) ? __ldg(aw + u) : 0u;
  uint8_t* dst = dst_tile + (r >> 3) * 1024 + (r & 7) * 128;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    uint32_t o[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int t = 4 * c + j;
      const uint32_t v = __funnelshift_r(w[t], w[t + 1], static_cast<uint32_t>(sh) * 8u);
      const int left = nv - 4 * t;                                // valid bytes of this word
      const uint32_t part = (1u << (8 * (left & 3))) - 1u;        // (used for left = 1..3 only)
      o[j] = left >= 4 ? v : (left <= 0 ? 0u : (v & part));
    }
    *reinterpret_cast<uint4*>(dst + ((c ^ (r & 7)) << 4)) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

}  // namespace gc
