// Internal declarations shared by the host-side planner (gc_api.cu) and the kernel translation units.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/gc.h"

namespace gc {

enum Act : int { ACT_NONE = 0, ACT_RELU = 1, ACT_GELU_TANH = 2, ACT_SIGMOID = 3 };

// What a fused op does to each accumulator element before it is stored (the post-op anchor of the
// fused-op template, Section IV).  Order is fixed:
//   t = acc                      (float accumulator)            or
//   t = (float)acc * dq          (s32 accumulator, has_dq)      or   raw s32 store (no has_dq)
//   t = t + bias[n]              (bias != nullptr)
//   t = act(t)
//   out = t                      (f32)  |  bf16(t)  |  saturate(rne(t * inv) + zp)  (u8 / s8)
// On the integer path every multiply/add is a separately rounded fp32 operation.
struct Epilogue {
  int acc_is_int;
  int has_dq;
  float dq;
  const float* dqv;  // per-output-column dequantisation scales (per-channel weight scales), or null: `dq` applies
  const int* comp;   // per-output-column s32 compensation a_z * colsum(W), subtracted from the raw accumulator
                     // of a kernel that multiplies the stored (not zero-point-shifted) activation codes; or null
  const float* bias;
  int act;
  int out_dtype;   // gc_dtype_t
  float inv;       // 1.0f / scale_out
  int zp;          // zero point of the quantised output
};

struct GemmTcParams {
  int M, N, K;
  int num_k_blocks, m_tiles, n_tiles;
  uint32_t idesc;      // tcgen05 instruction descriptor (filled by the launcher)
  void* out;
  int64_t out_pitch;   // elements
  Epilogue epi;
  uint32_t* status;
};

struct GemmSimtParams {
  const void* A;       // [batch][M][a_pitch]
  const void* Wt;      // [batch][N][w_pitch]   (reduction axis contiguous)
  int64_t a_pitch, w_pitch, a_batch_stride, w_batch_stride, out_batch_stride;
  int M, N, K, batch;
  int a_dtype, w_dtype;  // gc_dtype_t
  int a_zp, w_zp;
  void* out;
  int64_t out_pitch;
  Epilogue epi;
};

struct SdpaParams {
  const void* Q;
  const void* K;
  const void* V;
  const float* mask;   // [B, S_kv] or nullptr
  void* O;
  void* P_out;         // optional second graph output: the probabilities as the second MatMul consumes them
                       // (u8 codes or bf16), [B,H,S,S]; nullptr when not requested
  int B, H, S, D;
  int is_int8;         // u8/s8 operands (else bf16)
  int zp_q, zp_k, zp_v;
  float dq1;           // scale_q * scale_k   (int8)
  float scalar;        // the Mul op's constant (1/sqrt(d)); 1 if absent
  int p_is_quant;      // probabilities quantised (int8 path)
  float inv_p;         // 1 / scale_p
  int zp_p;
  float dq2;           // scale_p * scale_v
  float inv_o;         // 1 / scale_o
  int zp_o;
  int out_dtype;       // GC_BF16 or GC_U8 / GC_S8
  int q_signed, k_signed, v_signed;   // s8 instead of u8 storage
  float skip_thr;      // int8: a 32-key chunk whose mask values times log2(e) are all <= -skip_thr contributes exactly
                       // zero to the softmax of any row that has an unmasked key (bound derived from the largest
                       // possible integer score); 0 disables the skipping of such chunks
  int max_free;        // int8, no mask, scores bounded at compile time: exponentials without a row maximum (Section VII's
                       // "fast softmax"); only the kernel for 64-wide heads with resident K/V implements it
  uint32_t* status;
};

// One layer, or two consecutive large fused ops in one launch, of the CTA-pair GEMM (kernels_gemm_tc2.cu).
struct GemmPairLayer {
  int N, num_k_blocks, n_tiles;   // n_tiles: 256-column tiles per 256-row block
  uint32_t idesc;                 // tcgen05 instruction descriptor (filled by the launcher)
  Epilogue epi;
};
struct GemmPairParams {
  GemmPairLayer L[2];
  const int* sched;               // [clusters][sched_pitch]: (layer << 24) | tile, a negative entry ends a list;
  int sched_pitch;                // null: one layer whose implicit_tiles tiles the clusters take round robin
  int implicit_tiles;
  int m_pairs, raster_rows;       // one layer: 256-row blocks in all, and how many of them form a group of the tile order
  unsigned long long* ready;      // null for one layer.  [0] = launches completed so far (the epoch: bumped by the
                                  // last CTA to finish; keeping it on the device, not in the launch parameters, is
                                  // what makes a captured launch replayable), [1] = CTAs finished in this launch,
                                  // [2 + tile] = one counter per first-layer tile: epilogue warps whose stores of the
                                  // tile have completed (16 per launch; only grows)
  uint32_t* status;
  alignas(64) CUtensorMap tm[6];  // A, Wt, D of the first layer, then of the second
};
cudaError_t launch_gemm_tc2_fused(int kind, int a_signed, const GemmPairParams& p, int grid, cudaStream_t s);

// One layer of the fused small-batch chain kernel (kernels_chain.cu).
constexpr int CHAIN_MAX_LAYERS = 8;
struct ChainLayer {
  int M, N, K, nkb;        // nkb: 128-byte blocks along the reduction axis
  int active_ctas;         // CTAs that own 32 output columns each; 0 = this layer runs on CUDA cores
  int a_tm, b_tm;          // indices into ChainParams::tmaps (A operand, prepacked weight)
  uint32_t idesc;          // tcgen05 instruction descriptor
  uint32_t w_smem_off;     // where this layer's weight slice lives in shared memory
  const void* a_ptr;       // CUDA-core layers: activation and prepacked weight in global memory
  const void* wt_ptr;
  int64_t a_pitch, w_pitch;
  int a_dtype, w_dtype, a_zp;
  void* out;
  int64_t out_pitch;       // elements
  int out_elem;            // bytes per stored element
  Epilogue epi;
  // one-cluster variant only (kernels_chain_cluster.cu): parts this layer's reduction axis is split into, and the rows
  // of the tile each CTA of such a group finishes (a multiple of 8)
  int ks_l, rows_per;
};
struct ChainParams {
  int n_layers;
  ChainLayer L[CHAIN_MAX_LAYERS];
  uint32_t w_smem_bytes;   // shared memory taken by the resident weight slices
  int a_stages;            // A-operand ring: stages and bytes per stage (round_up(M, 8) rows of 128 bytes)
  int a_stage_bytes;
  const void* pack_src;    // graph-entry reorder: the first layer's input when TMA cannot address its row pitch
  int pack_rows;           // its rows (0: the first layer is fed by TMA like the others)
  int64_t pack_src_pitch;  // bytes
  unsigned long long* barrier;              // grid-barrier counter (only grows)
                                            // its value at the start of a launch is derived from the counter itself on
                                            // the device, so that a captured launch can be replayed
  int n_barriers;                           // grid barriers one launch passes
  int ks;                                   // CTAs per cluster = parts the reduction axis of every layer is split into
  int slices;                               // 32-column slices per row tile: grid = row tiles x slices x ks
  int early_weights;                        // 1: the prepacked weights were written by an earlier call, so their loads
                                            // need not wait for the kernel that precedes this one on the stream
  int fold_tail;                            // grid-wide variant: the last layer has one output column and is folded into
                                            // the finishing step of the layer before it (partial dot products added
                                            // per row with atomics; the last contributor of a row applies the post-ops)
  int* tail_acc;                            // [M] s32 sums, zero between launches
  unsigned int* tail_cnt;                   // [M] contributions counted so far, zero between launches
  int recompute_first;                      // one-cluster variant: every CTA of the second layer computes the first
                                            // layer's columns it needs itself (no hand-over between the two)
  uint32_t* status;
  // TMA descriptors travel in the kernel parameter space (fetched once, cached by the TMA unit); descriptors
  // kept in global memory cost a fetch of several hundred clocks on every load instruction.
  alignas(64) CUtensorMap tmaps[2 * CHAIN_MAX_LAYERS];
};
size_t mlp_chain_smem_bytes(size_t w_smem_bytes, int a_stages, int a_stage_bytes, int ks);
cudaError_t launch_mlp_chain(int kind, const ChainParams& p, int grid, cudaStream_t s);
// clusters of `ks` CTAs of the chain kernel that can be resident together on the current device (0 on error)
int mlp_chain_max_clusters(int kind, int ks, size_t smem);

// The same chain inside ONE thread-block cluster (fp32 / tf32 chains small enough for it): activations travel from
// layer to layer through distributed shared memory, no grid barrier, no round trip through the L2.  Uses
// ChainParams with a_stages = stages per A-operand region (two regions, alternating by layer) and the per-layer
// ks_l / rows_per; `cluster` = CTAs of the launch = cluster size (8 or 16).
size_t mlp_cluster_smem_bytes(size_t w_smem_bytes, int a_stages, int a_stage_bytes);
cudaError_t launch_mlp_cluster(const ChainParams& p, int cluster, cudaStream_t s);
int mlp_cluster_max_clusters(int cluster, size_t smem);

// Raise a kernel's dynamic shared-memory limit to at least `smem` bytes on the current device.  The driver call is made
// once per (kernel, device) and size, not on every launch.
cudaError_t ensure_dynamic_smem(const void* kern, size_t smem);

// ---- launchers (each enqueues exactly one kernel on the stream and returns cudaGetLastError) ----
cudaError_t launch_pack_rows(const void* src, void* dst, int rows, int64_t src_pitch_bytes, int64_t dst_pitch_bytes,
                             cudaStream_t s);
// W given as [K,N] (transposed = 0) or [N,K] (transposed = 1), dense; writes Wt[N][Kp] with the
// reduction axis contiguous and zero padded.  f32 weights are rounded to tf32 (nearest, ties away).
cudaError_t launch_prepack_weight(const void* W, void* Wt, int K, int N, int Kp, int transposed, int dtype,
                                  cudaStream_t s);
// comp[n] = a_zp * sum_k Wt[n][k] for a prepacked s8 weight (zero padded to Kp)
cudaError_t launch_weight_compensation(const void* Wt, int N, int Kp, int a_zp, int* comp, cudaStream_t s);
cudaError_t launch_gemm_simt(const GemmSimtParams& p, cudaStream_t s);
// one small kernel that waits on a barrier nobody arrives on, gives up after limit_ns and records a timeout code
cudaError_t launch_bounded_wait_selftest(uint32_t* status, uint64_t limit_ns, cudaStream_t s);
cudaError_t launch_sdpa_simt(const SdpaParams& p, cudaStream_t s);

// kind: 0 = i8 (u8/s8 x s8 -> s32), 1 = bf16, 2 = tf32.  a_signed only matters for kind 0.
bool gemm_tc_supported_block_n(int block_n);
size_t gemm_tc_smem_bytes(int block_n);
// Columns per TMA-store box for this tile width and output element size, or 0 when the kernel stores
// with plain vector stores (tile rows shorter than 128 bytes) and tmD is ignored.
int gemm_tc_store_box_cols(int block_n, int out_elem_bytes);
cudaError_t launch_gemm_tc(int kind, int block_n, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB,
                           const CUtensorMap& tmD, const GemmTcParams& p, int grid, bool pdl, cudaStream_t s);

// CTA-pair variant (cta_group::2): 256 x 256 tiles per cluster of two CTAs; tmB must have a 128-row box.
// `grid` must be even.
size_t gemm_tc2_smem_bytes();
// clusters of two CTAs of the CTA-pair kernel that can be resident together on the current device (0 on error)
int gemm_tc2_max_clusters(int kind, int out_dtype);
cudaError_t launch_gemm_tc2(int kind, int a_signed, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmD,
                            const GemmTcParams& p, int grid, bool pdl, cudaStream_t s);

size_t sdpa_tc_smem_bytes(int S, int is_int8);
// Attention for rows longer than tensor memory holds (kernels_sdpa_long.cu): head dimension 64 / 96 / 128, any number of
// keys, scores computed twice around a blockwise softmax.  Takes the 3-D tensor maps of the streaming kernel
// (sdpa_wide_box).  Dynamic shared memory it needs (0 = shape not supported).
size_t sdpa_long_smem_bytes(int S, int D, int is_int8);
cudaError_t launch_sdpa_long(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                             int num_sms, cudaStream_t s);
// Streaming attention kernel (head dimension 64 / 96 / 128, up to 512 keys): dynamic shared memory it needs
// (0 = shape not supported), the TMA box (elements per row, swizzle bytes) its Q / K / V tensor maps must use
// (128 rows per box), and the launcher.
// One unit per CTA, several CTAs per SM (kernels_sdpa_small.cu): bf16, 128 keys, head width 64.
bool sdpa_small_supported(int S, int D, int is_int8);
cudaError_t launch_sdpa_small(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                              cudaStream_t s);
size_t sdpa_wide_smem_bytes(int S, int D, int is_int8);
void sdpa_wide_box(int D, int is_int8, int* box_elems, int* swizzle_bytes);
cudaError_t launch_sdpa_wide(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const SdpaParams& p,
                             int num_sms, cudaStream_t s);
// tmO: output [B*H*S, 64] with a [32 rows x 64 columns] box, swizzle = row bytes (64 for 8-bit, 128 for bf16)
cudaError_t launch_sdpa_tc(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmO,
                           const SdpaParams& p, int num_sms, cudaStream_t s);

}  // namespace gc
