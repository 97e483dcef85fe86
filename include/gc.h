/*
 * gc.h - C ABI of the B200 fused-subgraph executor.
 *
 * The boundary follows the paper's statement of the problem (Sections II, V and VII): a framework
 * hands over a *partition* - a list of ops over logical tensors with static shapes, dtypes, plain
 * row-major layouts and per-tensor quantisation attributes -, the partition is *compiled once*, and
 * the compiled object is *executed* many times on plain-layout inputs and outputs.  Constant
 * weights may be unknown at compile time; they are preprocessed when they first arrive and the
 * result is reused (Section V, "constant weight preprocessing").
 *
 * Two subgraph patterns are accepted; everything else fails at gc_compile with GC_ERR_UNSUPPORTED
 * (there is no CPU fallback - the paper leaves fallback to the framework, Section VII):
 *
 *   MLP chain   (Section VII "MLP"; Fig. 5):  L >= 1 layers, each
 *       MatMul(h, W) [-> Dequantize] [-> Add(bias)] [-> ReLU | GELU_TANH | Sigmoid]
 *                    [-> Quantize | TypeCast]
 *     h is the previous layer's result (graph input for the first layer), W a constant 2-D graph
 *     input [K,N] (or [N,K] with transpose_b), bias a constant 1-D fp32 graph input [N].
 *
 *   Attention   (Section VII "MHA": two batch matmuls, a softmax and the binary ops between):
 *       MatMul(Q, K, transpose_b) [-> Dequantize] [-> Mul(scalar)] [-> Add(mask)] -> SoftMax
 *           [-> Quantize | TypeCast] -> MatMul(P, V) [-> Dequantize -> Quantize | -> TypeCast]
 *     Q, K, V, O are [B,H,S,D] contiguous; mask is fp32 [B,1,1,S].  The tensor P that the second
 *     MatMul consumes (u8 codes or bf16, [B,H,S,S]) may be listed as a second graph output; it is
 *     then written out as well, which lets a caller verify the integer stage after the softmax exactly.
 *
 * Semantics of the ops (what an unfused, op-by-op evaluation gives, which the fused kernels must
 * reproduce):
 *   MatMul on u8/s8 operands: exact integer sum of zero-point-subtracted operands, s32 result whose
 *     implied scale is the fp32 product scale_a * scale_b.  On bf16/f32 operands: fp32 accumulation
 *     on tensor cores (f32 operands are consumed as tf32).
 *   Dequantize: (float)(q - zero_point) * scale, fp32.          Quantize: saturate(rne(x * inv) + zp)
 *     with inv = 1.0f / scale formed in fp32 (Section V: DQ scales and offsets, Q does the reverse).
 *   On the integer paths every fp32 multiply/add is a separately rounded IEEE operation (no fused
 *   multiply-add), so results are reproducible bit for bit.
 *
 * Conventions
 *   - Every call returns a gc_status_t; out-parameters are untouched on error; gc_last_error()
 *     returns a thread-local, library-owned message for the last failing call on this thread.
 *   - Pointers named *_dev are CUDA device pointers on the device given to gc_compile; pointers
 *     named *_host are host pointers.  The caller owns all tensor memory, the workspace and the
 *     stream; the library owns only host-side plan objects.  Input and output device pointers must
 *     be 16-byte aligned (GC_ERR_ALIGNMENT otherwise).
 *   - in_*[i] corresponds to input_ids[i] given at gc_partition_create, out_*[i] to output_ids[i].
 *   - gc_execute is asynchronous on the given stream.  One compiled object must not be executed
 *     concurrently on two streams (it owns one workspace).  Plans that run as ONE persistent kernel
 *     whose CTAs wait for one another (the small-batch chain, two large layers in one launch; the
 *     plan description names them) size their grid to what the device can hold resident at once,
 *     queried at gc_compile: work of another object, or of anything else, that occupies SMs at the
 *     same time can keep part of such a grid from starting.  Run these objects one at a time per
 *     GPU (one stream, or ordered streams); if they are overlapped anyway the bounded waits expire
 *     and gc_query_status reports GC_ERR_TIMEOUT - nothing hangs.
 *   - Device-side waits are bounded: if one expires the kernel records an error in a status word
 *     and returns; gc_query_status reports it as GC_ERR_TIMEOUT.  Nothing traps.
 */
#ifndef GC_B200_H_
#define GC_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  GC_OK = 0,
  GC_ERR_INVALID_ARG = 1,
  GC_ERR_UNSUPPORTED = 2,
  GC_ERR_SHAPE = 3,
  GC_ERR_STATE = 4,
  GC_ERR_CUDA = 5,
  GC_ERR_OOM = 6,
  GC_ERR_TIMEOUT = 7,
  GC_ERR_ALIGNMENT = 8
} gc_status_t;

typedef enum { GC_F32 = 0, GC_BF16 = 1, GC_U8 = 2, GC_S8 = 3, GC_S32 = 4 } gc_dtype_t;

typedef enum {
  GC_OP_MATMUL = 0,
  GC_OP_ADD = 1,
  GC_OP_MUL = 2,
  GC_OP_RELU = 3,
  GC_OP_GELU_TANH = 4,
  GC_OP_SIGMOID = 5,
  GC_OP_SOFTMAX = 6,
  GC_OP_QUANTIZE = 7,
  GC_OP_DEQUANTIZE = 8,
  GC_OP_TYPECAST = 9
} gc_op_kind_t;

#define GC_MAX_DIMS 6

/* Logical tensor (Section II: dtype, shape, layout metadata).  Layout is always dense row-major. */
typedef struct {
  int64_t id;
  int32_t dtype;          /* gc_dtype_t */
  int32_t ndims;
  int64_t dims[GC_MAX_DIMS];
  float scale;            /* per-tensor quantisation scale; ignored for float dtypes */
  int32_t zero_point;
  int32_t is_constant;    /* 1: same pointer and contents on every execution (weights, biases) */
  /* Per-channel quantisation (the weight scheme of Section VII's int8 evaluation: symmetric s8 weights with one
   * scale per output channel): a HOST array
   * of dims[channel_axis] scales, copied by gc_partition_create; NULL = the per-tensor `scale` applies.
   * Accepted only on the constant s8 weight of a 2-D MatMul, along its output-channel axis (1 for a [k,n]
   * weight, 0 for a transposed [n,k] one); anything else is GC_ERR_UNSUPPORTED. */
  const float* channel_scales;
  int32_t channel_axis;
  int32_t reserved_;
} gc_logical_tensor_t;

/* Op (Section II: kind, attributes, input and output logical tensors). */
typedef struct {
  int32_t kind;           /* gc_op_kind_t */
  int32_t n_in;           /* 1 or 2 */
  int64_t in[3];          /* logical tensor ids */
  int64_t out;            /* logical tensor id */
  int32_t transpose_b;    /* MATMUL: second operand stored [.., n, k] */
  int32_t axis;           /* SOFTMAX: must address the last axis (-1 or ndims-1) */
  float scalar;           /* MUL: the constant multiplier */
  int32_t has_scalar;     /* MUL: must be 1 */
} gc_op_t;

/* Options for gc_compile; pass NULL for the defaults (all zero). */
typedef struct {
  int32_t force_generic;  /* 1: use the shape-generic CUDA-core kernels instead of the tcgen05 ones
                             (ablation / debugging; results obey the same contracts) */
  int32_t no_chain_fusion;/* 1: one launch per fused op with full stream ordering between them, the
                             analogue of running with coarse-grain fusion disabled (Section VII) */
  int32_t streaming_attention; /* 1: attention always runs on the streaming tcgen05 kernel (K/V and P rings),
                             also for the shapes (head dimension 64, up to 384 keys) that by default use the
                             kernel with resident K/V (ablation) */
  int32_t exact_max_softmax;   /* 1: the softmax always subtracts the row maximum.  By default an 8-bit attention
                             block without a mask whose scores are bounded at compile time (|score| * log2(e) <= 60,
                             from the operand ranges and the folded scales) skips it: the "fast softmax" of
                             Section VII, equal in exact arithmetic (ablation) */
  int32_t grid_wide_chain;     /* 1: a small fp32 MLP chain that would run inside one thread-block cluster
                             (activations handed over through distributed shared memory) runs on the
                             grid-wide chain kernel instead (hand-over through the L2 behind a grid barrier;
                             ablation) */
  int32_t reserved[3];
} gc_compile_options_t;

typedef struct gc_partition gc_partition_t;
typedef struct gc_compiled gc_compiled_t;

/* Build a partition (Section II, graph of ops and logical tensors).  Host only; copies everything.
 * ops must be in topological order.  Errors: INVALID_ARG (null pointers, unknown ids, duplicate
 * ids, bad enum values), SHAPE (dims inconsistent with the op). */
gc_status_t gc_partition_create(gc_partition_t** out, const gc_op_t* ops, int32_t n_ops,
                                const gc_logical_tensor_t* tensors, int32_t n_tensors,
                                const int64_t* input_ids, int32_t n_in,
                                const int64_t* output_ids, int32_t n_out);
void gc_partition_destroy(gc_partition_t* p);

/* Pass as cuda_device to gc_compile to form the pattern and the plan for a nominal B200 (148 SMs)
 * without touching a device; the result answers the query calls but gc_execute returns GC_ERR_STATE. */
#define GC_DEVICE_PLAN_ONLY (-1)

/* Compile a partition for one CUDA device (Section V: pattern formation, constant folding of the
 * quantisation parameters, kernel/tile selection; Section VI: temporary buffers sized and reused
 * at compile time).  Host only; touches the device only to query its properties. */
gc_status_t gc_compile(const gc_partition_t* p, int32_t cuda_device, const gc_compile_options_t* opt,
                       gc_compiled_t** out);
void gc_compiled_destroy(gc_compiled_t* c);

/* Scratch memory the compiled object needs (Section VI: temporary buffers are sized, and reused
 * between fused ops whose life spans do not overlap, at compile time; Section V: the preprocessed
 * constant weights are kept for reuse): inter-layer activations, prepacked weights, padded input
 * copies, a status word.  The caller allocates it on the device (256-byte aligned), hands it over
 * once and keeps it alive until gc_compiled_destroy.  Contents need no initialisation. */
gc_status_t gc_workspace_bytes(const gc_compiled_t* c, size_t* bytes);
gc_status_t gc_set_workspace(gc_compiled_t* c, void* workspace_dev, size_t bytes);

/* Execute (Section VII: a subgraph costs one call into compiled code, not one per op).  Enqueues
 * all work on cuda_stream (a cudaStream_t, may be NULL for the default stream) and returns.  On
 * the first call, or when a constant input arrives at a new address, the constant weights are
 * prepacked on the same stream first and cached in the workspace (Section V).  A call that does
 * not prepack (same pointers as an earlier call) only enqueues kernel launches with parameters
 * that do not depend on how often the object has run (the kernels' synchronisation counters keep
 * their epochs on the device), so it may be recorded by stream capture and replayed as a CUDA
 * graph; the first call must come before the capture. */
gc_status_t gc_execute(gc_compiled_t* c, void* cuda_stream, const void* const* in_dev, int32_t n_in,
                       void* const* out_dev, int32_t n_out);

/* Same computation with HOST buffers: copies the inputs to a device staging area (constants only
 * when their host pointer changes), executes, copies the outputs back and synchronises the stream.
 * The staging area is caller-allocated device memory of gc_host_staging_bytes bytes. */
gc_status_t gc_host_staging_bytes(const gc_compiled_t* c, size_t* bytes);
gc_status_t gc_set_host_staging(gc_compiled_t* c, void* staging_dev, size_t bytes);
gc_status_t gc_execute_host(gc_compiled_t* c, void* cuda_stream, const void* const* in_host,
                            int32_t n_in, void* const* out_host, int32_t n_out);

/* No counterpart in the paper (its tensors live in host memory already): the same computation with
 * HOST buffers, but asynchronous, so that the copies of consecutive batches overlap each other and
 * the execution.  The staging area set by gc_set_host_staging holds one slot per multiple of
 * gc_host_staging_bytes (at most GC_HOST_SLOTS; three keep both copy directions busy when a batch
 * spends about as long in each copy as in the execution).  The call enqueues, for staging slot
 * `slot` (0 .. slots - 1): the
 * host-to-device copies of the non-constant inputs on a copy stream the object owns, the execute
 * on cuda_stream behind them, and the device-to-host copies of the outputs on a second copy stream
 * behind the execute; then it returns.  gc_host_wait(c, slot) blocks until that slot's outputs
 * have arrived in out_host; the host buffers must stay valid and untouched until then, and should
 * be page-locked (with pageable memory the copies are correct but do not overlap).  A slot that is
 * still in flight is refused with GC_ERR_STATE; constants are copied once, as in gc_execute_host,
 * and shared by both slots.  All calls on one object use the same cuda_stream. */
#define GC_HOST_SLOTS 4
gc_status_t gc_execute_host_async(gc_compiled_t* c, void* cuda_stream, int32_t slot,
                                  const void* const* in_host, int32_t n_in, void* const* out_host,
                                  int32_t n_out);
gc_status_t gc_host_wait(gc_compiled_t* c, int32_t slot);

/* No counterpart in the paper (its CPU kernels cannot time out).  Synchronise the stream and read
 * the device status word: GC_OK, GC_ERR_TIMEOUT (a bounded device-side wait expired) or
 * GC_ERR_CUDA (the stream reported an error).  A kernel that gave up leaves its synchronisation
 * counters mid-count, and the outputs of that execute (and of any later one issued before this
 * call) are undefined; when this call reports GC_ERR_TIMEOUT it has also zeroed the status word
 * and those counters, so the object can be executed again afterwards.  The cached prepacked
 * constants are kept. */
gc_status_t gc_query_status(gc_compiled_t* c, void* cuda_stream);

/* Constants are preprocessed once per address (Section V) and the result is cached; a caller that
 * rewrites a constant IN PLACE (same address, new contents) calls this to drop the cache: the next
 * execute preprocesses every constant again.  Host only; must not race with an execute. */
gc_status_t gc_invalidate_constants(gc_compiled_t* c);

/* No counterpart in the paper: introspection for tests and benchmarks.  Number of kernel launches
 * one gc_execute enqueues after prepacking, and a short text description of the plan (pattern,
 * per-layer kernel and tile).  The string is owned by the compiled object. */
gc_status_t gc_launches_per_execute(const gc_compiled_t* c, int32_t* n);
const char* gc_plan_description(const gc_compiled_t* c);

/* No counterpart in the paper: an entry point for callers that cannot allocate device memory.
 *
 * Some callers may not call cudaMalloc at all - a real-time loop with a fixed memory plan, a process
 * whose allocator owns the whole device and gives nothing back at run time, a component that is only
 * allowed to launch work on buffers it was handed.  The regular path asks such a caller for a
 * workspace it cannot provide.  gc_matmul_s32_noalloc computes
 *     out[m, n] (s32) = sum_k (a[m, k] - a_zero_point) * w[k, n]      a: u8 [m, k], w: s8 [k, n], row-major
 * exactly, like a MatMul-only partition, but keeps its scratch (the transposed, zero-padded weight
 * the kernel consumes) in a fixed array inside the library image.  It calls no allocating routine.
 *
 *   - Limit: n * round_up(k, 128) <= gc_noalloc_scratch_bytes() (1 MiB); larger problems are rejected
 *     with GC_ERR_UNSUPPORTED and a message - use gc_compile / gc_execute with a workspace instead.
 *     Also rejected: a_zero_point outside 0..255 (GC_ERR_INVALID_ARG), k > 65536 (the exact sum could
 *     leave s32) and m * n beyond what one launch covers (about 1.7e10), both GC_ERR_UNSUPPORTED.
 *   - The array costs every GPU that loads this library 1 MiB of device memory until the process exits.
 *   - All calls share the array.  Calls that can overlap on the GPU (different streams, or host threads
 *     racing on one stream) corrupt each other's scratch: keep them on one stream or serialise them.
 *     The array keeps the previous call's contents; every byte that is read is rewritten first, so no
 *     clearing is needed between calls.
 *   - The first call on each device looks up the array's device address (with that device current) and
 *     caches it; make that first call before any stream capture begins.
 *   - All three pointers are device pointers on the current device; out must be 4-byte aligned.
 *     Asynchronous on cuda_stream like gc_execute. */
gc_status_t gc_matmul_s32_noalloc(void* cuda_stream, const void* a_dev, const void* w_dev, void* out_dev,
                                  int32_t m, int32_t k, int32_t n, int32_t a_zero_point);
size_t gc_noalloc_scratch_bytes(void);

/* No counterpart in the paper: a self-test of the error path of the kernels' bounded waits.  Every wait inside
 * the kernels (on an mbarrier, on a counter in global memory) gives up after a time limit, records a code in the
 * status word and lets the kernel return, so that the context stays usable and gc_query_status can report
 * GC_ERR_TIMEOUT.  This call launches one small kernel whose wait can never be satisfied (a barrier nobody arrives
 * on), limited to limit_us microseconds (at most 100 000), and which then writes its code to *status_dev
 * (a 4-byte device word the caller has zeroed).  Asynchronous on cuda_stream. */
gc_status_t gc_selftest_bounded_wait(void* cuda_stream, void* status_dev, uint32_t limit_us);

const char* gc_last_error(void);
const char* gc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* GC_B200_H_ */
