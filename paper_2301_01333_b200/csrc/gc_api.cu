// Host side of the C ABI: partition bookkeeping, pattern formation (the fixed analogue of the paper's
// fine-grain fusion: one Tunable op plus the Fusible ops that follow it, Section V), constant folding of
// the quantisation parameters, kernel and tile selection (the role of the template heuristic, Section
// III), compile-time buffer planning with reuse (Section VI) and the execute path that enqueues the
// prepack (first call only) and the fused kernels on the caller's stream.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "gc_internal.h"

using namespace gc;

// ------------------------------------------------------------------------------------------------
// errors
// ------------------------------------------------------------------------------------------------
static thread_local char g_err[512] = "";

static gc_status_t fail(gc_status_t st, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return st;
}
#define CUDA_TRY(expr)                                                                          \
  do {                                                                                          \
    cudaError_t e__ = (expr);                                                                   \
    if (e__ != cudaSuccess) return fail(GC_ERR_CUDA, "%s: %s", #expr, cudaGetErrorString(e__)); \
  } while (0)

// for the other translation units of the library: record a message for gc_last_error() and pass the status on
gc_status_t gc_set_error(gc_status_t st, const char* msg) { return fail(st, "%s", msg); }

extern "C" const char* gc_last_error(void) { return g_err; }
extern "C" const char* gc_version(void) { return "gc-b200 0.1 (sm_100a)"; }

// ------------------------------------------------------------------------------------------------
// partition
// ------------------------------------------------------------------------------------------------
struct gc_partition {
  std::vector<gc_op_t> ops;
  std::vector<gc_logical_tensor_t> tensors;
  std::map<int64_t, int> index;   // tensor id -> position in `tensors`
  std::map<int64_t, std::vector<float>> channel_scales;   // copies of the callers' per-channel scale arrays
  const std::vector<float>* ch_scales(int64_t id) const {
    auto it = channel_scales.find(id);
    return it == channel_scales.end() ? nullptr : &it->second;
  }
  std::vector<int64_t> in_ids, out_ids;
  const gc_logical_tensor_t* lt(int64_t id) const {
    auto it = index.find(id);
    return it == index.end() ? nullptr : &tensors[it->second];
  }
  int input_pos(int64_t id) const {
    for (size_t i = 0; i < in_ids.size(); ++i)
      if (in_ids[i] == id) return static_cast<int>(i);
    return -1;
  }
  int output_pos(int64_t id) const {
    for (size_t i = 0; i < out_ids.size(); ++i)
      if (out_ids[i] == id) return static_cast<int>(i);
    return -1;
  }
  int consumers(int64_t id) const {
    int n = 0;
    for (const auto& op : ops)
      for (int i = 0; i < op.n_in; ++i) n += op.in[i] == id;
    return n;
  }
};

static int dtype_bytes(int dt) { return dt == GC_F32 || dt == GC_S32 ? 4 : (dt == GC_BF16 ? 2 : 1); }
static bool is_int8(int dt) { return dt == GC_U8 || dt == GC_S8; }
static int64_t numel(const gc_logical_tensor_t& t) {
  int64_t n = 1;
  for (int i = 0; i < t.ndims; ++i) n *= t.dims[i];
  return n;
}
static bool same_dims(const gc_logical_tensor_t& a, const gc_logical_tensor_t& b) {
  if (a.ndims != b.ndims) return false;
  for (int i = 0; i < a.ndims; ++i)
    if (a.dims[i] != b.dims[i]) return false;
  return true;
}

extern "C" gc_status_t gc_partition_create(gc_partition_t** out, const gc_op_t* ops, int32_t n_ops,
                                           const gc_logical_tensor_t* tensors, int32_t n_tensors,
                                           const int64_t* input_ids, int32_t n_in, const int64_t* output_ids,
                                           int32_t n_out) {
  if (!out || !ops || !tensors || !input_ids || !output_ids) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (n_ops <= 0 || n_tensors <= 0 || n_in <= 0 || n_out <= 0) return fail(GC_ERR_INVALID_ARG, "empty partition");
  auto p = new gc_partition();
  auto bail = [&](gc_status_t st) {
    delete p;
    return st;
  };
  for (int i = 0; i < n_tensors; ++i) {
    const auto& t = tensors[i];
    if (t.dtype < GC_F32 || t.dtype > GC_S32) return bail(fail(GC_ERR_INVALID_ARG, "tensor %lld: bad dtype", (long long)t.id));
    if (t.ndims < 1 || t.ndims > GC_MAX_DIMS) return bail(fail(GC_ERR_INVALID_ARG, "tensor %lld: bad ndims", (long long)t.id));
    for (int d = 0; d < t.ndims; ++d)
      if (t.dims[d] <= 0) return bail(fail(GC_ERR_SHAPE, "tensor %lld: non-positive dimension", (long long)t.id));
    if (p->index.count(t.id)) return bail(fail(GC_ERR_INVALID_ARG, "duplicate tensor id %lld", (long long)t.id));
    if (is_int8(t.dtype) && !(t.scale > 0.f) ) return bail(fail(GC_ERR_INVALID_ARG, "tensor %lld: scale must be positive", (long long)t.id));
    p->index[t.id] = static_cast<int>(p->tensors.size());
    p->tensors.push_back(t);
    p->tensors.back().channel_scales = nullptr;       // the caller's array is not kept; see p->channel_scales
    if (t.channel_scales) {
      if (t.dtype != GC_S8 || !t.is_constant || t.ndims != 2 || t.channel_axis < 0 || t.channel_axis > 1)
        return bail(fail(GC_ERR_UNSUPPORTED, "tensor %lld: per-channel scales need a constant 2-D s8 weight and axis 0 or 1",
                         (long long)t.id));
      std::vector<float> cs(t.channel_scales, t.channel_scales + t.dims[t.channel_axis]);
      for (float s : cs)
        if (!(s > 0.f)) return bail(fail(GC_ERR_INVALID_ARG, "tensor %lld: channel scales must be positive", (long long)t.id));
      p->channel_scales[t.id] = std::move(cs);
    }
  }
  std::map<int64_t, bool> defined;
  for (int i = 0; i < n_in; ++i) {
    if (!p->lt(input_ids[i])) return bail(fail(GC_ERR_INVALID_ARG, "unknown input id %lld", (long long)input_ids[i]));
    if (defined.count(input_ids[i])) return bail(fail(GC_ERR_INVALID_ARG, "duplicate input id"));
    defined[input_ids[i]] = true;
    p->in_ids.push_back(input_ids[i]);
  }
  for (int i = 0; i < n_ops; ++i) {
    const auto& op = ops[i];
    if (op.kind < GC_OP_MATMUL || op.kind > GC_OP_TYPECAST) return bail(fail(GC_ERR_INVALID_ARG, "op %d: bad kind", i));
    const int want_in = (op.kind == GC_OP_MATMUL || op.kind == GC_OP_ADD) ? 2 : 1;
    if (op.n_in != want_in) return bail(fail(GC_ERR_INVALID_ARG, "op %d: expects %d inputs", i, want_in));
    for (int k = 0; k < op.n_in; ++k) {
      if (!p->lt(op.in[k])) return bail(fail(GC_ERR_INVALID_ARG, "op %d: unknown input tensor", i));
      if (!defined.count(op.in[k])) return bail(fail(GC_ERR_INVALID_ARG, "op %d: input used before it is defined (ops must be in topological order)", i));
    }
    const auto* o = p->lt(op.out);
    if (!o) return bail(fail(GC_ERR_INVALID_ARG, "op %d: unknown output tensor", i));
    if (defined.count(op.out)) return bail(fail(GC_ERR_INVALID_ARG, "op %d: output tensor defined twice", i));
    const auto* a = p->lt(op.in[0]);
    // shape checks
    if (op.kind == GC_OP_MATMUL) {
      const auto* b = p->lt(op.in[1]);
      if (a->ndims < 2 || b->ndims < 2 || o->ndims != a->ndims)
        return bail(fail(GC_ERR_SHAPE, "op %d: matmul needs >= 2-D operands", i));
      const int64_t m = a->dims[a->ndims - 2], k = a->dims[a->ndims - 1];
      const int64_t kb = op.transpose_b ? b->dims[b->ndims - 1] : b->dims[b->ndims - 2];
      const int64_t n = op.transpose_b ? b->dims[b->ndims - 2] : b->dims[b->ndims - 1];
      if (k != kb || o->dims[o->ndims - 2] != m || o->dims[o->ndims - 1] != n)
        return bail(fail(GC_ERR_SHAPE, "op %d: matmul shapes do not agree", i));
      if (b->ndims > 2) {
        if (b->ndims != a->ndims) return bail(fail(GC_ERR_SHAPE, "op %d: batched matmul rank mismatch", i));
        for (int d = 0; d < a->ndims - 2; ++d)
          if (a->dims[d] != b->dims[d] || a->dims[d] != o->dims[d])
            return bail(fail(GC_ERR_SHAPE, "op %d: batch dimensions differ", i));
      }
    } else if (op.kind == GC_OP_ADD) {
      const auto* b = p->lt(op.in[1]);
      if (!same_dims(*a, *o)) return bail(fail(GC_ERR_SHAPE, "op %d: add output shape", i));
      // second operand must broadcast onto the first (trailing alignment)
      if (b->ndims > a->ndims) return bail(fail(GC_ERR_SHAPE, "op %d: add broadcast rank", i));
      for (int d = 0; d < b->ndims; ++d) {
        const int64_t bd = b->dims[b->ndims - 1 - d], ad = a->dims[a->ndims - 1 - d];
        if (bd != 1 && bd != ad) return bail(fail(GC_ERR_SHAPE, "op %d: add operands do not broadcast", i));
      }
    } else {
      if (!same_dims(*a, *o)) return bail(fail(GC_ERR_SHAPE, "op %d: elementwise output shape differs", i));
      if (op.kind == GC_OP_MUL && !op.has_scalar) return bail(fail(GC_ERR_INVALID_ARG, "op %d: mul needs a scalar", i));
      if (op.kind == GC_OP_SOFTMAX && !(op.axis == -1 || op.axis == a->ndims - 1))
        return bail(fail(GC_ERR_UNSUPPORTED, "op %d: softmax over the last axis only", i));
    }
    defined[op.out] = true;
    p->ops.push_back(op);
  }
  for (int i = 0; i < n_out; ++i) {
    if (!p->lt(output_ids[i]) || !defined.count(output_ids[i]))
      return bail(fail(GC_ERR_INVALID_ARG, "output id %lld is not produced by the partition", (long long)output_ids[i]));
    p->out_ids.push_back(output_ids[i]);
  }
  *out = p;
  return GC_OK;
}

extern "C" void gc_partition_destroy(gc_partition_t* p) { delete p; }

// ------------------------------------------------------------------------------------------------
// compiled object
// ------------------------------------------------------------------------------------------------
enum Pattern { PAT_MLP = 1, PAT_SDPA = 2, PAT_BATCHED_MATMUL = 3 };

struct LayerPlan {
  int M = 0, K = 0, N = 0;
  int a_dtype = 0, w_dtype = 0, a_zp = 0;
  int transposed_w = 0;
  int a_input = -1;          // graph input position of the activation (first layer) or -1
  int w_input = -1, bias_input = -1;
  Epilogue epi = {};
  int out_pos = -1;          // graph output position, or -1 for an intermediate
  int out_elem = 0;          // bytes per stored element
  int64_t out_pitch = 0;     // elements
  size_t out_off = 0;        // workspace offset of an intermediate
  size_t in_off = 0;         // workspace offset of the previous intermediate
  int64_t a_pitch = 0;       // elements
  bool use_tc = false;
  bool cta2 = false;         // CTA-pair kernel (256 x 256 tiles per cluster of two)
  int kind = 0, block_n = 0, grid = 0, m_tiles = 0, n_tiles = 0, nkb = 0;
  bool need_pack = false;
  size_t pack_off = 0;
  int64_t pack_pitch = 0;    // elements
  size_t wt_off = 0;
  int Kp = 0;
  std::vector<float> dqv_host;   // per-channel weights: float32(a_scale) * float32(w_scale[n]) per output column
  size_t dqv_off = 0;            // workspace offset of their device copy
  // this layer and the next one run as one launch of the CTA-pair GEMM (kernels_gemm_tc2.cu)
  bool fused_first = false;
  std::vector<int> pair_sched;   // [clusters][pair_pitch] tile lists: (layer << 24) | tile, -1 terminated
  int pair_pitch = 0, pair_clusters = 0;
  size_t pair_sched_off = 0, pair_ready_off = 0, pair_ready_words = 0;
  bool need_comp = false;        // tcgen05 path with a non-zero activation zero point
  size_t comp_off = 0;           // workspace offset of a_zp * colsum(W), s32 per output column
  // cached tensor maps
  CUtensorMap tmA, tmB, tmD;
  const void* tmA_ptr = nullptr;
  const void* tmD_ptr = nullptr;
  bool tmB_valid = false;
};

struct SdpaPlan {
  SdpaParams prm = {};
  int q_input = -1, k_input = -1, v_input = -1, mask_input = -1, out_pos = 0;
  int p_out_pos = -1;        // graph output position of the probabilities tensor, if it is an output too
  bool use_tc = false;
  bool wide = false;         // streaming kernel (wider heads, 512 keys) instead of the D = 64 kernel
  bool two_pass = false;     // more than 512 keys: blockwise softmax with the scores computed twice
  bool small = false;        // bf16, 128 keys, width 64: one unit per CTA, several CTAs per SM
  CUtensorMap tmQ, tmK, tmV, tmO;
  const void *q_ptr = nullptr, *k_ptr = nullptr, *v_ptr = nullptr, *o_ptr = nullptr;
};

struct gc_compiled {
  int device = 0, num_sms = 148;
  int pattern = 0;
  gc_compile_options_t opt = {};
  std::vector<LayerPlan> layers;
  SdpaPlan sdpa;
  GemmSimtParams bmm = {};   // PAT_BATCHED_MATMUL
  int n_in = 0, n_out = 0;
  std::vector<size_t> in_bytes, out_bytes;
  std::vector<int> in_constant;
  size_t ws_bytes = 0;
  void* ws = nullptr;
  bool status_cleared = false;
  bool prepacked = false;
  std::vector<const void*> const_ptrs;   // constant input pointers seen at the last prepack
  int launches = 0;
  std::string desc;
  // fused small-batch chain (one persistent kernel for all layers)
  bool chain_fused = false;
  int chain_kind = 0, chain_grid = 0, chain_barriers = 0, chain_ks = 1, chain_slices = 0;
  size_t chain_tmap_off = 0;                 // workspace offset of the tensor-map array
  uint32_t chain_w_smem = 0;
  int chain_a_stages = 0, chain_a_stage_bytes = 0, chain_a_rows = 0;
  std::vector<uint32_t> chain_w_off;         // per layer: offset of its weight slice in shared memory
  std::vector<CUtensorMap> chain_tmaps;      // host copy of the tensor-map array
  const void* chain_a0_ptr = nullptr;        // first-layer A pointer the array was built for
  bool chain_tmaps_valid = false;
  bool chain_fold_tail = false;              // the one-column last layer is folded into the layer before it
  size_t chain_tail_off = 0;                 // workspace offset of its per-row sums and counters (2 x 4 bytes x M)
  // the same chain inside one thread-block cluster (small fp32 chains)
  int chain_cluster = 0;                     // cluster size (0: the grid-wide kernel)
  bool chain_recompute_first = false;
  std::vector<int> chain_ks_l, chain_rows_per;
  // host staging
  size_t staging_bytes = 0;
  void* staging = nullptr;
  std::vector<size_t> in_stage_off, out_stage_off;
  std::vector<const void*> host_const_seen;
  // overlapped host execution: up to GC_HOST_SLOTS staging slots, copy streams of their own, one event triple per slot
  int staging_slots = 0;
  bool pipe_ready = false;
  cudaStream_t h2d_stream = nullptr, d2h_stream = nullptr;
  cudaEvent_t ev_in[GC_HOST_SLOTS] = {}, ev_exec[GC_HOST_SLOTS] = {}, ev_out[GC_HOST_SLOTS] = {};
  bool slot_busy[GC_HOST_SLOTS] = {};
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// 2-D row-major tensor [rows][inner] with a row pitch in bytes; box = [box_rows][box_inner].
static gc_status_t make_tmap(CUtensorMap* m, const void* ptr, int dtype, uint64_t inner, uint64_t rows,
                             uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows, int swizzle_bytes) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return fail(GC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  CUtensorMapDataType dt = dtype == GC_F32    ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
                           : dtype == GC_S32  ? CU_TENSOR_MAP_DATA_TYPE_INT32
                           : dtype == GC_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16
                                              : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t gdim[2] = {inner, rows};
  cuuint64_t gstr[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMapSwizzle sw = swizzle_bytes == 128  ? CU_TENSOR_MAP_SWIZZLE_128B
                          : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                          : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                : CU_TENSOR_MAP_SWIZZLE_NONE;
  CUresult r = enc(m, dt, 2, const_cast<void*>(ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(GC_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
  return GC_OK;
}

// 3-D tensor [slices][rows][inner], dense; box = [1][box_rows][box_inner].  Rows past a slice's end (and columns past
// `inner`) read as zeros.
static gc_status_t make_tmap3(CUtensorMap* m, const void* ptr, int dtype, uint64_t inner, uint64_t rows, uint64_t slices,
                              uint32_t box_inner, uint32_t box_rows, int swizzle_bytes) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return fail(GC_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const uint64_t esz = static_cast<uint64_t>(dtype_bytes(dtype));
  CUtensorMapDataType dt = dtype == GC_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  cuuint64_t gdim[3] = {inner, rows, slices};
  cuuint64_t gstr[2] = {inner * esz, inner * esz * rows};
  cuuint32_t box[3] = {box_inner, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  CUresult r = enc(m, dt, 3, const_cast<void*>(ptr), gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(GC_ERR_CUDA, "cuTensorMapEncodeTiled (3-D) failed with code %d", (int)r);
  return GC_OK;
}

// ------------------------------------------------------------------------------------------------
// pattern formation
// ------------------------------------------------------------------------------------------------
static int act_of(int kind) {
  return kind == GC_OP_RELU ? ACT_RELU : kind == GC_OP_GELU_TANH ? ACT_GELU_TANH : kind == GC_OP_SIGMOID ? ACT_SIGMOID : -1;
}

static gc_status_t match_mlp(const gc_partition& p, gc_compiled& c) {
  size_t i = 0;
  int64_t cur = -1;
  while (i < p.ops.size()) {
    const gc_op_t& mm = p.ops[i];
    if (mm.kind != GC_OP_MATMUL) return fail(GC_ERR_UNSUPPORTED, "op %zu: expected a matmul to start a fused op", i);
    const auto* a = p.lt(mm.in[0]);
    const auto* w = p.lt(mm.in[1]);
    if (a->ndims != 2 || w->ndims != 2) return fail(GC_ERR_UNSUPPORTED, "MLP layers need 2-D operands");
    LayerPlan L;
    if (c.layers.empty()) {
      L.a_input = p.input_pos(mm.in[0]);
      if (L.a_input < 0) return fail(GC_ERR_UNSUPPORTED, "first matmul must read a graph input");
    } else if (mm.in[0] != cur) {
      return fail(GC_ERR_UNSUPPORTED, "op %zu: matmul does not consume the previous fused op (not a chain)", i);
    }
    L.w_input = p.input_pos(mm.in[1]);
    if (L.w_input < 0 || !w->is_constant) return fail(GC_ERR_UNSUPPORTED, "op %zu: weights must be a constant graph input", i);
    L.M = static_cast<int>(a->dims[0]);
    L.K = static_cast<int>(a->dims[1]);
    L.N = static_cast<int>(p.lt(mm.out)->dims[1]);
    L.a_dtype = a->dtype;
    L.w_dtype = w->dtype;
    L.transposed_w = mm.transpose_b;
    const bool int_path = is_int8(a->dtype) && is_int8(w->dtype);
    const bool flt_path = (a->dtype == GC_BF16 && w->dtype == GC_BF16) || (a->dtype == GC_F32 && w->dtype == GC_F32);
    if (!int_path && !flt_path) return fail(GC_ERR_UNSUPPORTED, "op %zu: unsupported matmul operand dtypes", i);
    if (int_path && w->zero_point != 0) return fail(GC_ERR_UNSUPPORTED, "weights must be symmetric (zero point 0)");
    if (p.lt(mm.out)->dtype != (int_path ? GC_S32 : GC_F32))
      return fail(GC_ERR_UNSUPPORTED, "op %zu: matmul result must be %s", i, int_path ? "s32" : "f32");
    L.a_zp = int_path ? a->zero_point : 0;
    L.epi.acc_is_int = int_path;
    L.epi.out_dtype = int_path ? GC_S32 : GC_F32;
    int64_t t = mm.out;
    ++i;
    auto next_is = [&](int kind) { return i < p.ops.size() && p.ops[i].kind == kind && p.ops[i].in[0] == t; };
    if (next_is(GC_OP_DEQUANTIZE)) {
      if (!int_path) return fail(GC_ERR_UNSUPPORTED, "dequantize after a float matmul");
      L.epi.has_dq = 1;
      L.epi.dq = a->scale * w->scale;   // fp32 product, the scale of the s32 result
      if (const std::vector<float>* cs = p.ch_scales(mm.in[1])) {
        if (w->channel_axis != (mm.transpose_b ? 0 : 1))
          return fail(GC_ERR_UNSUPPORTED, "op %zu: per-channel scales must run along the weight's output-channel axis", i);
        L.dqv_host.resize(cs->size());
        for (size_t n = 0; n < cs->size(); ++n) L.dqv_host[n] = a->scale * (*cs)[n];
      }
      L.epi.out_dtype = GC_F32;
      t = p.ops[i++].out;
    }
    if (i < p.ops.size() && p.ops[i].kind == GC_OP_ADD && (p.ops[i].in[0] == t || p.ops[i].in[1] == t)) {
      const int64_t other = p.ops[i].in[0] == t ? p.ops[i].in[1] : p.ops[i].in[0];
      const auto* b = p.lt(other);
      const int pos = p.input_pos(other);
      if (pos >= 0 && b->dtype == GC_F32 && numel(*b) == L.N && b->dims[b->ndims - 1] == L.N) {
        if (int_path && !L.epi.has_dq) return fail(GC_ERR_UNSUPPORTED, "bias add on an s32 tensor");
        L.bias_input = pos;
        t = p.ops[i++].out;
      } else {
        return fail(GC_ERR_UNSUPPORTED, "op %zu: add operand is not a per-column fp32 bias", i);
      }
    }
    if (i < p.ops.size() && act_of(p.ops[i].kind) >= 0 && p.ops[i].in[0] == t) {
      if (int_path && !L.epi.has_dq) return fail(GC_ERR_UNSUPPORTED, "activation on an s32 tensor");
      L.epi.act = act_of(p.ops[i].kind);
      t = p.ops[i++].out;
    }
    if (next_is(GC_OP_QUANTIZE)) {
      const auto* o = p.lt(p.ops[i].out);
      if (!is_int8(o->dtype)) return fail(GC_ERR_UNSUPPORTED, "quantize must produce u8 or s8");
      if (int_path && !L.epi.has_dq) return fail(GC_ERR_UNSUPPORTED, "quantize on an s32 tensor");
      L.epi.out_dtype = o->dtype;
      L.epi.inv = 1.0f / o->scale;
      L.epi.zp = o->zero_point;
      t = p.ops[i++].out;
    } else if (next_is(GC_OP_TYPECAST)) {
      const auto* o = p.lt(p.ops[i].out);
      if (o->dtype != GC_BF16 && o->dtype != GC_F32) return fail(GC_ERR_UNSUPPORTED, "typecast target must be bf16 or f32");
      if (int_path && !L.epi.has_dq) return fail(GC_ERR_UNSUPPORTED, "typecast on an s32 tensor");
      L.epi.out_dtype = o->dtype;
      t = p.ops[i++].out;
    }
    if (p.lt(t)->dtype != L.epi.out_dtype) return fail(GC_ERR_UNSUPPORTED, "fused op result dtype does not match its logical tensor");
    const bool last = i == p.ops.size();
    if (last) {
      L.out_pos = p.output_pos(t);
      if (L.out_pos < 0 || p.out_ids.size() != 1) return fail(GC_ERR_UNSUPPORTED, "the chain's last tensor must be the only graph output");
    } else {
      if (p.output_pos(t) >= 0 || p.consumers(t) != 1)
        return fail(GC_ERR_UNSUPPORTED, "intermediate tensors must have exactly one consumer and not be outputs");
      if (L.epi.out_dtype == GC_S32) return fail(GC_ERR_UNSUPPORTED, "an s32 tensor cannot feed the next matmul");
    }
    L.out_elem = dtype_bytes(L.epi.out_dtype);
    cur = t;
    c.layers.push_back(L);
  }
  return c.layers.empty() ? fail(GC_ERR_UNSUPPORTED, "no matmul found") : GC_OK;
}

static gc_status_t match_sdpa(const gc_partition& p, gc_compiled& c) {
  SdpaPlan& s = c.sdpa;
  SdpaParams& prm = s.prm;
  size_t i = 0;
  const gc_op_t& m1 = p.ops[0];
  const auto *q = p.lt(m1.in[0]), *k = p.lt(m1.in[1]);
  if (!m1.transpose_b || q->ndims != 4 || !same_dims(*q, *k)) return fail(GC_ERR_UNSUPPORTED, "attention: Q and K must be [B,H,S,D] with transpose_b");
  s.q_input = p.input_pos(m1.in[0]);
  s.k_input = p.input_pos(m1.in[1]);
  if (s.q_input < 0 || s.k_input < 0) return fail(GC_ERR_UNSUPPORTED, "attention: Q and K must be graph inputs");
  prm.B = static_cast<int>(q->dims[0]);
  prm.H = static_cast<int>(q->dims[1]);
  prm.S = static_cast<int>(q->dims[2]);
  prm.D = static_cast<int>(q->dims[3]);
  const bool i8 = is_int8(q->dtype) && is_int8(k->dtype);
  if (!i8 && !(q->dtype == GC_BF16 && k->dtype == GC_BF16)) return fail(GC_ERR_UNSUPPORTED, "attention: operands must be bf16 or 8-bit");
  prm.is_int8 = i8;
  prm.zp_q = i8 ? q->zero_point : 0;
  prm.zp_k = i8 ? k->zero_point : 0;
  prm.q_signed = q->dtype == GC_S8;
  prm.k_signed = k->dtype == GC_S8;
  prm.dq1 = i8 ? q->scale * k->scale : 1.0f;
  prm.scalar = 1.0f;
  int64_t t = m1.out;
  ++i;
  auto next_is = [&](int kind) { return i < p.ops.size() && p.ops[i].kind == kind && p.ops[i].in[0] == t; };
  if (i8) {
    if (!next_is(GC_OP_DEQUANTIZE)) return fail(GC_ERR_UNSUPPORTED, "attention: int8 scores must be dequantized");
    t = p.ops[i++].out;
  }
  if (next_is(GC_OP_MUL)) {
    prm.scalar = p.ops[i].scalar;
    t = p.ops[i++].out;
  }
  if (i < p.ops.size() && p.ops[i].kind == GC_OP_ADD && p.ops[i].in[0] == t) {
    const auto* mk = p.lt(p.ops[i].in[1]);
    s.mask_input = p.input_pos(p.ops[i].in[1]);
    if (s.mask_input < 0 || mk->dtype != GC_F32 || mk->ndims != 4 || mk->dims[0] != prm.B || mk->dims[1] != 1 ||
        mk->dims[2] != 1 || mk->dims[3] != prm.S)
      return fail(GC_ERR_UNSUPPORTED, "attention: mask must be an fp32 graph input [B,1,1,S]");
    t = p.ops[i++].out;
  }
  if (!next_is(GC_OP_SOFTMAX)) return fail(GC_ERR_UNSUPPORTED, "attention: expected softmax");
  t = p.ops[i++].out;
  if (i8) {
    if (!next_is(GC_OP_QUANTIZE)) return fail(GC_ERR_UNSUPPORTED, "attention: int8 probabilities must be quantized");
    const auto* pq = p.lt(p.ops[i].out);
    if (pq->dtype != GC_U8) return fail(GC_ERR_UNSUPPORTED, "attention: quantized probabilities must be u8");
    prm.p_is_quant = 1;
    prm.inv_p = 1.0f / pq->scale;
    {
      // Largest |score| in log2 units: |q - 128| <= 128, |k code| <= 255 over D terms, times the folded scale.
      // A key whose mask term is below -(2 bound + 1 + 150) sits more than 150 binades under any row maximum
      // that an unmasked key (mask term >= -1) sets, so its fp32 exponential is exactly zero.
      const double bound = 128.0 * 255.0 * static_cast<double>(prm.D) *
                           std::fabs(static_cast<double>(prm.dq1) * prm.scalar) * 1.4426950408889634;
      prm.skip_thr = static_cast<float>(2.0 * bound + 151.0);
    }
    prm.zp_p = pq->zero_point;
    t = p.ops[i++].out;
  } else {
    if (!next_is(GC_OP_TYPECAST) || p.lt(p.ops[i].out)->dtype != GC_BF16)
      return fail(GC_ERR_UNSUPPORTED, "attention: bf16 path expects the probabilities cast to bf16");
    t = p.ops[i++].out;
  }
  if (!(i < p.ops.size() && p.ops[i].kind == GC_OP_MATMUL && p.ops[i].in[0] == t && !p.ops[i].transpose_b))
    return fail(GC_ERR_UNSUPPORTED, "attention: expected the P.V matmul");
  const auto* pt = p.lt(t);
  const int64_t p_tensor = t;
  const auto* v = p.lt(p.ops[i].in[1]);
  s.v_input = p.input_pos(p.ops[i].in[1]);
  if (s.v_input < 0 || !same_dims(*v, *q) || (i8 ? !is_int8(v->dtype) : v->dtype != GC_BF16))
    return fail(GC_ERR_UNSUPPORTED, "attention: V must be a graph input shaped and typed like Q");
  prm.zp_v = i8 ? v->zero_point : 0;
  prm.v_signed = v->dtype == GC_S8;
  prm.dq2 = i8 ? pt->scale * v->scale : 1.0f;
  t = p.ops[i++].out;
  if (i8) {
    if (!next_is(GC_OP_DEQUANTIZE)) return fail(GC_ERR_UNSUPPORTED, "attention: int8 output must be dequantized");
    t = p.ops[i++].out;
    if (!next_is(GC_OP_QUANTIZE)) return fail(GC_ERR_UNSUPPORTED, "attention: int8 output must be requantized");
    const auto* o = p.lt(p.ops[i].out);
    if (!is_int8(o->dtype)) return fail(GC_ERR_UNSUPPORTED, "attention: output must be u8 or s8");
    prm.out_dtype = o->dtype;
    prm.inv_o = 1.0f / o->scale;
    prm.zp_o = o->zero_point;
    t = p.ops[i++].out;
  } else {
    if (!next_is(GC_OP_TYPECAST) || p.lt(p.ops[i].out)->dtype != GC_BF16)
      return fail(GC_ERR_UNSUPPORTED, "attention: bf16 path expects a bf16 output");
    prm.out_dtype = GC_BF16;
    t = p.ops[i++].out;
  }
  // outputs: the attention result, optionally followed by the probabilities tensor (for inspection: it lets
  // a caller check the integer stage after the softmax exactly, given the probabilities the kernel used)
  if (i != p.ops.size() || p.output_pos(t) != 0 || p.out_ids.size() > 2 ||
      (p.out_ids.size() == 2 && p.output_pos(p_tensor) != 1))
    return fail(GC_ERR_UNSUPPORTED, "attention: trailing ops or wrong outputs");
  s.p_out_pos = p.out_ids.size() == 2 ? 1 : -1;
  return GC_OK;
}

static void choose_tile(LayerPlan& L, int num_sms) {
  const int esz = dtype_bytes(L.a_dtype);
  const int k_elems = 128 / esz;
  L.m_tiles = (L.M + 127) / 128;
  L.nkb = (L.K + k_elems - 1) / k_elems;
  const int cands[4] = {256, 128, 64, 32};
  int pick = 0;
  for (int bn : cands) {
    if (bn > 32 && bn > L.N) continue;
    const int tiles = L.m_tiles * ((L.N + bn - 1) / bn);
    if (tiles >= num_sms) {
      pick = bn;
      break;
    }
  }
  if (!pick) pick = 32;
  L.block_n = pick;
  L.n_tiles = (L.N + pick - 1) / pick;
  const int tiles = L.m_tiles * L.n_tiles;
  L.grid = tiles < num_sms ? tiles : num_sms;
  // Large problems: pair the CTAs.  A pair loads 32 KB per CTA and k-block instead of 48 KB, which lifts the
  // operand-fetch bound of the one-CTA 128 x 256 tile.
  L.cta2 = pick == 256 && L.m_tiles >= 2 && tiles >= num_sms;
  if (L.cta2) {
    const int pair_tiles = ((L.m_tiles + 1) / 2) * L.n_tiles;
    const int clusters = pair_tiles < num_sms / 2 ? pair_tiles : num_sms / 2;
    L.grid = 2 * clusters;
  }
}

extern "C" gc_status_t gc_compile(const gc_partition_t* p, int32_t cuda_device, const gc_compile_options_t* opt,
                                  gc_compiled_t** out) {
  if (!p || !out) return fail(GC_ERR_INVALID_ARG, "null argument");
  cudaDeviceProp prop = {};
  if (cuda_device == GC_DEVICE_PLAN_ONLY) {
    // plan for a nominal B200 without touching any device; the result cannot be executed
    prop.major = 10;
    prop.multiProcessorCount = 148;
    prop.sharedMemPerBlockOptin = 227 * 1024;
  } else {
    int ndev = 0;
    CUDA_TRY(cudaGetDeviceCount(&ndev));
    if (cuda_device < 0 || cuda_device >= ndev) return fail(GC_ERR_INVALID_ARG, "no such CUDA device %d", cuda_device);
    CUDA_TRY(cudaGetDeviceProperties(&prop, cuda_device));
    if (prop.major != 10) return fail(GC_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only", cuda_device, prop.major, prop.minor);
  }
  auto c = new gc_compiled();
  auto bail = [&](gc_status_t st) {
    delete c;
    return st;
  };
  c->device = cuda_device;
  c->num_sms = prop.multiProcessorCount;
  if (opt) c->opt = *opt;
  c->n_in = static_cast<int>(p->in_ids.size());
  c->n_out = static_cast<int>(p->out_ids.size());
  for (auto id : p->in_ids) {
    c->in_bytes.push_back(static_cast<size_t>(numel(*p->lt(id))) * dtype_bytes(p->lt(id)->dtype));
    c->in_constant.push_back(p->lt(id)->is_constant);
  }
  for (auto id : p->out_ids) c->out_bytes.push_back(static_cast<size_t>(numel(*p->lt(id))) * dtype_bytes(p->lt(id)->dtype));
  c->const_ptrs.assign(c->n_in, nullptr);
  c->host_const_seen.assign(c->n_in, nullptr);

  size_t ws = 256;   // [0,4): status word
  char line[256];
  const gc_op_t& first = p->ops[0];
  const bool batched = first.kind == GC_OP_MATMUL && p->lt(first.in[1])->ndims > 2;
  if (batched && p->ops.size() == 1) {
    // a bare batched matmul: the raw accumulator is the output
    const auto *a = p->lt(first.in[0]), *b = p->lt(first.in[1]), *o = p->lt(first.out);
    const bool i8 = is_int8(a->dtype) && is_int8(b->dtype);
    if (!first.transpose_b) return bail(fail(GC_ERR_UNSUPPORTED, "batched matmul needs transpose_b"));
    if (!i8 && !((a->dtype == GC_BF16 || a->dtype == GC_F32) && a->dtype == b->dtype))
      return bail(fail(GC_ERR_UNSUPPORTED, "batched matmul operand dtypes"));
    if (o->dtype != (i8 ? GC_S32 : GC_F32) || p->input_pos(first.in[0]) != 0 || p->input_pos(first.in[1]) != 1 ||
        p->output_pos(first.out) != 0)
      return bail(fail(GC_ERR_UNSUPPORTED, "batched matmul: inputs must be (A, B) and the result the output"));
    c->pattern = PAT_BATCHED_MATMUL;
    GemmSimtParams& g = c->bmm;
    g.M = static_cast<int>(a->dims[a->ndims - 2]);
    g.K = static_cast<int>(a->dims[a->ndims - 1]);
    g.N = static_cast<int>(b->dims[b->ndims - 2]);
    g.batch = static_cast<int>(numel(*a) / (static_cast<int64_t>(g.M) * g.K));
    g.a_pitch = g.K;
    g.w_pitch = g.K;
    g.a_batch_stride = static_cast<int64_t>(g.M) * g.K;
    g.w_batch_stride = static_cast<int64_t>(g.N) * g.K;
    g.out_batch_stride = static_cast<int64_t>(g.M) * g.N;
    g.out_pitch = g.N;
    g.a_dtype = a->dtype;
    g.w_dtype = b->dtype;
    g.a_zp = i8 ? a->zero_point : 0;
    g.w_zp = i8 ? b->zero_point : 0;
    g.epi.acc_is_int = i8;
    g.epi.out_dtype = o->dtype;
    c->launches = 1;
    c->desc = "pattern=batched_matmul kernel=cuda-core\n";
  } else if (batched) {
    gc_status_t st = match_sdpa(*p, *c);
    if (st != GC_OK) return bail(st);
    c->pattern = PAT_SDPA;
    SdpaParams& s = c->sdpa.prm;
    bool tc = !c->opt.force_generic && !c->opt.streaming_attention && s.D == 64 && s.S % 128 == 0 && s.S <= 384 &&
              sdpa_tc_smem_bytes(s.S, s.is_int8) <= static_cast<size_t>(prop.sharedMemPerBlockOptin);
    bool wide = false;
    if (!tc && !c->opt.force_generic) {
      const size_t need = sdpa_wide_smem_bytes(s.S, s.D, s.is_int8);
      wide = tc = need > 0 && need <= static_cast<size_t>(prop.sharedMemPerBlockOptin);
    }
    bool two_pass = false;
    if (!tc && !c->opt.force_generic && s.S > 512 && c->sdpa.p_out_pos < 0) {
      const size_t need = sdpa_long_smem_bytes(s.S, s.D, s.is_int8);
      two_pass = wide = tc = need > 0 && need <= static_cast<size_t>(prop.sharedMemPerBlockOptin);
    }
    if (!s.is_int8 && c->sdpa.p_out_pos >= 0) tc = false;   // the bf16 tcgen05 kernels never form normalised P
    // the probabilities as a second output: written in 16-byte pieces, which needs whole key blocks
    if (c->sdpa.p_out_pos >= 0 && s.S % 128 != 0) tc = false;
    if (s.is_int8)
      // Q must be exactly centred (s8 / zero point 0, or u8 / zero point 128); a zero point on K only
      // shifts every score of a row by the same amount, which softmax cancels
      tc = tc && s.zp_p == 0 && ((s.q_signed && s.zp_q == 0) || (!s.q_signed && s.zp_q == 128));
    if (!tc && s.S > 8192) return bail(fail(GC_ERR_UNSUPPORTED, "attention: sequence length %d not supported", s.S));
    c->sdpa.use_tc = tc;
    c->sdpa.wide = tc && wide;
    c->sdpa.two_pass = tc && two_pass;
    c->sdpa.small = tc && !wide && c->sdpa.p_out_pos < 0 && sdpa_small_supported(s.S, s.D, s.is_int8);
    c->launches = 1;
    // The paper's max-free softmax, where it is safe: 8-bit operands bound every score at compile time; with
    // |score| log2(e) <= 60 neither an exponential nor a row sum can leave fp32's range, and without a mask no row
    // can be pushed out of it at run time.  skip_thr = 2 bound + 151 (see match_sdpa).
    s.max_free = tc && !wide && s.is_int8 && c->sdpa.mask_input < 0 && !c->opt.exact_max_softmax && s.skip_thr > 0.f &&
                 (static_cast<double>(s.skip_thr) - 151.0) * 0.5 <= 60.0;
    snprintf(line, sizeof(line), "pattern=attention %s B=%d H=%d S=%d D=%d kernel=%s%s\n", s.is_int8 ? "int8" : "bf16", s.B,
             s.H, s.S, s.D, tc ? (two_pass ? "tcgen05.two-pass" : (wide ? "tcgen05.streaming" : (c->sdpa.small ? "tcgen05.unit-per-cta" : "tcgen05"))) : "cuda-core",
             s.max_free ? " softmax=max-free" : "");
    c->desc = line;
  } else {
    gc_status_t st = match_mlp(*p, *c);
    if (st != GC_OK) return bail(st);
    c->pattern = PAT_MLP;
    c->desc = "pattern=mlp_chain\n";
    // prepacked weights
    for (auto& L : c->layers) {
      const int esz = dtype_bytes(L.w_dtype);
      L.Kp = static_cast<int>(align_up(static_cast<size_t>(L.K) * esz, 128) / esz);
      L.wt_off = ws;
      ws = align_up(ws + static_cast<size_t>(L.N) * L.Kp * esz, 1024);
      // constants derived from the quantisation parameters and the weight: per-column scales, compensation
      if (!L.dqv_host.empty()) {
        L.dqv_off = ws;
        ws = align_up(ws + align_up(static_cast<size_t>(L.N), 16) * sizeof(float), 256);
      }
      if (L.epi.acc_is_int && L.a_zp != 0) {
        L.comp_off = ws;
        ws = align_up(ws + align_up(static_cast<size_t>(L.N), 16) * sizeof(int), 256);
      }
    }
    // temporaries between fused ops: two buffers reused alternately (life spans never overlap by
    // more than one layer), each sized for the largest tensor it ever holds
    size_t act_bytes[2] = {0, 0};
    for (size_t l = 0; l + 1 < c->layers.size(); ++l) {
      LayerPlan& L = c->layers[l];
      L.out_pitch = static_cast<int64_t>(align_up(static_cast<size_t>(L.N), 16));
      const size_t b = static_cast<size_t>(L.M) * L.out_pitch * L.out_elem;
      if (b > act_bytes[l & 1]) act_bytes[l & 1] = b;
    }
    size_t act_off[2];
    act_off[0] = ws;
    ws = align_up(ws + act_bytes[0], 1024);
    act_off[1] = ws;
    ws = align_up(ws + act_bytes[1], 1024);
    for (size_t l = 0; l < c->layers.size(); ++l) {
      LayerPlan& L = c->layers[l];
      const int esz = dtype_bytes(L.a_dtype);
      if (l + 1 < c->layers.size()) L.out_off = act_off[l & 1];
      else L.out_pitch = L.N;
      if (l > 0) {
        L.in_off = act_off[(l - 1) & 1];
        L.a_pitch = c->layers[l - 1].out_pitch;
      } else {
        L.a_pitch = L.K;
      }
      // 8-bit operands go to the tensor cores as stored; a non-zero activation zero point is removed afterwards
      // with the compensation term, which needs |sum_k a_k w_kn| and |a_z colsum(W)_n| to stay inside s32
      const bool dt_ok = (is_int8(L.a_dtype) && L.w_dtype == GC_S8 && (L.a_zp == 0 || L.K <= 65536)) ||
                         L.a_dtype == GC_BF16 || L.a_dtype == GC_F32;
      L.use_tc = !c->opt.force_generic && dt_ok && L.N >= 16 && L.N % 16 == 0;
      L.need_comp = L.use_tc && is_int8(L.a_dtype) && L.a_zp != 0;
      if (L.use_tc) {
        L.kind = is_int8(L.a_dtype) ? 0 : (L.a_dtype == GC_BF16 ? 1 : 2);
        choose_tile(L, c->num_sms);
        if ((L.a_pitch * esz) % 16 != 0) {   // graph-entry reorder: TMA needs 16-byte row pitches
          L.need_pack = true;
          L.pack_pitch = static_cast<int64_t>(align_up(static_cast<size_t>(L.K) * esz, 16) / esz);
          L.pack_off = ws;
          ws = align_up(ws + static_cast<size_t>(L.M) * L.pack_pitch * esz, 1024);
          c->launches += 1;
        }
      }
      c->launches += 1;
      snprintf(line, sizeof(line), "  layer %zu: M=%d K=%d N=%d kernel=%s block_n=%d grid=%d%s act=%d out=%d\n", l, L.M, L.K,
               L.N, L.use_tc ? (L.kind == 0 ? "tcgen05.i8" : L.kind == 1 ? "tcgen05.bf16" : "tcgen05.tf32") : "cuda-core",
               L.block_n, L.grid, L.cta2 ? " cta_pair" : (L.need_pack ? " +pack" : ""), L.epi.act, L.epi.out_dtype);
      c->desc += line;
    }
  }
  if (c->pattern == PAT_MLP && !c->opt.no_chain_fusion && !c->opt.force_generic && c->layers.size() >= 2 &&
      c->layers.size() <= static_cast<size_t>(CHAIN_MAX_LAYERS)) {
    // Small-batch chains run as one persistent kernel when every layer fits one MMA row tile and all
    // weight slices of a CTA fit in shared memory next to the activation ring.
    bool ok = true;
    c->chain_w_off.assign(c->layers.size(), 0);
    int kind = -1, max_ctas = 0, max_nkb = 1, a_rows = 8;
    for (size_t l = 0; l < c->layers.size() && ok; ++l) {
      LayerPlan& L = c->layers[l];
      ok = L.M <= 512;
      const int lk = is_int8(L.a_dtype) ? 0 : (L.a_dtype == GC_BF16 ? 1 : 2);
      if (kind < 0) kind = lk;
      ok = ok && lk == kind;
      const int rows = L.M < 128 ? (L.M + 7) / 8 * 8 : 128;       // rows of one row tile
      a_rows = rows > a_rows ? rows : a_rows;
      if (L.use_tc) {
        const int ctas = (L.N + 31) / 32;
        max_ctas = ctas > max_ctas ? ctas : max_ctas;
        max_nkb = L.nkb > max_nkb ? L.nkb : max_nkb;
      }
    }
    // The reduction axis is split over a cluster of ks CTAs (each multiplies its share of the k-blocks, the
    // partial sums meet in distributed shared memory): worth it when the longest reduction has enough k-blocks.
    // A-operand ring: round_up(M, 8) rows per stage and one stage per k-block a CTA handles in the deepest
    // layer, so every layer fetches its whole A operand in one burst.
    const int a_stage_bytes = a_rows * 128;
    const int row_tiles = c->layers.empty() ? 1 : (c->layers[0].M + 127) / 128;   // all layers of a chain share M
    int ks = max_nkb >= 8 ? 4 : (max_nkb >= 4 ? 2 : 1);
    while (ks > 1 && max_ctas * ks * row_tiles > c->num_sms) ks >>= 1;   // row tiles come before splitting the reduction
    int a_stages = 0;
    uint32_t w_smem = 0;
    ok = ok && max_ctas > 0;
    for (; ok; ks >>= 1) {
      w_smem = 0;
      for (size_t l = 0; l < c->layers.size(); ++l) {
        const LayerPlan& L = c->layers[l];
        c->chain_w_off[l] = w_smem;
        if (L.use_tc) w_smem += static_cast<uint32_t>((L.nkb + ks - 1) / ks) * 32 * 128;
      }
      a_stages = (max_nkb + ks - 1) / ks;
      const size_t smem = mlp_chain_smem_bytes(w_smem, a_stages, a_stage_bytes, ks);
      bool fits = a_stages <= 32 && max_ctas * ks * row_tiles <= c->num_sms && smem <= static_cast<size_t>(prop.sharedMemPerBlockOptin);
      // all clusters must be resident together (the layers are separated by a grid-wide barrier)
      if (fits && cuda_device != GC_DEVICE_PLAN_ONLY) {
        int cur = -1;
        cudaGetDevice(&cur);
        if (cur != cuda_device) cudaSetDevice(cuda_device);     // the occupancy query answers for the current device
        fits = mlp_chain_max_clusters(kind, ks, smem) >= max_ctas * row_tiles;
        if (cur >= 0 && cur != cuda_device) cudaSetDevice(cur);
      }
      if (fits) break;
      if (ks == 1) ok = false;
    }
    if (ok) {
      c->chain_a_stages = a_stages;
      c->chain_a_stage_bytes = a_stage_bytes;
      c->chain_a_rows = a_rows;
      c->chain_fused = true;
      c->chain_kind = kind;
      c->chain_grid = max_ctas * ks * row_tiles;
      c->chain_ks = ks;
      c->chain_slices = max_ctas;
      c->chain_w_smem = w_smem;
      c->chain_barriers = static_cast<int>(c->layers.size()) - 1;   // one grid barrier between consecutive layers
      c->chain_tmap_off = ws;
      ws = align_up(ws + 2 * CHAIN_MAX_LAYERS * sizeof(CUtensorMap), 1024);
      // An 8-bit chain that ends in a single output column (the 256 -> 1 tail of a recommender's top MLP): that
      // column is a dot product over the row the layer before it has just finished, so its finishing threads add
      // their part of it per row instead of storing the row, and the barrier and the separate layer go away.
      {
        const size_t nl = c->layers.size();
        const LayerPlan& T = c->layers[nl - 1];
        const LayerPlan& P = c->layers[nl - 2];
        if (kind == 0 && ks > 1 && !T.use_tc && T.N == 1 && P.use_tc && P.out_pos < 0 && T.K == P.N && P.N % 32 == 0 &&
            (P.epi.out_dtype == GC_U8 || P.epi.out_dtype == GC_S8) && T.w_dtype == GC_S8 && !T.need_comp) {
          c->chain_fold_tail = true;
          c->chain_barriers -= 1;
          c->chain_tail_off = ws;
          ws = align_up(ws + 2 * sizeof(int) * static_cast<size_t>(T.M), 1024);
          c->desc += "  the one-column last layer is folded into the finishing step of the layer before it\n";
        }
      }
      c->launches = 1;
      snprintf(line, sizeof(line), "  fused chain: one persistent kernel, %d CTAs in clusters of %d (split reduction axis), %u KB of resident weight slices per CTA, %d grid barriers\n",
               max_ctas * ks * row_tiles, ks, w_smem / 1024, c->chain_barriers);
      c->desc += line;
    }
    // The smallest fp32 chains fit ONE thread-block cluster: weights of every layer resident in its CTAs, activations
    // handed from layer to layer through distributed shared memory (no grid barrier, no round trip through the L2).
    // Layer l uses slices_l = N_l / 32 column slices times ks_l parts of the reduction axis.
    if (ok && kind == 2 && row_tiles == 1 && !c->opt.grid_wide_chain) {
      // A first layer with a short reduction axis is recomputed by the CTAs of the second layer (each produces the
      // columns that form its own part of that layer's reduction axis) instead of being distributed and handed over.
      const bool can_recompute = c->layers.size() >= 2 && c->layers[0].nkb <= 2;
      for (int attempt = can_recompute ? 0 : 1; attempt < 2 && !c->chain_cluster; ++attempt) {   // (not re-indented)
      const bool recompute = attempt == 0;
      const size_t l_first = recompute ? 1 : 0;
      bool fit = c->layers[0].M <= 64;
      int want = 0;                                               // CTAs the widest distributed layer can use
      for (size_t l = 0; l < c->layers.size(); ++l) {
        const LayerPlan& L = c->layers[l];
        fit = fit && L.use_tc && L.N % 32 == 0 && L.epi.out_dtype == GC_F32 && !L.epi.acc_is_int;
        if (l >= l_first) want = std::max(want, (L.N / 32) * std::min(4, L.nkb));
      }
      const int C = want > 8 ? 16 : 8;
      const int rows_pad = (c->layers[0].M + 7) / 8 * 8;
      std::vector<int> ks_l(c->layers.size(), 1), rows_per(c->layers.size(), rows_pad);
      std::vector<uint32_t> w_off(c->layers.size(), 0);
      uint32_t cw = 0;
      int stages = 1, stage_rows = rows_pad;
      for (size_t l = l_first; fit && l < c->layers.size(); ++l) {
        const LayerPlan& L = c->layers[l];
        fit = L.N / 32 <= C;
        int ks = 1;
        while (ks < 4 && 2 * ks * (L.N / 32) <= C && 2 * ks <= L.nkb) ks *= 2;
        ks_l[l] = ks;
        rows_per[l] = ((rows_pad + ks - 1) / ks + 7) / 8 * 8;
        fit = fit && rows_per[l] <= 64;                           // two finishing threads per row, 128 of them
        stage_rows = std::max(stage_rows, ks * rows_per[l]);
        const int my_nkb = (L.nkb + ks - 1) / ks;
        stages = std::max(stages, my_nkb);
        w_off[l] = cw;
        cw += static_cast<uint32_t>(my_nkb) * 32 * 128;
      }
      if (fit && recompute) {
        const LayerPlan& L0 = c->layers[0];
        const LayerPlan& L1 = c->layers[1];
        const int n1 = (L1.nkb + ks_l[1] - 1) / ks_l[1];         // k-blocks of the second layer per CTA = 32-column groups to produce
        fit = n1 * 32 <= 256;                                     // one accumulator, one MMA N
        stages = std::max(stages, L0.nkb);
        w_off[0] = cw;
        cw += static_cast<uint32_t>(L0.nkb * n1) * 32 * 128;
      }
      size_t csmem = 0;
      if (fit) {
        csmem = mlp_cluster_smem_bytes(cw, stages, stage_rows * 128);
        fit = csmem <= static_cast<size_t>(prop.sharedMemPerBlockOptin);
      }
      if (fit && cuda_device != GC_DEVICE_PLAN_ONLY) {
        int cur = -1;
        cudaGetDevice(&cur);
        if (cur != cuda_device) cudaSetDevice(cuda_device);
        fit = mlp_cluster_max_clusters(C, csmem) >= 1;
        if (cur >= 0 && cur != cuda_device) cudaSetDevice(cur);
      }
      if (fit) {
        c->chain_cluster = C;
        c->chain_ks_l = ks_l;
        c->chain_rows_per = rows_per;
        c->chain_recompute_first = recompute;
        c->chain_w_off = w_off;
        c->chain_w_smem = cw;
        c->chain_a_stages = stages;
        c->chain_a_stage_bytes = stage_rows * 128;
        c->chain_grid = C;
        c->chain_barriers = 0;
        snprintf(line, sizeof(line), "  -> inside one cluster of %d CTAs instead: activations through distributed shared memory, %u KB of resident weight slices per CTA, no grid barrier%s\n",
                 C, cw / 1024, recompute ? "; first layer recomputed by the CTAs of the second" : "");
        c->desc += line;
      }
      }
    }
  }
  // Two consecutive large layers on CTA pairs: one launch with a tile schedule over both (see the kernel's header).
  if (c->pattern == PAT_MLP && !c->chain_fused && !c->opt.no_chain_fusion && !c->opt.force_generic) {
    auto out_kind = [](const LayerPlan& L) {
      return L.epi.out_dtype == GC_BF16 ? 1 : (L.epi.out_dtype == GC_F32 ? 2 : ((L.epi.acc_is_int && !L.epi.has_dq) ? 3 : 0));
    };
    for (size_t l = 0; l + 1 < c->layers.size(); ++l) {
      LayerPlan& A = c->layers[l];
      LayerPlan& B = c->layers[l + 1];
      if (l > 0 && c->layers[l - 1].fused_first) continue;       // A is already the second half of a pair
      const bool kinds_ok = A.use_tc && B.use_tc && A.cta2 && B.cta2 && A.kind == B.kind && A.M == B.M && !B.need_pack &&
                            out_kind(A) == out_kind(B) && out_kind(A) == A.kind;   // i8 -> 8-bit, bf16 -> bf16, tf32 -> f32
      if (!kinds_ok) continue;
      // Second-layer tiles wait on counters that first-layer tiles of OTHER clusters advance, so every cluster of the
      // launch must be resident at once: no more clusters than the device can hold of this kernel.
      int C = c->num_sms / 2;
      if (cuda_device != GC_DEVICE_PLAN_ONLY) {
        int cur = -1;
        cudaGetDevice(&cur);
        if (cur != cuda_device) cudaSetDevice(cuda_device);
        const int resident = gemm_tc2_max_clusters(A.kind, A.epi.out_dtype);
        if (cur >= 0 && cur != cuda_device) cudaSetDevice(cur);
        if (resident < C) C = resident;
      }
      if (C < 1) continue;
      const int m_pairs = (A.m_tiles + 1) / 2;
      const long T0 = static_cast<long>(m_pairs) * A.n_tiles, T1 = static_cast<long>(m_pairs) * B.n_tiles;
      const long w0 = A.nkb, w1 = B.nkb;
      if (T0 + T1 < 2L * C || T0 >= (1L << 24) || T1 >= (1L << 24)) continue;
      // Schedule (static, built here).  Every cluster's list holds its first-layer tiles, then its second-layer
      // tiles, so first-layer work never waits and the waits of the second layer cannot deadlock.  A second-layer
      // tile reads its A operand (256 hidden rows) in groups of k-blocks, one group per first-layer tile of that row
      // block, and waits group by group, so it can run right behind the tiles that produce its operand.  A tile
      // becomes readable a while after its main loop ends (epilogue, store completion, counter, the poll: about 24
      // k-block times measured on the FFN workload).  Candidates are built two ways and the step is simulated for
      // each; the shortest one wins:
      //  * "even": first-layer tiles round robin in row-block order; the clusters that will take one second-layer
      //    tile fewer take e = 0..4 extra first-layer tiles; second-layer tiles to whichever cluster is free first;
      //  * "balanced": second-layer quotas differ by at most one, first-layer quotas fill every cluster up to the
      //    same total work; the first-layer tiles of the slots in which only the clusters with large quotas are
      //    still busy (the tail) are dealt out column by column over the remaining row blocks, so that each of
      //    those row blocks becomes readable group by group in the order its consumers read it.
      const long lat = 24, lat_next = 20;
      const long kpg = B.kind == 0 ? 2 : (B.kind == 1 ? 4 : 8);   // (i8, bf16, tf32) second-layer k-blocks per first-layer tile
      const int heavy = T1 % C ? C - static_cast<int>(T1 % C) : 0;   // clusters with one second-layer tile fewer
      long best_span = -1;
      std::vector<int> best_sched;
      int best_pitch = 0;
      // simulate the second layer over given first-layer lists; quota[k] < 0: no limit
      auto finish = [&](std::vector<std::vector<int>>& list, std::vector<long> quota) {
        // when a first-layer tile becomes readable: the last one of a list lat after its main loop; the others
        // are announced at the end of the epilogue of the tile that follows them (see the kernel)
        std::vector<long> ready0(T0, 0), avail(C);
        for (int k = 0; k < C; ++k) {
          const size_t n = list[k].size();
          for (size_t i = 0; i < n; ++i)
            ready0[list[k][i]] = i + 1 == n ? static_cast<long>(i + 1) * w0 + lat : static_cast<long>(i + 2) * w0 + lat_next;
          avail[k] = static_cast<long>(n) * w0;
        }
        for (long t = 0; t < T1; ++t) {
          int bestk = -1;
          for (int k = 0; k < C; ++k)
            if (quota[k] != 0 && (bestk < 0 || avail[k] < avail[bestk])) bestk = k;
          if (bestk < 0) return;
          const long mp = t / B.n_tiles;
          long tt = avail[bestk];
          for (long j = 0; j < A.n_tiles; ++j) {
            const long r = ready0[mp * A.n_tiles + j];
            tt = (tt > r ? tt : r) + kpg;
          }
          tt += w1 - kpg * A.n_tiles > 0 ? w1 - kpg * A.n_tiles : 0;
          avail[bestk] = tt;
          if (quota[bestk] > 0) --quota[bestk];
          list[bestk].push_back((1 << 24) | static_cast<int>(t));
        }
        long span = 0;
        size_t longest = 0;
        for (int k = 0; k < C; ++k) {
          span = avail[k] > span ? avail[k] : span;
          longest = list[k].size() > longest ? list[k].size() : longest;
        }
        if (best_span < 0 || span < best_span) {
          best_span = span;
          best_pitch = static_cast<int>(longest) + 1;
          best_sched.assign(static_cast<size_t>(C) * best_pitch, -1);
          for (int k = 0; k < C; ++k)
            for (size_t i = 0; i < list[k].size(); ++i) best_sched[static_cast<size_t>(k) * best_pitch + i] = list[k][i];
        }
      };
      for (int e = 0; e <= 4; ++e) {                                // "even"
        if (e > 0 && heavy == 0) break;
        std::vector<long> n0(C, 0);
        const long light = C - heavy;
        long base = (T0 - static_cast<long>(heavy) * e) / C;
        if (base < 0) break;
        long rest = T0 - base * C - static_cast<long>(heavy) * e;
        for (int k = 0; k < C; ++k) n0[k] = base + (k >= light ? e : 0);
        for (int k = 0; rest > 0; k = (k + 1) % C, --rest) ++n0[k];
        std::vector<std::vector<int>> list(C);
        long next0 = 0;
        while (next0 < T0)
          for (int k = 0; k < C && next0 < T0; ++k)
            if (static_cast<long>(list[k].size()) < n0[k]) list[k].push_back(static_cast<int>(next0++));
        finish(list, std::vector<long>(C, -1));
      }
      {                                                             // "balanced"
        const double target = static_cast<double>(T0 * w0 + T1 * w1) / C;
        std::vector<long> b1(C), a0(C);
        long sum = 0;
        for (int k = 0; k < C; ++k) {
          b1[k] = T1 / C + (k < T1 % C ? 1 : 0);
          const double room = (target - static_cast<double>(b1[k] * w1)) / static_cast<double>(w0);
          a0[k] = room > 0 ? static_cast<long>(room + 0.5) : 0;
          sum += a0[k];
        }
        while (sum != T0) {                                         // rounding: take from the fullest / give to the emptiest
          int pick = -1;
          for (int k = 0; k < C; ++k) {
            if (sum > T0 && a0[k] == 0) continue;
            if (pick < 0) { pick = k; continue; }
            const long lk = a0[k] * w0 + b1[k] * w1, lp = a0[pick] * w0 + b1[pick] * w1;
            if (sum > T0 ? lk > lp : lk < lp) pick = k;
          }
          if (sum > T0) { --a0[pick]; --sum; } else { ++a0[pick]; ++sum; }
        }
        long amin = a0[0];
        for (int k = 1; k < C; ++k) amin = a0[k] < amin ? a0[k] : amin;
        std::vector<std::vector<int>> list(C);
        const long n_body = amin * C;
        for (long t = 0; t < n_body; ++t) list[t % C].push_back(static_cast<int>(t));
        // the tail: column by column (j-major) over the remaining tiles, slot by slot over the clusters with quota left
        std::vector<int> tail;
        for (long j = 0; j < A.n_tiles; ++j)
          for (long mp = 0; mp < m_pairs; ++mp)
            if (mp * A.n_tiles + j >= n_body) tail.push_back(static_cast<int>(mp * A.n_tiles + j));
        long amax = amin;
        for (int k = 0; k < C; ++k) amax = a0[k] > amax ? a0[k] : amax;
        size_t idx = 0;
        for (long slot = amin; slot < amax && idx < tail.size(); ++slot)
          for (int k = 0; k < C && idx < tail.size(); ++k)
            if (static_cast<long>(list[k].size()) == slot && slot < a0[k]) list[k].push_back(tail[idx++]);
        if (idx == tail.size()) finish(list, b1);
      }
      if (best_span < 0) continue;
      A.pair_pitch = best_pitch;
      A.pair_clusters = C;
      A.pair_sched = best_sched;
      const long worst = best_span;
      const double target = static_cast<double>(T0 * w0 + T1 * w1) / C;
      A.fused_first = true;
      A.pair_sched_off = ws;
      ws = align_up(ws + A.pair_sched.size() * sizeof(int), 256);
      A.pair_ready_off = ws;
      // epoch, finished CTAs, then one counter per first-layer tile
      A.pair_ready_words = 2 + static_cast<size_t>(T0);
      ws = align_up(ws + A.pair_ready_words * sizeof(unsigned long long), 256);
      c->launches -= 1;
      snprintf(line, sizeof(line), "  layers %zu+%zu: one launch, %d clusters, tile schedule over both (longest list %ld of %.1f k-blocks ideal)\n",
               l, l + 1, C, worst, target);
      c->desc += line;
    }
  }
  c->ws_bytes = align_up(ws, 1024);
  // host staging layout
  size_t so = 0;
  for (int i = 0; i < c->n_in; ++i) {
    c->in_stage_off.push_back(so);
    so = align_up(so + c->in_bytes[i], 256);
  }
  for (int i = 0; i < c->n_out; ++i) {
    c->out_stage_off.push_back(so);
    so = align_up(so + c->out_bytes[i], 256);
  }
  c->staging_bytes = so;
  *out = c;
  return GC_OK;
}

extern "C" void gc_compiled_destroy(gc_compiled_t* c) {
  if (!c) return;
  if (c->pipe_ready) {
    for (int s = 0; s < GC_HOST_SLOTS; ++s) {
      if (c->slot_busy[s]) cudaEventSynchronize(c->ev_out[s]);
      cudaEventDestroy(c->ev_in[s]);
      cudaEventDestroy(c->ev_exec[s]);
      cudaEventDestroy(c->ev_out[s]);
    }
    cudaStreamDestroy(c->h2d_stream);
    cudaStreamDestroy(c->d2h_stream);
  }
  delete c;
}

extern "C" gc_status_t gc_workspace_bytes(const gc_compiled_t* c, size_t* bytes) {
  if (!c || !bytes) return fail(GC_ERR_INVALID_ARG, "null argument");
  *bytes = c->ws_bytes;
  return GC_OK;
}

extern "C" gc_status_t gc_set_workspace(gc_compiled_t* c, void* ws, size_t bytes) {
  if (!c || !ws) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (bytes < c->ws_bytes) return fail(GC_ERR_INVALID_ARG, "workspace too small: %zu < %zu", bytes, c->ws_bytes);
  if (reinterpret_cast<uintptr_t>(ws) % 256) return fail(GC_ERR_ALIGNMENT, "workspace must be 256-byte aligned");
  c->ws = ws;
  c->prepacked = false;
  c->status_cleared = false;
  c->chain_tmaps_valid = false;
  for (auto& L : c->layers) {
    L.tmA_ptr = nullptr;
    L.tmD_ptr = nullptr;
    L.tmB_valid = false;
  }
  return GC_OK;
}

extern "C" gc_status_t gc_host_staging_bytes(const gc_compiled_t* c, size_t* bytes) {
  if (!c || !bytes) return fail(GC_ERR_INVALID_ARG, "null argument");
  *bytes = c->staging_bytes;
  return GC_OK;
}

extern "C" gc_status_t gc_set_host_staging(gc_compiled_t* c, void* p, size_t bytes) {
  if (!c || !p) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (bytes < c->staging_bytes) return fail(GC_ERR_INVALID_ARG, "staging area too small");
  if (reinterpret_cast<uintptr_t>(p) % 256) return fail(GC_ERR_ALIGNMENT, "staging area must be 256-byte aligned");
  for (int s = 0; s < GC_HOST_SLOTS; ++s)
    if (c->slot_busy[s]) return fail(GC_ERR_STATE, "a host execute is still in flight: call gc_host_wait first");
  c->staging = p;
  c->staging_slots = c->staging_bytes ? static_cast<int>(std::min<size_t>(GC_HOST_SLOTS, bytes / c->staging_bytes)) : 1;
  std::fill(c->host_const_seen.begin(), c->host_const_seen.end(), nullptr);
  return GC_OK;
}

extern "C" gc_status_t gc_launches_per_execute(const gc_compiled_t* c, int32_t* n) {
  if (!c || !n) return fail(GC_ERR_INVALID_ARG, "null argument");
  *n = c->launches;
  return GC_OK;
}

extern "C" const char* gc_plan_description(const gc_compiled_t* c) { return c ? c->desc.c_str() : ""; }

// ------------------------------------------------------------------------------------------------
// execute
// ------------------------------------------------------------------------------------------------
static gc_status_t run_mlp(gc_compiled& c, cudaStream_t st, const void* const* in, void* const* out) {
  char* ws = static_cast<char*>(c.ws);
  uint32_t* status = reinterpret_cast<uint32_t*>(ws);
  // constant-weight preprocessing: once, and again only if a constant arrives at a new address
  bool need = !c.prepacked;
  for (auto& L : c.layers) need = need || c.const_ptrs[L.w_input] != in[L.w_input];
  if (need) {
    for (auto& L : c.layers) {
      CUDA_TRY(launch_prepack_weight(in[L.w_input], ws + L.wt_off, L.K, L.N, L.Kp, L.transposed_w, L.w_dtype, st));
      if (!L.dqv_host.empty())
        CUDA_TRY(cudaMemcpyAsync(ws + L.dqv_off, L.dqv_host.data(), L.dqv_host.size() * sizeof(float), cudaMemcpyHostToDevice, st));
      if (L.need_comp)
        CUDA_TRY(launch_weight_compensation(ws + L.wt_off, L.N, L.Kp, L.a_zp, reinterpret_cast<int*>(ws + L.comp_off), st));
      c.const_ptrs[L.w_input] = in[L.w_input];
      if (L.fused_first) {
        CUDA_TRY(cudaMemcpyAsync(ws + L.pair_sched_off, L.pair_sched.data(), L.pair_sched.size() * sizeof(int),
                                 cudaMemcpyHostToDevice, st));
        CUDA_TRY(cudaMemsetAsync(ws + L.pair_ready_off, 0, L.pair_ready_words * sizeof(unsigned long long), st));
      }
    }
    c.prepacked = true;
  }
  if (c.chain_fused) {
    ChainParams cp = {};
    cp.n_layers = static_cast<int>(c.layers.size());
    cp.w_smem_bytes = c.chain_w_smem;
    cp.a_stages = c.chain_a_stages;
    cp.a_stage_bytes = c.chain_a_stage_bytes;
    cp.status = status;
    cp.barrier = reinterpret_cast<unsigned long long*>(ws + 64);
    cp.n_barriers = c.chain_barriers;
    cp.early_weights = need ? 0 : 1;
    cp.ks = c.chain_ks;
    cp.slices = c.chain_slices;
    const LayerPlan& L0 = c.layers[0];
    const void* a0 = in[L0.a_input];
    if (L0.need_pack) {
      const int esz0 = dtype_bytes(L0.a_dtype);
      cp.pack_src = a0;
      cp.pack_rows = L0.M;
      cp.pack_src_pitch = L0.a_pitch * esz0;
    }
    const bool rebuild = !c.chain_tmaps_valid || (!L0.need_pack && c.chain_a0_ptr != a0);
    if (rebuild) c.chain_tmaps.assign(2 * CHAIN_MAX_LAYERS, CUtensorMap());
    for (size_t l = 0; l < c.layers.size(); ++l) {
      const LayerPlan& L = c.layers[l];
      const int esz = dtype_bytes(L.a_dtype);
      ChainLayer& cl = cp.L[l];
      const void* A = l == 0 ? (L.need_pack ? static_cast<const void*>(ws + L.pack_off) : a0)
                             : static_cast<const void*>(ws + L.in_off);
      const int64_t a_pitch = (l == 0 && L.need_pack) ? L.pack_pitch : L.a_pitch;
      cl.M = L.M;
      cl.N = L.N;
      cl.K = L.K;
      cl.nkb = L.nkb;
      cl.active_ctas = L.use_tc ? (L.N + 31) / 32 : 0;
      cl.a_tm = static_cast<int>(2 * l);
      cl.b_tm = static_cast<int>(2 * l + 1);
      cl.w_smem_off = c.chain_w_off[l];
      cl.a_ptr = A;
      cl.wt_ptr = ws + L.wt_off;
      cl.a_pitch = a_pitch;
      cl.w_pitch = L.Kp;
      cl.a_dtype = L.a_dtype;
      cl.w_dtype = L.w_dtype;
      cl.a_zp = L.a_zp;
      cl.out = L.out_pos >= 0 ? out[L.out_pos] : static_cast<void*>(ws + L.out_off);
      cl.out_pitch = L.out_pitch;
      cl.out_elem = L.out_elem;
      cl.epi = L.epi;
      cl.epi.bias = L.bias_input >= 0 ? static_cast<const float*>(in[L.bias_input]) : nullptr;
      cl.epi.dqv = L.dqv_host.empty() ? nullptr : reinterpret_cast<const float*>(ws + L.dqv_off);
      cl.epi.comp = L.need_comp ? reinterpret_cast<const int*>(ws + L.comp_off) : nullptr;
      if (c.chain_cluster) {
        cl.ks_l = c.chain_ks_l[l];
        cl.rows_per = c.chain_rows_per[l];
      }
      if (L.use_tc) {
        const uint32_t afmt = L.a_dtype == GC_S8 ? 1u : 0u;
        cl.idesc = L.kind == 0   ? ((2u << 4) | (afmt << 7) | (1u << 10) | ((32u >> 3) << 17) | ((128u >> 4) << 24))
                   : L.kind == 1 ? ((1u << 4) | (1u << 7) | (1u << 10) | ((32u >> 3) << 17) | ((128u >> 4) << 24))
                                 : ((1u << 4) | (2u << 7) | (2u << 10) | ((32u >> 3) << 17) | ((128u >> 4) << 24));
        if (rebuild) {
          const int k_elems = 128 / esz;
          gc_status_t s = make_tmap(&c.chain_tmaps[2 * l], A, L.a_dtype, L.K, L.M, a_pitch * esz, k_elems, c.chain_a_rows, 128);
          if (s != GC_OK) return s;
          s = make_tmap(&c.chain_tmaps[2 * l + 1], ws + L.wt_off, L.w_dtype, L.Kp, L.N, static_cast<uint64_t>(L.Kp) * esz,
                        k_elems, 32, 128);
          if (s != GC_OK) return s;
        }
      }
    }
    if (rebuild) {
      c.chain_tmaps_valid = true;
      c.chain_a0_ptr = a0;
    }
    memcpy(cp.tmaps, c.chain_tmaps.data(), sizeof(cp.tmaps));
    cp.recompute_first = c.chain_recompute_first ? 1 : 0;
    cp.fold_tail = (c.chain_fold_tail && !c.chain_cluster) ? 1 : 0;
    cp.tail_acc = reinterpret_cast<int*>(ws + c.chain_tail_off);
    cp.tail_cnt = reinterpret_cast<unsigned int*>(ws + c.chain_tail_off) + c.layers.back().M;
    if (c.chain_cluster)
      CUDA_TRY(launch_mlp_cluster(cp, c.chain_cluster, st));
    else
      CUDA_TRY(launch_mlp_chain(c.chain_kind, cp, c.chain_grid, st));
    return GC_OK;
  }
  GemmTcParams pair_first = {};
  for (size_t l = 0; l < c.layers.size(); ++l) {
    LayerPlan& L = c.layers[l];
    const int esz = dtype_bytes(L.a_dtype);
    const void* A = l == 0 ? in[L.a_input] : ws + L.in_off;
    int64_t a_pitch = L.a_pitch;
    void* O = L.out_pos >= 0 ? out[L.out_pos] : ws + L.out_off;
    Epilogue e = L.epi;
    e.bias = L.bias_input >= 0 ? static_cast<const float*>(in[L.bias_input]) : nullptr;
    e.dqv = L.dqv_host.empty() ? nullptr : reinterpret_cast<const float*>(ws + L.dqv_off);
    e.comp = L.need_comp ? reinterpret_cast<const int*>(ws + L.comp_off) : nullptr;
    if (L.use_tc) {
      if (L.need_pack) {
        CUDA_TRY(launch_pack_rows(A, ws + L.pack_off, L.M, L.a_pitch * esz, L.pack_pitch * esz, st));
        A = ws + L.pack_off;
        a_pitch = L.pack_pitch;
      }
      const int k_elems = 128 / esz;
      if (L.tmA_ptr != A) {
        gc_status_t s = make_tmap(&L.tmA, A, L.a_dtype, L.K, L.M, a_pitch * esz, k_elems, 128, 128);
        if (s != GC_OK) return s;
        L.tmA_ptr = A;
      }
      if (!L.tmB_valid) {
        gc_status_t s = make_tmap(&L.tmB, ws + L.wt_off, L.w_dtype, L.Kp, L.N, static_cast<uint64_t>(L.Kp) * esz, k_elems,
                                  L.cta2 ? 128 : L.block_n, 128);
        if (s != GC_OK) return s;
        L.tmB_valid = true;
      }
      GemmTcParams g = {};
      g.M = L.M;
      g.N = L.N;
      g.K = L.K;
      g.num_k_blocks = L.nkb;
      g.m_tiles = L.m_tiles;
      g.n_tiles = L.n_tiles;
      g.out = O;
      g.out_pitch = L.out_pitch;
      g.epi = e;
      g.status = status;
      const int box_cols = gemm_tc_store_box_cols(L.block_n, L.out_elem);
      if (box_cols && L.tmD_ptr != O) {
        gc_status_t s = make_tmap(&L.tmD, O, L.epi.out_dtype, L.N, L.M, static_cast<uint64_t>(L.out_pitch) * L.out_elem,
                                  box_cols, 32, 128);
        if (s != GC_OK) return s;
        L.tmD_ptr = O;
      }
      // Programmatic dependent launch, also for the first layer: whatever ran before on the stream, this kernel's
      // set-up overlaps its tail and the kernel waits for it to complete before it touches global memory
      const bool pdl = !c.opt.no_chain_fusion && !L.need_pack;
      if (L.fused_first) {
        pair_first = g;                                            // launched together with the next layer
        continue;
      }
      if (l > 0 && c.layers[l - 1].fused_first) {
        LayerPlan& F = c.layers[l - 1];
        GemmPairParams pp = {};
        const GemmTcParams* gs[2] = {&pair_first, &g};
        const LayerPlan* ls[2] = {&F, &L};
        for (int k = 0; k < 2; ++k) {
          pp.L[k].N = gs[k]->N;
          pp.L[k].num_k_blocks = gs[k]->num_k_blocks;
          pp.L[k].n_tiles = gs[k]->n_tiles;
          pp.L[k].epi = gs[k]->epi;
          pp.tm[3 * k] = ls[k]->tmA;
          pp.tm[3 * k + 1] = ls[k]->tmB;
          pp.tm[3 * k + 2] = ls[k]->tmD;
        }
        pp.sched = reinterpret_cast<const int*>(ws + F.pair_sched_off);
        pp.sched_pitch = F.pair_pitch;
        pp.ready = reinterpret_cast<unsigned long long*>(ws + F.pair_ready_off);
        pp.status = status;
        CUDA_TRY(launch_gemm_tc2_fused(L.kind, F.a_dtype == GC_S8, pp, 2 * F.pair_clusters, st));
        continue;
      }
      if (L.cta2)
        CUDA_TRY(launch_gemm_tc2(L.kind, L.a_dtype == GC_S8, L.tmA, L.tmB, L.tmD, g, L.grid, pdl, st));
      else
        CUDA_TRY(launch_gemm_tc(L.kind, L.block_n, L.a_dtype == GC_S8, L.tmA, L.tmB, box_cols ? L.tmD : L.tmA, g, L.grid,
                                pdl, st));
    } else {
      GemmSimtParams g = {};
      g.A = A;
      g.Wt = ws + L.wt_off;
      g.a_pitch = a_pitch;
      g.w_pitch = L.Kp;
      g.M = L.M;
      g.N = L.N;
      g.K = L.K;
      g.batch = 1;
      g.a_dtype = L.a_dtype;
      g.w_dtype = L.w_dtype;
      g.a_zp = L.a_zp;
      g.w_zp = 0;
      g.out = O;
      g.out_pitch = L.out_pitch;
      g.epi = e;
      CUDA_TRY(launch_gemm_simt(g, st));
    }
  }
  return GC_OK;
}

static gc_status_t run_sdpa(gc_compiled& c, cudaStream_t st, const void* const* in, void* const* out) {
  SdpaPlan& s = c.sdpa;
  SdpaParams prm = s.prm;
  prm.Q = in[s.q_input];
  prm.K = in[s.k_input];
  prm.V = in[s.v_input];
  prm.mask = s.mask_input >= 0 ? static_cast<const float*>(in[s.mask_input]) : nullptr;
  prm.O = out[0];
  prm.P_out = s.p_out_pos >= 0 ? out[s.p_out_pos] : nullptr;
  prm.status = reinterpret_cast<uint32_t*>(c.ws);
  if (!s.use_tc) {
    CUDA_TRY(launch_sdpa_simt(prm, st));
    return GC_OK;
  }
  const int dt = prm.is_int8 ? GC_U8 : GC_BF16;
  const int esz = prm.is_int8 ? 1 : 2;
  const uint64_t rows = static_cast<uint64_t>(prm.B) * prm.H * prm.S;
  if (s.wide) {
    int box = 0, swz = 0;
    sdpa_wide_box(prm.D, prm.is_int8, &box, &swz);
    const void* ptrs[3] = {prm.Q, prm.K, prm.V};
    const void** cached[3] = {&s.q_ptr, &s.k_ptr, &s.v_ptr};
    CUtensorMap* maps[3] = {&s.tmQ, &s.tmK, &s.tmV};
    for (int i = 0; i < 3; ++i) {
      if (*cached[i] == ptrs[i]) continue;
      // a box wider than the head (D = 96) reads zeros past the tensor's edge, and so does a box that reaches past
      // the end of a head's sequence (sequence lengths that are not a multiple of 128)
      gc_status_t r = make_tmap3(maps[i], ptrs[i], dt, prm.D, prm.S, static_cast<uint64_t>(prm.B) * prm.H, box, 128, swz);
      if (r != GC_OK) return r;
      *cached[i] = ptrs[i];
    }
    if (s.two_pass)
      CUDA_TRY(launch_sdpa_long(s.tmQ, s.tmK, s.tmV, prm, c.num_sms, st));
    else
      CUDA_TRY(launch_sdpa_wide(s.tmQ, s.tmK, s.tmV, prm, c.num_sms, st));
    return GC_OK;
  }
  const int swz = prm.is_int8 ? 64 : 128;
  if (s.q_ptr != prm.Q) {
    gc_status_t r = make_tmap(&s.tmQ, prm.Q, dt, prm.D, rows, static_cast<uint64_t>(prm.D) * esz, prm.D, 128, swz);
    if (r != GC_OK) return r;
    s.q_ptr = prm.Q;
  }
  if (s.k_ptr != prm.K) {
    gc_status_t r = make_tmap(&s.tmK, prm.K, dt, prm.D, rows, static_cast<uint64_t>(prm.D) * esz, prm.D, 128, swz);
    if (r != GC_OK) return r;
    s.k_ptr = prm.K;
  }
  if (s.v_ptr != prm.V) {
    gc_status_t r = make_tmap(&s.tmV, prm.V, dt, prm.D, rows, static_cast<uint64_t>(prm.D) * esz, prm.D, 128, swz);
    if (r != GC_OK) return r;
    s.v_ptr = prm.V;
  }
  if (s.small) {
    CUDA_TRY(launch_sdpa_small(s.tmQ, s.tmK, s.tmV, prm, st));
    return GC_OK;
  }
  if (s.o_ptr != prm.O) {
    gc_status_t r = make_tmap(&s.tmO, prm.O, dt, prm.D, rows, static_cast<uint64_t>(prm.D) * esz, prm.D, 32, prm.D * esz);
    if (r != GC_OK) return r;
    s.o_ptr = prm.O;
  }
  CUDA_TRY(launch_sdpa_tc(s.tmQ, s.tmK, s.tmV, s.tmO, prm, c.num_sms, st));
  return GC_OK;
}

// Zero the status word, the chain kernel's grid-barrier counter (both in the first 256 bytes of the workspace) and
// the counters of every fused two-layer launch.
static gc_status_t reset_device_state(gc_compiled& c, cudaStream_t st) {
  CUDA_TRY(cudaMemsetAsync(c.ws, 0, 256, st));
  if (c.chain_fold_tail)
    CUDA_TRY(cudaMemsetAsync(static_cast<char*>(c.ws) + c.chain_tail_off, 0, 2 * sizeof(int) * static_cast<size_t>(c.layers.back().M), st));
  for (auto& L : c.layers)
    if (L.fused_first)
      CUDA_TRY(cudaMemsetAsync(static_cast<char*>(c.ws) + L.pair_ready_off, 0, L.pair_ready_words * sizeof(unsigned long long), st));
  return GC_OK;
}

extern "C" gc_status_t gc_execute(gc_compiled_t* c, void* cuda_stream, const void* const* in_dev, int32_t n_in,
                                  void* const* out_dev, int32_t n_out) {
  if (!c || !in_dev || !out_dev) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (n_in != c->n_in || n_out != c->n_out)
    return fail(GC_ERR_INVALID_ARG, "expected %d inputs and %d outputs, got %d and %d", c->n_in, c->n_out, n_in, n_out);
  if (c->device < 0) return fail(GC_ERR_STATE, "compiled with GC_DEVICE_PLAN_ONLY: cannot execute");
  if (!c->ws) return fail(GC_ERR_STATE, "gc_set_workspace has not been called");
  for (int i = 0; i < n_in; ++i) {
    if (!in_dev[i]) return fail(GC_ERR_INVALID_ARG, "input %d is null", i);
    if (reinterpret_cast<uintptr_t>(in_dev[i]) % 16) return fail(GC_ERR_ALIGNMENT, "input %d is not 16-byte aligned", i);
  }
  for (int i = 0; i < n_out; ++i) {
    if (!out_dev[i]) return fail(GC_ERR_INVALID_ARG, "output %d is null", i);
    if (reinterpret_cast<uintptr_t>(out_dev[i]) % 16) return fail(GC_ERR_ALIGNMENT, "output %d is not 16-byte aligned", i);
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  int cur = -1;
  CUDA_TRY(cudaGetDevice(&cur));
  if (cur != c->device) CUDA_TRY(cudaSetDevice(c->device));
  if (!c->status_cleared) {
    CUDA_TRY(cudaMemsetAsync(c->ws, 0, 256, st));
    if (c->chain_fold_tail)
      CUDA_TRY(cudaMemsetAsync(static_cast<char*>(c->ws) + c->chain_tail_off, 0, 2 * sizeof(int) * static_cast<size_t>(c->layers.back().M), st));
    c->status_cleared = true;
  }
  gc_status_t r;
  if (c->pattern == PAT_MLP) {
    r = run_mlp(*c, st, in_dev, out_dev);
  } else if (c->pattern == PAT_SDPA) {
    r = run_sdpa(*c, st, in_dev, out_dev);
  } else {
    GemmSimtParams g = c->bmm;
    g.A = in_dev[0];
    g.Wt = in_dev[1];
    g.out = out_dev[0];
    cudaError_t e = launch_gemm_simt(g, st);
    r = e == cudaSuccess ? GC_OK : fail(GC_ERR_CUDA, "launch_gemm_simt: %s", cudaGetErrorString(e));
  }
  return r;
}

// Enqueue one host-buffer execute on staging slot `slot`: inputs -> slot (on `in_st`), execute (on `st`), slot -> host
// (on `out_st`).  With in_st == st == out_st everything is ordered by the stream alone; otherwise the three are chained
// by the slot's events.  The constants live in slot 0 only (one device address, so the prepack cache stays valid).
static gc_status_t host_enqueue(gc_compiled_t* c, cudaStream_t st, cudaStream_t in_st, cudaStream_t out_st, int slot,
                                const void* const* in_host, int32_t n_in, void* const* out_host, int32_t n_out) {
  char* base0 = static_cast<char*>(c->staging);
  char* sg = base0 + static_cast<size_t>(slot) * c->staging_bytes;
  std::vector<const void*> din(n_in);
  std::vector<void*> dout(n_out);
  for (int i = 0; i < n_in; ++i)
    if (!in_host[i]) return fail(GC_ERR_INVALID_ARG, "input %d is null", i);
  for (int i = 0; i < n_out; ++i)
    if (!out_host[i]) return fail(GC_ERR_INVALID_ARG, "output %d is null", i);
  for (int i = 0; i < n_in; ++i) {
    if (c->in_constant[i]) {
      din[i] = base0 + c->in_stage_off[i];
      if (c->host_const_seen[i] != in_host[i]) {
        CUDA_TRY(cudaMemcpyAsync(base0 + c->in_stage_off[i], in_host[i], c->in_bytes[i], cudaMemcpyHostToDevice, st));
        // A constant that arrives at a new host address lands at the same staging address: forget the device
        // pointer recorded at the last prepack, so that the execute below preprocesses the new contents.
        if (c->host_const_seen[i] != nullptr) c->const_ptrs[i] = nullptr;
        c->host_const_seen[i] = in_host[i];
      }
    } else {
      din[i] = sg + c->in_stage_off[i];
      CUDA_TRY(cudaMemcpyAsync(sg + c->in_stage_off[i], in_host[i], c->in_bytes[i], cudaMemcpyHostToDevice, in_st));
    }
  }
  if (in_st != st) {
    CUDA_TRY(cudaEventRecord(c->ev_in[slot], in_st));
    CUDA_TRY(cudaStreamWaitEvent(st, c->ev_in[slot], 0));
  }
  for (int i = 0; i < n_out; ++i) dout[i] = sg + c->out_stage_off[i];
  gc_status_t r = gc_execute(c, st, din.data(), n_in, dout.data(), n_out);
  if (r != GC_OK) return r;
  if (out_st != st) {
    CUDA_TRY(cudaEventRecord(c->ev_exec[slot], st));
    CUDA_TRY(cudaStreamWaitEvent(out_st, c->ev_exec[slot], 0));
  }
  for (int i = 0; i < n_out; ++i)
    CUDA_TRY(cudaMemcpyAsync(out_host[i], sg + c->out_stage_off[i], c->out_bytes[i], cudaMemcpyDeviceToHost, out_st));
  return GC_OK;
}

extern "C" gc_status_t gc_execute_host(gc_compiled_t* c, void* cuda_stream, const void* const* in_host, int32_t n_in,
                                       void* const* out_host, int32_t n_out) {
  if (!c || !in_host || !out_host) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (n_in != c->n_in || n_out != c->n_out) return fail(GC_ERR_INVALID_ARG, "wrong number of inputs or outputs");
  if (!c->staging) return fail(GC_ERR_STATE, "gc_set_host_staging has not been called");
  if (c->slot_busy[0]) return fail(GC_ERR_STATE, "staging slot 0 is in flight: call gc_host_wait first");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  gc_status_t r = host_enqueue(c, st, st, st, 0, in_host, n_in, out_host, n_out);
  if (r != GC_OK) return r;
  CUDA_TRY(cudaStreamSynchronize(st));
  return GC_OK;
}

extern "C" gc_status_t gc_execute_host_async(gc_compiled_t* c, void* cuda_stream, int32_t slot, const void* const* in_host,
                                             int32_t n_in, void* const* out_host, int32_t n_out) {
  if (!c || !in_host || !out_host) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (n_in != c->n_in || n_out != c->n_out) return fail(GC_ERR_INVALID_ARG, "wrong number of inputs or outputs");
  if (!c->staging) return fail(GC_ERR_STATE, "gc_set_host_staging has not been called");
  if (slot < 0 || slot >= c->staging_slots)
    return fail(GC_ERR_INVALID_ARG, "slot %d: the staging area holds %d slot(s) of gc_host_staging_bytes each", slot,
                c->staging_slots);
  if (c->slot_busy[slot]) return fail(GC_ERR_STATE, "slot %d is still in flight: call gc_host_wait first", slot);
  int cur = -1;
  CUDA_TRY(cudaGetDevice(&cur));
  if (cur != c->device) CUDA_TRY(cudaSetDevice(c->device));
  if (!c->pipe_ready) {
    CUDA_TRY(cudaStreamCreateWithFlags(&c->h2d_stream, cudaStreamNonBlocking));
    CUDA_TRY(cudaStreamCreateWithFlags(&c->d2h_stream, cudaStreamNonBlocking));
    for (int s = 0; s < GC_HOST_SLOTS; ++s) {
      CUDA_TRY(cudaEventCreateWithFlags(&c->ev_in[s], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&c->ev_exec[s], cudaEventDisableTiming));
      CUDA_TRY(cudaEventCreateWithFlags(&c->ev_out[s], cudaEventDisableTiming));
    }
    c->pipe_ready = true;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  gc_status_t r = host_enqueue(c, st, c->h2d_stream, c->d2h_stream, slot, in_host, n_in, out_host, n_out);
  if (r != GC_OK) {
    // whatever was enqueued before the failure must not outlive the caller's buffers
    cudaStreamSynchronize(c->h2d_stream);
    cudaStreamSynchronize(st);
    cudaStreamSynchronize(c->d2h_stream);
    return r;
  }
  CUDA_TRY(cudaEventRecord(c->ev_out[slot], c->d2h_stream));
  c->slot_busy[slot] = true;
  return GC_OK;
}

extern "C" gc_status_t gc_host_wait(gc_compiled_t* c, int32_t slot) {
  if (!c) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (slot < 0 || slot >= GC_HOST_SLOTS) return fail(GC_ERR_INVALID_ARG, "slot %d out of range", slot);
  if (!c->slot_busy[slot]) return GC_OK;
  c->slot_busy[slot] = false;
  CUDA_TRY(cudaEventSynchronize(c->ev_out[slot]));
  return GC_OK;
}

extern "C" gc_status_t gc_selftest_bounded_wait(void* cuda_stream, void* status_dev, uint32_t limit_us) {
  if (!status_dev) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (reinterpret_cast<uintptr_t>(status_dev) % 4) return fail(GC_ERR_ALIGNMENT, "status word must be 4-byte aligned");
  if (limit_us > 100000u) limit_us = 100000u;
  CUDA_TRY(launch_bounded_wait_selftest(static_cast<uint32_t*>(status_dev), static_cast<uint64_t>(limit_us) * 1000ull,
                                        static_cast<cudaStream_t>(cuda_stream)));
  return GC_OK;
}

extern "C" gc_status_t gc_query_status(gc_compiled_t* c, void* cuda_stream) {
  if (!c) return fail(GC_ERR_INVALID_ARG, "null argument");
  if (!c->ws) return fail(GC_ERR_STATE, "gc_set_workspace has not been called");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint32_t word = 0;
  CUDA_TRY(cudaMemcpyAsync(&word, c->ws, sizeof(word), cudaMemcpyDeviceToHost, st));
  CUDA_TRY(cudaStreamSynchronize(st));
  if (word != 0) {
    // The kernels that gave up left their synchronisation counters (grid-barrier count, the fused two-layer
    // launch's epoch and per-tile counters) mid-count.  The stream is idle here: zero them together with the status
    // word, so that the next execute starts from a clean state; the cached prepacked weights stay valid.
    gc_status_t r = reset_device_state(*c, st);
    if (r != GC_OK) return r;
    CUDA_TRY(cudaStreamSynchronize(st));
    return fail(GC_ERR_TIMEOUT, "a bounded device-side wait expired (code 0x%x); the object's device state has been reset",
                word);
  }
  return GC_OK;
}

extern "C" gc_status_t gc_invalidate_constants(gc_compiled_t* c) {
  if (!c) return fail(GC_ERR_INVALID_ARG, "null argument");
  c->prepacked = false;
  std::fill(c->const_ptrs.begin(), c->const_ptrs.end(), nullptr);
  std::fill(c->host_const_seen.begin(), c->host_const_seen.end(), nullptr);
  return GC_OK;
}
