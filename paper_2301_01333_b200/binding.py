"""ctypes binding of the C ABI in ``include/gc.h``: argument marshalling only.

Every function here has the name of the C entry point it forwards to.  PyTorch is used for device
memory and streams (``CompiledPartition`` allocates the workspace with torch and passes raw pointers);
all computation happens in the CUDA library.  Loading fails loudly when the library has not been
built - there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import numpy as np

from .graph import Graph

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgc_b200.so")

GC_OK, GC_ERR_INVALID_ARG, GC_ERR_UNSUPPORTED, GC_ERR_SHAPE, GC_ERR_STATE, GC_ERR_CUDA, GC_ERR_OOM, \
    GC_ERR_TIMEOUT, GC_ERR_ALIGNMENT = range(9)
STATUS_NAMES = ["GC_OK", "GC_ERR_INVALID_ARG", "GC_ERR_UNSUPPORTED", "GC_ERR_SHAPE", "GC_ERR_STATE",
                "GC_ERR_CUDA", "GC_ERR_OOM", "GC_ERR_TIMEOUT", "GC_ERR_ALIGNMENT"]
GC_DEVICE_PLAN_ONLY = -1
DTYPE_CODE = {"f32": 0, "bf16": 1, "u8": 2, "s8": 3, "s32": 4}
OP_CODE = {"matmul": 0, "add": 1, "mul": 2, "relu": 3, "gelu_tanh": 4, "sigmoid": 5, "softmax": 6,
           "quantize": 7, "dequantize": 8, "typecast": 9}
NP_DTYPE = {"f32": np.float32, "bf16": np.uint16, "u8": np.uint8, "s8": np.int8, "s32": np.int32}

# every symbol include/gc.h declares
EXPORTS = [
    "gc_partition_create", "gc_partition_destroy", "gc_compile", "gc_compiled_destroy", "gc_workspace_bytes",
    "gc_set_workspace", "gc_execute", "gc_host_staging_bytes", "gc_set_host_staging", "gc_execute_host",
    "gc_execute_host_async", "gc_host_wait",
    "gc_query_status", "gc_launches_per_execute", "gc_plan_description", "gc_last_error", "gc_version",
    "gc_matmul_s32_noalloc", "gc_noalloc_scratch_bytes", "gc_selftest_bounded_wait", "gc_invalidate_constants",
]


class gc_logical_tensor_t(C.Structure):
    _fields_ = [("id", C.c_int64), ("dtype", C.c_int32), ("ndims", C.c_int32), ("dims", C.c_int64 * 6),
                ("scale", C.c_float), ("zero_point", C.c_int32), ("is_constant", C.c_int32),
                ("channel_scales", C.POINTER(C.c_float)), ("channel_axis", C.c_int32), ("reserved_", C.c_int32)]


class gc_op_t(C.Structure):
    _fields_ = [("kind", C.c_int32), ("n_in", C.c_int32), ("in_", C.c_int64 * 3), ("out", C.c_int64),
                ("transpose_b", C.c_int32), ("axis", C.c_int32), ("scalar", C.c_float), ("has_scalar", C.c_int32)]


class gc_compile_options_t(C.Structure):
    _fields_ = [("force_generic", C.c_int32), ("no_chain_fusion", C.c_int32), ("streaming_attention", C.c_int32),
                ("exact_max_softmax", C.c_int32), ("grid_wide_chain", C.c_int32), ("reserved", C.c_int32 * 3)]


class GcError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {message}")
        self.status = status


_lib = None


def load_library() -> C.CDLL:
    """dlopen the in-tree CUDA library; raise if it is missing (run ``python -m paper_2301_01333_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2301_01333_b200.build`; "
                          "there is no non-CUDA fallback")
    lib = C.CDLL(LIB_PATH)
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    lib.gc_partition_create.argtypes = [C.POINTER(vp), C.POINTER(gc_op_t), i32, C.POINTER(gc_logical_tensor_t), i32,
                                        C.POINTER(C.c_int64), i32, C.POINTER(C.c_int64), i32]
    lib.gc_partition_destroy.argtypes = [vp]
    lib.gc_partition_destroy.restype = None
    lib.gc_compile.argtypes = [vp, i32, C.POINTER(gc_compile_options_t), C.POINTER(vp)]
    lib.gc_compiled_destroy.argtypes = [vp]
    lib.gc_compiled_destroy.restype = None
    lib.gc_workspace_bytes.argtypes = [vp, C.POINTER(sz)]
    lib.gc_set_workspace.argtypes = [vp, vp, sz]
    lib.gc_execute.argtypes = [vp, vp, C.POINTER(vp), i32, C.POINTER(vp), i32]
    lib.gc_host_staging_bytes.argtypes = [vp, C.POINTER(sz)]
    lib.gc_set_host_staging.argtypes = [vp, vp, sz]
    lib.gc_execute_host.argtypes = [vp, vp, C.POINTER(vp), i32, C.POINTER(vp), i32]
    lib.gc_execute_host_async.argtypes = [vp, vp, i32, C.POINTER(vp), i32, C.POINTER(vp), i32]
    lib.gc_host_wait.argtypes = [vp, i32]
    lib.gc_query_status.argtypes = [vp, vp]
    lib.gc_launches_per_execute.argtypes = [vp, C.POINTER(i32)]
    lib.gc_plan_description.argtypes = [vp]
    lib.gc_plan_description.restype = C.c_char_p
    lib.gc_last_error.restype = C.c_char_p
    lib.gc_version.restype = C.c_char_p
    lib.gc_matmul_s32_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32]
    lib.gc_matmul_s32_noalloc.restype = i32
    lib.gc_noalloc_scratch_bytes.restype = sz
    lib.gc_invalidate_constants.argtypes = [vp]
    lib.gc_invalidate_constants.restype = i32
    lib.gc_selftest_bounded_wait.argtypes = [vp, vp, C.c_uint32]
    lib.gc_selftest_bounded_wait.restype = i32
    for name in ("gc_partition_create", "gc_compile", "gc_workspace_bytes", "gc_set_workspace", "gc_execute",
                 "gc_host_staging_bytes", "gc_set_host_staging", "gc_execute_host", "gc_execute_host_async",
                 "gc_host_wait", "gc_query_status", "gc_launches_per_execute"):
        getattr(lib, name).restype = i32
    _lib = lib
    return lib


def _check(st: int) -> None:
    if st != GC_OK:
        raise GcError(st, gc_last_error())


def gc_last_error() -> str:
    return load_library().gc_last_error().decode()


def gc_version() -> str:
    return load_library().gc_version().decode()


def marshal_graph(g: Graph):
    """Graph -> (ops array, tensors array, input ids, output ids) in the C layout."""
    tensors = (gc_logical_tensor_t * len(g.tensors))()
    keep = []
    for i, t in enumerate(g.tensors.values()):
        tensors[i].id = t.id
        tensors[i].dtype = DTYPE_CODE[t.dtype]
        tensors[i].ndims = len(t.dims)
        for d, v in enumerate(t.dims):
            tensors[i].dims[d] = v
        tensors[i].scale = t.scale
        tensors[i].zero_point = t.zero_point
        tensors[i].is_constant = int(t.is_constant)
        if t.channel_scales is not None:
            cs = (C.c_float * len(t.channel_scales))(*t.channel_scales)
            keep.append(cs)                      # alive until gc_partition_create has copied it
            tensors[i].channel_scales = C.cast(cs, C.POINTER(C.c_float))
            tensors[i].channel_axis = t.channel_axis
    tensors._channel_scale_arrays = keep
    ops = (gc_op_t * len(g.ops))()
    for i, op in enumerate(g.ops):
        ops[i].kind = OP_CODE[op.kind]
        ops[i].n_in = len(op.inputs)
        for k, v in enumerate(op.inputs):
            ops[i].in_[k] = v
        ops[i].out = op.output
        ops[i].transpose_b = int(op.transpose_b)
        ops[i].axis = op.axis
        ops[i].scalar = 0.0 if op.scalar is None else op.scalar
        ops[i].has_scalar = int(op.scalar is not None)
    ins = (C.c_int64 * len(g.inputs))(*g.inputs)
    outs = (C.c_int64 * len(g.outputs))(*g.outputs)
    return ops, tensors, ins, outs


def gc_partition_create(g: Graph) -> C.c_void_p:
    lib = load_library()
    ops, tensors, ins, outs = marshal_graph(g)
    h = C.c_void_p()
    _check(lib.gc_partition_create(C.byref(h), ops, len(ops), tensors, len(tensors), ins, len(ins), outs, len(outs)))
    return h


def gc_partition_destroy(p) -> None:
    load_library().gc_partition_destroy(p)


def gc_compile(p, cuda_device: int = 0, force_generic: bool = False, no_chain_fusion: bool = False,
               streaming_attention: bool = False, exact_max_softmax: bool = False,
               grid_wide_chain: bool = False) -> C.c_void_p:
    lib = load_library()
    opt = gc_compile_options_t()
    opt.force_generic = int(force_generic)
    opt.no_chain_fusion = int(no_chain_fusion)
    opt.streaming_attention = int(streaming_attention)
    opt.exact_max_softmax = int(exact_max_softmax)
    opt.grid_wide_chain = int(grid_wide_chain)
    h = C.c_void_p()
    _check(lib.gc_compile(p, cuda_device, C.byref(opt), C.byref(h)))
    return h


def gc_compiled_destroy(c) -> None:
    load_library().gc_compiled_destroy(c)


def gc_workspace_bytes(c) -> int:
    n = C.c_size_t()
    _check(load_library().gc_workspace_bytes(c, C.byref(n)))
    return n.value


def gc_set_workspace(c, dev_ptr: int, nbytes: int) -> None:
    _check(load_library().gc_set_workspace(c, C.c_void_p(dev_ptr), nbytes))


def gc_host_staging_bytes(c) -> int:
    n = C.c_size_t()
    _check(load_library().gc_host_staging_bytes(c, C.byref(n)))
    return n.value


def gc_set_host_staging(c, dev_ptr: int, nbytes: int) -> None:
    _check(load_library().gc_set_host_staging(c, C.c_void_p(dev_ptr), nbytes))


def _ptr_array(ptrs: Sequence[int]):
    return (C.c_void_p * len(ptrs))(*[C.c_void_p(p) for p in ptrs])


def gc_execute(c, stream: int, in_ptrs: Sequence[int], out_ptrs: Sequence[int]) -> None:
    _check(load_library().gc_execute(c, C.c_void_p(stream), _ptr_array(in_ptrs), len(in_ptrs), _ptr_array(out_ptrs),
                                     len(out_ptrs)))


def gc_execute_host(c, stream: int, in_ptrs: Sequence[int], out_ptrs: Sequence[int]) -> None:
    _check(load_library().gc_execute_host(c, C.c_void_p(stream), _ptr_array(in_ptrs), len(in_ptrs),
                                          _ptr_array(out_ptrs), len(out_ptrs)))


def gc_execute_host_async(c, stream: int, slot: int, in_ptrs: Sequence[int], out_ptrs: Sequence[int]) -> None:
    _check(load_library().gc_execute_host_async(c, C.c_void_p(stream), slot, _ptr_array(in_ptrs), len(in_ptrs),
                                                _ptr_array(out_ptrs), len(out_ptrs)))


def gc_host_wait(c, slot: int) -> None:
    _check(load_library().gc_host_wait(c, slot))


def gc_query_status(c, stream: int = 0) -> None:
    _check(load_library().gc_query_status(c, C.c_void_p(stream)))


def gc_invalidate_constants(c) -> None:
    _check(load_library().gc_invalidate_constants(c))


def gc_launches_per_execute(c) -> int:
    n = C.c_int32()
    _check(load_library().gc_launches_per_execute(c, C.byref(n)))
    return n.value


def gc_plan_description(c) -> str:
    return load_library().gc_plan_description(c).decode()


def gc_noalloc_scratch_bytes() -> int:
    return load_library().gc_noalloc_scratch_bytes()


def gc_matmul_s32_noalloc(stream: int, a_ptr: int, w_ptr: int, out_ptr: int, m: int, k: int, n: int,
                          a_zero_point: int = 0) -> None:
    """out[m,n] (s32) = (a - zp) @ w for u8 a [m,k] and s8 w [k,n], all device pointers.  For callers
    that cannot allocate: the scratch is a fixed 1 MiB array inside the library, shared by all calls."""
    _check(load_library().gc_matmul_s32_noalloc(C.c_void_p(stream), C.c_void_p(a_ptr), C.c_void_p(w_ptr),
                                                C.c_void_p(out_ptr), m, k, n, a_zero_point))


def gc_selftest_bounded_wait(stream: int, status_ptr: int, limit_us: int) -> None:
    """Launch the kernel whose wait cannot be satisfied; after limit_us it writes a timeout code to *status_ptr."""
    _check(load_library().gc_selftest_bounded_wait(C.c_void_p(stream), C.c_void_p(status_ptr), limit_us))


class CompiledPartition:
    """Convenience owner: partition + compiled object + torch-allocated workspace."""

    def __init__(self, g: Graph, device: int = 0, force_generic: bool = False, no_chain_fusion: bool = False,
                 streaming_attention: bool = False, exact_max_softmax: bool = False, grid_wide_chain: bool = False):
        import torch
        self.graph = g
        self.device = device
        self._part = gc_partition_create(g)
        try:
            self._comp = gc_compile(self._part, device, force_generic, no_chain_fusion, streaming_attention,
                                    exact_max_softmax, grid_wide_chain)
        except Exception:
            gc_partition_destroy(self._part)
            self._part = None
            raise
        self._ws = None
        self._staging = None
        if device >= 0:
            n = gc_workspace_bytes(self._comp)
            self._ws = torch.empty(max(n, 256), dtype=torch.uint8, device=f"cuda:{device}")
            gc_set_workspace(self._comp, self._ws.data_ptr(), self._ws.numel())
        self._in_arrays = (C.c_void_p * len(g.inputs))()
        self._out_arrays = (C.c_void_p * len(g.outputs))()
        self._lib = load_library()

    # -- queries ----------------------------------------------------------------------------------
    @property
    def launches(self) -> int:
        return gc_launches_per_execute(self._comp)

    @property
    def plan(self) -> str:
        return gc_plan_description(self._comp)

    @property
    def workspace_bytes(self) -> int:
        return gc_workspace_bytes(self._comp)

    # -- device execution -------------------------------------------------------------------------
    def execute(self, inputs, outputs, stream: Optional[int] = None) -> None:
        """inputs / outputs: torch CUDA tensors (any dtype view; only data_ptr() is used)."""
        import torch
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        for i, t in enumerate(inputs):
            self._in_arrays[i] = t.data_ptr()
        for i, t in enumerate(outputs):
            self._out_arrays[i] = t.data_ptr()
        st = self._lib.gc_execute(self._comp, C.c_void_p(stream), self._in_arrays, len(inputs), self._out_arrays,
                                  len(outputs))
        if st != GC_OK:
            raise GcError(st, gc_last_error())

    def execute_ptrs(self, in_ptrs, out_ptrs, stream: int) -> None:
        gc_execute(self._comp, stream, in_ptrs, out_ptrs)

    def query_status(self, stream: Optional[int] = None) -> None:
        import torch
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        gc_query_status(self._comp, stream)

    def invalidate_constants(self) -> None:
        gc_invalidate_constants(self._comp)

    # -- host execution ---------------------------------------------------------------------------
    def execute_host(self, in_arrays: List[np.ndarray], out_arrays: List[np.ndarray], stream: Optional[int] = None):
        """Host numpy / pinned buffers in, host buffers out (copies run inside the call)."""
        import torch
        if self._staging is None:
            n = gc_host_staging_bytes(self._comp)
            self._staging = torch.empty(max(n, 256), dtype=torch.uint8, device=f"cuda:{self.device}")
            gc_set_host_staging(self._comp, self._staging.data_ptr(), self._staging.numel())
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        gc_execute_host(self._comp, stream, [_host_ptr(a) for a in in_arrays], [_host_ptr(a) for a in out_arrays])

    HOST_SLOTS = 3

    def execute_host_async(self, slot: int, in_arrays: List[np.ndarray], out_arrays: List[np.ndarray],
                           stream: Optional[int] = None):
        """Enqueue copies in, execute and copies out for staging slot 0 .. HOST_SLOTS - 1 and return; host_wait(slot)
        completes it.  Several slots in flight overlap the copies of one batch with the execution and the copies of
        its neighbours."""
        import torch
        n = gc_host_staging_bytes(self._comp)
        if self._staging is None or self._staging.numel() < self.HOST_SLOTS * n:
            for s in range(self.HOST_SLOTS):
                self.host_wait(s)
            self._staging = torch.empty(max(self.HOST_SLOTS * n, 256), dtype=torch.uint8, device=f"cuda:{self.device}")
            gc_set_host_staging(self._comp, self._staging.data_ptr(), self._staging.numel())
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        gc_execute_host_async(self._comp, stream, slot, [_host_ptr(a) for a in in_arrays],
                              [_host_ptr(a) for a in out_arrays])

    def host_wait(self, slot: int) -> None:
        gc_host_wait(self._comp, slot)

    def close(self) -> None:
        if getattr(self, "_comp", None):
            gc_compiled_destroy(self._comp)
            self._comp = None
        if getattr(self, "_part", None):
            gc_partition_destroy(self._part)
            self._part = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _host_ptr(a) -> int:
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()   # a pinned torch CPU tensor


def device_inputs(w, device: int = 0):
    """Upload a workload's host arrays (in graph-input order) as raw-byte torch tensors."""
    import torch
    outs = []
    for tid in w.graph.inputs:
        a = np.ascontiguousarray(w.feeds[tid])
        outs.append(torch.from_numpy(a.view(np.uint8).reshape(-1)).to(f"cuda:{device}"))
    return outs


def device_outputs(g: Graph, device: int = 0):
    import torch
    return [torch.empty(g.tensors[t].nbytes, dtype=torch.uint8, device=f"cuda:{device}") for t in g.outputs]


def output_to_numpy(g: Graph, tid: int, t) -> np.ndarray:
    lt = g.tensors[tid]
    return t.cpu().numpy().view(NP_DTYPE[lt.dtype]).reshape(lt.dims)
