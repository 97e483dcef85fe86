"""Plain-data description of a partition: logical tensors, ops, graph inputs and outputs.

This mirrors the paper's Graph IR vocabulary (Section II: a graph is a set of ops and logical
tensors; a logical tensor carries dtype, shape and layout metadata; an op has a kind, attributes
and input/output logical tensors).  It holds no arithmetic: it is the neutral form that the
seeded workload builders emit, that the ctypes binding marshals into the C structs of
``include/gc.h`` and that the CPU oracle interprets on its own.

Layouts are always plain row-major and dense (the paper keeps graph inputs and outputs in plain
layout, Section V "layout propagation" and Section VII).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

DTYPES = ("f32", "bf16", "u8", "s8", "s32")
DTYPE_BYTES = {"f32": 4, "bf16": 2, "u8": 1, "s8": 1, "s32": 4}

OP_KINDS = (
    "matmul",      # Tunable op (Section III)
    "add",         # broadcast add: bias, additive mask
    "mul",         # multiply by a scalar attribute
    "relu",
    "gelu_tanh",
    "sigmoid",
    "softmax",     # over the last axis
    "quantize",    # f32 -> u8/s8 using the OUTPUT tensor's scale / zero point
    "dequantize",  # u8/s8/s32 -> f32 using the INPUT tensor's scale / zero point
    "typecast",    # f32 <-> bf16
)


@dataclass
class LogicalTensor:
    id: int
    dtype: str
    dims: Tuple[int, ...]
    scale: float = 1.0       # per-tensor quantisation scale (ignored for float dtypes)
    zero_point: int = 0
    is_constant: bool = False  # same pointer and contents on every execution (weights, biases)
    name: str = ""
    # per-channel quantisation of a constant s8 weight (the symmetric per-output-channel weight scheme of
    # Section VII's int8 evaluation): one scale per index of `channel_axis`, which must be the output-channel axis of the
    # MatMul that consumes the tensor.  None = the per-tensor `scale` applies.
    channel_scales: Optional[Tuple[float, ...]] = None
    channel_axis: int = -1

    @property
    def numel(self) -> int:
        n = 1
        for d in self.dims:
            n *= d
        return n

    @property
    def nbytes(self) -> int:
        return self.numel * DTYPE_BYTES[self.dtype]


@dataclass
class Op:
    kind: str
    inputs: Tuple[int, ...]
    output: int
    transpose_b: bool = False       # matmul: second operand is stored [.., n, k]
    scalar: Optional[float] = None  # mul
    axis: int = -1                  # softmax


@dataclass
class Graph:
    tensors: Dict[int, LogicalTensor] = field(default_factory=dict)
    ops: List[Op] = field(default_factory=list)
    inputs: List[int] = field(default_factory=list)
    outputs: List[int] = field(default_factory=list)
    name: str = ""

    # -- small builder helpers (bookkeeping only) ---------------------------------------------
    def tensor(self, dtype: str, dims: Sequence[int], *, scale: float = 1.0, zero_point: int = 0,
               is_constant: bool = False, name: str = "", channel_scales: Optional[Sequence[float]] = None,
               channel_axis: int = -1) -> int:
        assert dtype in DTYPES, dtype
        tid = len(self.tensors)
        dims = tuple(int(d) for d in dims)
        cs = None
        if channel_scales is not None:
            channel_axis = channel_axis % len(dims)
            cs = tuple(float(s) for s in channel_scales)
            assert len(cs) == dims[channel_axis], "one scale per channel"
        self.tensors[tid] = LogicalTensor(tid, dtype, dims, float(scale), int(zero_point), bool(is_constant), name,
                                          cs, int(channel_axis))
        return tid

    def input(self, *a, **k) -> int:
        tid = self.tensor(*a, **k)
        self.inputs.append(tid)
        return tid

    def op(self, kind: str, inputs: Sequence[int], out: int, **attrs) -> int:
        assert kind in OP_KINDS, kind
        self.ops.append(Op(kind, tuple(inputs), out, **attrs))
        return out

    def mark_output(self, tid: int) -> int:
        self.outputs.append(tid)
        return tid
