"""CPU oracle: an unfused, op-by-op interpreter of a partition.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; it
shares no code with the CUDA path and never calls it.

What it computes is the plain definition of the graph the paper's compiler starts from: every op
reads whole tensors and materialises a whole tensor, in topological (list) order, with no fusion,
blocking or reordering.  All of the paper's optimisations (low-precision conversion, fine- and
coarse-grain fusion, Section V) are stated there to preserve this result, so this is what a
fused kernel must reproduce.

Arithmetic domains
  * 8-bit x 8-bit MatMul: exact integers.  Operands have their zero point subtracted first
    (asymmetric activations: Section V's dequantisation removes the zero point a_z); the sum is taken in
    int64 and checked to fit s32, which is the accumulator type of an int8 matmul.
  * Dequantize / Add / Mul / ReLU / Quantize applied to values that are exactly representable in
    fp32 (integer accumulators, fp32 graph inputs): IEEE fp32, one rounding per op, no fused
    multiply-add.  This is the "fp32 multiply, round-half-to-even, saturate" requantisation;
    both sides can reproduce it bit for bit.  Such values are tagged ``f32x``.
  * Float MatMul, SoftMax, GELU, Sigmoid: fp64 from exactly promoted inputs; their results are
    tagged ``wide`` and everything downstream of a wide value stays in fp64.  TypeCast is the
    identity on a wide value unless ``faithful=True`` (diagnostic mode: every tensor is rounded to
    its declared dtype).

Constants derived from logical-tensor attributes are formed in fp32 exactly like this:
    dq  = float32(scale_a) * float32(scale_b)         (scale of an s32 MatMul result; with per-channel
                                                       weight scales one such product per output column)
    inv = float32(1) / float32(scale_out)              (Quantize multiplies by the reciprocal)

Parity pins: tests/test_oracle_pins.py (brute force with Python integers, closed forms, rounding
boundary vectors, softmax invariants, independent straight-line restatements of each workload).
The paper prints no worked numeric example, so beyond those pins parity is unpinned by the paper.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional

import numpy as np

_INT_RANGE = {"u8": (0, 255), "s8": (-128, 127), "s32": (-(2 ** 31), 2 ** 31 - 1)}


@dataclass
class Value:
    data: np.ndarray          # int64 | float32 | float64
    kind: str                 # "int" | "f32x" | "wide"
    qscale: Optional[np.float32] = None   # for "int": scale that Dequantize applies; a per-channel weight
                                          # carries a float32 vector and `qaxis`, a MatMul result of one a
                                          # vector over its last axis
    zero_point: int = 0                   # for "int": offset that MatMul / Dequantize subtract
    qaxis: int = -1                       # axis a vector-valued qscale runs along


def _bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Nearest-even rounding of fp32/fp64 values to bf16, returned as fp32."""
    f = np.asarray(x, dtype=np.float64).astype(np.float32)
    # fp64 -> fp32 -> bf16 double rounding is avoided by rounding the fp64 value directly:
    # a bf16 neighbour pair is found in fp32 and the nearer one (ties to even) is chosen in fp64.
    u = f.view(np.uint32)
    lo = (u & np.uint32(0xFFFF0000)).view(np.float32).astype(np.float64)
    hi = ((u & np.uint32(0xFFFF0000)) + np.uint32(0x10000)).view(np.float32).astype(np.float64)
    xd = np.asarray(x, dtype=np.float64)
    # lo and hi bracket f (towards larger magnitude); pick by distance in fp64
    dlo, dhi = np.abs(xd - lo), np.abs(hi - xd)
    lo_even = ((u >> 16) & 1) == 0
    pick_hi = (dhi < dlo) | ((dhi == dlo) & ~lo_even)
    out = np.where(pick_hi, hi, lo)
    return out.astype(np.float32)


def load_input(lt, arr) -> Value:
    """Wrap a host array as an oracle value according to its logical tensor."""
    if lt.dtype in ("u8", "s8", "s32"):
        data = np.asarray(arr).astype(np.int64).reshape(lt.dims)
        if getattr(lt, "channel_scales", None) is not None:
            # per-channel weight scales (Section VII, the int8 scheme of the evaluation)
            return Value(data, "int", np.asarray(lt.channel_scales, dtype=np.float32), int(lt.zero_point),
                         int(lt.channel_axis) % len(lt.dims))
        return Value(data, "int", np.float32(lt.scale), int(lt.zero_point))
    if lt.dtype == "bf16":
        return Value(_bf16_bits_to_f32(arr).reshape(lt.dims), "f32x")
    if lt.dtype == "f32":
        return Value(np.asarray(arr, dtype=np.float32).reshape(lt.dims), "f32x")
    raise ValueError(lt.dtype)


def _as_f64(v: Value) -> np.ndarray:
    if v.kind == "int":
        raise TypeError("integer tensor used where a float tensor is required (missing Dequantize)")
    return v.data.astype(np.float64)


# ------------------------------------------------------------------------------------------------
# op definitions
# ------------------------------------------------------------------------------------------------
def op_matmul(a: Value, b: Value, transpose_b: bool) -> Value:
    """C[..., m, n] = sum_k A[..., m, k] * B[..., k, n]   (Section III: A[M,K] x B[K,N] -> C[M,N])."""
    if a.kind == "int" and b.kind == "int":
        A = a.data - a.zero_point
        B = b.data - b.zero_point
        if transpose_b:
            B = np.swapaxes(B, -1, -2)
        C = np.matmul(A, B)                       # int64, exact
        if C.size and (C.max() > 2 ** 31 - 1 or C.min() < -(2 ** 31)):
            raise OverflowError("int8 matmul result does not fit the s32 accumulator")
        if np.ndim(a.qscale) != 0:
            raise TypeError("per-channel scales are defined for the weight operand only")
        if np.ndim(b.qscale) != 0:
            # the scales must run along the weight's output-channel axis (n): the last axis of [.., k, n],
            # the one before it when the weight is stored transposed
            n_axis = b.data.ndim - (2 if transpose_b else 1)
            if b.qaxis != n_axis:
                raise TypeError("per-channel scales must follow the output-channel axis of the weight")
            return Value(C, "int", np.float32(a.qscale) * b.qscale.astype(np.float32), 0, C.ndim - 1)
        return Value(C, "int", np.float32(a.qscale) * np.float32(b.qscale), 0)
    if a.kind == "int" or b.kind == "int":
        raise TypeError("mixed integer/float MatMul")
    A, B = _as_f64(a), _as_f64(b)
    if transpose_b:
        B = np.swapaxes(B, -1, -2)
    return Value(np.matmul(A, B), "wide")


def op_dequantize(x: Value) -> Value:
    """y = (q - zero_point) * scale in fp32 (Section V, the DQ op)."""
    if x.kind != "int":
        raise TypeError("Dequantize needs an integer tensor")
    t = (x.data - x.zero_point).astype(np.float32)      # round-to-nearest-even for |.| > 2^24
    if np.ndim(x.qscale) != 0:                          # one scale per index of axis `qaxis`
        shape = [1] * t.ndim
        shape[x.qaxis] = -1
        return Value((t * x.qscale.astype(np.float32).reshape(shape)).astype(np.float32), "f32x")
    return Value(t * np.float32(x.qscale), "f32x")


def op_quantize(x: Value, out_lt) -> Value:
    """q = saturate(rne(x * inv) + zero_point), inv = 1.0f / scale (Section V, the Q op; rounding
    and saturation rule: fp32 multiply, round half to even, saturate)."""
    lo, hi = _INT_RANGE[out_lt.dtype]
    inv = np.float32(1.0) / np.float32(out_lt.scale)
    if x.kind == "f32x":
        r = np.rint(x.data * inv)
    elif x.kind == "wide":
        r = np.rint(x.data * np.float64(inv))
    else:
        raise TypeError("Quantize needs a float tensor")
    r = np.clip(r.astype(np.float64), -2.0 ** 31, 2.0 ** 31 - 1).astype(np.int64)
    q = np.clip(r + int(out_lt.zero_point), lo, hi)
    return Value(q, "int", np.float32(out_lt.scale), int(out_lt.zero_point))


def _binary(a: Value, b: Value, fn) -> Value:
    if a.kind == "int" or b.kind == "int":
        raise TypeError("elementwise op on an integer tensor (missing Dequantize)")
    if a.kind == "f32x" and b.kind == "f32x":
        return Value(fn(a.data, b.data).astype(np.float32), "f32x")
    return Value(fn(_as_f64(a), _as_f64(b)), "wide")


def op_add(a: Value, b: Value) -> Value:
    """Broadcast add (bias, additive attention mask)."""
    return _binary(a, b, np.add)


def op_mul_scalar(x: Value, scalar: float) -> Value:
    c = np.float32(scalar)
    if x.kind == "f32x":
        return Value(x.data * c, "f32x")
    return Value(_as_f64(x) * np.float64(c), "wide")


def op_relu(x: Value) -> Value:
    """max(x, 0)  (the ReLU post-op of Fig. 6)."""
    if x.kind == "int":
        raise TypeError("ReLU on an integer tensor")
    return Value(np.maximum(x.data, x.data.dtype.type(0)), x.kind)


def op_gelu_tanh(x: Value) -> Value:
    z = _as_f64(x)
    return Value(0.5 * z * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (z + 0.044715 * z ** 3))), "wide")


def op_sigmoid(x: Value) -> Value:
    z = _as_f64(x)
    return Value(1.0 / (1.0 + np.exp(-z)), "wide")


def op_softmax(x: Value, axis: int) -> Value:
    """p_j = exp(x_j - max x) / sum_j exp(x_j - max x) over the last axis."""
    z = _as_f64(x)
    if axis not in (-1, z.ndim - 1):
        raise ValueError("softmax over the last axis only")
    m = z.max(axis=-1, keepdims=True)
    e = np.exp(z - m)
    return Value(e / e.sum(axis=-1, keepdims=True), "wide")


def op_typecast(x: Value, out_lt, faithful: bool) -> Value:
    if x.kind == "int":
        raise TypeError("TypeCast on an integer tensor")
    if not faithful:
        return x
    if out_lt.dtype == "bf16":
        return Value(_round_to_bf16(x.data), "f32x")
    return Value(x.data.astype(np.float32), "f32x")


# ------------------------------------------------------------------------------------------------
# interpreter
# ------------------------------------------------------------------------------------------------
def run(graph, feeds: Dict[int, np.ndarray], faithful: bool = False,
        keep_all: bool = False) -> Dict[int, np.ndarray]:
    """Interpret ``graph`` (objects with .tensors/.ops/.inputs/.outputs as in the workload builders)
    on host arrays ``feeds`` (tensor id -> array).  Returns tensor id -> array for the graph outputs
    (all tensors if ``keep_all``): int64 for integer tensors, float32 for pinned-fp32 values,
    float64 otherwise."""
    env: Dict[int, Value] = {}
    for tid in graph.inputs:
        env[tid] = load_input(graph.tensors[tid], feeds[tid])
    for op in graph.ops:
        ins = [env[i] for i in op.inputs]
        olt = graph.tensors[op.output]
        k = op.kind
        if k == "matmul":
            out = op_matmul(ins[0], ins[1], op.transpose_b)
        elif k == "dequantize":
            out = op_dequantize(ins[0])
        elif k == "quantize":
            out = op_quantize(ins[0], olt)
        elif k == "add":
            out = op_add(ins[0], ins[1])
        elif k == "mul":
            out = op_mul_scalar(ins[0], op.scalar)
        elif k == "relu":
            out = op_relu(ins[0])
        elif k == "gelu_tanh":
            out = op_gelu_tanh(ins[0])
        elif k == "sigmoid":
            out = op_sigmoid(ins[0])
        elif k == "softmax":
            out = op_softmax(ins[0], op.axis)
        elif k == "typecast":
            out = op_typecast(ins[0], olt, faithful)
        else:
            raise ValueError(f"unknown op kind {k}")
        if tuple(out.data.shape) != tuple(olt.dims):
            raise ValueError(f"op {k}: result shape {out.data.shape} != declared {olt.dims}")
        if faithful and out.kind == "wide":
            out = (Value(_round_to_bf16(out.data), "f32x") if olt.dtype == "bf16"
                   else Value(out.data.astype(np.float32), "f32x"))
        env[op.output] = out
    ids = list(env.keys()) if keep_all else list(graph.outputs)
    return {tid: env[tid].data for tid in ids}
