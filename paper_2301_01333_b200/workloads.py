"""Seeded synthetic workloads: the partition (op list) and the host input arrays for each config.

This module serves both the CUDA path (through the binding) and the CPU oracle (through the
tests and the bench), so it contains no arithmetic of the method itself: it only builds graph
descriptions and draws random inputs.  Shapes follow the paper's Table I (MLP-1 = 13x512x256x128,
MLP-2 = 479x1024x1024x512x256x1, MHA with sequence 128/384 and head size 64); the inputs are
synthetic stand-ins with the stated distributions, never items of a dataset.

Recipe (fixed): one ``numpy.random.default_rng(seed)`` stream per workload; tensors are drawn in
the order activations (X or Q, K, V) -> weights layer by layer -> biases layer by layer -> valid
lengths.  bf16 tensors are drawn in fp32 and rounded to nearest-even; the bf16 values (carried as
uint16 bit patterns) are the inputs.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, Sequence

import numpy as np

from .graph import Graph


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = ((u >> 16) & 1) + 0x7FFF
    return ((u + r) >> 16).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


@dataclass
class Workload:
    name: str
    graph: Graph
    feeds: Dict[int, np.ndarray]            # tensor id -> host array (bf16 as uint16 bits)
    ops: int = 0                            # algorithmic multiply-add ops x2 of all matmuls
    bytes: int = 0                          # graph inputs + outputs, each counted once
    info: dict = field(default_factory=dict)

    def finish(self) -> "Workload":
        g = self.graph
        self.bytes = sum(g.tensors[t].nbytes for t in list(g.inputs) + list(g.outputs))
        ops = 0
        for op in g.ops:
            if op.kind == "matmul":
                a = g.tensors[op.inputs[0]].dims
                o = g.tensors[op.output].dims
                n_out = 1
                for d in o:
                    n_out *= d
                ops += 2 * n_out * a[-1]
        self.ops = ops
        return self


# ------------------------------------------------------------------------------------------------
# MLP chains
# ------------------------------------------------------------------------------------------------
def mlp_f32(batch: int = 32, dims: Sequence[int] = (13, 512, 256, 128), seed: int = 0) -> Workload:
    """fp32 MLP: every layer is matmul + bias + ReLU (config 1 at the defaults)."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"mlp_f32_b{batch}_" + "x".join(map(str, dims)))
    feeds = {}
    x = g.input("f32", (batch, dims[0]), name="x")
    feeds[x] = rng.uniform(-1.0, 1.0, size=(batch, dims[0])).astype(np.float32)
    ws, bs = [], []
    for l in range(len(dims) - 1):
        k, n = dims[l], dims[l + 1]
        w = g.input("f32", (k, n), is_constant=True, name=f"w{l}")
        feeds[w] = (rng.standard_normal((k, n)) * np.sqrt(1.0 / k)).astype(np.float32)
        ws.append(w)
    for l in range(len(dims) - 1):
        n = dims[l + 1]
        b = g.input("f32", (n,), is_constant=True, name=f"b{l}")
        feeds[b] = rng.uniform(-0.1, 0.1, size=(n,)).astype(np.float32)
        bs.append(b)
    h = x
    for l in range(len(dims) - 1):
        n = dims[l + 1]
        z = g.op("matmul", (h, ws[l]), g.tensor("f32", (batch, n)))
        z = g.op("add", (z, bs[l]), g.tensor("f32", (batch, n)))
        h = g.op("relu", (z,), g.tensor("f32", (batch, n)))
    g.mark_output(h)
    return Workload(g.name, g, feeds).finish()


def mlp_int8(batch: int = 128, dims: Sequence[int] = (479, 1024, 1024, 512, 256, 1), seed: int = 0,
             s_x: float = 0.02, s_w: float = 0.005, s_act: float = 0.05,
             final: str = "sigmoid", per_channel: bool = False, x_zp: int = 0, act_zp: int = 0) -> Workload:
    """int8 MLP (config 2 at the defaults): u8 activations, s8 weights, s32 accumulation;
    hidden layers dequantize + bias + ReLU + requantize to u8; the last layer dequantizes,
    adds its bias and applies ``final`` ("sigmoid", or "none" to expose the fp32 logits).
    ``per_channel`` gives every weight one scale per output column (drawn in [0.5, 1.5] x s_w), ``x_zp`` /
    ``act_zp`` are the zero points of the input and of the requantised hidden activations: together the
    evaluation's scheme of asymmetric u8 activations and per-channel symmetric s8 weights."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"mlp_int8_b{batch}_" + "x".join(map(str, dims)) + ("_pc" if per_channel else "") +
              (f"_zp{x_zp}_{act_zp}" if (x_zp or act_zp) else ""))
    feeds = {}
    x = g.input("u8", (batch, dims[0]), scale=s_x, zero_point=x_zp, name="x")
    feeds[x] = rng.integers(0, 256, size=(batch, dims[0]), dtype=np.int64).astype(np.uint8)
    nl = len(dims) - 1
    ws, bs = [], []
    for l in range(nl):
        k, n = dims[l], dims[l + 1]
        if per_channel:
            cs = (s_w * np.random.default_rng(seed + 1000 + l).uniform(0.5, 1.5, size=n)).astype(np.float32)
            w = g.input("s8", (k, n), scale=s_w, is_constant=True, name=f"w{l}", channel_scales=cs, channel_axis=1)
        else:
            w = g.input("s8", (k, n), scale=s_w, is_constant=True, name=f"w{l}")
        feeds[w] = rng.integers(-127, 128, size=(k, n), dtype=np.int64).astype(np.int8)
        ws.append(w)
    for l in range(nl):
        n = dims[l + 1]
        b = g.input("f32", (n,), is_constant=True, name=f"b{l}")
        feeds[b] = rng.uniform(-0.1, 0.1, size=(n,)).astype(np.float32)
        bs.append(b)
    h = x
    for l in range(nl):
        n = dims[l + 1]
        acc = g.op("matmul", (h, ws[l]), g.tensor("s32", (batch, n)))
        z = g.op("dequantize", (acc,), g.tensor("f32", (batch, n)))
        z = g.op("add", (z, bs[l]), g.tensor("f32", (batch, n)))
        if l < nl - 1:
            z = g.op("relu", (z,), g.tensor("f32", (batch, n)))
            h = g.op("quantize", (z,), g.tensor("u8", (batch, n), scale=s_act, zero_point=act_zp))
        else:
            h = z if final == "none" else g.op(final, (z,), g.tensor("f32", (batch, n)))
    g.mark_output(h)
    return Workload(g.name, g, feeds).finish()


def ffn_bf16(tokens: int = 8192, d_model: int = 1024, d_ff: int = 4096, seed: int = 0) -> Workload:
    """bf16 transformer FFN (config 5 at the defaults): matmul + bias + GELU(tanh), bf16 hidden
    tensor, matmul + bias, bf16 output."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"ffn_bf16_t{tokens}_{d_model}x{d_ff}x{d_model}")
    feeds = {}
    x = g.input("bf16", (tokens, d_model), name="x")
    feeds[x] = f32_to_bf16_bits(rng.standard_normal((tokens, d_model), dtype=np.float32))
    w1 = g.input("bf16", (d_model, d_ff), is_constant=True, name="w1")
    feeds[w1] = f32_to_bf16_bits(rng.standard_normal((d_model, d_ff), dtype=np.float32) * np.float32(0.02))
    w2 = g.input("bf16", (d_ff, d_model), is_constant=True, name="w2")
    feeds[w2] = f32_to_bf16_bits(rng.standard_normal((d_ff, d_model), dtype=np.float32) * np.float32(0.02))
    b1 = g.input("f32", (d_ff,), is_constant=True, name="b1")
    feeds[b1] = rng.uniform(-0.1, 0.1, size=(d_ff,)).astype(np.float32)
    b2 = g.input("f32", (d_model,), is_constant=True, name="b2")
    feeds[b2] = rng.uniform(-0.1, 0.1, size=(d_model,)).astype(np.float32)
    z = g.op("matmul", (x, w1), g.tensor("f32", (tokens, d_ff)))
    z = g.op("add", (z, b1), g.tensor("f32", (tokens, d_ff)))
    z = g.op("gelu_tanh", (z,), g.tensor("f32", (tokens, d_ff)))
    h = g.op("typecast", (z,), g.tensor("bf16", (tokens, d_ff)))
    z = g.op("matmul", (h, w2), g.tensor("f32", (tokens, d_model)))
    z = g.op("add", (z, b2), g.tensor("f32", (tokens, d_model)))
    y = g.op("typecast", (z,), g.tensor("bf16", (tokens, d_model)))
    g.mark_output(y)
    return Workload(g.name, g, feeds).finish()


def plain_gemm_bf16(m: int = 8192, k: int = 8192, n: int = 8192, seed: int = 0) -> Workload:
    """One bf16 matmul with a bf16 result and nothing fused: the shape library GEMM peaks are quoted on."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"gemm_bf16_{m}x{k}x{n}")
    feeds = {}
    x = g.input("bf16", (m, k), name="x")
    feeds[x] = f32_to_bf16_bits(rng.standard_normal((m, k), dtype=np.float32))
    w = g.input("bf16", (k, n), is_constant=True, name="w")
    feeds[w] = f32_to_bf16_bits(rng.standard_normal((k, n), dtype=np.float32) * np.float32(0.02))
    z = g.op("matmul", (x, w), g.tensor("f32", (m, n)))
    y = g.op("typecast", (z,), g.tensor("bf16", (m, n)))
    g.mark_output(y)
    return Workload(g.name, g, feeds).finish()


# ------------------------------------------------------------------------------------------------
# Scaled-dot-product attention blocks
# ------------------------------------------------------------------------------------------------
def _mask_from_valid(valid: np.ndarray, seq: int) -> np.ndarray:
    j = np.arange(seq)[None, :]
    m = np.where(j < valid[:, None], np.float32(0.0), np.float32(-10000.0)).astype(np.float32)
    return m.reshape(valid.shape[0], 1, 1, seq)


def mha_bf16(batch: int = 32, heads: int = 12, seq: int = 128, head_dim: int = 64, seed: int = 0,
             valid_lo: int | None = None, valid_hi: int | None = None) -> Workload:
    """bf16 attention block (config 3 at the defaults): Q.K^T, x 1/sqrt(d), + additive mask,
    softmax, cast to bf16, .V, bf16 output.  Layout [B, H, S, D]."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"mha_bf16_b{batch}_h{heads}_s{seq}_d{head_dim}")
    feeds = {}
    shp = (batch, heads, seq, head_dim)
    q = g.input("bf16", shp, name="q")
    k = g.input("bf16", shp, name="k")
    v = g.input("bf16", shp, name="v")
    for t in (q, k, v):
        feeds[t] = f32_to_bf16_bits(rng.standard_normal(shp, dtype=np.float32))
    mask = g.input("f32", (batch, 1, 1, seq), name="mask")
    lo = seq // 2 if valid_lo is None else valid_lo
    hi = seq if valid_hi is None else valid_hi
    valid = rng.integers(lo, hi + 1, size=(batch,))
    feeds[mask] = _mask_from_valid(valid, seq)
    sshape = (batch, heads, seq, seq)
    s = g.op("matmul", (q, k), g.tensor("f32", sshape), transpose_b=True)
    s = g.op("mul", (s,), g.tensor("f32", sshape), scalar=float(1.0 / np.sqrt(head_dim)))
    s = g.op("add", (s, mask), g.tensor("f32", sshape))
    p = g.op("softmax", (s,), g.tensor("f32", sshape), axis=-1)
    p = g.op("typecast", (p,), g.tensor("bf16", sshape))
    o = g.op("matmul", (p, v), g.tensor("f32", shp))
    o = g.op("typecast", (o,), g.tensor("bf16", shp))
    g.mark_output(o)
    w = Workload(g.name, g, feeds, info={"valid": valid}).finish()
    return w


def mha_int8(batch: int = 64, heads: int = 16, seq: int = 384, head_dim: int = 64, seed: int = 0,
             s_qkv: float = 0.03, zp_qkv: int = 128, s_out: float = 0.02, zp_out: int = 128,
             valid_lo: int | None = None, valid_hi: int | None = None,
             all_value: int | None = None, with_mask: bool = True) -> Workload:
    """int8 attention block (config 4 at the defaults): u8 Q, K, V (zero point 128), exact s32
    Q.K^T, dequantize, x 1/sqrt(d), + mask, softmax, probabilities quantised to u8 (scale
    1/255), exact s32 P.V, dequantize, requantize to u8."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"mha_int8_b{batch}_h{heads}_s{seq}_d{head_dim}")
    feeds = {}
    shp = (batch, heads, seq, head_dim)
    q = g.input("u8", shp, scale=s_qkv, zero_point=zp_qkv, name="q")
    k = g.input("u8", shp, scale=s_qkv, zero_point=zp_qkv, name="k")
    v = g.input("u8", shp, scale=s_qkv, zero_point=zp_qkv, name="v")
    for t in (q, k, v):
        if all_value is None:
            feeds[t] = rng.integers(0, 256, size=shp, dtype=np.int64).astype(np.uint8)
        else:
            feeds[t] = np.full(shp, all_value, dtype=np.uint8)
    lo = seq // 2 if valid_lo is None else valid_lo
    hi = seq if valid_hi is None else valid_hi
    valid = rng.integers(lo, hi + 1, size=(batch,))
    if with_mask:
        mask = g.input("f32", (batch, 1, 1, seq), name="mask")
        feeds[mask] = _mask_from_valid(valid, seq)
    sshape = (batch, heads, seq, seq)
    s_p = float(np.float32(1.0 / 255.0))
    a = g.op("matmul", (q, k), g.tensor("s32", sshape), transpose_b=True)
    s = g.op("dequantize", (a,), g.tensor("f32", sshape))
    s = g.op("mul", (s,), g.tensor("f32", sshape), scalar=float(1.0 / np.sqrt(head_dim)))
    if with_mask:
        s = g.op("add", (s, mask), g.tensor("f32", sshape))
    p = g.op("softmax", (s,), g.tensor("f32", sshape), axis=-1)
    pq = g.op("quantize", (p,), g.tensor("u8", sshape, scale=s_p, zero_point=0))
    a2 = g.op("matmul", (pq, v), g.tensor("s32", shp))
    o = g.op("dequantize", (a2,), g.tensor("f32", shp))
    o = g.op("quantize", (o,), g.tensor("u8", shp, scale=s_out, zero_point=zp_out))
    g.mark_output(o)
    return Workload(g.name, g, feeds, info={"valid": valid, "p_quant": pq}).finish()


def single_matmul(a_dtype: str, b_dtype: str, m: int, k: int, n: int, seed: int = 0,
                  transpose_b: bool = False, a_zp: int = 0, batch: Sequence[int] = ()) -> Workload:
    """A MatMul-only partition whose output is the raw accumulator (s32 for 8-bit operands,
    fp32 otherwise).  Used to show that accumulators are exact."""
    rng = np.random.default_rng(seed)
    g = Graph(name=f"matmul_{a_dtype}_{b_dtype}_{m}x{k}x{n}")
    feeds = {}
    bt = tuple(batch)
    ashape = bt + (m, k)
    bshape = bt + ((n, k) if transpose_b else (k, n))

    def draw(dtype, shape):
        if dtype == "u8":
            return rng.integers(0, 256, size=shape, dtype=np.int64).astype(np.uint8)
        if dtype == "s8":
            return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)
        x = rng.standard_normal(shape, dtype=np.float32)
        return f32_to_bf16_bits(x) if dtype == "bf16" else x

    a = g.input(a_dtype, ashape, scale=0.02, zero_point=a_zp, name="a")
    feeds[a] = draw(a_dtype, ashape)
    b = g.input(b_dtype, bshape, scale=0.005, is_constant=not bt, name="b")
    feeds[b] = draw(b_dtype, bshape)
    out_dtype = "s32" if a_dtype in ("u8", "s8") else "f32"
    o = g.op("matmul", (a, b), g.tensor(out_dtype, bt + (m, n)), transpose_b=transpose_b)
    g.mark_output(o)
    return Workload(g.name, g, feeds).finish()


CONFIGS = {
    "c1": lambda: mlp_f32(),
    "c2": lambda: mlp_int8(),
    "c3": lambda: mha_bf16(),
    "c4": lambda: mha_int8(),
    "c5": lambda: ffn_bf16(),
}

# The independent units a config shards over when several GPUs split ONE batch (rows of an MLP chain, sequences of
# an attention block; Section V's outer parallel loop over the batch and Section VII's independent (batch, head)
# units): builder keyword that sets the unit count, and the full count.
CONFIG_UNITS = {
    "c1": (mlp_f32, "batch", 32),
    "c2": (mlp_int8, "batch", 128),
    "c3": (mha_bf16, "batch", 32),
    "c4": (mha_int8, "batch", 64),
    "c5": (ffn_bf16, "tokens", 8192),
}


def shard_config(name: str, full: Workload, first: int, count: int) -> Workload:
    """Units [first, first + count) of config `name`: a workload of `count` units whose per-unit inputs are that
    slice of the full workload's inputs (leading axis) and whose constants are the full workload's."""
    make, key, total = CONFIG_UNITS[name]
    shard = make(**{key: count})
    for a, b in zip(shard.graph.inputs, full.graph.inputs):
        src = full.feeds[b]
        if not full.graph.tensors[b].is_constant and src.shape[0] == total:
            shard.feeds[a] = np.ascontiguousarray(src[first:first + count])
        else:
            shard.feeds[a] = src
    shard.info = dict(shard.info, first=first, count=count, of=total)
    return shard
