"""Pins for the CPU oracle: it is checked against things other than itself - brute force with
Python integers and math.fsum, closed forms, hand-derived rounding vectors, softmax invariants and
independent straight-line restatements of each workload on reduced shapes."""
import math
import os

import numpy as np
import pytest

from oracle import interp
from paper_2301_01333_b200 import workloads as W
from paper_2301_01333_b200.graph import Graph

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run1(w, **kw):
    out = interp.run(w.graph, w.feeds, **kw)
    return out[w.graph.outputs[0]]


# ---------------------------------------------------------------------------- integer matmul
@pytest.mark.parametrize("m,k,n,tb,zp", [(3, 5, 4, False, 0), (1, 479, 1, False, 0), (4, 33, 6, True, 0),
                                         (2, 17, 3, False, 128)])
def test_int_matmul_brute_force(m, k, n, tb, zp):
    w = W.single_matmul("u8", "s8", m, k, n, seed=3, transpose_b=tb, a_zp=zp)
    got = run1(w)
    a = w.feeds[w.graph.inputs[0]].tolist()
    b = w.feeds[w.graph.inputs[1]].tolist()
    for i in range(m):
        for j in range(n):
            s = 0
            for kk in range(k):
                bv = b[j][kk] if tb else b[kk][j]
                s += (a[i][kk] - zp) * bv
            assert int(got[i, j]) == s


def test_int_matmul_extreme_value():
    # all-255 activations against all-(-127) weights over K=1024: -255*127*1024
    w = W.single_matmul("u8", "s8", 2, 1024, 3)
    w.feeds[w.graph.inputs[0]][:] = 255
    w.feeds[w.graph.inputs[1]][:] = -127
    got = run1(w)
    assert (got == -33162240).all()


def test_int_matmul_overflow_detected():
    g = Graph()
    a = g.input("s32", (1, 2))
    b = g.input("s32", (2, 1))
    g.mark_output(g.op("matmul", (a, b), g.tensor("s32", (1, 1))))
    feeds = {a: np.array([[2 ** 30, 2 ** 30]]), b: np.array([[2], [2]])}
    with pytest.raises(OverflowError):
        interp.run(g, feeds)


def test_int_matmul_identity_and_one_hot():
    k = 16
    w = W.single_matmul("u8", "s8", 5, k, k, a_zp=7)
    a = w.feeds[w.graph.inputs[0]]
    w.feeds[w.graph.inputs[1]] = np.eye(k, dtype=np.int8)
    assert (run1(w) == a.astype(np.int64) - 7).all()
    onehot = np.zeros((k, k), dtype=np.int8)
    onehot[3, :] = 1          # every output column selects activation 3
    w.feeds[w.graph.inputs[1]] = onehot
    assert (run1(w) == (a[:, 3:4].astype(np.int64) - 7)).all()


# ---------------------------------------------------------------------------- requantisation
def _quant_graph(scale, zp, n):
    g = Graph()
    x = g.input("f32", (n,))
    g.mark_output(g.op("quantize", (x,), g.tensor("u8", (n,), scale=scale, zero_point=zp)))
    return g, x


def test_requant_boundary_vectors_golden():
    """tests/golden/requant_boundaries.txt: value-before-rounding, zero point, expected u8; derived
    by hand from 'round half to even, add zero point, saturate to [0,255]'."""
    rows = []
    with open(os.path.join(GOLDEN, "requant_boundaries.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                u, zp, q = line.split()
                rows.append((float(u), int(zp), int(q)))
    assert len(rows) >= 12
    for zp in sorted({r[1] for r in rows}):
        sel = [r for r in rows if r[1] == zp]
        g, x = _quant_graph(1.0, zp, len(sel))
        got = interp.run(g, {x: np.array([r[0] for r in sel], dtype=np.float32)})[g.outputs[0]]
        assert got.tolist() == [r[2] for r in sel]


def test_requant_boundary_vectors_signed_golden():
    """tests/golden/requant_boundaries_s8.txt: the same rule with an s8 result - the range is [-128, 127],
    both bounds are reachable without saturation, and ties go to even on the negative side too."""
    rows = []
    with open(os.path.join(GOLDEN, "requant_boundaries_s8.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                u, zp, q = line.split()
                rows.append((float(u), int(zp), int(q)))
    assert len(rows) >= 16 and min(r[2] for r in rows) == -128 and max(r[2] for r in rows) == 127
    for zp in sorted({r[1] for r in rows}):
        sel = [r for r in rows if r[1] == zp]
        g = Graph()
        x = g.input("f32", (len(sel),))
        g.mark_output(g.op("quantize", (x,), g.tensor("s8", (len(sel),), scale=1.0, zero_point=zp)))
        got = interp.run(g, {x: np.array([r[0] for r in sel], dtype=np.float32)})[g.outputs[0]]
        assert got.tolist() == [r[2] for r in sel]


def test_bf16_rounding_ties_to_even_and_no_double_rounding_golden():
    """tests/golden/bf16_rounding.txt: exact ties between two bf16 neighbours (lower neighbour even, and odd), both
    signs, and fp64 values just above a tie, which a detour through fp32 would round the other way."""
    vals, bits = [], []
    with open(os.path.join(GOLDEN, "bf16_rounding.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                sign, exps, b = line.split()
                v = math.fsum(2.0 ** int(t) for t in exps.split(","))
                vals.append(-v if sign == "-" else v)
                bits.append(int(b, 16))
    assert len(vals) >= 10
    got = interp._round_to_bf16(np.array(vals, dtype=np.float64))
    assert got.dtype == np.float32
    assert (got.view(np.uint32) & 0xFFFF == 0).all()                    # bf16 values
    assert (got.view(np.uint32) >> 16).tolist() == bits
    # the faithful TypeCast goes through the same routine
    g = Graph()
    x = g.input("f32", (2,))
    g.mark_output(g.op("typecast", (x,), g.tensor("bf16", (2,))))
    out = interp.run(g, {x: np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)}, faithful=True)[g.outputs[0]]
    assert (out.view(np.uint32) >> 16).tolist() == [0x3F80, 0x3F82]


def test_requant_reciprocal_constants():
    # the reciprocal is formed in fp32; for the workloads' scales it is exactly these values
    assert np.float32(1.0) / np.float32(0.05) == np.float32(20.0)
    assert np.float32(1.0) / np.float32(0.02) == np.float32(50.0)
    inv_p = np.float32(1.0) / np.float32(1.0 / 255.0)
    assert inv_p != np.float32(255.0) and abs(float(inv_p) - 254.99998) < 1e-5
    # scale 0.05: x = 0.125 -> u = 2.5 -> 2 (tie to even); x = 0.175 -> 3.5 (fp32: 3.4999998) -> 3
    g, x = _quant_graph(0.05, 0, 3)
    got = interp.run(g, {x: np.array([0.125, 0.075, 1000.0], dtype=np.float32)})[g.outputs[0]]
    assert got.tolist() == [2, 2, 255]   # 0.075f*20 = 1.5000001 -> 2


def test_dequantize_large_accumulator_rounds_to_nearest_even():
    g = Graph()
    a = g.input("s32", (3,), scale=1.0)
    g.mark_output(g.op("dequantize", (a,), g.tensor("f32", (3,))))
    got = interp.run(g, {a: np.array([16777217, 16777219, -16777217])})[g.outputs[0]]
    assert got.dtype == np.float32
    assert got.tolist() == [16777216.0, 16777220.0, -16777216.0]


def test_dequantize_scale_is_fp32_product():
    # the scale of an int8 matmul result is float32(s_a) * float32(s_b), a single fp32 product
    w = W.single_matmul("u8", "s8", 1, 1, 1)
    w.feeds[w.graph.inputs[0]][:] = 200
    w.feeds[w.graph.inputs[1]][:] = 100
    g = w.graph
    g.outputs.clear()
    g.mark_output(g.op("dequantize", (g.ops[0].output,), g.tensor("f32", (1, 1))))
    got = run1(w)
    expect = np.float32(20000.0) * (np.float32(0.02) * np.float32(0.005))
    assert got.dtype == np.float32 and got[0, 0] == expect
    assert np.float32(0.02) * np.float32(0.005) == np.float32(1e-4)


# ---------------------------------------------------------------------------- float matmul
def test_float_matmul_brute_force_fsum():
    w = W.single_matmul("f32", "f32", 3, 7, 4, seed=5)
    got = run1(w)
    a = w.feeds[w.graph.inputs[0]].astype(np.float64).tolist()
    b = w.feeds[w.graph.inputs[1]].astype(np.float64).tolist()
    for i in range(3):
        for j in range(4):
            ref = math.fsum(a[i][k] * b[k][j] for k in range(7))
            assert abs(got[i, j] - ref) <= 1e-12 * max(1.0, abs(ref))


def test_float_matmul_bf16_inputs_identity_and_transpose():
    w = W.single_matmul("bf16", "bf16", 4, 8, 8, seed=2, transpose_b=True)
    a = W.bf16_bits_to_f32(w.feeds[w.graph.inputs[0]])
    w.feeds[w.graph.inputs[1]] = W.f32_to_bf16_bits(np.eye(8, dtype=np.float32))
    assert np.array_equal(run1(w), a.astype(np.float64))
    # a non-symmetric B distinguishes B from B^T: B[n,k] = 1 iff k == 0 -> C[m,n] = A[m,0]
    b = np.zeros((8, 8), dtype=np.float32)
    b[:, 0] = 1.0
    w.feeds[w.graph.inputs[1]] = W.f32_to_bf16_bits(b)
    assert np.array_equal(run1(w), np.repeat(a[:, :1].astype(np.float64), 8, axis=1))


# ---------------------------------------------------------------------------- activations
def _unary_graph(kind, xs):
    g = Graph()
    x = g.input("f32", (len(xs),))
    g.mark_output(g.op(kind, (x,), g.tensor("f32", (len(xs),))))
    return interp.run(g, {x: np.array(xs, dtype=np.float32)})[g.outputs[0]]


def test_relu_gelu_sigmoid_invariants():
    xs = [-8.0, -3.0, -1.0, -0.25, 0.0, 0.25, 1.0, 3.0, 8.0]
    r = _unary_graph("relu", xs)
    assert (r >= 0).all() and r.tolist() == [max(x, 0.0) for x in xs]
    ge = _unary_graph("gelu_tanh", xs)
    assert ge[4] == 0.0
    assert abs(ge[-1] - 8.0) < 1e-9                      # GELU(x) -> x for large x
    for i, x in enumerate(xs):                            # GELU(x) - GELU(-x) = x
        assert abs((ge[i] - ge[len(xs) - 1 - i]) - x) < 1e-12
        ref = 0.5 * x * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x * x * x)))
        assert abs(ge[i] - ref) < 1e-12
    s = _unary_graph("sigmoid", xs)
    assert s[4] == 0.5
    for i, x in enumerate(xs):
        assert abs(s[i] + s[len(xs) - 1 - i] - 1.0) < 1e-15
        assert abs(s[i] - 1.0 / (1.0 + math.exp(-x))) < 1e-15


def test_zero_weights_give_activation_of_bias():
    w = W.mlp_f32(batch=4, dims=(6, 5))
    g = w.graph
    w.feeds[g.inputs[1]][:] = 0.0
    bias = w.feeds[g.inputs[2]]
    out = run1(w)
    assert np.array_equal(out, np.broadcast_to(np.maximum(bias, 0).astype(np.float64), out.shape))


# ---------------------------------------------------------------------------- softmax / attention
def test_softmax_rows_sum_to_one_and_shift_invariant():
    g = Graph()
    x = g.input("f32", (5, 37))
    g.mark_output(g.op("softmax", (x,), g.tensor("f32", (5, 37))))
    rng = np.random.default_rng(1)
    a = (rng.standard_normal((5, 37)) * 10).astype(np.float32)
    p = interp.run(g, {x: a})[g.outputs[0]]
    assert np.abs(p.sum(-1) - 1.0).max() < 1e-12
    p2 = interp.run(g, {x: (a + np.float32(64.0)).astype(np.float32)})[g.outputs[0]]
    # adding 64 to fp32 inputs is not exact in general; use values where it is
    a3 = np.round(a * 8) / 8
    p3 = interp.run(g, {x: a3.astype(np.float32)})[g.outputs[0]]
    p4 = interp.run(g, {x: (a3 + 64.0).astype(np.float32)})[g.outputs[0]]
    assert np.abs(p3 - p4).max() < 1e-15
    assert p2.shape == p.shape
    # brute force on one row
    row = a[0].astype(np.float64).tolist()
    m = max(row)
    e = [math.exp(v - m) for v in row]
    s = math.fsum(e)
    assert max(abs(p[0, j] - e[j] / s) for j in range(37)) < 1e-15


def test_attention_q_zero_gives_mean_of_valid_values():
    w = W.mha_bf16(batch=2, heads=2, seq=16, head_dim=8, seed=4, valid_lo=5, valid_hi=11)
    g = w.graph
    q, k, v, mask = g.inputs
    w.feeds[q][:] = 0
    out = run1(w)
    vv = W.bf16_bits_to_f32(w.feeds[v]).astype(np.float64)
    for b in range(2):
        L = int(w.info["valid"][b])
        assert 5 <= L <= 11
        ref = vv[b, :, :L, :].mean(axis=1)                # [heads, d]
        assert np.abs(out[b] - ref[:, None, :]).max() < 1e-12


def test_attention_equal_value_rows_and_masked_weight_zero():
    w = W.mha_bf16(batch=2, heads=1, seq=12, head_dim=4, seed=6, valid_lo=3, valid_hi=9)
    g = w.graph
    q, k, v, mask = g.inputs
    vrow = np.array([0.5, -1.25, 2.0, 3.0], dtype=np.float32)
    w.feeds[v] = W.f32_to_bf16_bits(np.broadcast_to(vrow, (2, 1, 12, 4)).copy())
    out = run1(w)
    assert np.abs(out - vrow.astype(np.float64)).max() < 1e-12
    allv = interp.run(g, w.feeds, keep_all=True)
    p = allv[[op.output for op in g.ops if op.kind == "softmax"][0]]
    for b in range(2):
        L = int(w.info["valid"][b])
        assert (p[b, :, :, L:] == 0.0).all()              # exp(-10000 + delta) underflows to 0
        assert (p[b, :, :, :L] > 0.0).all()


def test_int8_attention_all_128_inputs_give_zero_point():
    w = W.mha_int8(batch=1, heads=2, seq=24, head_dim=8, all_value=128, valid_lo=10, valid_hi=20)
    out = run1(w)
    assert (out == 128).all()


def test_int8_attention_prob_row_sums():
    w = W.mha_int8(batch=2, heads=2, seq=48, head_dim=16, seed=9)
    allv = interp.run(w.graph, w.feeds, keep_all=True)
    p = allv[w.info["p_quant"]]
    rs = p.sum(-1)
    assert rs.min() >= 255 - 24 and rs.max() <= 255 + 24
    assert p.min() >= 0 and p.max() <= 255


# ---------------------------------------------------------------------------- whole graphs, restated
def test_mlp_int8_against_straight_line_restatement():
    w = W.mlp_int8(batch=3, dims=(7, 8, 4, 1), seed=11, final="none")
    got = run1(w)
    g = w.graph
    x = w.feeds[g.inputs[0]].tolist()
    ws = [w.feeds[g.inputs[1 + l]].tolist() for l in range(3)]
    bs = [w.feeds[g.inputs[4 + l]] for l in range(3)]
    f = np.float32
    dq = [f(0.02) * f(0.005), f(0.05) * f(0.005), f(0.05) * f(0.005)]
    inv = f(1.0) / f(0.05)
    for m in range(3):
        act = x[m]
        for l in range(3):
            K, N = len(ws[l]), len(ws[l][0])
            nxt = []
            for n in range(N):
                acc = sum(act[k] * ws[l][k][n] for k in range(K))
                t = f(acc)
                t = f(t * dq[l])
                t = f(t + bs[l][n])
                if l < 2:
                    t = t if t > 0 else f(0.0)
                    u = f(t * inv)
                    r = int(np.rint(u))
                    nxt.append(min(max(r, 0), 255))
                else:
                    nxt.append(t)
            act = nxt
        assert got.dtype == np.float32
        assert got[m, 0] == act[0]
    # sigmoid variant = fp64 sigmoid of the same logits
    ws_ = W.mlp_int8(batch=3, dims=(7, 8, 4, 1), seed=11)
    sg = run1(ws_)
    for m in range(3):
        assert abs(sg[m, 0] - 1.0 / (1.0 + math.exp(-float(got[m, 0])))) < 1e-15


def test_mlp_int8_per_channel_asymmetric_against_straight_line_restatement():
    # the evaluation's scheme (Section VII): asymmetric u8 activations, per-channel symmetric s8 weights.
    # Python integers for the sums, struct-rounded fp32 for every float step.
    import struct

    def r32(v):
        return struct.unpack("f", struct.pack("f", v))[0]

    w = W.mlp_int8(batch=3, dims=(9, 8, 5), seed=5, final="none", per_channel=True, x_zp=7, act_zp=3)
    got = run1(w)
    g = w.graph
    x = w.feeds[g.inputs[0]].tolist()
    ws = [w.feeds[g.inputs[1 + l]].tolist() for l in range(2)]
    bs = [[float(v) for v in w.feeds[g.inputs[3 + l]]] for l in range(2)]
    cs = [[r32(v) for v in g.tensors[g.inputs[1 + l]].channel_scales] for l in range(2)]
    assert len(set(cs[0])) > 1                       # the scales really differ per column
    a_scale, a_zp = [r32(0.02), r32(0.05)], [7, 3]
    inv = r32(1.0 / r32(0.05))
    for m in range(3):
        act = x[m]
        for l in range(2):
            K, N = len(ws[l]), len(ws[l][0])
            nxt = []
            for n in range(N):
                acc = sum((act[k] - a_zp[l]) * ws[l][k][n] for k in range(K))
                # the identity the low-precision conversion relies on: the zero point leaves the sum as a
                # per-column constant, a_z * colsum(W)
                assert acc == sum(act[k] * ws[l][k][n] for k in range(K)) - a_zp[l] * sum(ws[l][k][n] for k in range(K))
                dq = r32(a_scale[l] * cs[l][n])      # product of two fp32 values is exact in fp64: one rounding
                t = r32(r32(float(acc)) * dq)
                t = r32(t + bs[l][n])
                if l == 0:
                    t = max(t, 0.0)
                    u = r32(t * inv)
                    r = int(np.rint(np.float64(u)))
                    nxt.append(min(max(r + 3, 0), 255))
                else:
                    nxt.append(t)
            act = nxt
        assert got.dtype == np.float32
        assert got[m].tolist() == act


def test_per_channel_scales_reduce_to_per_tensor_and_follow_the_n_axis():
    # equal channel scales are the per-tensor case; a transposed weight carries them on axis 0
    base = W.mlp_int8(batch=4, dims=(12, 6), seed=2, final="none")
    ref = run1(base)
    for transposed in (False, True):
        g = Graph()
        feeds = {}
        x = g.input("u8", (4, 12), scale=0.02, name="x")
        wshape = (6, 12) if transposed else (12, 6)
        wt = g.input("s8", wshape, scale=123.0, is_constant=True, channel_scales=[0.005] * 6,
                     channel_axis=0 if transposed else 1)
        b = g.input("f32", (6,), is_constant=True)
        wv = base.feeds[base.graph.inputs[1]]
        feeds[x], feeds[wt], feeds[b] = base.feeds[base.graph.inputs[0]], (wv.T.copy() if transposed else wv), \
            base.feeds[base.graph.inputs[2]]
        acc = g.op("matmul", (x, wt), g.tensor("s32", (4, 6)), transpose_b=transposed)
        z = g.op("dequantize", (acc,), g.tensor("f32", (4, 6)))
        g.mark_output(g.op("add", (z, b), g.tensor("f32", (4, 6))))
        got = interp.run(g, feeds)[g.outputs[0]]
        assert np.array_equal(got, ref)
    # scales on the reduction axis are meaningless and refused
    g = Graph()
    x = g.input("u8", (2, 4), scale=0.02)
    wt = g.input("s8", (4, 3), is_constant=True, channel_scales=[0.1] * 4, channel_axis=0)
    g.mark_output(g.op("matmul", (x, wt), g.tensor("s32", (2, 3))))
    with pytest.raises(TypeError):
        interp.run(g, {x: np.zeros((2, 4), np.uint8), wt: np.zeros((4, 3), np.int8)})


def test_mlp_f32_against_straight_line_restatement():
    w = W.mlp_f32(batch=2, dims=(5, 6, 3), seed=12)
    got = run1(w)
    g = w.graph
    x = w.feeds[g.inputs[0]].astype(np.float64).tolist()
    ws = [w.feeds[g.inputs[1 + l]].astype(np.float64).tolist() for l in range(2)]
    bs = [w.feeds[g.inputs[3 + l]].astype(np.float64).tolist() for l in range(2)]
    for m in range(2):
        act = x[m]
        for l in range(2):
            act = [max(math.fsum(act[k] * ws[l][k][n] for k in range(len(act))) + bs[l][n], 0.0)
                   for n in range(len(bs[l]))]
        assert max(abs(got[m, n] - act[n]) for n in range(3)) < 1e-12


def test_ffn_bf16_against_straight_line_restatement():
    w = W.ffn_bf16(tokens=2, d_model=6, d_ff=10, seed=13)
    got = run1(w)
    g = w.graph
    x, w1, w2, b1, b2 = (w.feeds[i] for i in g.inputs)
    x = W.bf16_bits_to_f32(x).astype(np.float64).tolist()
    w1 = W.bf16_bits_to_f32(w1).astype(np.float64).tolist()
    w2 = W.bf16_bits_to_f32(w2).astype(np.float64).tolist()
    c = math.sqrt(2.0 / math.pi)
    for m in range(2):
        h = []
        for n in range(10):
            z = math.fsum(x[m][k] * w1[k][n] for k in range(6)) + float(b1[n])
            h.append(0.5 * z * (1.0 + math.tanh(c * (z + 0.044715 * z ** 3))))
        for n in range(6):
            y = math.fsum(h[k] * w2[k][n] for k in range(10)) + float(b2[n])
            assert abs(got[m, n] - y) < 1e-12


def test_mha_bf16_against_straight_line_restatement():
    w = W.mha_bf16(batch=1, heads=2, seq=6, head_dim=4, seed=14, valid_lo=3, valid_hi=5)
    got = run1(w)
    g = w.graph
    q, k, v = (W.bf16_bits_to_f32(w.feeds[i]).astype(np.float64) for i in g.inputs[:3])
    mask = w.feeds[g.inputs[3]].astype(np.float64)
    for h in range(2):
        for i in range(6):
            x = [math.fsum(q[0, h, i, d] * k[0, h, j, d] for d in range(4)) * 0.5 + mask[0, 0, 0, j]
                 for j in range(6)]
            mx = max(x)
            e = [math.exp(t - mx) for t in x]
            s = math.fsum(e)
            for d in range(4):
                o = math.fsum(e[j] / s * v[0, h, j, d] for j in range(6))
                assert abs(got[0, h, i, d] - o) < 1e-12


def test_mha_int8_against_straight_line_restatement():
    w = W.mha_int8(batch=1, heads=2, seq=10, head_dim=4, seed=15, valid_lo=5, valid_hi=9)
    got = run1(w)
    g = w.graph
    q, k, v = (w.feeds[i].astype(np.int64) - 128 for i in g.inputs[:3])
    mask = w.feeds[g.inputs[3]]
    f = np.float32
    dq1 = f(0.03) * f(0.03)
    s_p = f(1.0 / 255.0)
    inv_p = f(1.0) / s_p
    dq2 = s_p * f(0.03)
    inv_o = f(1.0) / f(0.02)
    for h in range(2):
        for i in range(10):
            x = []
            for j in range(10):
                acc = int(sum(int(q[0, h, i, d]) * int(k[0, h, j, d]) for d in range(4)))
                t = f(f(acc) * dq1)
                t = f(t * f(0.5))
                t = f(t + mask[0, 0, 0, j])
                x.append(float(t))
            mx = max(x)
            e = [math.exp(t - mx) for t in x]
            s = math.fsum(e)
            pq = [min(max(int(np.rint(e[j] / s * float(inv_p))), 0), 255) for j in range(10)]
            for d in range(4):
                acc2 = sum(pq[j] * int(v[0, h, j, d]) for j in range(10))
                t = f(f(acc2) * dq2)
                u = f(t * inv_o)
                o = min(max(int(np.rint(u)) + 128, 0), 255)
                assert int(got[0, h, i, d]) == o


def test_faithful_mode_rounds_to_declared_dtypes():
    w = W.ffn_bf16(tokens=4, d_model=8, d_ff=16, seed=1)
    pure = run1(w)
    faith = run1(w, faithful=True)
    assert faith.dtype == np.float32
    bits = W.f32_to_bf16_bits(faith)
    assert np.array_equal(W.bf16_bits_to_f32(bits), faith)      # already bf16 values
    assert np.abs(pure - faith).max() < 2e-2
