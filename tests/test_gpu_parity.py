"""Parity of the CUDA path (called through the C ABI) against the CPU oracle on the same seeded inputs.

Bars: integer results bit-exact; fp32 (tf32 matmuls) within 5e-3 * max|ref|; bf16 outputs within 2e-2
max-abs of the fp64 oracle; sigmoid outputs within 2e-6; int8 attention (an fp32 softmax between two
exact integer stages, quantised at rounding boundaries) within one code with at most 1e-3 of the
outputs differing."""
import numpy as np
import pytest

from oracle import interp
from paper_2301_01333_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2301_01333_b200 import build as gc_build
    gc_build.build()
    from paper_2301_01333_b200 import binding
    return binding


def run_gpu(B, w, n_runs=1, **opts):
    import torch
    c = B.CompiledPartition(w.graph, 0, **opts)
    ins = B.device_inputs(w)
    # canary guard bands around the output: 256 bytes on each side must stay untouched
    lt = w.graph.tensors[w.graph.outputs[0]]
    guard = 256
    buf = torch.full((lt.nbytes + 2 * guard,), 0xAB, dtype=torch.uint8, device="cuda:0")
    out = buf[guard:guard + lt.nbytes]
    results = []
    for _ in range(n_runs):
        out.fill_(0xCD)
        c.execute(ins, [out])
        c.query_status()
        results.append(B.output_to_numpy(w.graph, w.graph.outputs[0], out).copy())
    torch.cuda.synchronize()
    assert bool((buf[:guard] == 0xAB).all()) and bool((buf[guard + lt.nbytes:] == 0xAB).all()), "guard band overwritten"
    plan = c.plan
    c.close()
    return (results[0] if n_runs == 1 else results), plan


def oracle(w):
    return interp.run(w.graph, w.feeds)[w.graph.outputs[0]]


def bf16_to_f64(a):
    return W.bf16_bits_to_f32(a).astype(np.float64)


# ------------------------------------------------------------------------------ single matmuls
@pytest.mark.parametrize("m,k,n", [(128, 128, 64), (128, 1024, 256), (300, 479, 1024), (1, 256, 16), (77, 130, 48),
                                   (256, 4096, 512)])
@pytest.mark.parametrize("generic", [False, True])
def test_int8_matmul_accumulators_exact(B, m, k, n, generic):
    w = W.single_matmul("u8", "s8", m, k, n, seed=m + k + n)
    got, plan = run_gpu(B, w, force_generic=generic)
    assert ("tcgen05.i8" in plan) == (not generic)
    assert np.array_equal(got.astype(np.int64), oracle(w))


@pytest.mark.parametrize("m,k,n", [(5, 33, 7), (1, 479, 1), (3, 256, 1), (130, 64, 17)])
def test_int8_matmul_ragged_shapes_exact(B, m, k, n):
    w = W.single_matmul("u8", "s8", m, k, n, seed=1, a_zp=3)
    got, plan = run_gpu(B, w)
    assert "cuda-core" in plan
    assert np.array_equal(got.astype(np.int64), oracle(w))


def test_int8_matmul_transposed_weights_and_signed_activations(B):
    w = W.single_matmul("s8", "s8", 64, 200, 32, seed=2, transpose_b=True)
    got, plan = run_gpu(B, w)
    assert "tcgen05.i8" in plan
    assert np.array_equal(got.astype(np.int64), oracle(w))


def test_int8_matmul_extreme_values(B):
    w = W.single_matmul("u8", "s8", 128, 1024, 64)
    w.feeds[w.graph.inputs[0]][:] = 255
    w.feeds[w.graph.inputs[1]][:] = -127
    got, _ = run_gpu(B, w)
    assert (got == -33162240).all()


@pytest.mark.parametrize("m,k,n", [(128, 64, 64), (200, 1000, 272), (32, 13, 512), (1024, 1024, 1024)])
@pytest.mark.parametrize("dtype,tol", [("bf16", 2e-4), ("f32", 5e-3)])
def test_float_matmul(B, m, k, n, dtype, tol):
    if dtype == "bf16" and k % 8:
        k += 8 - k % 8          # keep the bf16 case on the tcgen05 path (row pitch multiple of 16 bytes)
    w = W.single_matmul(dtype, dtype, m, k, n, seed=7)
    got, plan = run_gpu(B, w)
    assert "tcgen05" in plan
    ref = oracle(w)
    assert np.abs(got - ref).max() <= tol * np.abs(ref).max()


@pytest.mark.parametrize("m,k,n", [(2600, 512, 2048), (4096, 200, 1280)])
def test_cta_pair_gemm_int8_exact(B, m, k, n):
    # large enough for the CTA-pair kernel; 2600 rows = 21 row blocks, so the last pair has an empty partner
    w = W.single_matmul("u8", "s8", m, k, n, seed=11)
    got, plan = run_gpu(B, w)
    assert "cta_pair" in plan
    assert np.array_equal(got.astype(np.int64), oracle(w))


def test_cta_pair_gemm_bf16_with_epilogue(B):
    w = W.ffn_bf16(tokens=2600, d_model=256, d_ff=2048)
    got, plan = run_gpu(B, w)
    assert "cta_pair" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


def test_cta_pair_gemm_bf16_grouped_tile_order_sampled_rows(B):
    # a plain GEMM large enough for the grouped tile order of the CTA-pair kernel: 20 row blocks of 256 = two full
    # groups of eight and a short one, 16 column tiles; every row block is sampled, the last one is ragged
    w = W.plain_gemm_bf16(5000, 1024, 4096, seed=5)
    got, plan = run_gpu(B, w)
    assert "cta_pair" in plan
    rows = np.unique(np.concatenate([np.arange(0, 5000, 19), [127, 128, 255, 256, 2047, 2048, 4095, 4096, 4863, 4864, 4999]]))
    sub = W.plain_gemm_bf16(len(rows), 1024, 4096, seed=5)
    for a, b in zip(sub.graph.inputs, w.graph.inputs):
        sub.feeds[a] = w.feeds[b][rows] if a == sub.graph.inputs[0] else w.feeds[b]
    ref = oracle(sub)
    assert np.abs(bf16_to_f64(got)[rows] - ref).max() <= 2e-2
    assert np.isfinite(bf16_to_f64(got)).all()


def test_batched_matmul_int8_exact(B):
    w = W.single_matmul("u8", "u8", 24, 16, 24, seed=3, transpose_b=True, a_zp=128, batch=(2, 3))
    w.graph.tensors[w.graph.inputs[1]].zero_point = 128
    got, _ = run_gpu(B, w)
    assert np.array_equal(got.astype(np.int64), oracle(w))


# ------------------------------------------------------------------------------ MLP chains
@pytest.mark.parametrize("batch,dims", [(32, (13, 512, 256, 128)), (7, (13, 32, 16)), (200, (40, 64, 48, 16))])
@pytest.mark.parametrize("generic", [False, True])
def test_mlp_f32(B, batch, dims, generic):
    w = W.mlp_f32(batch=batch, dims=dims)
    got, _ = run_gpu(B, w, force_generic=generic)
    ref = oracle(w)
    assert (got >= 0).all()
    assert np.abs(got - ref).max() <= 5e-3 * np.abs(ref).max()


@pytest.mark.parametrize("batch,dims", [(128, (479, 1024, 1024, 512, 256, 1)), (5, (30, 32, 16, 1)), (300, (479, 64, 48, 32))])
@pytest.mark.parametrize("opts", [{}, {"force_generic": True}, {"no_chain_fusion": True}])
def test_mlp_int8_logits_bit_exact_and_sigmoid(B, batch, dims, opts):
    w = W.mlp_int8(batch=batch, dims=dims, final="none")
    got, _ = run_gpu(B, w, **opts)
    ref = oracle(w)
    assert ref.dtype == np.float32
    assert np.array_equal(got, ref)                      # separately rounded fp32 ops: bit-exact
    ws = W.mlp_int8(batch=batch, dims=dims)
    gs, _ = run_gpu(B, ws, **opts)
    assert np.abs(gs.astype(np.float64) - oracle(ws)).max() <= 2e-6


@pytest.mark.parametrize("batch,dims", [(128, (479, 1024, 1024, 512, 256, 1)), (37, (100, 80, 48, 16)),
                                        (2600, (512, 2048, 256))])
@pytest.mark.parametrize("opts", [{}, {"force_generic": True}, {"no_chain_fusion": True}])
def test_mlp_int8_per_channel_scales_and_zero_points_bit_exact(B, batch, dims, opts):
    # the evaluation's scheme (Section VII): asymmetric u8 activations, per-channel s8 weight scales; the tensor
    # cores multiply the stored codes and the zero point leaves through the compensated-weight term
    w = W.mlp_int8(batch=batch, dims=dims, final="none", per_channel=True, x_zp=12, act_zp=5)
    got, plan = run_gpu(B, w, **opts)
    if not opts.get("force_generic"):
        assert "tcgen05.i8" in plan
    ref = oracle(w)
    assert ref.dtype == np.float32
    assert np.array_equal(got, ref)


@pytest.mark.parametrize("m,k,n,zp", [(128, 1024, 256, 128), (77, 130, 48, 3), (2600, 512, 2048, 200)])
def test_int8_matmul_nonzero_zero_point_on_tensor_cores_exact(B, m, k, n, zp):
    w = W.single_matmul("u8", "s8", m, k, n, seed=zp, a_zp=zp)
    got, plan = run_gpu(B, w)
    assert "tcgen05.i8" in plan
    assert np.array_equal(got.astype(np.int64), oracle(w))


@pytest.mark.parametrize("batch,dims,ks", [(64, (600, 256, 64), 2), (77, (700, 128, 32), 2), (33, (131, 64, 16), 1),
                                           (128, (1030, 512, 256, 32), 4), (1, (479, 1024, 16), 4),
                                           (256, (479, 1024, 1024, 512, 256, 1), 2), (512, (100, 304, 32), 1), (512, (100, 512, 32), 2),
                                           (300, (13, 512, 256, 128), 2), (130, (70, 64, 32), 1)])
def test_mlp_int8_chain_kernel_cluster_sizes_and_entry_reorder(B, batch, dims, ks):
    # the fused chain kernel with the reduction axis split over 1, 2 and 4 CTAs, inputs whose rows start at every
    # byte alignment (the graph-entry reorder inside the kernel) and reductions that end inside a k-block
    w = W.mlp_int8(batch=batch, dims=dims, final="none", per_channel=True, x_zp=3, act_zp=7)
    got, plan = run_gpu(B, w)
    assert f"clusters of {ks}" in plan
    assert np.array_equal(got, oracle(w))


@pytest.mark.parametrize("batch,dims,ks,final", [
    (128, (479, 1024, 1024, 512, 256, 1), 4, "sigmoid"),   # config 2: four threads per finished row
    (300, (600, 512, 64, 1), 2, "none"),                   # two threads per row, three row tiles, the last one ragged
    (512, (1024, 256, 1), 4, "sigmoid"),                   # four row tiles: 32 slices x 4 x 4 CTAs would not fit -> ks shrinks
    (7, (700, 96, 32, 1), 2, "none"),                      # a handful of rows, one slice in the folded layer
])
def test_mlp_int8_one_column_tail_folded_into_the_layer_before(B, batch, dims, ks, final):
    w = W.mlp_int8(batch=batch, dims=dims, final=final, per_channel=True, x_zp=3, act_zp=7)
    got, plan = run_gpu(B, w, n_runs=3)
    assert "folded into the finishing step" in plan, plan
    assert np.array_equal(got[0], got[1]) and np.array_equal(got[0], got[2])      # sums and counters are left at zero
    ref = oracle(w)
    if final == "none":
        assert np.array_equal(got[0], ref)
    else:
        assert np.abs(got[0].astype(np.float64) - ref).max() <= 2e-6
    sep, plan2 = run_gpu(B, w, no_chain_fusion=True)
    assert "folded" not in plan2
    assert np.array_equal(sep, got[0]) if final == "none" else np.abs(sep.astype(np.float64) - ref).max() <= 2e-6


@pytest.mark.parametrize("batch,dims,ks", [(16, (160, 64, 32), 2), (100, (13, 1024, 48), 4), (128, (37, 32, 16), 1)])
def test_mlp_f32_chain_kernel_cluster_sizes(B, batch, dims, ks):
    w = W.mlp_f32(batch=batch, dims=dims)
    got, plan = run_gpu(B, w, grid_wide_chain=True)
    assert f"clusters of {ks}" in plan and "inside one cluster" not in plan
    ref = oracle(w)
    assert np.abs(got.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()


@pytest.mark.parametrize("batch,dims,cluster", [
    (32, (13, 512, 256, 128), 16),        # config 1: 16 x 1, 8 x 2 and 4 x 4 (slices x parts of the reduction axis)
    (64, (13, 512, 256, 128), 16),        # the most rows the kernel takes
    (1, (32, 32, 32), 8),                 # one row, one slice
    (17, (45, 96, 64), 8),                # ragged rows and a first layer whose row pitch TMA cannot address
    (8, (64, 128, 64), 8),                # first layer fed by TMA
    (24, (200, 160, 288, 32, 64), 16),    # five k-blocks over two parts, nine slices, a one-slice layer in the middle
    (32, (13, 1024, 64), 8),              # recomputed first layer at its widest (256 columns per CTA)
    (40, (100, 256, 256, 128, 32), 16),   # first layer too deep to recompute: distributed like the others
    (32, (60, 64, 32), 8),                # recomputed first layer with two k-blocks
])
def test_mlp_f32_chain_inside_one_cluster(B, batch, dims, cluster):
    w = W.mlp_f32(batch=batch, dims=dims)
    got, plan = run_gpu(B, w, n_runs=3)
    assert f"inside one cluster of {cluster} CTAs" in plan
    assert np.array_equal(got[0], got[1]) and np.array_equal(got[0], got[2])      # deterministic, no state carried over
    ref = oracle(w)
    assert np.abs(got[0].astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()
    wide, plan_w = run_gpu(B, w, grid_wide_chain=True)
    assert "inside one cluster" not in plan_w
    assert np.abs(wide.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()


def test_mlp_f32_too_large_for_one_cluster_stays_grid_wide(B):
    for batch, dims in ((65, (13, 512, 256, 128)), (32, (13, 1024, 1024, 64)), (48, (300, 512, 512, 256, 128))):
        w = W.mlp_f32(batch=batch, dims=dims)
        got, plan = run_gpu(B, w)
        assert "fused chain" in plan and "inside one cluster" not in plan
        ref = oracle(w)
        assert np.abs(got.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()


def test_two_large_layers_in_one_launch_bf16(B):
    # both GEMMs on CTA pairs in one persistent launch (row-block counters between them); 39 row tiles: the last
    # pair is half empty
    w = W.ffn_bf16(tokens=4900, d_model=1024, d_ff=1024)
    got, plan = run_gpu(B, w, n_runs=2)
    assert "one launch" in plan
    assert np.array_equal(got[0], got[1])
    assert np.abs(bf16_to_f64(got[0]) - oracle(w)).max() <= 2e-2
    sep, plan2 = run_gpu(B, w, no_chain_fusion=True)
    assert "one launch" not in plan2
    assert np.array_equal(sep, got[0])                   # same tiles, same arithmetic: identical bits


def test_two_large_layers_in_one_launch_ragged_hidden_width(B):
    # hidden width 1008: the fourth 256-column tile of the first layer is clipped and the second layer's last group of
    # k-blocks is partly padding; 75 row tiles: the last pair is half empty.  bf16 (4 k-blocks per first-layer tile)
    # and tf32 (8 per tile).
    w = W.ffn_bf16(tokens=9500, d_model=512, d_ff=1008)
    got, plan = run_gpu(B, w, n_runs=2)
    assert "one launch" in plan
    assert np.array_equal(got[0], got[1])
    assert np.abs(bf16_to_f64(got[0]) - oracle(w)).max() <= 2e-2
    w = W.mlp_f32(batch=9500, dims=(256, 1008, 512), seed=4)
    got, plan = run_gpu(B, w)
    assert "one launch" in plan
    ref = oracle(w)
    assert np.abs(got.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()


def test_two_large_layers_in_one_launch_int8_bit_exact(B):
    w = W.mlp_int8(batch=4900, dims=(1024, 1024, 1024, 16), final="none", per_channel=True, x_zp=9, act_zp=4)
    got, plan = run_gpu(B, w)
    assert "layers 0+1: one launch" in plan
    assert np.array_equal(got, oracle(w))


def _mlp_variant(kind, batch, dims, bias=True, act="relu", transposed=False, hidden="u8", per_channel=False, seed=3):
    """An MLP chain with optional pieces changed: no bias, another activation, weights stored [n, k] (with the
    per-channel scales on axis 0), s8 hidden activations."""
    from paper_2301_01333_b200.graph import Graph
    from paper_2301_01333_b200.workloads import Workload, f32_to_bf16_bits
    rng = np.random.default_rng(seed)
    g = Graph(name="mlp_variant")
    feeds = {}
    if kind == "int8":
        x = g.input("u8", (batch, dims[0]), scale=0.02, zero_point=5)
        feeds[x] = rng.integers(0, 256, size=(batch, dims[0])).astype(np.uint8)
    elif kind == "bf16":
        x = g.input("bf16", (batch, dims[0]))
        feeds[x] = f32_to_bf16_bits(rng.standard_normal((batch, dims[0]), dtype=np.float32))
    else:
        x = g.input("f32", (batch, dims[0]))
        feeds[x] = rng.standard_normal((batch, dims[0]), dtype=np.float32)
    h = x
    nl = len(dims) - 1
    for l in range(nl):
        k, n = dims[l], dims[l + 1]
        wshape = (n, k) if transposed else (k, n)
        if kind == "int8":
            kw = {}
            if per_channel:
                kw = dict(channel_scales=(0.005 * rng.uniform(0.5, 1.5, size=n)).astype(np.float32),
                          channel_axis=0 if transposed else 1)
            w = g.input("s8", wshape, scale=0.005, is_constant=True, **kw)
            feeds[w] = rng.integers(-127, 128, size=wshape).astype(np.int8)
        else:
            w = g.input(kind, wshape, is_constant=True)
            wv = (rng.standard_normal(wshape) * np.sqrt(1.0 / k)).astype(np.float32)
            feeds[w] = f32_to_bf16_bits(wv) if kind == "bf16" else wv
        z = g.op("matmul", (h, w), g.tensor("s32" if kind == "int8" else "f32", (batch, n)), transpose_b=transposed)
        if kind == "int8":
            z = g.op("dequantize", (z,), g.tensor("f32", (batch, n)))
        if bias:
            b = g.input("f32", (n,), is_constant=True)
            feeds[b] = rng.uniform(-0.1, 0.1, size=(n,)).astype(np.float32)
            z = g.op("add", (z, b), g.tensor("f32", (batch, n)))
        if l < nl - 1:
            z = g.op(act, (z,), g.tensor("f32", (batch, n)))
            if kind == "int8":
                h = g.op("quantize", (z,), g.tensor(hidden, (batch, n), scale=0.05, zero_point=3 if hidden == "u8" else 0))
            elif kind == "bf16":
                h = g.op("typecast", (z,), g.tensor("bf16", (batch, n)))
            else:
                h = z
        else:
            h = g.op("typecast", (z,), g.tensor("bf16", (batch, n))) if kind == "bf16" else z
    g.mark_output(h)
    return Workload(g.name, g, feeds).finish()


@pytest.mark.parametrize("kind,batch,dims,kw", [
    ("int8", 64, (300, 256, 64, 32), dict(transposed=True, hidden="s8", per_channel=True)),
    ("int8", 3000, (512, 1024, 1024, 32), dict(transposed=True, per_channel=True)),
    ("int8", 3000, (512, 1024, 1024, 32), dict(hidden="s8", bias=False)),
    ("bf16", 96, (256, 512, 128), dict(bias=False, act="gelu_tanh")),
    ("bf16", 5000, (1024, 1024, 1024), dict(transposed=True, act="gelu_tanh")),
    ("f32", 32, (100, 256, 64), dict(act="sigmoid")),
    ("f32", 16, (40, 128, 64, 32), dict(act="gelu_tanh")),        # one cluster, first layer recomputed, out-of-line activation
    ("f32", 8, (20, 64, 32), dict(bias=False, act="sigmoid")),
    ("f32", 600, (64, 512, 128), dict(bias=False, transposed=True))])
@pytest.mark.parametrize("opts", [{}, {"no_chain_fusion": True}])
def test_mlp_graph_variants(B, kind, batch, dims, kw, opts):
    w = _mlp_variant(kind, batch, dims, **kw)
    got, _ = run_gpu(B, w, **opts)
    ref = oracle(w)
    if kind == "int8":
        assert np.array_equal(got, ref)
    elif kind == "bf16":
        assert np.abs(bf16_to_f64(got) - ref).max() <= 2e-2
    else:
        assert np.abs(got.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()


def test_ffn_bf16_chain_kernel_with_split_reduction(B):
    w = W.ffn_bf16(tokens=96, d_model=512, d_ff=256)
    got, plan = run_gpu(B, w)
    assert "clusters of 4" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


def test_mlp_int8_hidden_layer_codes_bit_exact(B):
    # a chain that ends on a requantised u8 tensor: compares the codes themselves
    w = W.mlp_int8(batch=128, dims=(479, 1024, 512), final="none")
    g = w.graph
    # drop the last layer's dequantize/add and end after the first layer's quantize instead
    first_q = [i for i, op in enumerate(g.ops) if op.kind == "quantize"][0]
    del g.ops[first_q + 1:]
    g.outputs[:] = [g.ops[first_q].output]
    g.inputs[:] = [t for t in g.inputs if any(t in op.inputs for op in g.ops)]
    got, plan = run_gpu(B, w)
    assert "tcgen05.i8" in plan
    ref = oracle(w)
    assert np.array_equal(got.astype(np.int64), ref)
    assert (ref == 255).mean() > 0.05 and (ref == 0).mean() > 0.05     # saturation is exercised


@pytest.mark.parametrize("tokens,d_model,d_ff", [(256, 128, 512), (100, 64, 272)])
def test_ffn_bf16_reduced(B, tokens, d_model, d_ff):
    w = W.ffn_bf16(tokens=tokens, d_model=d_model, d_ff=d_ff)
    got, _ = run_gpu(B, w)
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


def test_ffn_bf16_full_size_every_output(B):
    # the benchmark's headline configuration in the launch configuration the benchmark times (both GEMMs in one
    # launch over the 640-tile schedule): all 8192 x 1024 outputs against the oracle
    w = W.ffn_bf16()                                      # 8192 x (1024 -> 4096 -> 1024)
    got, plan = run_gpu(B, w)
    assert plan.count("tcgen05.bf16") == 2 and "one launch" in plan
    ref = oracle(w)
    assert ref.shape == (8192, 1024)
    assert np.abs(bf16_to_f64(got) - ref).max() <= 2e-2


# ------------------------------------------------------------------------------ attention
@pytest.mark.parametrize("b,h,s,d", [(32, 12, 128, 64), (2, 3, 256, 64), (1, 2, 384, 64), (2, 2, 48, 32), (1, 1, 200, 64)])
def test_mha_bf16(B, b, h, s, d):
    w = W.mha_bf16(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w)
    assert ("tcgen05" in plan) == (d == 64)                  # any sequence length up to 512 keys; head width 32 is CUDA-core
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


@pytest.mark.parametrize("b,h,valid", [(32, 12, None), (1, 1, None), (50, 12, None), (3, 5, (1, 128)), (2, 4, (0, 40))])
def test_mha_bf16_one_unit_per_cta(B, b, h, valid):
    # 128 keys, head width 64: one (batch, head) unit per CTA, three CTAs per SM.  600 units are more than the 444 that
    # are resident at once (a second wave); padding masks from a single valid key up, and rows whose mask is minus
    # infinity for most keys
    kw = {} if valid is None else {"valid_lo": valid[0], "valid_hi": valid[1]}
    w = W.mha_bf16(batch=b, heads=h, seq=128, head_dim=64, seed=b + h, **kw)
    if valid == (0, 40):
        mask = w.feeds[w.graph.inputs[3]]
        mask[mask < 0] = -np.inf
        mask[..., :1] = 0.0                                     # every row keeps one key
    got, plan = run_gpu(B, w)
    assert "tcgen05.unit-per-cta" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


# the other head dimensions and sequence lengths of the evaluation's workload table, on the streaming kernel;
# the larger cases give every CTA more than one work unit, so the rings and barrier phases wrap
WIDE_SHAPES = [(1, 2, 128, 96), (1, 2, 384, 128), (1, 2, 512, 64), (2, 1, 256, 128), (1, 1, 512, 128), (1, 1, 256, 96),
               (4, 40, 128, 96), (2, 30, 384, 128), (1, 50, 512, 64)]


@pytest.mark.parametrize("b,h,s,d", WIDE_SHAPES)
def test_mha_bf16_streaming_kernel(B, b, h, s, d):
    w = W.mha_bf16(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w)
    assert "tcgen05.streaming" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


# sequence lengths that are not a multiple of the 128-key block (a batch padded to 200 or 320 keys, fewer keys than one
# block, one key short of or past a block): the kernel runs the next multiple, the keys past the end must get weight
# exactly zero, the query rows past the end must not be stored (the guard bands around the output check that)
RAGGED_SHAPES = [(1, 1, 200, 64), (2, 2, 320, 64), (1, 2, 72, 64), (2, 3, 127, 96), (1, 2, 129, 128), (3, 20, 200, 64),
                 (1, 2, 500, 64), (1, 1, 8, 64)]


@pytest.mark.parametrize("b,h,s,d", RAGGED_SHAPES)
@pytest.mark.parametrize("kind", ["bf16", "int8"])
def test_mha_ragged_sequence_lengths_on_tensor_cores(B, kind, b, h, s, d):
    w = W.mha_bf16(batch=b, heads=h, seq=s, head_dim=d) if kind == "bf16" else W.mha_int8(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w)
    assert "tcgen05.streaming" in plan
    if kind == "bf16":
        assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2
    else:
        check_int8_attention(got, oracle(w))


def test_mha_ragged_without_a_mask_and_with_minus_infinity(B):
    # no mask op at all (the kernel still has to mask the keys past the end), and a user mask that already holds -inf
    w = _attention_variant("int8", 2, 3, 200, 64, False, True, False)
    got, plan = run_gpu(B, w)
    assert "tcgen05.streaming" in plan
    check_int8_attention(got, oracle(w))
    w = W.mha_bf16(batch=2, heads=2, seq=300, head_dim=64, seed=4)
    mid = [t for t in w.graph.inputs if w.graph.tensors[t].name == "mask"][0]
    m = w.feeds[mid].copy()
    m[m < 0] = -np.inf
    w.feeds[mid] = m
    got, plan = run_gpu(B, w)
    assert "tcgen05.streaming" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


# rows of more than 512 keys do not fit tensor memory next to the output: blockwise softmax with the scores computed
# twice; several units per CTA on the larger cases (rings and barrier phases wrap), a ragged length, every head width
LONG_SHAPES = [(1, 2, 640, 64), (1, 2, 1024, 128), (1, 1, 1000, 96), (1, 40, 640, 64), (1, 40, 768, 128), (1, 1, 2048, 64)]


@pytest.mark.parametrize("b,h,s,d", LONG_SHAPES)
@pytest.mark.parametrize("kind", ["bf16", "int8"])
def test_mha_more_than_512_keys_on_tensor_cores(B, kind, b, h, s, d):
    w = W.mha_bf16(batch=b, heads=h, seq=s, head_dim=d) if kind == "bf16" else W.mha_int8(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w)
    assert "tcgen05.two-pass" in plan
    if kind == "bf16":
        assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2
    else:
        check_int8_attention(got, oracle(w))


@pytest.mark.parametrize("b,h,s,d", WIDE_SHAPES)
def test_mha_int8_streaming_kernel(B, b, h, s, d):
    w = W.mha_int8(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w)
    assert "tcgen05.streaming" in plan
    check_int8_attention(got, oracle(w))


def test_mha_int8_streaming_kernel_stages_around_the_softmax(B):
    import torch
    w = W.mha_int8(batch=2, heads=2, seq=512, head_dim=64, seed=9)
    g = w.graph
    g.mark_output(w.info["p_quant"])
    c = B.CompiledPartition(g, 0)
    assert "tcgen05.streaming" in c.plan
    ins = B.device_inputs(w)
    outs = B.device_outputs(g)
    c.execute(ins, outs)
    c.query_status()
    torch.cuda.synchronize()
    o_gpu = B.output_to_numpy(g, g.outputs[0], outs[0]).copy()
    p_gpu = B.output_to_numpy(g, g.outputs[1], outs[1]).copy()
    c.close()
    ref = interp.run(g, w.feeds)
    dp = np.abs(p_gpu.astype(np.int64) - ref[g.outputs[1]])
    assert dp.max() <= 1 and (dp != 0).mean() <= 1e-3
    assert_stage_after_softmax_exact(w, o_gpu, p_gpu)


def _attention_variant(kind, b, h, s, d, mask, mul, q_signed, seed=1):
    """An attention partition with optional pieces left out (no mask, no scaling) or s8 queries."""
    from paper_2301_01333_b200.graph import Graph
    from paper_2301_01333_b200.workloads import Workload, _mask_from_valid, f32_to_bf16_bits
    rng = np.random.default_rng(seed)
    g = Graph(name="attention_variant")
    feeds = {}
    shp, ss = (b, h, s, d), (b, h, s, s)
    if kind == "bf16":
        q, k, v = (g.input("bf16", shp) for _ in range(3))
        for t in (q, k, v):
            feeds[t] = f32_to_bf16_bits(rng.standard_normal(shp, dtype=np.float32))
        x = g.op("matmul", (q, k), g.tensor("f32", ss), transpose_b=True)
    else:
        q = g.input("s8" if q_signed else "u8", shp, scale=0.03, zero_point=0 if q_signed else 128)
        k = g.input("u8", shp, scale=0.03, zero_point=128)
        v = g.input("u8", shp, scale=0.03, zero_point=128)
        feeds[q] = rng.integers(-128, 128, size=shp).astype(np.int8) if q_signed else rng.integers(0, 256, size=shp).astype(np.uint8)
        feeds[k] = rng.integers(0, 256, size=shp).astype(np.uint8)
        feeds[v] = rng.integers(0, 256, size=shp).astype(np.uint8)
        a = g.op("matmul", (q, k), g.tensor("s32", ss), transpose_b=True)
        x = g.op("dequantize", (a,), g.tensor("f32", ss))
    if mul:
        x = g.op("mul", (x,), g.tensor("f32", ss), scalar=float(1 / np.sqrt(d)))
    if mask:
        m = g.input("f32", (b, 1, 1, s))
        feeds[m] = _mask_from_valid(rng.integers(s // 2, s + 1, size=(b,)), s)
        x = g.op("add", (x, m), g.tensor("f32", ss))
    p = g.op("softmax", (x,), g.tensor("f32", ss), axis=-1)
    if kind == "bf16":
        pb = g.op("typecast", (p,), g.tensor("bf16", ss))
        o = g.op("matmul", (pb, v), g.tensor("f32", shp))
        o = g.op("typecast", (o,), g.tensor("bf16", shp))
    else:
        pq = g.op("quantize", (p,), g.tensor("u8", ss, scale=float(np.float32(1 / 255)), zero_point=0))
        a2 = g.op("matmul", (pq, v), g.tensor("s32", shp))
        o = g.op("dequantize", (a2,), g.tensor("f32", shp))
        o = g.op("quantize", (o,), g.tensor("u8", shp, scale=0.02, zero_point=128))
    g.mark_output(o)
    return Workload(g.name, g, feeds).finish()


@pytest.mark.parametrize("kind,s,d,mask,mul,q_signed", [
    ("bf16", 128, 64, False, True, False), ("bf16", 256, 128, True, False, False), ("bf16", 512, 64, False, False, False),
    ("int8", 384, 64, False, False, True), ("int8", 512, 64, True, True, True), ("int8", 128, 96, False, True, False),
    ("int8", 256, 128, True, False, True)])
def test_attention_graph_variants(B, kind, s, d, mask, mul, q_signed):
    # the optional ops of the pattern left out (no mask, no scaling) and signed queries, on both tcgen05 kernels
    w = _attention_variant(kind, 2, 3, s, d, mask, mul, q_signed)
    got, plan = run_gpu(B, w)
    assert "tcgen05" in plan
    if kind == "bf16":
        assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2
    else:
        check_int8_attention(got, oracle(w))


def test_mha_bf16_generic_kernel(B):
    w = W.mha_bf16(batch=2, heads=2, seq=128, head_dim=64)
    got, plan = run_gpu(B, w, force_generic=True)
    assert "cuda-core" in plan
    assert np.abs(bf16_to_f64(got) - oracle(w)).max() <= 2e-2


def check_int8_attention(got, ref):
    diff = np.abs(got.astype(np.int64) - ref)
    assert diff.max() <= 1, f"max code difference {diff.max()}"
    frac = (diff != 0).mean()
    assert frac <= 1e-3, f"mismatch fraction {frac}"
    return frac


@pytest.mark.parametrize("b,h,s,d", [(2, 2, 128, 64), (1, 3, 384, 64), (2, 2, 256, 64), (1, 2, 40, 16)])
@pytest.mark.parametrize("generic", [False, True])
def test_mha_int8_reduced(B, b, h, s, d, generic):
    w = W.mha_int8(batch=b, heads=h, seq=s, head_dim=d)
    got, plan = run_gpu(B, w, force_generic=generic)
    assert ("tcgen05" in plan) == (not generic and d == 64 and s % 128 == 0)
    check_int8_attention(got, oracle(w))


@pytest.mark.parametrize("s", [128, 384])
def test_mha_int8_max_free_softmax(B, s):
    # 8-bit attention without a mask and with scales small enough that every score is bounded at compile time
    # (|score| log2(e) <= 60): the planner picks the max-free softmax (Section VII); same results as with the row
    # maximum (the option switches it off), both within the int8 bar of the oracle
    w = W.mha_int8(batch=2, heads=3, seq=s, head_dim=64, s_qkv=0.012, with_mask=False, seed=7)
    got, plan = run_gpu(B, w)
    assert "softmax=max-free" in plan
    ref = oracle(w)
    check_int8_attention(got, ref)
    exact, plan2 = run_gpu(B, w, exact_max_softmax=True)
    assert "max-free" not in plan2
    check_int8_attention(exact, ref)
    assert (np.abs(got.astype(np.int64) - exact.astype(np.int64)) <= 1).all()
    # larger scales or a mask: the bound does not hold, the row maximum stays
    for kw in (dict(s_qkv=0.03, with_mask=False), dict(s_qkv=0.012, with_mask=True)):
        w2 = W.mha_int8(batch=1, heads=1, seq=s, head_dim=64, **kw)
        assert "max-free" not in B.CompiledPartition(w2.graph, 0).plan


def test_mha_int8_masked_chunk_skipping_edge_cases(B):
    # the tcgen05 kernel leaves out 32-key chunks whose keys are all masked; rows must not notice.  Batches:
    # everything masked (no skipping allowed: the mask then cancels in the softmax), one valid key, a valid
    # length inside a chunk, a whole masked 128-key block, nothing masked, a mild mask value that is not
    # skippable, masked keys in the middle of the row, and -inf.
    w = W.mha_int8(batch=8, heads=2, seq=384, head_dim=64, seed=3)
    g = w.graph
    mid = [t for t in g.inputs if g.tensors[t].name == "mask"][0]
    mask = np.zeros((8, 1, 1, 384), dtype=np.float32)
    mask[0] = -10000.0
    mask[1, ..., 1:] = -10000.0
    mask[2, ..., 211:] = -10000.0
    mask[3, ..., 256:] = -10000.0
    mask[5, ..., 100:] = -3.0
    mask[6, ..., 64:160] = -10000.0
    mask[7, ..., 130:] = -np.inf
    w.feeds[mid] = mask
    g.mark_output(w.info["p_quant"])
    import torch
    c = B.CompiledPartition(g, 0)
    assert "tcgen05" in c.plan
    ins = B.device_inputs(w)
    outs = B.device_outputs(g)
    c.execute(ins, outs)
    c.query_status()
    torch.cuda.synchronize()
    got_o = B.output_to_numpy(g, g.outputs[0], outs[0])
    got_p = B.output_to_numpy(g, g.outputs[1], outs[1]).astype(np.int64)
    c.close()
    ref = interp.run(g, w.feeds)
    # the rows of this test sit on many more rounding boundaries than random data (a handful of equal large
    # probabilities per row): the codes may differ by one more often, the output by one code at most
    dp = np.abs(got_p - ref[g.outputs[1]])
    assert dp.max() <= 1 and (dp != 0).mean() <= 1e-3
    assert np.abs(got_o.astype(np.int64) - ref[g.outputs[0]]).max() <= 1
    assert_stage_after_softmax_exact(w, got_o, got_p.astype(np.uint8))
    assert not got_p[2, :, :, 211:].any() and not got_p[3, :, :, 256:].any() and not got_p[6, :, :, 64:160].any()
    assert not got_p[7, :, :, 130:].any()
    assert got_p[0].any(axis=-2).all()               # fully masked batch: every key still receives weight


@pytest.mark.parametrize("generic", [False, True])
def test_mha_int8_stages_around_the_softmax(B, generic):
    """The fp32 softmax sits between two exact integer stages.  With the probabilities as a second output:
    (a) the codes differ from the oracle's by at most one, rarely; (b) given the codes the kernel itself used,
    the integer stage after the softmax (P.V, dequantize, requantize) is reproduced by the oracle bit for bit."""
    import torch
    from paper_2301_01333_b200.graph import Graph
    w = W.mha_int8(batch=1, heads=3, seq=384, head_dim=64, seed=5)
    g = w.graph
    g.mark_output(w.info["p_quant"])
    c = B.CompiledPartition(g, 0, force_generic=generic)
    assert ("tcgen05" in c.plan) == (not generic)
    ins = B.device_inputs(w)
    outs = B.device_outputs(g)
    c.execute(ins, outs)
    c.query_status()
    torch.cuda.synchronize()
    o_gpu = B.output_to_numpy(g, g.outputs[0], outs[0]).copy()
    p_gpu = B.output_to_numpy(g, g.outputs[1], outs[1]).copy()
    c.close()
    ref = interp.run(g, w.feeds)
    dp = np.abs(p_gpu.astype(np.int64) - ref[g.outputs[1]])
    assert dp.max() <= 1 and (dp != 0).mean() <= 1e-3
    check_int8_attention(o_gpu, ref[g.outputs[0]])
    assert_stage_after_softmax_exact(w, o_gpu, p_gpu)


def assert_stage_after_softmax_exact(w, o_gpu, p_gpu):
    """P.V, dequantize, requantize recomputed by the oracle from the kernel's own probability codes."""
    from paper_2301_01333_b200.graph import Graph
    g = w.graph
    v_id = g.inputs[2]
    g3 = Graph()
    pin = g3.input("u8", g.tensors[g.outputs[1]].dims, scale=g.tensors[g.outputs[1]].scale, zero_point=0)
    vin = g3.input("u8", g.tensors[v_id].dims, scale=g.tensors[v_id].scale, zero_point=g.tensors[v_id].zero_point)
    a2 = g3.op("matmul", (pin, vin), g3.tensor("s32", g.tensors[g.outputs[0]].dims))
    d2 = g3.op("dequantize", (a2,), g3.tensor("f32", g.tensors[g.outputs[0]].dims))
    ot = g.tensors[g.outputs[0]]
    g3.mark_output(g3.op("quantize", (d2,), g3.tensor("u8", ot.dims, scale=ot.scale, zero_point=ot.zero_point)))
    exact = interp.run(g3, {pin: p_gpu, vin: w.feeds[v_id]})[g3.outputs[0]]
    assert np.array_equal(o_gpu.astype(np.int64), exact)


def test_mha_bf16_probabilities_output(B):
    w = W.mha_bf16(batch=1, heads=2, seq=128, head_dim=64, seed=8)
    g = w.graph
    p_id = [op.output for op in g.ops if op.kind == "typecast"][0]
    g.mark_output(p_id)
    c = B.CompiledPartition(g, 0)
    ins = B.device_inputs(w)
    outs = B.device_outputs(g)
    c.execute(ins, outs)
    c.query_status()
    p_gpu = bf16_to_f64(B.output_to_numpy(g, p_id, outs[1]))
    o_gpu = bf16_to_f64(B.output_to_numpy(g, g.outputs[0], outs[0]))
    c.close()
    ref = interp.run(g, w.feeds)
    assert np.abs(p_gpu - ref[p_id]).max() <= 4e-3 and np.abs(p_gpu.sum(-1) - 1.0).max() <= 2e-2
    assert np.abs(o_gpu - ref[g.outputs[0]]).max() <= 2e-2


def test_mha_int8_all_128_inputs_give_zero_point(B):
    w = W.mha_int8(batch=1, heads=2, seq=128, head_dim=64, all_value=128)
    got, _ = run_gpu(B, w)
    assert (got == 128).all()


def test_mha_int8_full_size_sampled_heads(B):
    w = W.mha_int8()                                      # B64 S384 H16 D64
    got, plan = run_gpu(B, w)
    assert "tcgen05" in plan
    g = w.graph
    for b0 in (0, 9, 18, 27, 37, 46, 55, 63):             # eight sequences spread over the batch, all 16 heads each
        sub = W.mha_int8(batch=1, heads=16)
        for a, bb in zip(sub.graph.inputs, g.inputs):
            sub.feeds[a] = w.feeds[bb][b0:b0 + 1]
        check_int8_attention(got[b0:b0 + 1], oracle(sub))
    # a property that holds at any size: every output is a valid code and not all saturated
    assert got.min() >= 0 and got.max() <= 255 and 100 < got.mean() < 156


# ------------------------------------------------------------------------------ determinism
def test_repeated_runs_are_bitwise_identical(B):
    for w in (W.mlp_f32(), W.mha_bf16(batch=4), W.mha_int8(batch=1, heads=4), W.ffn_bf16(tokens=512)):
        res, _ = run_gpu(B, w, n_runs=3)
        assert np.array_equal(res[0], res[1]) and np.array_equal(res[0], res[2])


@pytest.mark.parametrize("which", ["chain", "chain_folded_tail", "chain_in_one_cluster", "two_layers_one_launch", "attention"])
def test_captured_executes_replay_correctly(B, which):
    # gc_execute after the first call is a pure sequence of kernel launches: captured into a CUDA graph and replayed,
    # it must give the same results, also for the kernels that synchronise through counters in global memory
    # (their epochs live on the device, not in the launch parameters), and with new input contents per replay
    import torch
    if which == "chain":
        w = W.mlp_int8(batch=128, dims=(479, 1024, 512, 32), final="none", per_channel=True, x_zp=3, act_zp=2)
    elif which == "chain_in_one_cluster":
        w = W.mlp_f32()
    elif which == "chain_folded_tail":
        w = W.mlp_int8(batch=128, dims=(479, 1024, 256, 1), final="none", per_channel=True, x_zp=3, act_zp=2)
    elif which == "two_layers_one_launch":
        w = W.ffn_bf16(tokens=4900, d_model=1024, d_ff=1024)
    else:
        w = W.mha_int8(batch=2, heads=4, seq=384, head_dim=64)
    c = B.CompiledPartition(w.graph, 0)
    if which == "chain_in_one_cluster":
        assert "inside one cluster" in c.plan
    if which == "chain_folded_tail":
        assert "folded into the finishing step" in c.plan
    ins = B.device_inputs(w)
    outs = B.device_outputs(w.graph)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        c.execute(ins, outs, s.cuda_stream)                 # first call: constant preprocessing, outside the graph
    s.synchronize()
    first = B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]).copy()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for _ in range(3):
            c.execute(ins, outs, s.cuda_stream)
    for _ in range(2):
        outs[0].zero_()
        g.replay()
        torch.cuda.synchronize()
        assert np.array_equal(B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]), first)
    # new activations in the same buffer, one more replay, then an ordinary call again
    x_pos = 0
    x_id = w.graph.inputs[x_pos]
    new_x = np.roll(w.feeds[x_id], 1, axis=0).copy()
    ins[x_pos].copy_(torch.from_numpy(np.ascontiguousarray(new_x).view(np.uint8).reshape(-1)))
    g.replay()
    torch.cuda.synchronize()
    replayed = B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]).copy()
    c.execute(ins, outs)
    c.query_status()
    torch.cuda.synchronize()
    assert np.array_equal(B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]), replayed)
    assert not np.array_equal(replayed, first)
    w.feeds[x_id] = new_x
    ref = oracle(w)
    if which in ("chain", "chain_folded_tail"):
        assert np.array_equal(replayed, ref)
    elif which == "chain_in_one_cluster":
        assert np.abs(replayed.astype(np.float64) - ref).max() <= 5e-3 * np.abs(ref).max()
    elif which == "attention":
        check_int8_attention(replayed, ref)
    else:
        assert np.abs(bf16_to_f64(replayed) - ref).max() <= 2e-2
    c.close()


def test_bounded_wait_gives_up_records_a_code_and_leaves_the_context_usable(B):
    # the error path every kernel wait has: a wait that cannot be satisfied ends after its time limit, the kernel
    # writes its code and returns; the context keeps working
    import time
    import torch
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    B.gc_selftest_bounded_wait(torch.cuda.current_stream(0).cuda_stream, status.data_ptr(), 20000)   # 20 ms
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert int(status.item()) != 0
    assert 0.015 <= dt < 1.0
    w = W.single_matmul("u8", "s8", 128, 128, 64, seed=1)
    got, _ = run_gpu(B, w)
    assert np.array_equal(got.astype(np.int64), oracle(w))


def test_host_buffer_entry_point_matches_device_entry_point(B):
    import torch
    w = W.mlp_int8()
    got, _ = run_gpu(B, w)
    c = B.CompiledPartition(w.graph, 0)
    ins = [np.ascontiguousarray(w.feeds[t]) for t in w.graph.inputs]
    out = np.zeros((128, 1), dtype=np.float32)
    for _ in range(2):
        c.execute_host(ins, [out])
        assert np.array_equal(out, got)
    c.close()
    torch.cuda.synchronize()


def test_overlapped_host_entry_point_batches_in_flight(B):
    # different activations per staging slot, the constants shared; each slot's result must be its own batch's
    import torch
    ws = []
    for s in range(7):
        w = W.mlp_int8(batch=128, dims=(479, 256, 64, 1), seed=1)      # same weights, own activations
        x = w.graph.inputs[0]
        w.feeds[x] = np.random.default_rng(100 + s).integers(0, 256, size=w.feeds[x].shape).astype(np.uint8)
        ws.append(w)
    g = ws[0].graph
    c = B.CompiledPartition(g, 0)
    ns = c.HOST_SLOTS
    assert 2 <= ns < len(ws)
    refs = [interp.run(w.graph, w.feeds)[w.graph.outputs[0]] for w in ws]
    assert not np.array_equal(refs[0], refs[1])
    consts = [np.ascontiguousarray(ws[0].feeds[t]) for t in g.inputs[1:]]
    pinned_in = [torch.empty(ws[0].feeds[g.inputs[0]].nbytes, dtype=torch.uint8).pin_memory() for _ in range(ns)]
    pinned_out = [torch.empty(g.tensors[g.outputs[0]].nbytes, dtype=torch.uint8).pin_memory() for _ in range(ns)]
    got = [None] * len(ws)

    def collect(i):
        c.host_wait(i % ns)
        got[i] = pinned_out[i % ns].numpy().view(np.float32).reshape(refs[i].shape).copy()

    for i, w in enumerate(ws):
        if i >= ns:
            collect(i - ns)
        pinned_in[i % ns].numpy()[:] = np.ascontiguousarray(w.feeds[g.inputs[0]]).view(np.uint8).reshape(-1)
        c.execute_host_async(i % ns, [pinned_in[i % ns]] + consts, [pinned_out[i % ns]])
    # a slot in flight is refused, and so is a slot the staging area does not have
    with pytest.raises(B.GcError):
        c.execute_host_async((len(ws) - 1) % ns, [pinned_in[0]] + consts, [pinned_out[0]])
    with pytest.raises(B.GcError):
        c.execute_host_async(ns, [pinned_in[0]] + consts, [pinned_out[0]])
    for i in range(len(ws) - ns, len(ws)):
        collect(i)
    for i in range(len(ws)):
        assert np.abs(got[i] - refs[i]).max() <= 2e-6, i
    # the synchronous call still works on the same object afterwards
    out = np.zeros(refs[0].shape, dtype=np.float32)
    c.execute_host([np.ascontiguousarray(ws[3].feeds[g.inputs[0]])] + consts, [out])
    assert np.array_equal(out, got[3])
    c.close()
    torch.cuda.synchronize()


def test_overlapped_host_entry_point_with_pageable_buffers_and_attention(B):
    # pageable numpy buffers (the copies are then synchronous inside the call, the results the same) on the attention
    # pattern: every slot in flight at once, each with its own Q
    import torch
    ws = [W.mha_bf16(batch=2, heads=3, seed=s) for s in (1, 2, 3)]
    g = ws[0].graph
    c = B.CompiledPartition(g, 0)
    ns = c.HOST_SLOTS
    ins = [[np.ascontiguousarray(w.feeds[t]) for t in g.inputs] for w in ws[:ns]]
    outs = [np.zeros(g.tensors[g.outputs[0]].dims, dtype=np.uint16) for _ in range(ns)]
    for k in range(ns):
        c.execute_host_async(k, ins[k], [outs[k]])
    for k in range(ns):
        c.host_wait(k)
        ref = interp.run(ws[k].graph, ws[k].feeds)[ws[k].graph.outputs[0]]
        assert np.abs(bf16_to_f64(outs[k]) - ref).max() <= 2e-2
    c.host_wait(0)                                          # waiting for an idle slot returns at once
    c.close()
    torch.cuda.synchronize()


def test_host_buffer_entry_point_picks_up_a_constant_at_a_new_host_address(B):
    # a constant that arrives at a new host address is copied to the same staging address: the weights must be
    # preprocessed again, not only the bias re-read
    import torch
    w1 = W.mlp_int8(batch=64, dims=(200, 128, 64, 1), seed=1)
    w2 = W.mlp_int8(batch=64, dims=(200, 128, 64, 1), seed=2)
    c = B.CompiledPartition(w1.graph, 0)
    out = np.zeros((64, 1), dtype=np.float32)
    ins1 = [np.ascontiguousarray(w1.feeds[t]) for t in w1.graph.inputs]
    ins2 = [np.ascontiguousarray(w2.feeds[t]) for t in w2.graph.inputs]
    mixed = [ins1[0]] + ins2[1:]                            # same activations, every constant at a new address
    ref1 = interp.run(w1.graph, w1.feeds)[w1.graph.outputs[0]]
    feeds = dict(w2.feeds)
    feeds[w2.graph.inputs[0]] = w1.feeds[w1.graph.inputs[0]]
    ref_mixed = interp.run(w2.graph, feeds)[w2.graph.outputs[0]]
    assert not np.allclose(ref1, ref_mixed)
    for ins, ref in ((ins1, ref1), (mixed, ref_mixed), (ins1, ref1)):
        c.execute_host(ins, [out])
        assert np.abs(out - ref).max() <= 2e-6
    c.close()
    torch.cuda.synchronize()


def test_invalidate_constants_repacks_a_weight_rewritten_in_place(B):
    import torch
    w = W.mlp_int8(batch=128, dims=(479, 256, 64, 1), final="none")
    c = B.CompiledPartition(w.graph, 0)
    ins = B.device_inputs(w)
    outs = B.device_outputs(w.graph)
    c.execute(ins, outs)
    first = B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]).copy()
    assert np.array_equal(first, oracle(w))
    wid = w.graph.inputs[1]                                 # first-layer weight: new contents at the same address
    w.feeds[wid] = np.ascontiguousarray(w.feeds[wid][::-1])
    ins[1].copy_(torch.from_numpy(w.feeds[wid].view(np.uint8).reshape(-1)))
    c.execute(ins, outs)                                    # the cache is keyed by address: still the old weight
    assert np.array_equal(B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]), first)
    c.invalidate_constants()
    c.execute(ins, outs)
    c.query_status()
    ref = oracle(w)
    assert not np.array_equal(ref, first)
    assert np.array_equal(B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]), ref)
    c.close()


@pytest.mark.parametrize("which", ["chain", "two_layers_one_launch"])
def test_object_is_usable_again_after_a_reported_timeout(B, which):
    # A kernel whose bounded wait expired leaves a code in the status word and its counters mid-count.  Injected from
    # the host (no kernel is made to wait): a non-zero status word and garbage in the counters, written with copies.
    # gc_query_status must report the timeout once, reset the device state, and the next execute must be correct.
    import torch
    if which == "chain":
        w = W.mlp_int8(batch=128, dims=(479, 1024, 512, 32), final="none")
    else:
        w = W.ffn_bf16(tokens=4900, d_model=1024, d_ff=1024)
    c = B.CompiledPartition(w.graph, 0)
    assert ("fused chain" in c.plan) if which == "chain" else ("one launch" in c.plan)
    ins = B.device_inputs(w)
    outs = B.device_outputs(w.graph)
    c.execute(ins, outs)
    c.query_status()
    good = B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]).copy()
    torch.cuda.synchronize()
    ws32 = c._ws[:256].view(torch.int32)
    ws32[0] = 0x102                                         # status word: "a wait expired"
    ws32[16] = 12345                                        # grid-barrier counter of the chain kernel: not a multiple of a launch's count
    # (the fused two-layer launch keeps its epoch and per-tile counters elsewhere in the workspace; the reset zeroes
    # them too, which the correct result of the next execute shows: a stale count against a zeroed epoch would not
    # let its second-layer tiles start)
    torch.cuda.synchronize()
    with pytest.raises(B.GcError) as e:
        c.query_status()
    assert e.value.status == B.GC_ERR_TIMEOUT
    c.query_status()                                        # reported once; the state has been reset
    outs[0].zero_()
    c.execute(ins, outs)
    c.query_status()
    assert np.array_equal(B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]), good)
    c.close()


def test_misaligned_pointer_is_rejected(B):
    w = W.mlp_f32()
    c = B.CompiledPartition(w.graph, 0)
    ins = B.device_inputs(w)
    outs = B.device_outputs(w.graph)
    ptrs = [t.data_ptr() for t in ins]
    ptrs[0] += 4
    with pytest.raises(B.GcError) as e:
        c.execute_ptrs(ptrs, [outs[0].data_ptr()], 0)
    assert e.value.status == B.GC_ERR_ALIGNMENT
    c.close()
