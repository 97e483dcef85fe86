"""Host-side checks that need no GPU: the C-ABI library loads and exports every symbol the header
declares, argument validation, pattern formation and planning (plan-only compile)."""
import os
import re

import pytest

from paper_2301_01333_b200 import binding as B
from paper_2301_01333_b200 import build as gc_build
from paper_2301_01333_b200 import workloads as W
from paper_2301_01333_b200.graph import Graph

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    gc_build.build()


def test_library_exports_every_declared_symbol():
    text = open(os.path.join(ROOT, "include", "gc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(gc_[a-z0-9_]+)\s*\(", text))
    assert declared == set(B.EXPORTS)
    lib = B.load_library()
    for name in declared:
        assert hasattr(lib, name), name
    assert "sm_100a" in B.gc_version()


def plan(g, **kw):
    return B.CompiledPartition(g, device=B.GC_DEVICE_PLAN_ONLY, **kw)


def test_plans_for_the_five_configs():
    c1 = plan(W.mlp_f32().graph)
    assert c1.plan.count("tcgen05.tf32") == 3 and "+pack" in c1.plan
    c2 = plan(W.mlp_int8().graph)
    assert c2.plan.count("tcgen05.i8") == 4 and c2.plan.count("cuda-core") == 1      # 256 -> 1 is a GEMV
    c5 = plan(W.ffn_bf16().graph)
    assert c5.plan.count("tcgen05.bf16") == 2 and c5.plan.count("block_n=256") == 2
    assert c5.launches == 1 and "one launch" in c5.plan          # both GEMMs in one persistent launch
    assert plan(W.ffn_bf16().graph, no_chain_fusion=True).launches == 2
    c3 = plan(W.mha_bf16().graph)
    assert "attention bf16" in c3.plan and "tcgen05" in c3.plan
    c4 = plan(W.mha_int8().graph)
    assert "attention int8" in c4.plan and "S=384" in c4.plan and "tcgen05" in c4.plan
    # workspace: prepacked weights + two reused activation buffers (+ padded input copy)
    assert c5.workspace_bytes >= 16 * 2 ** 20 + 64 * 2 ** 20
    assert c2.workspace_bytes < 4 * 2 ** 20
    for c in (c1, c2, c3, c4, c5):
        c.close()


def test_force_generic_and_ragged_shapes_use_cuda_core_kernels():
    c = plan(W.mlp_int8().graph, force_generic=True)
    assert "tcgen05" not in c.plan
    c = plan(W.mlp_f32(batch=3, dims=(5, 7, 3)).graph)
    assert "tcgen05" not in c.plan           # N not a multiple of 16
    c = plan(W.mha_bf16(batch=1, heads=1, seq=48, head_dim=32).graph)
    assert "cuda-core" in c.plan


def test_plan_only_cannot_execute():
    c = plan(W.mlp_f32().graph)
    with pytest.raises(B.GcError) as e:
        B.gc_execute(c._comp, 0, [16] * 7, [16])
    assert e.value.status == B.GC_ERR_STATE


def test_partition_create_rejects_bad_graphs():
    g = W.mlp_f32(batch=4, dims=(8, 16)).graph
    g.ops[0].inputs = (g.ops[0].inputs[0], 999)
    with pytest.raises(B.GcError) as e:
        B.gc_partition_create(g)
    assert e.value.status == B.GC_ERR_INVALID_ARG
    g = W.mlp_f32(batch=4, dims=(8, 16)).graph
    g.tensors[g.ops[0].output].dims = (4, 17)
    with pytest.raises(B.GcError) as e:
        B.gc_partition_create(g)
    assert e.value.status == B.GC_ERR_SHAPE
    g = W.mlp_f32(batch=4, dims=(8, 16)).graph
    g.ops.reverse()                                  # not topological
    with pytest.raises(B.GcError) as e:
        B.gc_partition_create(g)
    assert e.value.status == B.GC_ERR_INVALID_ARG
    g = W.mlp_f32(batch=4, dims=(8, 16)).graph
    g.outputs = [g.inputs[0] + 1000]
    with pytest.raises(B.GcError):
        B.gc_partition_create(g)


def test_compile_rejects_unsupported_patterns():
    # softmax alone
    g = Graph()
    x = g.input("f32", (4, 8))
    g.mark_output(g.op("softmax", (x,), g.tensor("f32", (4, 8))))
    with pytest.raises(B.GcError) as e:
        plan(g)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
    # weights that are not constant
    w = W.mlp_f32(batch=4, dims=(8, 16))
    w.graph.tensors[w.graph.inputs[1]].is_constant = False
    with pytest.raises(B.GcError) as e:
        plan(w.graph)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
    # an intermediate that is also an output
    w = W.mlp_f32(batch=4, dims=(8, 16, 16))
    w.graph.outputs.append(w.graph.ops[2].output)
    with pytest.raises(B.GcError) as e:
        plan(w.graph)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
    # no such device
    p = B.gc_partition_create(W.mlp_f32().graph)
    with pytest.raises(B.GcError):
        B.gc_compile(p, 99)
    B.gc_partition_destroy(p)


def test_per_channel_scales_and_zero_points_plan_on_tensor_cores_and_bad_uses_are_refused():
    c = plan(W.mlp_int8(per_channel=True, x_zp=12, act_zp=5).graph)
    assert c.plan.count("tcgen05.i8") == 4          # a non-zero activation zero point no longer leaves the tcgen05 path
    # scales along the reduction axis
    w = W.mlp_int8(batch=4, dims=(16, 16), per_channel=True)
    w.graph.tensors[w.graph.inputs[1]].channel_axis = 0
    with pytest.raises(B.GcError) as e:
        plan(w.graph)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
    # scales on an activation
    w = W.mlp_int8(batch=4, dims=(16, 16))
    x = w.graph.tensors[w.graph.inputs[0]]
    x.channel_scales, x.channel_axis = (0.1,) * 16, 1
    with pytest.raises(B.GcError) as e:
        B.gc_partition_create(w.graph)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
    # a non-positive scale
    w = W.mlp_int8(batch=4, dims=(16, 16), per_channel=True)
    t = w.graph.tensors[w.graph.inputs[1]]
    t.channel_scales = (0.0,) + t.channel_scales[1:]
    with pytest.raises(B.GcError) as e:
        B.gc_partition_create(w.graph)
    assert e.value.status == B.GC_ERR_INVALID_ARG


def test_tile_schedules_of_the_two_layer_launch_over_a_range_of_shapes():
    # host logic only: the scheduler simulates the step and must never produce a list much longer than a perfect split
    # of the work when there is plenty of it, and must not fuse when a layer is too small for CTA pairs
    import re
    for tokens, d_model, d_ff, fused in [(8192, 1024, 4096, True), (16384, 1024, 4096, True), (8192, 2048, 8192, True),
                                         (9500, 512, 1008, True), (4900, 1024, 1024, True), (8192, 1024, 1024, True),
                                         (2048, 1024, 4096, False), (6400, 512, 1008, False)]:
        c = plan(W.ffn_bf16(tokens=tokens, d_model=d_model, d_ff=d_ff).graph)
        m = re.search(r"one launch, (\d+) clusters, .*longest list (\d+) of ([\d.]+) k-blocks ideal", c.plan)
        assert (m is not None) == fused, (tokens, d_model, d_ff, c.plan)
        if not fused:
            assert c.launches == 2
            continue
        assert c.launches == 1
        longest, ideal = int(m.group(2)), float(m.group(3))
        assert longest >= ideal
        if ideal >= 200:
            assert longest <= 1.03 * ideal, (tokens, d_model, d_ff, longest, ideal)


def test_reference_arm_of_the_bench_prints_the_contract_line_without_a_gpu():
    # `bench.py --impl reference` times the oracle on the host cores: no GPU, one JSON line with the contract's keys
    import json
    import subprocess
    import sys
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1",
                        "--workload", "c1"], capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("impl", "metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in line, key
    assert line["impl"] == "reference" and line["steps"] == 1 and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"] == "c1"


def test_max_free_softmax_is_planned_only_under_a_compile_time_score_bound():
    # Section VII's fast softmax: 8-bit operands, no mask, |score| log2(e) <= 60 from the ranges and the folded scales
    ok = plan(W.mha_int8(batch=2, heads=2, seq=384, s_qkv=0.01, with_mask=False).graph)
    assert "softmax=max-free" in ok.plan
    assert "max-free" not in plan(W.mha_int8(batch=2, heads=2, seq=384, s_qkv=0.01, with_mask=False).graph, exact_max_softmax=True).plan
    assert "max-free" not in plan(W.mha_int8(batch=2, heads=2, seq=384, s_qkv=0.03, with_mask=False).graph).plan
    assert "max-free" not in plan(W.mha_int8(batch=2, heads=2, seq=384, s_qkv=0.01).graph).plan          # masked
    assert "max-free" not in plan(W.mha_int8(batch=2, heads=2, seq=512, s_qkv=0.01, with_mask=False).graph).plan   # streaming kernel
    assert "max-free" not in plan(W.mha_bf16(batch=2, heads=2, seq=128).graph).plan
