"""The allocation-free entry point (gc_matmul_s32_noalloc) against the regular compile/execute path.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
It serves callers that may not call cudaMalloc (fixed memory plans, allocator-owned devices), so its
scratch is a fixed array inside the library that every call shares; the second call below runs a
different shape right after the first to show that what the first call left behind does no harm."""
import numpy as np
import pytest

from oracle import interp
from paper_2301_01333_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _regular_path(B, w):
    import torch
    c = B.CompiledPartition(w.graph, 0)
    ins = B.device_inputs(w)
    outs = B.device_outputs(w.graph)
    c.execute(ins, outs)
    c.query_status()
    torch.cuda.synchronize()
    got = B.output_to_numpy(w.graph, w.graph.outputs[0], outs[0]).copy()
    c.close()
    return got


def test_noalloc_matmul_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2301_01333_b200 import build as gc_build
    gc_build.build()
    from paper_2301_01333_b200 import binding as B

    assert B.gc_noalloc_scratch_bytes() == 1 << 20
    stream = torch.cuda.current_stream(0).cuda_stream
    # two calls in a row, the second smaller and with a zero point, reusing the shared scratch
    for (m, k, n, zp, seed) in [(96, 479, 1024, 0, 1), (33, 130, 48, 7, 2)]:
        w = W.single_matmul("u8", "s8", m, k, n, seed=seed, a_zp=zp)
        expect = _regular_path(B, w)
        a_dev, w_dev = B.device_inputs(w)
        out = torch.full((m * n,), -1, dtype=torch.int32, device="cuda:0")
        B.gc_matmul_s32_noalloc(stream, a_dev.data_ptr(), w_dev.data_ptr(), out.data_ptr(), m, k, n, zp)
        torch.cuda.synchronize()
        got = out.cpu().numpy().reshape(m, n)
        assert np.array_equal(got, expect)          # integer path: bit-exact, the tolerance the other tests use
        # and directly against the oracle's definition of the same matmul
        assert np.array_equal(got.astype(np.int64), interp.run(w.graph, w.feeds)[w.graph.outputs[0]])

    # beyond the built-in scratch: refused with a clear message, nothing launched
    with pytest.raises(B.GcError) as e:
        B.gc_matmul_s32_noalloc(stream, a_dev.data_ptr(), w_dev.data_ptr(), out.data_ptr(), 8, 4096, 1024, 0)
    assert e.value.status == B.GC_ERR_UNSUPPORTED and "1 MiB" in str(e.value)
    # a zero point no u8 operand can have, and a reduction long enough to leave s32: refused as well
    for bad_zp in (-1, 256):
        with pytest.raises(B.GcError) as e:
            B.gc_matmul_s32_noalloc(stream, a_dev.data_ptr(), w_dev.data_ptr(), out.data_ptr(), 8, 64, 16, bad_zp)
        assert e.value.status == B.GC_ERR_INVALID_ARG
    with pytest.raises(B.GcError) as e:
        B.gc_matmul_s32_noalloc(stream, a_dev.data_ptr(), w_dev.data_ptr(), out.data_ptr(), 8, 70000, 8, 0)
    assert e.value.status == B.GC_ERR_UNSUPPORTED
