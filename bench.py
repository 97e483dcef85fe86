#!/usr/bin/env python
"""Benchmark of the fused-subgraph executor on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c5] [--impl reference]

A step is one gc_execute of one compiled subgraph on one batch of synthetic input.  The headline
workload (default c5, the large-batch bf16 FFN - the tensor-bound config) gives `value`; the other four
configs are timed the same way and reported under "configs".  Inputs are resident in HBM before the
timed region; steps rotate through enough independent replicas (own weights, workspace, inputs,
outputs) that their total footprint exceeds L2, so every step streams from HBM.  `e2e` repeats the
measurement through gc_execute_host with pinned host buffers (copies inside the timed region).
With N > 1 (torchrun) every rank runs the same per-GPU work on its own GPU: no data-path collective,
weak scaling; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2301_01333_b200 import workloads as W  # noqa: E402

L2_BYTES = 126 * 2 ** 20
NOMINAL = {"bf16_tflops": 2250.0, "hbm_gbs": 8000.0}
FALLBACK = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# tensor peak of each config's MMA kind relative to dense bf16 (nominal ratios)
KIND_RATIO = {"c1": 0.5, "c2": 2.0, "c3": 1.0, "c4": 2.0, "c5": 1.0}
UNIT = {"c1": "TFLOP/s", "c2": "TOP/s", "c3": "TFLOP/s", "c4": "TOP/s", "c5": "TFLOP/s"}
DTYPE = {"c1": "tf32", "c2": "u8xs8->s32", "c3": "bf16", "c4": "u8xu8->s32", "c5": "bf16"}
# c5 runs for about a second so that the clocks settle under the power cap (the regime the "sustained" peak
# was measured in) and the clock sampler sees the timed region
DEFAULT_STEPS = {"c1": 2000, "c2": 2000, "c3": 500, "c4": 100, "c5": 8000}
GRAPH_STEPS = {"c1": 256, "c2": 256, "c3": 256, "c4": 50, "c5": 50}     # executes captured into one CUDA graph
# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum) from the newest ncu
# capture of each, which TRAFFIC_SOURCE names; a profiler figure cannot be re-measured inside an untimed run, so the
# line carries the capture it comes from.  c5: one launch per step, the 64 MiB hidden tensor is written back.
TRAFFIC_BYTES_PER_LAUNCH = {"c5": 126.65e6, "c3": 18.9e6, "c4": 84.8e6}
TRAFFIC_SOURCE = {"c5": "profiles/gemm_tc2_bf16_c5_ffn_one_launch.md (capture of the one-launch FFN, 70.0 MB read + 56.7 MB written)",
                  "c3": "profiles/sdpa_small_c3_attention.md (reads; the 6.3 MB of output were still in the L2 when the launch ended)", "c4": "profiles/sdpa_tc_c3_c4_attention.md"}
DOMINANT_KERNEL = {"c1": "mlp_cluster_kernel (tf32, whole chain inside one thread-block cluster)", "c2": "mlp_chain_kernel<i8>", "c3": "sdpa_small_kernel (bf16, one unit per CTA)",
                   "c4": "sdpa_tc_kernel<int8>", "c5": "gemm_tc2_kernel<bf16, bf16 out> (both FFN GEMMs in one launch)"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows = []
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


class Replica:
    def __init__(self, B, w, seed_shift, device, **opts):
        import torch
        self.c = B.CompiledPartition(w.graph, device, **opts)
        self.ins = B.device_inputs(w, device)
        if seed_shift:   # distinct activations per replica (weights may repeat: only addresses matter)
            for t, tid in zip(self.ins, w.graph.inputs):
                if not w.graph.tensors[tid].is_constant and w.graph.tensors[tid].dtype in ("u8", "s8"):
                    t.add_(seed_shift)
        self.outs = B.device_outputs(w.graph, device)
        self.bytes = sum(t.numel() for t in self.ins) + sum(t.numel() for t in self.outs) + self.c.workspace_bytes
        self.torch = torch

    def step(self, stream):
        self.c.execute(self.ins, self.outs, stream)


def time_config(B, name, steps, warmup, device, shard=None, **opts):
    """Builds the rotating replicas of one config (total footprint above the L2 size) and warms them up.
    shard = (first, count): this rank's units of the config's one batch instead of the whole batch."""
    import torch
    w = W.CONFIGS[name]()
    if shard is not None:
        w = W.shard_config(name, w, shard[0], shard[1])
    stream = torch.cuda.current_stream(device).cuda_stream
    first = Replica(B, w, 0, device, **opts)
    n_rep = int(min(64, max(2, -(-int(1.25 * L2_BYTES) // first.bytes))))
    reps = [first] + [Replica(B, w, i + 1, device, **opts) for i in range(n_rep - 1)]
    for r in reps:                      # first call prepacks the constant weights: outside the timing
        r.step(stream)
    torch.cuda.synchronize(device)
    for i in range(max(warmup, 3)):
        reps[i % n_rep].step(stream)
    torch.cuda.synchronize(device)
    return w, reps, n_rep


def run_timed(reps, n_rep, steps, device, barrier):
    import torch
    stream = torch.cuda.current_stream(device).cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize(device)
    e0.record()
    for i in range(steps):
        reps[i % n_rep].step(stream)
    e1.record()
    torch.cuda.synchronize(device)
    barrier()
    return e0.elapsed_time(e1)          # ms


def library_two_gemms_us(w, n_rep, steps, device):
    """Context for the FFN config, not a baseline of the path: the two GEMMs of the block as plain library calls
    (torch.matmul = cuBLAS, bf16, no bias, no GELU, hidden tensor through memory), on random data of the same shapes,
    rotating through as many buffer sets as the timed run rotates replicas, timed the same way."""
    import torch
    g = w.graph
    shapes = [g.tensors[t].dims for t in g.inputs]
    tokens, d_model = shapes[0]
    d_ff = [s for s in shapes[1:] if len(s) == 2][0]
    d_ff = d_ff[1] if d_ff[0] == d_model else d_ff[0]
    dev = f"cuda:{device}"
    sets = []
    for _ in range(n_rep):
        sets.append((torch.randn(tokens, d_model, device=dev, dtype=torch.bfloat16),
                     torch.randn(d_model, d_ff, device=dev, dtype=torch.bfloat16) * 0.03,
                     torch.randn(d_ff, d_model, device=dev, dtype=torch.bfloat16) * 0.03,
                     torch.empty(tokens, d_ff, device=dev, dtype=torch.bfloat16),
                     torch.empty(tokens, d_model, device=dev, dtype=torch.bfloat16)))
    def step(i):
        x, w1, w2, h, y = sets[i % n_rep]
        torch.matmul(x, w1, out=h)
        torch.matmul(h, w2, out=y)
    for i in range(max(3, n_rep)):
        step(i)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize(device)
    del sets
    return e0.elapsed_time(e1) * 1e3 / steps


def library_sdpa_us(w, n_rep, steps, device):
    """Context for the bf16 attention config, not a baseline of the path: torch's scaled_dot_product_attention (whatever
    fused library kernel it selects) on random data of the same shapes with an additive mask of the same form, rotating
    through as many buffer sets as the timed run rotates replicas, timed the same way."""
    import torch
    import torch.nn.functional as F
    g = w.graph
    q_dims = g.tensors[g.inputs[0]].dims                     # [B, H, S, D]
    Bn, H, S, D = q_dims
    dev = f"cuda:{device}"
    sets = []
    for _ in range(n_rep):
        q, k, v = (torch.randn(Bn, H, S, D, device=dev, dtype=torch.bfloat16) for _ in range(3))
        mask = torch.zeros(Bn, 1, 1, S, device=dev, dtype=torch.bfloat16)
        mask[:, :, :, S - S // 8:] = float("-inf")
        sets.append((q, k, v, mask))
    def step(i):
        q, k, v, mask = sets[i % n_rep]
        return F.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=0.125)
    for i in range(max(3, n_rep)):
        step(i)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        step(i)
    e1.record()
    torch.cuda.synchronize(device)
    del sets
    return e0.elapsed_time(e1) * 1e3 / steps


def launch_floor_us(B, device, steps=2000):
    """Back-to-back launches of the smallest partition (a 16x16x16 matmul on one CTA): the per-launch cost that
    bounds the small-batch configs from below however fast their kernels are."""
    import torch
    w = W.single_matmul("u8", "s8", 16, 16, 16)
    r = Replica(B, w, 0, device)
    stream = torch.cuda.current_stream(device).cuda_stream
    for _ in range(20):
        r.step(stream)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        r.step(stream)
    e1.record()
    torch.cuda.synchronize(device)
    n = r.c.launches
    r.c.close()
    return e0.elapsed_time(e1) * 1e3 / steps / max(n, 1)


# exp2 evaluations per second of the special-function units: 16 per clock per SM (4 per sub-partition) x 148 SMs
def exp_peak_per_s(sm_mhz):
    return 148 * 16 * sm_mhz * 1e6


def softmax_scores(w):
    """Number of attention scores (one exponential each) of an attention workload, else 0."""
    for op in w.graph.ops:
        if op.kind == "softmax":
            return int(np.prod(w.graph.tensors[op.inputs[0]].dims))
    return 0


def sweep_cases():
    """The shapes of the evaluation's workload table (Section VII, Table I): MLP-1 / MLP-2 at batch 32..512 and
    MHA-1..4 at batch 32..128, in the 8-bit scheme and in this build's float types (tf32 MLP, bf16 attention)."""
    cases = []
    for b in (32, 64, 128, 256, 512):
        cases.append((f"MLP-1 int8 b{b}", lambda b=b: W.mlp_int8(batch=b, dims=(13, 512, 256, 128), final="none")))
        cases.append((f"MLP-1 f32 b{b}", lambda b=b: W.mlp_f32(batch=b)))
        cases.append((f"MLP-2 int8 b{b}", lambda b=b: W.mlp_int8(batch=b)))
        cases.append((f"MLP-2 f32 b{b}", lambda b=b: W.mlp_f32(batch=b, dims=(479, 1024, 1024, 512, 256, 1))))
    for tag, seq, heads, hd in (("MHA-1", 128, 8, 96), ("MHA-2", 128, 12, 64), ("MHA-3", 384, 8, 128), ("MHA-4", 512, 16, 64)):
        for b in (32, 64, 128):
            cases.append((f"{tag} int8 b{b}", lambda b=b, s=seq, h=heads, d=hd: W.mha_int8(batch=b, heads=h, seq=s, head_dim=d)))
            cases.append((f"{tag} bf16 b{b}", lambda b=b, s=seq, h=heads, d=hd: W.mha_bf16(batch=b, heads=h, seq=s, head_dim=d)))
    return cases


def run_plain_gemm(B, device, peaks):
    """A plain 8192^3 bf16 GEMM through the same library, timed the way the measured cuBLAS peaks were (best of 10
    single calls; back-to-back calls for about 3 s), next to those peaks: how the GEMM kernel alone compares."""
    import torch
    w = W.plain_gemm_bf16()
    r = Replica(B, w, 0, device)
    stream = torch.cuda.current_stream(device).cuda_stream
    for _ in range(3):
        r.step(stream)
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = 1e30
    for _ in range(10):
        e0.record()
        r.step(stream)
        e1.record()
        torch.cuda.synchronize(device)
        best = min(best, e0.elapsed_time(e1))
    time.sleep(2.0)
    n = int(3000.0 / best)
    e0.record()
    for _ in range(n):
        r.step(stream)
    e1.record()
    torch.cuda.synchronize(device)
    sustained = e0.elapsed_time(e1) / n
    r.c.query_status()
    out = {"graph": w.name, "kernel": r.c.plan.strip().splitlines()[-1].strip(), "burst_us": best * 1e3,
           "burst_tflops": w.ops / (best * 1e-3) / 1e12, "sustained_us": sustained * 1e3, "sustained_calls": n,
           "sustained_tflops": w.ops / (sustained * 1e-3) / 1e12,
           "measured_library_peak_tflops": {"burst": peaks.get("bf16_tflops"), "sustained": peaks.get("bf16_tflops_sustained")}}
    out["frac_of_burst_peak"] = out["burst_tflops"] / peaks["bf16_tflops"]
    out["frac_of_sustained_peak"] = out["sustained_tflops"] / peaks["bf16_tflops_sustained"]
    r.c.close()
    return out


def run_sweep(B, device, peaks, only=""):
    """One line per shape: cold time (rotating replicas above the L2 size), kernels chosen, HBM-roofline time."""
    import torch
    out = []
    stream = torch.cuda.current_stream(device).cuda_stream
    for label, make in sweep_cases():
        if only and only not in label:
            continue
        w = make()
        first = Replica(B, w, 0, device)
        n_rep = int(min(32, max(2, -(-int(1.25 * L2_BYTES) // first.bytes))))
        reps = [first] + [Replica(B, w, i + 1, device) for i in range(n_rep - 1)]
        for r in reps:
            r.step(stream)
        torch.cuda.synchronize(device)
        # size the timed loop from one measured step: about 50 ms, at least 10 steps
        t1 = run_timed(reps, n_rep, 3, device, lambda: None) / 3
        steps = int(max(10, min(2000, 50.0 / max(t1, 1e-3))))
        us = run_timed(reps, n_rep, steps, device, lambda: None) * 1e3 / steps
        reps[0].c.query_status()
        kernels = sorted({tok for tok in reps[0].c.plan.replace("=", " ").split() if tok.startswith(("tcgen05", "cuda-core", "chain"))})
        out.append({"case": label, "graph": w.name, "us": us, "steps": steps, "replicas": n_rep, "launches": reps[0].c.launches,
                    "kernels": kernels, "ops": w.ops, "bytes": w.bytes, "t_hbm_us": w.bytes / (peaks["hbm_gbs"] * 1e9) * 1e6,
                    "tops": w.ops / (us * 1e-6) / 1e12})
        for r in reps:
            r.c.close()
        del reps, first
        torch.cuda.empty_cache()
    return out


def run_graph_replay(reps, n_rep, steps, device):
    """The same rotation of executes captured once into a CUDA graph and replayed (no per-call host work at all):
    microseconds per subgraph.  gc_execute after its first call only enqueues kernels, so it can be captured."""
    import torch
    s = torch.cuda.Stream(device)
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for i in range(steps):
            reps[i % n_rep].c.execute(reps[i % n_rep].ins, reps[i % n_rep].outs, s.cuda_stream)
    for _ in range(2):
        g.replay()
    torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        g.replay()
    e1.record()
    torch.cuda.synchronize(device)
    del g
    return e0.elapsed_time(e1) * 1e3 / (3 * steps)


def run_e2e(w, rep, steps, warmup, device):
    """End to end through the host-buffer entry points, pinned host buffers, copies inside the timed region.
    Returns (seconds per step with several batches in flight, seconds per step one batch at a time, h2d bytes, d2h bytes,
    whether both staging slots and the serial path returned identical bytes for the identical inputs).
    Overlapped: gc_execute_host_async on rotating staging slots; before a slot is reused gc_host_wait returns its
    outputs, so every step's input copy, execution and output copy happen inside the region - the copies of one batch
    run beside the execution and the copies of its neighbours.  Serial: gc_execute_host, which synchronises per call."""
    import torch
    g = w.graph
    host_in, host_out = [], []
    c = rep.c
    ns = c.HOST_SLOTS
    for slot in range(ns):
        ins = []
        for tid in g.inputs:
            a = np.ascontiguousarray(w.feeds[tid])
            if g.tensors[tid].is_constant and slot > 0:
                ins.append(host_in[0][len(ins)])              # constants: one host buffer (copied once)
            else:
                ins.append(torch.from_numpy(a.view(np.uint8).reshape(-1).copy()).pin_memory())
        host_in.append(ins)
        host_out.append([torch.empty(g.tensors[t].nbytes, dtype=torch.uint8).pin_memory() for t in g.outputs])
    h2d = sum(g.tensors[t].nbytes for t in g.inputs if not g.tensors[t].is_constant)
    d2h = sum(g.tensors[t].nbytes for t in g.outputs)

    def overlapped(n):
        for i in range(n):
            c.host_wait(i % ns)                                # the batch that used this slot ns steps ago
            c.execute_host_async(i % ns, host_in[i % ns], host_out[i % ns])
        for s in range(ns):
            c.host_wait(s)

    overlapped(max(3, warmup))
    torch.cuda.synchronize(device)
    t0 = time.perf_counter()
    overlapped(steps)
    torch.cuda.synchronize(device)
    dt_pipe = (time.perf_counter() - t0) / steps
    same = all(torch.equal(a, b) for k in range(1, ns) for a, b in zip(host_out[0], host_out[k]))
    for _ in range(max(3, warmup)):
        c.execute_host(host_in[0], host_out[0])
    torch.cuda.synchronize(device)
    t0 = time.perf_counter()
    for _ in range(steps):
        c.execute_host(host_in[0], host_out[0])
    torch.cuda.synchronize(device)
    dt_serial = (time.perf_counter() - t0) / steps
    same = same and all(torch.equal(a, b) for a, b in zip(host_out[0], host_out[1]))   # serial result in [0]
    return dt_pipe, dt_serial, h2d, d2h, same


def parity_check(B, name, w, rep):
    """Outside the timed region: the output one timed replica last produced against the oracle on the same inputs -
    every output for the small-batch chains, 256 sampled rows for the FFN, one sequence (all heads) for attention -
    at the tolerances of the parity tests.  Uses the oracle, so it belongs to the CPU-baseline leg."""
    from oracle import interp
    make, key, _ = W.CONFIG_UNITS[name]
    g = w.graph
    total = g.tensors[g.inputs[0]].dims[0]
    if name in ("c1", "c2"):
        idx = np.arange(total)
    elif name == "c5":
        idx = np.sort(np.random.default_rng(1).choice(total, size=min(256, total), replace=False))
    else:
        idx = np.array([total // 2])
    sub = make(**{key: len(idx)})
    for a, b in zip(sub.graph.inputs, g.inputs):
        src = w.feeds[b]
        sub.feeds[a] = np.ascontiguousarray(src[idx]) if (not g.tensors[b].is_constant and src.shape[0] == total) else src
    ref = interp.run(sub.graph, sub.feeds)[sub.graph.outputs[0]]
    got = B.output_to_numpy(g, g.outputs[0], rep.outs[0])[idx]
    if name == "c4":
        d = np.abs(got.astype(np.int64) - ref)
        err, frac = float(d.max()), float((d != 0).mean())
        ok = err <= 1 and frac <= 1e-3
        return {"rows": int(len(idx)), "unit": "sequences (all heads)", "max_err": err, "mismatch_frac": frac,
                "tolerance": "codes within 1, at most 1e-3 of them different", "ok": bool(ok)}
    if name in ("c3", "c5"):
        err = float(np.abs(W.bf16_bits_to_f32(got).astype(np.float64) - ref).max())
        tol = 2e-2
    elif name == "c1":
        err = float(np.abs(got - ref).max())
        tol = 5e-3 * float(np.abs(ref).max())
    else:
        err = float(np.abs(got.astype(np.float64) - ref).max())
        tol = 2e-6
    return {"rows": int(len(idx)), "unit": "sequences (all heads)" if name == "c3" else "rows", "max_err": err,
            "tolerance": tol, "ok": bool(err <= tol)}


def cpu_sample(name):
    """A bounded sample of the config for the oracle: returns (workload, fraction of the full ops, text)."""
    if name == "c1":
        return W.mlp_f32(), 1.0, "full config"
    if name == "c2":
        return W.mlp_int8(), 1.0, "full config"
    if name == "c3":
        return W.mha_bf16(), 1.0, "full config"
    if name == "c4":
        return W.mha_int8(batch=2), 2 / 64, "2 of 64 sequences (32 of 1024 (batch, head) units)"
    return W.ffn_bf16(), 1.0, "full config (8192 tokens)"


def time_oracle(name, repeats=1):
    from oracle import interp
    w, frac, text = cpu_sample(name)
    interp.run(w.graph, w.feeds)      # warm-up (BLAS threads, page faults)
    t0 = time.perf_counter()
    for _ in range(repeats):
        interp.run(w.graph, w.feeds)
    dt = (time.perf_counter() - t0) / repeats
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        nt = [p.get("num_threads", 1) for p in threadpool_info()]
        if nt:
            cores = max(nt)
    except Exception:
        pass
    return w.ops / dt / 1e12, cores, text, dt


def reference_arm(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.workload
    full = W.CONFIGS[name]()
    vals = []
    for _ in range(max(1, args.warmup)):
        time_oracle(name)
    for _ in range(max(1, args.steps)):
        v, cores, text, dt = time_oracle(name)
        vals.append((v, dt))
    v = float(np.mean([x[0] for x in vals]))
    dt = float(np.mean([x[1] for x in vals]))
    line = {
        "impl": "reference", "metric": "fused_subgraph_throughput", "value": v, "unit": UNIT[name], "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64/int64 (oracle)", "data": "synthetic",
        "config": {"workload": name, "graph": full.name, "sample": text},
        "cpu_baseline": {"value": v, "unit": UNIT[name], "cores": cores, "kind": "oracle", "sample": text},
        "e2e": {"value": v, "unit": UNIT[name], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="c5", choices=list(W.CONFIGS))
    ap.add_argument("--only", action="store_true", help="time only the headline workload")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU oracle baseline")
    ap.add_argument("--sweep", action="store_true",
                    help="instead of the headline run, time every shape of the evaluation's workload table (1 GPU)")
    ap.add_argument("--gemm", action="store_true",
                    help="instead of the benchmark: one plain 8192^3 bf16 GEMM, timed like the measured library peaks")
    ap.add_argument("--sweep-filter", default="", help="with --sweep: only the cases whose name contains this text")
    ap.add_argument("--split", action="store_true",
                    help="with N ranks: split the config's ONE batch evenly over the ranks (8192/N tokens, 64/N sequences; "
                         "strong scaling) instead of one full batch per rank")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 0:
            args.steps = 2
        return reference_arm(args)

    import torch
    from paper_2301_01333_b200 import build as gc_build
    from paper_2301_01333_b200 import multi
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    ranks = multi.init_ranks("nccl", f"cuda:{local}")
    rank, world = ranks.rank, ranks.world
    multi.build_on_local_root(ranks, gc_build.build)
    from paper_2301_01333_b200 import binding as B

    def barrier():
        multi.barrier(ranks)

    def max_over_ranks(x):
        return multi.max_over_ranks(ranks, x, f"cuda:{local}")

    peaks, peak_src = load_peaks()
    if args.gemm:
        if rank == 0:
            print(json.dumps({"plain_gemm": run_plain_gemm(B, local, peaks), "data": "synthetic"}))
        if world > 1:
            barrier()
            multi.finish(ranks)
        return
    if args.sweep:
        if rank == 0:
            print(json.dumps({"sweep": run_sweep(B, local, peaks, args.sweep_filter), "unit": "us per subgraph, cold L2", "data": "synthetic"}))
        if world > 1:
            barrier()
            multi.finish(ranks)
        return
    head = args.workload
    names = [head] if args.only else [head] + [n for n in W.CONFIGS if n != head]
    results = {}
    floor_us = launch_floor_us(B, local) if (rank == 0 and not args.only) else 0.0
    sm_max_mhz = 1965.0
    clocks = None
    launches_total = 0
    e2e = None
    for name in names:
        steps = args.steps if (args.steps and name == head) else DEFAULT_STEPS[name]
        shard = None
        if args.split and world > 1:
            shard = multi.split_units(W.CONFIG_UNITS[name][2], world, rank)
        w, reps, n_rep = time_config(B, name, steps, args.warmup, local, shard=shard)
        job_ops = multi.sum_over_ranks(ranks, float(w.ops), f"cuda:{local}")     # what all ranks process per step
        sampler = None
        if name == head and rank == 0:
            sampler = ClockSampler(local)
            sampler.start()
            time.sleep(0.3)
        ms = run_timed(reps, n_rep, steps, local, barrier)
        if sampler:
            clocks = sampler.stop()
        ms = max_over_ranks(ms)
        reps[0].c.query_status()
        us = ms * 1e3 / steps
        t_tensor = w.ops / (NOMINAL["bf16_tflops"] * KIND_RATIO[name] * 1e12)
        t_hbm_meas = w.bytes / (peaks["hbm_gbs"] * 1e9)
        # a timed region of half a second or more runs under the power cap: compare with the sustained peak;
        # shorter bursts with the burst peak
        peak_key = "bf16_tflops_sustained" if ms >= 500.0 else "bf16_tflops"
        tensor_meas = peaks.get(peak_key, 1590.0) * KIND_RATIO[name]
        t_tensor_meas = w.ops / (tensor_meas * 1e12)
        bound = "tensor" if t_tensor_meas > t_hbm_meas else "hbm"
        res = {
            "graph": w.name, "us_per_subgraph": us, "value": job_ops / (us * 1e-6) / 1e12, "unit": UNIT[name],
            "steps": steps, "replicas": n_rep, "launches_per_step": reps[0].c.launches,
            "algorithmic_ops": w.ops, "algorithmic_bytes": w.bytes,
            "achieved_gbs": w.bytes / (us * 1e-6) / 1e9,
            "roofline_bound": bound,
            "roofline_frac_measured_peak": max(t_tensor_meas, t_hbm_meas) / (us * 1e-6),
            "roofline_frac_nominal_peak": max(t_tensor, w.bytes / (NOMINAL["hbm_gbs"] * 1e9)) / (us * 1e-6),
        }
        res["launch_floor_us"] = floor_us * reps[0].c.launches
        # warm: the same buffers every call, so weights and small activations stay in L2
        warm_steps = max(20, steps // 4)
        res["us_per_subgraph_warm"] = max_over_ranks(run_timed(reps[:1], 1, warm_steps, local, barrier)) * 1e3 / warm_steps
        if not args.only:
            res["us_per_subgraph_graph"] = run_graph_replay(reps, n_rep, min(steps, GRAPH_STEPS[name]), local)
        if name == "c5" and rank == 0 and not args.only and not args.split:
            try:
                res["library_two_gemms_us"] = library_two_gemms_us(w, n_rep, steps, local)   # same steps: same power regime
                res["library_two_gemms_note"] = ("torch.matmul (cuBLAS) on the two GEMMs alone, same shapes and replica "
                                                 "rotation, no bias and no GELU: context, not part of the path")
            except Exception as exc:                    # context only: never fail the bench over it
                res["library_two_gemms_us"] = None
                res["library_two_gemms_note"] = f"not measured: {exc}"
        if name == "c3" and rank == 0 and not args.only and not args.split:
            try:
                res["library_sdpa_us"] = library_sdpa_us(w, n_rep, min(steps, 500), local)
                res["library_sdpa_note"] = ("torch.nn.functional.scaled_dot_product_attention (the fused library kernel it "
                                            "selects), same shapes, mask form and replica rotation: context, not part of the path")
            except Exception as exc:                    # context only: never fail the bench over it
                res["library_sdpa_us"] = None
                res["library_sdpa_note"] = f"not measured: {exc}"
        if name in ("c1", "c2") and not args.only:
            # coarse-grain fusion ablation (Section VII, Fig. 8): the whole chain in one persistent launch, one
            # launch per layer (fine-grain fusion only), and the CUDA-core kernels
            abl = {"fused_chain": {"us_cold": us, "us_warm": res["us_per_subgraph_warm"], "launches": reps[0].c.launches}}
            variants = [("per_layer", {"no_chain_fusion": True}), ("cuda_core_per_layer", {"force_generic": True})]
            if "inside one cluster" in reps[0].c.plan:
                # the same chain spread over the whole GPU, activations through the L2 behind a grid barrier
                variants.insert(0, ("grid_wide_chain", {"grid_wide_chain": True}))
            for label, opts in variants:
                _, areps, an = time_config(B, name, steps, args.warmup, local, **opts)
                cold = max_over_ranks(run_timed(areps, an, steps, local, barrier)) * 1e3 / steps
                warm = max_over_ranks(run_timed(areps[:1], 1, warm_steps, local, barrier)) * 1e3 / warm_steps
                abl[label] = {"us_cold": cold, "us_warm": warm, "launches": areps[0].c.launches}
                for r in areps:
                    r.c.close()
                del areps
            res["ablation"] = abl
        n_exp = softmax_scores(w)
        if n_exp:
            # attention: one exponential per score on the special-function units bounds the softmax from below
            t_exp = n_exp / exp_peak_per_s(sm_max_mhz)
            res["exp_bound_us"] = t_exp * 1e6
            res["exp_bound_frac"] = t_exp / (us * 1e-6)
            res["scores"] = n_exp
        if rank == 0 and not args.no_cpu:
            res["parity_checked"] = parity_check(B, name, w, reps[0])
        if name == head and ms < 500.0 and not args.only:
            # A short timed region (the requested K steps) runs at boost clocks.  The same step for about a second
            # more shows the regime under the power cap, next to the sustained library peak measured the same way.
            s_steps = int(min(20000, max(steps, 1000.0 / max(ms / steps, 1e-3))))
            s_sampler = None
            if rank == 0:
                s_sampler = ClockSampler(local)
                s_sampler.start()
                time.sleep(0.3)
            s_ms = run_timed(reps, n_rep, s_steps, local, barrier)
            s_clocks = s_sampler.stop() if s_sampler else None
            s_ms = max_over_ranks(s_ms)
            s_us = s_ms * 1e3 / s_steps
            s_peak = peaks.get("bf16_tflops_sustained", 1400.0) * KIND_RATIO[name]
            res["sustained"] = {"steps": s_steps, "ms": s_ms, "us_per_subgraph": s_us,
                                "value": job_ops / (s_us * 1e-6) / 1e12, "unit": UNIT[name],
                                "frac_of_measured_sustained_peak": (job_ops / (s_us * 1e-6) / 1e12) / s_peak if bound == "tensor" else None,
                                "clocks": s_clocks}
        if name == head:
            launches_total = steps * reps[0].c.launches
            e2e_s, e2e_serial, h2d, d2h, e2e_same = run_e2e(w, reps[0], max(4, min(steps, 50)), args.warmup, local)
            e2e_s = max_over_ranks(e2e_s)
            e2e_serial = max_over_ranks(e2e_serial)
            e2e = {"value": job_ops / e2e_s / 1e12, "unit": UNIT[name], "h2d_bytes_per_step": h2d,
                   "d2h_bytes_per_step": d2h, "us_per_subgraph": e2e_s * 1e6,
                   "mode": f"gc_execute_host_async, {reps[0].c.HOST_SLOTS} batches in flight (copies overlap execution and each other)",
                   "outputs_identical_across_slots_and_serial": bool(e2e_same),
                   "one_batch_at_a_time": {"value": job_ops / e2e_serial / 1e12, "us_per_subgraph": e2e_serial * 1e6,
                                           "call": "gc_execute_host"}}
            head_w, head_ms, head_steps, head_reps, head_peak_key = w, ms, steps, n_rep, peak_key
        results[name] = res
        for r in reps:
            r.c.close()
        del reps
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            multi.finish(ranks)
        return
    hr = results[head]
    us = hr["us_per_subgraph"]
    n_launch = hr["launches_per_step"]
    if "exp_bound_us" in hr and hr["exp_bound_us"] > us * hr["roofline_frac_measured_peak"]:
        # attention: neither DRAM nor the tensor pipe but the exponentials bound it
        peak = exp_peak_per_s(sm_max_mhz) / 1e12
        achieved = hr["scores"] / (us * 1e-6) / 1e12
        roof = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "Texp/s", "frac": achieved / peak,
                "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(head), "traffic_source": TRAFFIC_SOURCE.get(head),
                "peak_source": "derived: 148 SMs x 16 ex2 per clock x 1965 MHz (one exponential per attention score)",
                "kernel": DOMINANT_KERNEL[head], "launches_per_step": n_launch, "avg_launch_us": us / n_launch,
                "hbm_frac_measured_peak": hr["roofline_frac_measured_peak"]}
    elif hr["roofline_bound"] == "tensor":
        peak = peaks.get(head_peak_key, 1590.0) * KIND_RATIO[head]
        achieved = head_w.ops / (us * 1e-6) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s" if "FLOP" in UNIT[head] else "TOP/s",
                "frac": achieved / peak, "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(head), "traffic_source": TRAFFIC_SOURCE.get(head),
                "peak_source": f"{peak_src} cuBLAS {head_peak_key} (timed region {head_ms:.0f} ms) x kind ratio {KIND_RATIO[head]}",
                "kernel": DOMINANT_KERNEL[head], "launches_per_step": n_launch, "avg_launch_us": us / n_launch,
                "algorithmic_flops_per_launch": head_w.ops / n_launch,
                "frac_of_burst_peak": achieved / (peaks.get("bf16_tflops", 1590.0) * KIND_RATIO[head]),
                "frac_of_nominal": achieved / (NOMINAL["bf16_tflops"] * KIND_RATIO[head])}
        if hr.get("library_two_gemms_us"):
            # context: the library's two bare GEMMs on these very shapes (the peak above is its 8192^3 figure)
            roof["library_two_gemms_same_shapes_us"] = hr["library_two_gemms_us"]
            roof["vs_library_two_gemms"] = hr["library_two_gemms_us"] / us
    else:
        achieved = head_w.bytes / (us * 1e-6) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(head), "traffic_source": TRAFFIC_SOURCE.get(head), "peak_source": peak_src, "kernel": DOMINANT_KERNEL[head],
                "launches_per_step": n_launch, "avg_launch_us": us / n_launch,
                "algorithmic_bytes_per_launch": head_w.bytes / n_launch}
    cpu = None
    if not args.no_cpu:
        v, cores, text, dt = time_oracle(head)
        cpu = {"value": v, "unit": UNIT[head], "cores": cores, "kind": "oracle", "sample": text, "seconds": dt}
    line = {
        "metric": "fused_subgraph_throughput", "value": hr["value"], "unit": UNIT[head], "n_gpus": world,
        "steps": head_steps, "warmup": max(args.warmup, 3), "ms_per_step": head_ms / head_steps, "us_per_subgraph": us,
        "higher_is_better": True, "scaling": "strong" if (args.split and world > 1) else "weak", "vs_baseline": None,
        "dtype": DTYPE[head], "data": "synthetic",
        "config": {"workload": head, "graph": head_w.name,
                   "l2": f"steps rotate through {head_reps} independent replicas (weights, workspace, inputs, outputs) "
                         f"whose total footprint exceeds the 126 MB L2",
                   "parallelism": (f"one batch split evenly over {world} GPUs (rows / sequences are independent, no collective)"
                                   if (args.split and world > 1) else
                                   f"replicas x{world} (independent batches per GPU, no collective)")},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_total, "roofline": roof, "cpu_baseline": cpu,
        "parity_checked": hr.get("parity_checked"),
        "sustained": hr.get("sustained"),
        "configs": results,
    }
    print(json.dumps(line))
    if world > 1:
        multi.finish(ranks)
    bad = [n for n, r in results.items() if r.get("parity_checked") and not r["parity_checked"]["ok"]]
    if bad:
        raise SystemExit(f"parity check against the oracle failed for {bad}")


if __name__ == "__main__":
    main()
