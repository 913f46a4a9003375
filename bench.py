#!/usr/bin/env python
"""Benchmark of the W4A16 layer on B200: the batch sweep on one large layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extra]
    python bench.py --sustain SECONDS          # the same step replayed for that long, rate per SM-clock bin
    python bench.py --case M,K,N,G[,sparse|w8] # one layer shape a few times (for profiler captures)
    python bench.py --case C,K,N,G,quantize    # the quantiser with C clipping candidates on a K x N matrix

Workload (config 2 of this build): K = N = 8192, group size 128, M in {1,2,4,8,16,32,64,128};
A ~ fp16 N(0,1), codes uniform 0..15 (zero point 8), scales uniform in [0.005, 0.02]; synthetic.
One step = one pass of the layer at every M of the sweep (pack is offline and not in the step).
Weights are cold: every launch reads the next of several packed copies whose total size exceeds
twice the L2 capacity.

Prints ONE JSON line.  `value` = packed weight bytes (codes + scales) streamed per second over the
whole step, inputs resident in HBM, timed with CUDA events around a CUDA graph of K steps.
`e2e` = the same metric with every step's A copied from pinned host memory and its C copied back inside
the timed region (one transfer each way per step; weights stay resident: they are the model), through the
package's binding, run two ways of which the faster is reported and both are listed: eagerly on copy streams that
overlap the neighbouring steps' kernels, and as three CUDA graphs of one step each (copy in, eight calls, copy
out) replayed in turn on three streams.  `roofline` is that of the dominant kernel (the
instance that serves M = 1, 2, 4, 8): its algorithmic bytes (weights + scales + A + C, each once) per
second of its own live launch time against the measured HBM peak, with the same figure for the whole
step under `whole_step`.  `per_m` lists each
batch size: time, weight GB/s, TFLOP/s, fraction of its roofline, speedup over a cuBLAS fp16 GEMM
of the same shape (torch.matmul).  `cpu_baseline` times the CPU oracle on a bounded sample.

N > 1: the layer does not shard in this build (replicas only): every rank runs the same sweep on
its own GPU; `value` sums the ranks, time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2408_11743_b200 import inputs, replicas, roofline  # noqa: E402

K_DIM, N_DIM, GROUP = 8192, 8192, 128
SWEEP = (1, 2, 4, 8, 16, 32, 64, 128)
METRIC = "w4a16_gemm_weight_stream_rate_batch_sweep_M1-128_K8192_N8192_g128"
UNIT = "GB/s"
CPU_SAMPLE_MS = (1, 2, 4, 8, 16, 32, 64, 128)  # cpu_baseline leg of the GPU arm: one whole step (about 25 core-seconds)
REFERENCE_SAMPLE_MS = (16,)   # one step of --impl reference


def launches_for(M: int) -> int:
    """Kernels one marlin_gemm call launches on this layer: the warp-MMA kernel up to 16 rows, the tcgen05
    kernel (up to 128 rows per launch) above."""
    return 1 if M <= 128 else (M + 127) // 128


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, the instance that
# serves M <= 8, from the committed ncu capture of its M = 1 launch (profiles/gemm_dense_kernel_M1_K8192_N8192.md);
# the algorithmic bytes of that launch are 34.64e6
NCU_DRAM_BYTES_PER_LAUNCH = 34.69e6


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while a region runs (read-only queries)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()

    def summary(self, t0: float, t1: float):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.05] or [r for _, r in self.rows]
        for r in rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "reasons": sorted(reasons),
                "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# CPU oracle leg
# ------------------------------------------------------------------------------------------------
def time_oracle_sample(case_cache, Ms=CPU_SAMPLE_MS):
    """The oracle as it stands, on the host cores, on the full layer at a few batch sizes of the sweep."""
    import oracle
    oracle.build()
    t = 0.0
    wbytes = 0
    for M in Ms:
        case = case_cache(M)
        t0 = time.perf_counter()
        oracle.gemm(case.A, case.q_kpacked, case.S, case.G)
        t += time.perf_counter() - t0
        wbytes += roofline.weight_bytes(K_DIM, N_DIM, GROUP)
    return wbytes / t / 1e9, t, oracle.num_threads()


def make_case_cache():
    cache = {}
    base = inputs.make_dense(max(SWEEP), K_DIM, N_DIM, GROUP, inputs.case_seed(2, 0, 0))

    def get(M):
        if M not in cache:
            cache[M] = inputs.DenseCase(np.ascontiguousarray(base.A[:M]), base.q_kpacked, base.S, M, K_DIM, N_DIM,
                                        GROUP, base.seed)
        return cache[M]
    return get


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    get = make_case_cache()
    vals = []
    for i in range(args.warmup + args.steps):
        v, t, cores = time_oracle_sample(get, REFERENCE_SAMPLE_MS)
        if i >= args.warmup:
            vals.append((v, t))
    value = sum(v for v, _ in vals) / len(vals)
    ms = 1e3 * sum(t for _, t in vals) / len(vals)
    sample = f"full layer at M in {list(REFERENCE_SAMPLE_MS)} per step (1 of the 8 batch sizes of the sweep)"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "batch sweep K=8192 N=8192 g128 (CPU oracle on a bounded sample)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU leg
# ------------------------------------------------------------------------------------------------
class LayerBench:
    """One packed layer resident on the GPU (several cold copies) and its cuBLAS fp16 counterpart, timed per batch size."""

    def __init__(self, marlin, dev, stream, l2, K, N, G, sparse, rng, with_fp16=True, w8=False):
        import torch
        self.m, self.dev, self.stream, self.K, self.N, self.G, self.sparse = marlin, dev, stream, K, N, G, sparse
        self.w8 = w8
        self.wb = roofline.weight_bytes(K, N, G, sparse24=sparse, bits=8 if w8 else 4)
        self.copies = max(2, int(np.ceil(2.0 * l2 / self.wb)) + 1)
        S = torch.from_numpy(rng.uniform(0.005, 0.02, size=(K // G, N)).astype(np.float16)).to(dev)
        if w8:
            q8 = torch.from_numpy(rng.integers(0, 256, size=(K, N), dtype=np.uint8)).to(dev)
            packed0 = marlin.pack_w8(q8, S, G)
        elif sparse:
            qc = torch.from_numpy(rng.integers(-2**31, 2**31 - 1, size=(K // 16, N), dtype=np.int64).astype(np.int32)).to(dev)
            pat = rng.integers(0, 6, size=(K // 4, N))
            idx = np.empty((K // 2, N), dtype=np.uint8)
            idx[0::2], idx[1::2] = inputs._KEEP_PATTERNS[pat, 0], inputs._KEEP_PATTERNS[pat, 1]
            packed0 = marlin.pack_sparse24(qc, torch.from_numpy(idx).to(dev), S, G)
        else:
            q = torch.from_numpy(rng.integers(-2**31, 2**31 - 1, size=(K // 8, N), dtype=np.int64).astype(np.int32)).to(dev)
            packed0 = marlin.pack(q, S, G)
        self.packed = [tuple(t.clone() for t in packed0) for _ in range(self.copies)]
        self.W16 = None
        if with_fp16:
            n16 = max(2, int(np.ceil(2.0 * l2 / (2 * K * N))) + 1)
            self.W16 = [torch.randn((K, N), dtype=torch.float16, device=dev) * 0.05 for _ in range(n16)]
        self.rng = rng

    def time(self, M, capture, time_graph, peaks, reps_min=16):
        import torch
        marlin, dev, stream, K, N, G = self.m, self.dev, self.stream, self.K, self.N, self.G
        A = torch.from_numpy(self.rng.standard_normal((M, K), dtype=np.float32).astype(np.float16)).to(dev)
        C = torch.empty((M, N), dtype=torch.float16, device=dev)
        ws = marlin.new_workspace(M, K, N, device=dev)
        rot = [0]

        def call():
            pk = self.packed[rot[0] % self.copies]
            rot[0] += 1
            if self.w8:
                marlin.gemm_w8(A, pk[0], pk[1], K, N, G, ws, out=C, stream=stream)
            elif self.sparse:
                marlin.gemm_sparse24(A, pk[0], pk[1], pk[2], K, N, G, ws, out=C, stream=stream)
            else:
                marlin.gemm(A, pk[0], pk[1], K, N, G, ws, out=C, stream=stream)
        with torch.cuda.stream(stream):
            for _ in range(3):
                call()
        torch.cuda.synchronize(dev)
        reps = max(reps_min, 2 * self.copies)
        g = capture(call, reps)
        time_graph(g)
        t = min(time_graph(g) for _ in range(5)) / reps
        troof = roofline.roofline_seconds(M, K, N, G, peaks, sparse24=self.sparse, bits=8 if self.w8 else 4)
        if marlin.read_status(ws, stream=stream) != 0:
            raise RuntimeError("device-side wait expired")
        r = {"K": K, "N": N, "G": G, "M": M, "sparse24": self.sparse, "us": round(t * 1e6, 3),
             "weight_gbs": round(self.wb / t / 1e9, 1), "tflops": round(roofline.flops(M, K, N) / t / 1e12, 2),
             "roofline_frac": round(troof / t, 4)}
        if self.W16 is not None:
            o16 = torch.empty((M, N), dtype=torch.float16, device=dev)
            r16 = [0]

            def fp16():
                torch.matmul(A, self.W16[r16[0] % len(self.W16)], out=o16)
                r16[0] += 1
            with torch.cuda.stream(stream):
                for _ in range(3):
                    fp16()
            torch.cuda.synchronize(dev)
            g16 = capture(fp16, 2 * len(self.W16))
            time_graph(g16)
            t16 = min(time_graph(g16) for _ in range(5)) / (2 * len(self.W16))
            r["cublas_fp16_us"] = round(t16 * 1e6, 3)
            r["speedup_vs_fp16"] = round(t16 / t, 3)
        return r


def mlp_chain(marlin, dev, stream, l2, capture, time_graph, rng, K=4096, I=11008, N=4096, Ms=(1, 16, 64)):
    import torch
    G = GROUP

    def rand_layer(k, n):
        q = torch.from_numpy(rng.integers(-2**31, 2**31 - 1, size=(k // 8, n), dtype=np.int64).astype(np.int32)).to(dev)
        S = torch.from_numpy(rng.uniform(0.005, 0.02, size=(k // G, n)).astype(np.float16)).to(dev)
        return q, S
    qg, sg = rand_layer(K, I)
    qu, su = rand_layer(K, I)
    q_gu, s_gu = marlin.interleave_gate_up(qg, sg, qu, su, G)
    gu0 = marlin.pack(q_gu, s_gu, G)
    d0 = marlin.pack(*rand_layer(I, N), G)
    wb = roofline.weight_bytes(K, 2 * I, G) + roofline.weight_bytes(I, N, G)
    copies = max(2, int(np.ceil(2.0 * l2 / wb)) + 1)
    gus = [tuple(t.clone() for t in gu0) for _ in range(copies)]
    ds = [tuple(t.clone() for t in d0) for _ in range(copies)]
    res = []
    for M in Ms:
        A = torch.from_numpy(rng.standard_normal((M, K), dtype=np.float32).astype(np.float16)).to(dev)
        H = torch.empty((M, I), dtype=torch.float16, device=dev)
        H2 = torch.empty((M, 2 * I), dtype=torch.float16, device=dev)
        C = torch.empty((M, N), dtype=torch.float16, device=dev)
        ws = torch.zeros(max(marlin.workspace_bytes(M, K, 2 * I), marlin.workspace_bytes(M, I, N)), dtype=torch.uint8, device=dev)
        rot = [0]

        def fused():
            i = rot[0] % copies
            rot[0] += 1
            marlin.mlp_swiglu(A, gus[i][0], gus[i][1], ds[i][0], ds[i][1], K, I, N, G, ws, H=H, out=C, stream=stream)

        def unfused():
            i = rot[0] % copies
            rot[0] += 1
            marlin.gemm(A, gus[i][0], gus[i][1], K, 2 * I, G, ws, out=H2, stream=stream)
            v = H2.view(M, I // 8, 2, 8)
            torch.mul(torch.nn.functional.silu(v[:, :, 0, :]), v[:, :, 1, :], out=H.view(M, I // 8, 8))
            marlin.gemm(H, ds[i][0], ds[i][1], I, N, G, ws, out=C, stream=stream)
        t = {}
        for name, fn in (("fused", fused), ("unfused", unfused)):
            with torch.cuda.stream(stream):
                for _ in range(3):
                    fn()
            torch.cuda.synchronize(dev)
            reps = 2 * copies
            g = capture(fn, reps)
            time_graph(g)
            t[name] = min(time_graph(g) for _ in range(5)) / reps
        if marlin.read_status(ws, stream=stream) != 0:
            raise RuntimeError("device-side wait expired")
        res.append({"layer": "llama2-7b MLP chain (gate_up + SwiGLU + down)", "config": 3, "M": M, "K": K, "I": I, "N": N,
                    "G": G, "fused_us": round(t["fused"] * 1e6, 2), "unfused_us": round(t["unfused"] * 1e6, 2),
                    "weight_gbs": round(wb / t["fused"] / 1e9, 1)})
    return res


def extra_layers(marlin, dev, stream, l2, peaks, capture, time_graph):
    """Per-layer numbers outside the timed step: every layer and batch size of configs 3 (Llama-2-7B shapes), 4
    (Llama-2-70B shapes, group 128 and one scale per column) and 5 (the 2:4 layer, with the dense layer beside it),
    and batches of 256 to 4096 rows on two layers."""
    import torch
    out = []
    rng = np.random.default_rng(1234)

    def sweep(K, N, G, sparse, Ms, label, config, w8=False):
        layer = LayerBench(marlin, dev, stream, l2, K, N, G, sparse, rng, w8=w8)
        for M in Ms:
            r = layer.time(M, capture, time_graph, peaks)
            r["layer"], r["config"] = label, config
            out.append(r)
        del layer
        torch.cuda.empty_cache()

    for name, K, N in inputs.LLAMA7B_LAYERS:
        sweep(K, N, GROUP, False, (1, 16, 32, 64, 128), "llama2-7b " + name, 3)
    sweep(8192, 8192, GROUP, True, (16, 32, 64, 128), "2:4 sparse 8192x8192", 5)
    # batches above 128 rows (Section 5.1 "Large batch performance"): one launch, tensor-bound; roofline_frac is taken
    # against the measured dense bf16 GEMM peak there, cublas_fp16_us is the uncompressed layer through torch.matmul
    sweep(8192, 8192, GROUP, False, (256, 512, 1024, 2048, 4096), "large batch 8192x8192", 2)
    sweep(4096, 22016, GROUP, False, (256, 1024, 4096), "large batch llama2-7b gate_up", 3)
    # the offline quantiser in front of the pack (Section 3.5 (a)): fp16 weights -> codes and scales, 10 clipping
    # candidates per group; bounded by the arithmetic of the search (the algorithmic bytes are 2.5 per weight)
    for nc in (1, 10):
        Wq = torch.randn((8192, 8192), device=dev, dtype=torch.float32).mul_(0.02).half()
        with torch.cuda.stream(stream):
            marlin.quantize_rtn(Wq, GROUP, 20, nc, stream=stream)
        torch.cuda.synchronize(dev)
        g = capture(lambda: marlin.quantize_rtn(Wq, GROUP, 20, nc, stream=stream), 2)
        tq = min(time_graph(g) for _ in range(3)) / 2
        out.append({"layer": "quantize_rtn 8192x8192", "config": "front end", "G": GROUP, "n_grid": 20, "n_candidates": nc,
                    "us": round(tq * 1e6, 1), "gweights_per_s": round(8192 * 8192 / tq / 1e9, 1),
                    "algorithmic_gbs": round((8192 * 8192 * 2.5 + 2 * 64 * 8192) / tq / 1e9, 1)})
        del Wq
    # 8-bit weights on the same layer (twice the bytes per weight: the roofline time doubles)
    sweep(8192, 8192, GROUP, False, (1, 16, 64, 128), "8-bit weights 8192x8192", 2, w8=True)
    # the gated MLP of a Llama-2-7B layer as a chain: gate_up with the activation fused into its epilogue, then down
    # (two launches, the second under programmatic dependent launch), against the same layers with the activation
    # as separate elementwise kernels on the wide intermediate
    out.extend(mlp_chain(marlin, dev, stream, l2, capture, time_graph, rng))
    for name, K, N in inputs.LLAMA70B_LAYERS:
        for G in (GROUP, K):
            sweep(K, N, G, False, (1, 16, 64, 128),
                  "llama2-70b " + name + (" g128" if G == GROUP else " per-column scales"), 4)
    return out


def run_case(args):
    """One layer shape, a few launches: the small, self-contained command the profiler captures are made with."""
    import torch
    import paper_2408_11743_b200 as marlin
    parts = args.case.split(",")
    M, K, N, G = (int(x) for x in parts[:4])
    sparse = len(parts) > 4 and parts[4].startswith("sparse")
    w8 = len(parts) > 4 and parts[4].startswith("w8")
    if G <= 0:
        G = K
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    stream = torch.cuda.Stream(device=dev)
    if len(parts) > 4 and parts[4].startswith("quantize"):
        # M is the number of clipping candidates here: the quantiser on a K x N matrix, a few launches
        W = torch.randn((K, N), device=dev, dtype=torch.float32).mul_(0.02).half()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            marlin.quantize_rtn(W, G, 20, M, stream=stream)
            e0.record(stream)
            for _ in range(args.iters):
                marlin.quantize_rtn(W, G, 20, M, stream=stream)
            e1.record(stream)
        e1.synchronize()
        t = e0.elapsed_time(e1) * 1e-3 / args.iters
        print(json.dumps({"quantize_rtn": True, "K": K, "N": N, "G": G, "n_grid": 20, "n_candidates": M,
                          "us": round(t * 1e6, 1), "gweights_per_s": round(K * N / t / 1e9, 1)}), flush=True)
        return
    peaks = roofline.load_peaks(ROOT)
    l2 = args.copies_bytes
    layer = LayerBench(marlin, dev, stream, l2, K, N, G, sparse, np.random.default_rng(1), with_fp16=False, w8=w8)

    def capture(fn, reps):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                fn()
        return g

    def time_graph(g):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            g.replay()
            e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e-3
    r = layer.time(M, capture, time_graph, peaks, reps_min=args.iters)
    r["copies"] = layer.copies
    print(json.dumps(r), flush=True)


def run_ours(args):
    import torch
    import torch.distributed as dist
    import paper_2408_11743_b200 as marlin

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a GPU: this library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    marlin.lib()
    dev = torch.device("cuda", local_rank)
    props = torch.cuda.get_device_properties(dev)
    l2 = getattr(props, "L2_cache_size", 126 * 1024 * 1024)

    get = make_case_cache()
    base = get(max(SWEEP))
    wbytes = roofline.weight_bytes(K_DIM, N_DIM, GROUP)
    copies = max(2, int(np.ceil(2.0 * l2 / wbytes)) + 1)
    q_dev = torch.from_numpy(base.q_kpacked.view(np.int32)).to(dev)
    s_dev = torch.from_numpy(base.S).to(dev)
    w0, s0 = marlin.pack(q_dev, s_dev, GROUP)
    packed = [(w0.clone(), s0.clone()) for _ in range(copies)]
    del q_dev
    A_dev = {M: torch.from_numpy(get(M).A).to(dev) for M in SWEEP}
    C_dev = {M: torch.empty((M, N_DIM), dtype=torch.float16, device=dev) for M in SWEEP}
    ws = marlin.new_workspace(max(SWEEP), K_DIM, N_DIM, device=dev)
    stream = torch.cuda.Stream(device=dev)
    rot = [0]

    def one_gemm(M):
        w, s = packed[rot[0] % copies]
        rot[0] += 1
        marlin.gemm(A_dev[M], w, s, K_DIM, N_DIM, GROUP, ws, out=C_dev[M], stream=stream)

    def one_step():
        for M in SWEEP:
            one_gemm(M)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # warm-up (also sets kernel attributes before any capture)
    with torch.cuda.stream(stream):
        for _ in range(max(3, args.warmup)):
            one_step()
    torch.cuda.synchronize(dev)
    if marlin.read_status(ws, stream=stream) != 0:
        raise RuntimeError("device-side wait expired during warm-up")

    def capture(fn, reps):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(reps):
                fn()
        return g

    def time_graph(g, replays=1):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _ in range(replays):
                g.replay()
            e1.record(stream)
        e1.synchronize()
        return e0.elapsed_time(e1) * 1e-3

    # ---- main timed region: K steps, device time, max over ranks ----
    g_steps = capture(one_step, args.steps)
    with torch.cuda.stream(stream):
        g_steps.replay()  # instantiate / upload outside the timed region
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)
    barrier()
    t_wall0 = time.time()
    elapsed = time_graph(g_steps)
    # keep the same load running a little longer so that the 50 ms clock sampler sees it
    t_extra_end = time.time() + 0.6
    while time.time() < t_extra_end:
        time_graph(g_steps)
    t_wall1 = time.time()
    barrier()
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    elapsed = replicas.max_over_ranks(elapsed, dev)
    step_s = elapsed / args.steps
    step_wbytes = wbytes * len(SWEEP)
    value = replicas.job_throughput(step_wbytes, world, step_s) / 1e9
    step_alg_bytes = sum(roofline.algorithmic_bytes(M, K_DIM, N_DIM, GROUP) for M in SWEEP)
    launches_per_step = sum(launches_for(M) for M in SWEEP)

    # ---- sustained mode (Section 5.1 "Sustained performance"): the same graph replayed for seconds; the SM clock is
    # sampled beside it (read-only) and the rate is reported per clock bin and as time x clock ----
    sustained = None
    if args.sustain > 0:
        s2 = ClockSampler(local_rank)
        s2.start()
        time.sleep(0.3)
        barrier()
        batches = []
        t_end = time.time() + args.sustain
        while time.time() < t_end:
            w0 = time.time()
            dt = time_graph(g_steps, replays=10)
            batches.append((w0, time.time(), dt / (10 * args.steps)))
        barrier()
        s2.stop()
        if rank == 0 and batches:
            samples = []
            for t, row in s2.rows:
                parts = [x.strip() for x in row.split(",")]
                try:
                    samples.append((t, float(parts[0])))
                except (ValueError, IndexError):
                    pass
            bins = {}
            prods = []
            for w0, w1, step_t in batches:
                near = [mhz for t, mhz in samples if w0 - 0.06 <= t <= w1 + 0.06]
                if not near:
                    continue
                mhz = statistics.median(near)
                bins.setdefault(int(round(mhz / 50.0)) * 50, []).append(step_t)
                prods.append(step_t * mhz)
            all_t = [b[2] for b in batches]
            summ = s2.summary(batches[0][0], batches[-1][1])
            sustained = {
                "seconds": round(batches[-1][1] - batches[0][0], 2), "steps": len(batches) * 10 * args.steps,
                "ms_per_step": round(1e3 * statistics.median(all_t), 5),
                "value": round(world * step_wbytes / statistics.median(all_t) / 1e9, 2), "unit": UNIT,
                "sm_mhz_median": summ["sm_mhz"], "reasons": summ["reasons"],
                "us_per_step_x_ghz": round(1e3 * statistics.median(prods), 3) if prods else None,
                "by_clock": [{"sm_mhz": k, "batches": len(v), "ms_per_step": round(1e3 * statistics.median(v), 5),
                              "value": round(world * step_wbytes / statistics.median(v) / 1e9, 2)}
                             for k, v in sorted(bins.items())],
            }

    line = None
    if rank == 0:
        peaks = roofline.load_peaks(ROOT)
        # ---- per batch size: our kernel and cuBLAS fp16 on cold weights ----
        reps = 4 * copies
        W16 = [torch.randn((K_DIM, N_DIM), dtype=torch.float16, device=dev) * 0.05
               for _ in range(max(2, int(np.ceil(2.0 * l2 / (2 * K_DIM * N_DIM))) + 1))]
        rot16 = [0]
        per_m = []
        for M in SWEEP:
            g = capture(lambda: one_gemm(M), reps)
            time_graph(g)
            t_ours = min(time_graph(g) for _ in range(5)) / reps
            out16 = torch.empty((M, N_DIM), dtype=torch.float16, device=dev)

            def fp16_gemm():
                torch.matmul(A_dev[M], W16[rot16[0] % len(W16)], out=out16)
                rot16[0] += 1
            with torch.cuda.stream(stream):
                for _ in range(3):
                    fp16_gemm()
            torch.cuda.synchronize(dev)
            g16 = capture(fp16_gemm, 2 * len(W16))
            time_graph(g16)
            t_fp16 = min(time_graph(g16) for _ in range(5)) / (2 * len(W16))
            t_roof = roofline.roofline_seconds(M, K_DIM, N_DIM, GROUP, peaks)
            per_m.append({
                "M": M, "us": round(t_ours * 1e6, 3), "weight_gbs": round(wbytes / t_ours / 1e9, 1),
                "tflops": round(roofline.flops(M, K_DIM, N_DIM) / t_ours / 1e12, 2),
                "roofline_us": round(t_roof * 1e6, 3), "roofline_frac": round(t_roof / t_ours, 4),
                "cublas_fp16_us": round(t_fp16 * 1e6, 3), "speedup_vs_fp16": round(t_fp16 / t_ours, 3),
                "launches": launches_for(M),
            })
            del g, g16
        del W16

        # ---- context, not part of the step: Llama-2-7B-shaped layers and the 2:4 variant ----
        extra = []
        if not args.no_extra:
            extra = extra_layers(marlin, dev, stream, l2, peaks, capture, time_graph)

        # ---- end to end: host buffers, copies inside the timed region ----
        # The inputs of a step arrive in one pinned host buffer and its results leave in one: one copy each way
        # per step (all eight activation matrices, all eight results), the eight calls in between.  Copy-in,
        # compute and copy-out run on three streams over two sets of device buffers, so the copies of one step
        # overlap the kernels of its neighbours; every step still copies its own inputs in and its results out.
        rows = sum(SWEEP)
        A_host = torch.empty((rows, K_DIM), dtype=torch.float16).pin_memory()
        C_host = [torch.empty((rows, N_DIM), dtype=torch.float16).pin_memory() for _ in range(2)]
        A_all = [torch.empty((rows, K_DIM), dtype=torch.float16, device=dev) for _ in range(2)]
        C_all = [torch.empty((rows, N_DIM), dtype=torch.float16, device=dev) for _ in range(2)]
        A_e2e, C_e2e, r0 = [{}, {}], [{}, {}], 0
        for M in SWEEP:
            A_host[r0:r0 + M].copy_(torch.from_numpy(get(M).A))
            for b in range(2):
                A_e2e[b][M], C_e2e[b][M] = A_all[b][r0:r0 + M], C_all[b][r0:r0 + M]
            r0 += M
        # the packed copies of the layer as Layer objects of the public binding (buffers checked once, one foreign
        # call per use): what a caller that runs the same layers step after step holds
        e2e_layers = [marlin.Layer(w, s, K_DIM, N_DIM, GROUP, ws, max_M=max(SWEEP)) for w, s in packed]
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in range(2)]    # inputs of the buffer set are on the device
        ev_cmp = [torch.cuda.Event() for _ in range(2)]   # its kernels are done (A may be overwritten, C read)
        ev_out = [torch.cuda.Event() for _ in range(2)]   # its results are on the host (C may be overwritten)
        step_no = [0]
        # the device buffers of a step are fixed, so the calls are prepared once (buffers checked, pointers read)
        e2e_calls = [{M: [layer.prepare(A_e2e[b][M], out=C_e2e[b][M], stream=stream) for layer in e2e_layers]
                      for M in SWEEP} for b in range(2)]

        def e2e_step():
            # (torch.cuda.set_stream instead of the stream context manager, and the compute stream passed to the calls:
            # the host side of a step is a dozen short calls, and on a slow host it is what bounds this number)
            b = step_no[0] % 2
            first_use = step_no[0] < 2
            step_no[0] += 1
            torch.cuda.set_stream(s_in)
            if not first_use:
                s_in.wait_event(ev_cmp[b])
            A_all[b].copy_(A_host, non_blocking=True)
            ev_in[b].record(s_in)
            stream.wait_event(ev_in[b])
            if not first_use:
                stream.wait_event(ev_out[b])
            for M in SWEEP:
                e2e_calls[b][M][rot[0] % copies]()
                rot[0] += 1
            ev_cmp[b].record(stream)
            torch.cuda.set_stream(s_out)
            s_out.wait_event(ev_cmp[b])
            C_host[b].copy_(C_all[b], non_blocking=True)
            ev_out[b].record(s_out)

        for _ in range(4):
            e2e_step()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        # the timed region starts on the copy-in stream and ends when the last results are on the host
        e0.record(s_in)
        for _ in range(args.steps):
            e2e_step()
        s_out.wait_stream(stream)
        s_out.wait_stream(s_in)
        e1.record(s_out)
        e1.synchronize()
        torch.cuda.synchronize(dev)
        e2e_s = e0.elapsed_time(e1) * 1e-3 / args.steps
        torch.cuda.set_stream(torch.cuda.default_stream(dev))

        # The same step as a caller with fixed buffers runs it: captured once through the same binding into a CUDA
        # graph (copy in from the pinned buffer, the eight calls, copy out to a pinned buffer), three such graphs
        # with buffer sets, workspaces and streams of their own replayed in turn, so that the copies of one step run
        # under the kernels of the others.  Every step still moves its inputs in and its results out; the host makes
        # two torch calls per step instead of a dozen, so a slow host no longer bounds the number.
        NG = 3
        g_streams = [torch.cuda.Stream(device=dev) for _ in range(NG)]
        g_ws = [marlin.new_workspace(max(SWEEP), K_DIM, N_DIM, device=dev) for _ in range(NG)]
        g_A = [torch.empty((rows, K_DIM), dtype=torch.float16, device=dev) for _ in range(NG)]
        g_C = [torch.empty((rows, N_DIM), dtype=torch.float16, device=dev) for _ in range(NG)]
        g_Ch = [torch.empty((rows, N_DIM), dtype=torch.float16).pin_memory() for _ in range(NG)]
        graphs = []
        for gi in range(NG):
            layers_g = [marlin.Layer(w, s, K_DIM, N_DIM, GROUP, g_ws[gi], max_M=max(SWEEP)) for w, s in packed]

            def one_step(gi=gi, layers_g=layers_g):
                g_A[gi].copy_(A_host, non_blocking=True)
                r0 = 0
                for j, M in enumerate(SWEEP):
                    layers_g[(len(SWEEP) * gi + j) % copies](g_A[gi][r0:r0 + M], out=g_C[gi][r0:r0 + M], stream=g_streams[gi])
                    r0 += M
                g_Ch[gi].copy_(g_C[gi], non_blocking=True)
            with torch.cuda.stream(g_streams[gi]):
                one_step()
            g_streams[gi].synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=g_streams[gi]):
                one_step()
            graphs.append(g)
        torch.cuda.synchronize(dev)

        def graph_step(i):
            torch.cuda.set_stream(g_streams[i % NG])
            graphs[i % NG].replay()
        for i in range(2 * NG):
            graph_step(i)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(g_streams[0])
        for i in range(args.steps):
            graph_step(i)
        for st in g_streams[1:]:
            g_streams[0].wait_stream(st)
        e1.record(g_streams[0])
        e1.synchronize()
        torch.cuda.synchronize(dev)
        torch.cuda.set_stream(torch.cuda.default_stream(dev))
        e2e_graph_s = e0.elapsed_time(e1) * 1e-3 / args.steps
        for gi in range(NG):
            if marlin.read_status(g_ws[gi]) != 0:
                raise RuntimeError("device-side wait expired during the end-to-end run")
        # the results that came back to the host are those of the eager pipeline's buffers (same inputs, same layer)
        if not torch.equal(torch.nan_to_num(g_Ch[0][:16].float()), torch.nan_to_num(C_host[0][:16].float())):
            raise RuntimeError("graph-replayed step and eager step returned different results for M <= 16")
        h2d = sum(2 * M * K_DIM for M in SWEEP)
        d2h = sum(2 * M * N_DIM for M in SWEEP)

        if marlin.read_status(ws, stream=stream) != 0:
            raise RuntimeError("device-side wait expired during the benchmark")

        # ---- CPU oracle on a bounded sample ----
        cpu_v, cpu_t, cores = time_oracle_sample(get)

        step_achieved = step_alg_bytes / step_s / 1e9
        # the dominant kernel: the instance of gemm_dense_kernel that serves M = 1, 2, 4, 8 (four of the eight
        # launches of a step and the largest share of its time), timed live above, one graph per batch size
        dom = [r for r in per_m if r["M"] <= 8]
        dom_bytes = sum(roofline.algorithmic_bytes(r["M"], K_DIM, N_DIM, GROUP) for r in dom)
        dom_us = sum(r["us"] for r in dom)
        achieved = dom_bytes / (dom_us * 1e-6) / 1e9
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": round(step_s * 1e3, 5), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16 x int4 -> f32 accumulate -> f16",
            "data": "synthetic",
            "config": {"workload": "config 2: batch sweep M in {1,2,4,8,16,32,64,128} on K=8192 N=8192 g128",
                       "step": "one marlin_gemm per batch size (8 calls)", "cold_weights":
                       f"{copies} rotating packed copies ({copies * wbytes / 2**20:.0f} MiB > 2 x L2)",
                       "timing": "CUDA graph of K steps between CUDA events on the launch stream",
                       "multi_gpu": "replicas only"},
            "roofline": {"bound": "hbm", "achieved": round(achieved, 1), "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": round(achieved / peaks["hbm_gbs"], 4), "traffic": NCU_DRAM_BYTES_PER_LAUNCH,
                         "traffic_note": "ncu capture of the M=1 launch; algorithmic bytes of that launch 34.64e6",
                         "peak_source": peaks["source"],
                         "kernel": "gemm_dense_kernel<1,2,12,0>: the M = 1, 2, 4, 8 launches of the step",
                         "per_launch_us": round(dom_us / len(dom), 3),
                         "algorithmic_bytes_per_launch": round(dom_bytes / len(dom)),
                         "whole_step": {"achieved": round(step_achieved, 1),
                                        "frac": round(step_achieved / peaks["hbm_gbs"], 4),
                                        "per_launch_us": round(step_s * 1e6 / launches_per_step, 3),
                                        "algorithmic_bytes_per_step": step_alg_bytes,
                                        "kernels": "gemm_dense_kernel (M <= 16), gemm_dense_tc_kernel (M = 32, 64, 128)"}},
            "per_m": per_m,
            "other_layers": extra,
            "cpu_baseline": {"value": round(cpu_v, 4), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"one whole step: the full layer at M in {list(CPU_SAMPLE_MS)} ({cpu_t:.1f} s on {cores} threads)"},
            "e2e": {"value": round(world * step_wbytes / min(e2e_s, e2e_graph_s) / 1e9, 2), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": round(min(e2e_s, e2e_graph_s) * 1e3, 5),
                    "how": "the faster of two ways to run the step from pinned host buffers through the binding",
                    "eager_ms_per_step": round(e2e_s * 1e3, 5),
                    "eager": "a dozen torch calls and eight layer calls per step on three streams, two buffer sets",
                    "graph_ms_per_step": round(e2e_graph_s * 1e3, 5),
                    "graph": "the step (copy in, eight calls, copy out) captured once per buffer set, three graphs "
                             "replayed in turn on three streams"},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
        }
        if sustained is not None:
            line["sustained"] = sustained
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if line is not None:
        print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extra", action="store_true", help="skip the Llama-shaped and 2:4 context measurements")
    ap.add_argument("--sustain", type=float, default=0.0, metavar="SECONDS",
                    help="replay the step for this long and report the rate per sampled SM clock (Section 5.1, "
                         "sustained performance); clocks are only read, never set")
    ap.add_argument("--case", default=None, metavar="M,K,N,G[,sparse]", help="time one layer shape and exit")
    ap.add_argument("--iters", type=int, default=8, help="--case: launches per timed graph")
    ap.add_argument("--copies-bytes", type=int, default=126 * 1024 * 1024,
                    help="--case: the cold copies of the packed layer exceed twice this many bytes")
    args = ap.parse_args()
    if args.case:
        run_case(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
