#!/usr/bin/env python
"""Benchmark of the quantised-network forward hot path on B200.

One "step" = one Algorithm-4 forward pass of the MNIST-shaped binarised MLP
(784-4096-4096-4096-10, batch 10000 per GPU, 8-bit inputs as bit-planes,
hidden layers XNOR + folded threshold, int32 scores) through the C ABI.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--algo auto|popc|tc_i8|b1_mma]

Prints ONE JSON line (rank 0).  `value` is binary tera-ops per second,
2*M*N*K per 1-bit plane product, summed over the layers and over all ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

DIMS = (784, 4096, 4096, 4096, 10)
BATCH = 10000
IN_BITS = 8
E2E_CHUNKS = int(os.environ.get("QNN_BENCH_E2E_CHUNKS", "1"))   # pieces of the batch whose input copies overlap the previous piece's layers
E2E_GRAPH_MAX_BATCH = int(os.environ.get("QNN_BENCH_E2E_GRAPH_MAX_BATCH", "2048"))
METRIC = "binary_gemm_tops"
UNIT = "Tops/s (2*M*N*K per 1-bit plane product)"

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel, from
# the ncu capture of that kernel; None until a capture exists for the kernel the run selects.
NCU_TRAFFIC_BYTES = {
    # hidden layer 2 (the launch the live timing brackets): 28.96 MB read + 0.23 MB written per launch
    "tcgen05 kind::mxf4 xnor product 10000x4096x4096, threshold epilogue (gemm_tc_kernel<FP4>)": 29.20e6,
}


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


def _ops(M, count_planes=True):
    """Operations per layer: 2*M*N*K per 1-bit plane product (the paper's cost model, 8 planes in layer 1), or with
    count_planes=False per integer multiply-accumulate (layer 1 counted once: what the tensor cores issue)."""
    per_layer = []
    for l in range(len(DIMS) - 1):
        planes = IN_BITS if (l == 0 and count_planes) else 1
        per_layer.append(2.0 * M * DIMS[l + 1] * DIMS[l] * planes)
    return per_layer


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(prefix="qnn_clocks_", suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "50",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin=None, t_end=None):
        """Summarises the samples whose wall-clock timestamp lies in [t_begin, t_end] (all samples if none given)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()            # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            with open(self.path) as f:
                for ln in f:
                    c = [x.strip() for x in ln.split(",")]
                    if len(c) < 9:
                        continue
                    try:
                        ts = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        if t_begin is not None and not (t_begin - 0.05 <= ts <= t_end + 0.05):
                            continue
                        sm.append(float(c[1])); mx.append(float(c[2]))
                    except ValueError:
                        continue
                    for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                       c[5:9]):
                        if v.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(mx)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


def _dist_setup(n_gpus: int):
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    return rank, world, local


def shard_plan(world: int, rank: int, batch_per_gpu: int = BATCH):
    """Data-parallel plan: every rank owns an independent batch (weak scaling), same weights, no collective."""
    return {"stream": rank, "rows": batch_per_gpu, "global_rows": batch_per_gpu * world}


class MlpBench:
    def __init__(self, q, rank: int, algo: int, M: int = BATCH):
        from paper_1609_07061_b200 import workloads
        self.q, self.M, self.algo = q, M, algo
        plan = shard_plan(1, rank, M)
        wl = workloads.mnist_mlp(M=M, dims=DIMS, seed=1, stream=plan["stream"])
        self.wl = wl
        self.x_host = wl.X.contiguous().pin_memory()
        self.x = wl.X.cuda()
        self.packed, self.ldws = [], []
        for W in wl.Ws:                                   # weight packing = model load, outside the step
            K, N = W.shape
            ld = ((K + 31) // 32 + 3) // 4 * 4
            out = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
            q.qnn_quantize_pack_sign_t(W.cuda(), K, N, N, out, ld)
            self.packed.append(out); self.ldws.append(ld)
        self.thr = [t.cuda() for t in wl.Ts]
        self.layers = q.make_mlp_layers(self.packed, self.ldws, DIMS[:-1], DIMS[1:], self.thr, [None] * len(self.thr))
        # weights rewritten once in the tensor-core form of their layer (model load, outside the step)
        self.w_tc = q.prepack_mlp_weights(self.layers, self.packed, IN_BITS) if algo in (q.QNN_ALGO_AUTO,) else []
        self.ws = torch.empty(q.qnn_mlp_workspace_bytes(M, IN_BITS, self.layers, algo, 1), dtype=torch.uint8,
                              device="cuda")
        self.scores = torch.empty(M, DIMS[-1], dtype=torch.int32, device="cuda")
        self.scores_host = torch.empty(M, DIMS[-1], dtype=torch.int32).pin_memory()
        # per-call buffers for the instrumented step (same kernels as qnn_mlp_forward, one call per layer)
        self.kw0 = self.ldws[0]
        self.planes = torch.zeros(IN_BITS, M, self.kw0, dtype=torch.int32, device="cuda")
        self.act = [torch.zeros(M, 128, dtype=torch.int32, device="cuda") for _ in range(2)]
        self.actf = [torch.zeros(M, 4096 // 2, dtype=torch.uint8, device="cuda") for _ in range(2)]
        gw = max(q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, DIMS[1], DIMS[0], IN_BITS, 1, algo),
                 q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, 4096, 4096, 1, 1, algo), 256)
        self.gws = torch.empty(gw, dtype=torch.uint8, device="cuda")
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        self.flush_rd = torch.zeros(64 << 20, dtype=torch.int32, device="cuda")
        self.graph = None

    def flush_l2(self):
        """Writes a 256 MiB buffer (evicts every cached input), then reads another 256 MiB so that the dirty
        lines of that write are written back BEFORE the timed region instead of inside it."""
        self.flush_buf.fill_(1)
        self.flush_sink = self.flush_rd.sum()

    def step_calls(self, ev=None):
        """One Algorithm-4 pass on device buffers; `ev` (optional) brackets the dominant product kernel."""
        if self.algo == self.q.QNN_ALGO_AUTO:
            return self.step_forward(ev)
        return self.step_calls_bits(ev)

    def step_forward(self, ev=None):
        """qnn_mlp_forward with prepacked weights: the uint8 input is the int8-form operand of layer 1 (Eq. 8
        recomposed), hidden activations travel as e2m1 values written by the previous product's threshold
        epilogue, down to the 10-unit head, which runs on the tensor cores too since its weights are prepacked."""
        q = self.q
        if ev is not None:
            q.qnn_set_kernel_events_nth(ev[0], ev[1], 1)  # second product kernel = hidden layer 2 (10000 x 4096 x 4096)
        q.qnn_mlp_forward(self.x, self.M, IN_BITS, self.layers, self.scores, self.algo, self.ws)

    def step_calls_bits(self, ev=None):
        """The pass on packed bits with a forced algorithm (plane split, per-call operand rewriting)."""
        q, M = self.q, self.M
        q.qnn_pack_planes_u8(self.x, M, DIMS[0], DIMS[0], IN_BITS, self.planes, self.kw0, M * self.kw0)
        q.qnn_bitplane_gemm_threshold(self.planes, IN_BITS, q.QNN_MODE_U01, self.kw0, M * self.kw0, self.packed[0], 1,
                                      q.QNN_MODE_PM1, self.ldws[0], 0, M, DIMS[1], DIMS[0], self.thr[0], None,
                                      self.act[0], 128, self.algo, self.gws)
        if ev is not None:
            q.qnn_set_kernel_events(ev[0], ev[1])
        q.qnn_xnor_gemm_threshold(self.act[0], 128, self.packed[1], self.ldws[1], M, DIMS[2], DIMS[1], self.thr[1],
                                  None, self.act[1], 128, self.algo, self.gws)
        q.qnn_xnor_gemm_threshold(self.act[1], 128, self.packed[2], self.ldws[2], M, DIMS[3], DIMS[2], self.thr[2],
                                  None, self.act[0], 128, self.algo, self.gws)
        q.qnn_xnor_gemm(self.act[0], 128, self.packed[3], self.ldws[3], M, DIMS[4], DIMS[3], self.scores, DIMS[4],
                        self.algo, self.gws)

    def step_e2e(self):
        """One pass from pinned host memory to scores in pinned host memory.  Small batches (launch-bound) replay a CUDA
        graph built once (input copies, all kernels, the copy back; one launch per pass); large batches, where the input
        copy over PCIe and the layers dominate and the graph gains nothing (measured), use the call-by-call host entry
        point, which overlaps the second half-batch's copy with the first half's layers."""
        if self.algo == self.q.QNN_ALGO_AUTO and self.M <= E2E_GRAPH_MAX_BATCH:
            if self.graph is None:
                self.graph = self.q.MlpGraph(self.x_host, self.M, IN_BITS, self.layers, self.scores_host, self.algo, self.ws,
                                             chunks=E2E_CHUNKS)
            self.graph.launch()
            torch.cuda.current_stream().synchronize()
        else:
            self.q.qnn_mlp_forward_host(self.x_host, self.M, IN_BITS, self.layers, self.scores_host, self.algo, self.ws)

    def step_e2e_calls(self):
        self.q.qnn_mlp_forward_host(self.x_host, self.M, IN_BITS, self.layers, self.scores_host, self.algo, self.ws)


def backward_records(q, flush, rec, reps=5):
    M, Nu, K = BATCH, 4096, 4096                       # batch, units of the layer, its inputs
    emin, emax = -30, 0
    G = q.qnn_logquant_groups(emin, emax)
    g = torch.Generator(device="cuda").manual_seed(6)
    gs = torch.randn(M, Nu, device="cuda", generator=g) * torch.exp2(torch.randint(emin, emax + 1, (M, Nu), device="cuda", generator=g).float())
    for name, transposed, rows, kdim, ncols in (("g_a = LogQuant(g_s) W", 0, M, Nu, K), ("g_W = a^T LogQuant(g_s)", 1, Nu, M, K)):
        kz = (kdim + 31) // 32 * 32
        ld = (kz + 127) // 128 * 128
        a8 = torch.empty(G * rows, ld, dtype=torch.uint8, device="cuda")
        bits = torch.randint(-2**31, 2**31 - 1, (ncols, (kdim + 31) // 32), dtype=torch.int32, device="cuda", generator=g)
        if kdim % 32:
            bits[:, -1] &= (1 << (kdim % 32)) - 1
        b8 = torch.empty(ncols, ld, dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(bits, 1, q.QNN_MODE_PM1, (kdim + 31) // 32, 0, ncols, kdim, q.QNN_FORM_I8, b8, ld)
        part = torch.empty(G * rows, ncols, dtype=torch.int32, device="cuda")
        out = torch.empty(rows, ncols, dtype=torch.int64, device="cuda")
        A = q.tc_operand(a8, ld, q.QNN_FORM_I8, planes=7, mode=q.QNN_MODE_PM1)
        Bo = q.tc_operand(b8, ld, q.QNN_FORM_I8, planes=1, mode=q.QNN_MODE_PM1)
        tag = "g_a" if not transposed else "g_W"
        ms, best = _time_op(lambda: q.qnn_logquant_pack_groups(gs, rows, kdim, Nu, transposed, emin, emax, a8, ld), flush, reps=reps)
        rec(f"alg1_backward_{tag}_pack_groups", ms, best, bytes_=4.0 * M * Nu + float(G) * rows * ld,
            note=f"{name}: fp32 gradient -> {G} int8 group matrices ({'transposed' if transposed else 'row-major'})")

        def whole():
            q.qnn_logquant_pack_groups(gs, rows, kdim, Nu, transposed, emin, emax, a8, ld)
            q.qnn_tc_gemm(A, Bo, G * rows, ncols, kdim, out=part, ldo=ncols)
            q.qnn_logquant_combine(part, G, rows, ncols, ncols, out, ncols)
        ms, best = _time_op(whole, flush, reps=reps)
        rec(f"alg1_backward_{tag}_{rows}x{ncols}x{kdim}_6bit_log_gradients", ms, best, ops=2.0 * rows * ncols * kdim * G,
            note=f"{name}: pack, one int8 product of {G} stacked groups, int64 combine; rate counted per int8 multiply-accumulate issued "
                 f"({2.0 * rows * ncols * kdim / ms / 1e9:.0f} Top/s counted once per 6-bit product)")
        del a8, bits, b8, part, out


def _cpu_baseline(sample_rows: int = 0, budget_s: float = 15.0):
    """The oracle as it stands, on the host cores, on a bounded sample of batch rows of the same workload."""
    import oracle
    from paper_1609_07061_b200 import workloads
    wl = workloads.mnist_mlp(M=BATCH if sample_rows <= 0 else sample_rows, dims=DIMS, seed=1)
    Ws = [oracle.sign(w.numpy()) for w in wl.Ws]
    Ts = [t.numpy() for t in wl.Ts]
    x = wl.X.numpy().astype(np.int32)
    if sample_rows <= 0:
        t0 = time.perf_counter()
        oracle.mlp_forward(x[:8], Ws, Ts)
        t8 = time.perf_counter() - t0
        sample_rows = int(max(8, min(BATCH, 8 * budget_s / max(t8, 1e-3))))
    t0 = time.perf_counter()
    oracle.mlp_forward(x[:sample_rows], Ws, Ts)
    dt = time.perf_counter() - t0
    ops = sum(_ops(sample_rows))
    return {"value": ops / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{sample_rows} of {BATCH} batch rows through all {len(DIMS) - 1} layers, {dt:.2f} s",
            "seconds": dt, "rows": sample_rows}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = 24
    times = []
    base = None
    for i in range(args.warmup + args.steps):
        base = _cpu_baseline(sample_rows=rows)
        if i >= args.warmup:
            times.append(base["seconds"])
    ms = 1e3 * sum(times) / len(times)
    value = sum(_ops(rows)) / (ms / 1e3) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "int64", "data": "synthetic",
        "config": {"workload": "MNIST-shaped binarised MLP 784-4096-4096-4096-10 (Algorithm 4), seed 1; "
                               f"each step = {rows} of {BATCH} batch rows on the CPU oracle"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": base["cores"], "kind": "oracle",
                         "sample": f"{rows} of {BATCH} batch rows per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _time_op(fn, flush, reps=7, warm=3):
    """Median and best device time (ms) of fn(), L2 flushed before every timed call."""
    for _ in range(warm):
        fn()
    ts = []
    for _ in range(reps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts), min(ts)


def _time_graph(fn, flush, n=100, reps=5):
    """Per-call device time (ms) of n back-to-back calls of fn() captured in one CUDA graph: what remains of a small
    operation once launch latency is amortised (the calls inside a replay run warm)."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            for _ in range(n):
                fn()
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); g.replay(); b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b) / n)
    return statistics.median(ts), min(ts)


def convnet_record(q, Bn, flush, rec, reps=7):
    """Times one qnn_convnet_forward call of the Table 7 network at batch Bn (weights prepared once, L2 flushed)."""
    from paper_1609_07061_b200 import workloads
    wln = workloads.cifar_convnet(B=Bn)
    net = q.ConvNet(3, 32, 32, wln.conv_W, wln.conv_pool, wln.fc_W, wln.Ts, wln.flips)
    wsn = net.workspace(Bn)
    xn = wln.X.cuda()
    sn = torch.zeros(Bn, net.n_out, dtype=torch.int32, device="cuda")
    opsn, c_, h_, w_ = 0.0, 3, 32, 32
    for Wc, pool in zip(wln.conv_W, wln.conv_pool):
        opsn += 2.0 * Bn * h_ * w_ * Wc.shape[0] * 9 * c_ * (8 if c_ == 3 else 1)
        c_ = Wc.shape[0]
        if pool:
            h_, w_ = h_ // 2, w_ // 2
    for Wf in wln.fc_W:
        opsn += 2.0 * Bn * Wf.shape[0] * Wf.shape[1]
    ms, best = _time_op(lambda: net.forward(xn, sn, wsn), flush, reps=reps)
    rec(f"table7_convnet_forward_batch{Bn}", ms, best, ops=opsn,
        note=f"{Bn / ms * 1e3:.0f} images/s; 6 conv + 3 FC layers in one qnn_convnet_forward call, weights prepared once")
    # the same call replayed from a CUDA graph (the runner allocates nothing and never synchronises)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        net.forward(xn, sn, wsn)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            net.forward(xn, sn, wsn)
    torch.cuda.synchronize()
    ms, best = _time_op(graph.replay, flush, reps=reps)
    rec(f"table7_convnet_forward_batch{Bn}_one_graph", ms, best, ops=opsn, note=f"{Bn / ms * 1e3:.0f} images/s; the call captured once, one launch per pass")
    del graph


def pipe_peaks(q):
    """Issue-only rate of each pipe, measured in this run with the library's own measurement kernels (every SM
    re-multiplies one resident shared-memory tile pair, or runs xor/popc/add on registers): Tops/s, best of 5."""
    out = {}
    for name, pipe, iters in (("e2m1_tensor", q.QNN_PIPE_TENSOR_FP4, 1500), ("int8_tensor", q.QNN_PIPE_TENSOR_I8, 800),
                              ("popc_alu", q.QNN_PIPE_POPC, 400)):
        ops = q.qnn_pipe_peak_launch(pipe, iters)
        torch.cuda.synchronize()
        best = 1e30
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); q.qnn_pipe_peak_launch(pipe, iters); b.record()
            b.synchronize()
            best = min(best, a.elapsed_time(b))
        out[name] = {"Tops": round(ops / best / 1e9, 1), "ms": round(best, 4), "iters": iters}
    return out


def algo_matrix(q, flush):
    """The competing inner loops measured against each other on the same shapes (whole call from packed bits, L2
    flushed): xor/popc on the CUDA cores, 1-bit mma.sync, int8 and e2m1 on tcgen05 -- and what the library picks."""
    from paper_1609_07061_b200 import workloads
    names = {q.QNN_ALGO_POPC: "popc", q.QNN_ALGO_B1_MMA: "b1_mma", q.QNN_ALGO_TC_I8: "tc_i8", q.QNN_ALGO_TC_FP4: "tc_fp4",
             q.QNN_ALGO_TC_PACKED: "tc_packed"}
    rows = []

    def measure(label, M, N, K, ka, kb, call, ops, reps):
        r = {"shape": label, "binary_ops": ops, "ms": {}, "binary_Tops": {}}
        for al, nm in names.items():
            if al == q.QNN_ALGO_TC_PACKED and M > 1024:
                continue                                   # (re-expands the weights for every 128 rows: a small-batch kernel)
            try:
                ms, best = _time_op(lambda: call(al), flush, reps=reps, warm=2)
            except q.QnnError as e:
                if e.status != q.QNN_ERR_UNSUPPORTED:
                    raise
                continue
            r["ms"][nm] = round(ms, 5)
            r["binary_Tops"][nm] = round(ops / ms / 1e9, 1)
        picked = names[q.qnn_select_algo(M, N, K, ka, kb, q.QNN_MODE_PM1, q.QNN_MODE_PM1)]     # (with a workspace)
        fastest = min(r["ms"], key=r["ms"].get)
        r["selected"] = picked
        r["fastest"] = fastest
        r["selected_is_fastest"] = bool(picked == fastest or r["ms"][picked] <= 1.03 * r["ms"][fastest])
        rows.append(r)

    g = torch.Generator(device="cuda").manual_seed(4)
    for (M, N, K) in ((64, 256, 1024), (128, 256, 1024), (128, 512, 2048), (256, 1024, 1024), (512, 1024, 2048), (100, 4096, 4096),
                      (1024, 1024, 1024), (4096, 4096, 4096), (8192, 8192, 8192)):
        ld = K // 32
        a = torch.randint(-2**31, 2**31 - 1, (M, ld), dtype=torch.int32, device="cuda", generator=g)
        b = torch.randint(-2**31, 2**31 - 1, (N, ld), dtype=torch.int32, device="cuda", generator=g)
        o = torch.empty(M, N, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, q.QNN_ALGO_AUTO), 256), dtype=torch.uint8, device="cuda")
        measure(f"xnor {M}x{N}x{K}", M, N, K, 1, 1, lambda al: q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, o, N, al, ws), 2.0 * M * N * K,
                3 if M >= 8192 else 5)
        del a, b, o, ws
    M, N, K = 700, 4096, 2048
    ld = K // 32
    a = torch.randint(-2**31, 2**31 - 1, (4, M, ld), dtype=torch.int32, device="cuda", generator=g)
    b = torch.randint(-2**31, 2**31 - 1, (4, N, ld), dtype=torch.int32, device="cuda", generator=g)
    o = torch.empty(M, N, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, N, K, 4, 4, q.QNN_ALGO_AUTO), 256), dtype=torch.uint8, device="cuda")
    measure("4bit x 4bit 700x4096x2048", M, N, K, 4, 4,
            lambda al: q.qnn_bitplane_gemm(a, 4, q.QNN_MODE_PM1, ld, M * ld, b, 4, q.QNN_MODE_PM1, ld, N * ld, M, N, K, o, N, al, ws),
            2.0 * M * N * K * 16, 5)
    wl4 = workloads.cifar_conv()
    B, C, H, W = wl4.X.shape; Co = wl4.W.shape[0]
    xb = torch.randint(-2**31, 2**31 - 1, (B, H, W, C // 32), dtype=torch.int32, device="cuda", generator=g)
    wb = torch.randint(-2**31, 2**31 - 1, (Co, 9 * C // 32), dtype=torch.int32, device="cuda", generator=g)
    o4 = torch.empty(B, Co, H, W, dtype=torch.int32, device="cuda")
    w4 = torch.empty(q.qnn_workspace_bytes(q.QNN_OP_CONV2D, B * H * W, Co, 9 * C, 1, 1, q.QNN_ALGO_AUTO), dtype=torch.uint8, device="cuda")
    measure("conv3x3 128x256x16x16 -> 256", B * H * W, Co, 9 * C, 1, 1,
            lambda al: q.qnn_binary_conv2d(xb, B, C, H, W, wb, Co, 3, 3, 1, 1, 1, o4, None, None, None, al, w4), 2.0 * B * H * W * Co * 9 * C, 5)
    return rows


def run_extras(q, bench, peaks, algo):
    """Other paper-shaped workloads, one record each (device time, L2 flushed): packers against the HBM
    roofline, products in binary Tops/s."""
    from paper_1609_07061_b200 import workloads
    recs = []
    hbm = peaks["hbm_gbs"]
    flush = bench.flush_l2

    def rec(name, ms, best, bytes_=None, ops=None, note=None):
        r = {"name": name, "ms": round(ms, 5), "ms_best": round(best, 5)}
        if bytes_ is not None:
            r["GBps"] = round(bytes_ / ms / 1e6, 1)
            r["hbm_frac"] = round(bytes_ / ms / 1e6 / hbm, 4)
        if ops is not None:
            r["binary_Tops"] = round(ops / ms / 1e9, 2)
        if note:
            r["note"] = note
        recs.append(r)

    # config 1: single FC layer, incl. the "cold weights" variant (fp32 -> bits of X and W, then the product)
    wl = workloads.fc_single()
    M, K = wl.X.shape; N = wl.W.shape[1]; ld = K // 32
    Xd, Wd = wl.X.cuda(), wl.W.cuda()
    a = torch.zeros(M, ld, dtype=torch.int32, device="cuda"); b = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
    out = torch.empty(M, N, dtype=torch.int32, device="cuda")
    ws = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, algo), 256), dtype=torch.uint8, device="cuda")
    ms, best = _time_op(lambda: q.qnn_quantize_pack_sign_t(Wd, K, N, N, b, ld), flush)
    rec("c1_pack_W_4096x4096_transposed", ms, best, bytes_=K * N * 4.125)
    ms, best = _time_op(lambda: q.qnn_quantize_pack_sign(Xd, M, K, K, a, ld), flush)
    rec("c1_pack_X_100x4096", ms, best, bytes_=M * K * 4.125, note="roofline time below launch latency")
    ms, best = _time_op(lambda: q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out, N, algo, ws), flush)
    rec("c1_xnor_gemm_100x4096x4096", ms, best, bytes_=(M + N) * ld * 4 + M * N * 4, ops=2.0 * M * N * K)

    # static weights rewritten once in tensor-core form (qnn_tc_prepack); per call only the activations are
    form = q.qnn_tc_form(1, q.QNN_MODE_PM1, 1, q.QNN_MODE_PM1, K)
    rb = q.qnn_tc_row_bytes(K, form)
    wf = torch.empty(N, rb, dtype=torch.uint8, device="cuda"); af = torch.empty(M, rb, dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(b, 1, q.QNN_MODE_PM1, ld, 0, N, K, form, wf, rb)

    def warm_prepacked():
        q.qnn_tc_prepack(a, 1, q.QNN_MODE_PM1, ld, 0, M, K, form, af, rb)
        q.qnn_tc_gemm(q.tc_operand(af, rb, form), q.tc_operand(wf, rb, form), M, N, K, out, N)
    ms, best = _time_op(warm_prepacked, flush)
    rec("c1_xnor_gemm_100x4096x4096_prepacked_weights", ms, best, bytes_=(M + N) * ld * 4 + M * N * 4, ops=2.0 * M * N * K)

    def cold():
        q.qnn_quantize_pack_sign(Xd, M, K, K, a, ld)
        q.qnn_quantize_pack_sign_t(Wd, K, N, N, b, ld)
        q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out, N, algo, ws)
    ms, best = _time_op(cold, flush)
    rec("c1_layer_cold_weights", ms, best, bytes_=(M * K + K * N) * 4.0 + 2 * (M + N) * ld * 4 + M * N * 4,
        ops=2.0 * M * N * K)

    # the same cold layer without packed planes in between: fp32 -> tensor-core form (one pass each), then the product
    form1 = q.qnn_tc_form(1, q.QNN_MODE_PM1, 1, q.QNN_MODE_PM1, K)
    rb1 = q.qnn_tc_row_bytes(K, form1)
    xf1 = torch.empty(M, rb1, dtype=torch.uint8, device="cuda"); wf1 = torch.empty(N, rb1, dtype=torch.uint8, device="cuda")

    def cold_direct():
        q.qnn_quantize_form_sign(Xd, M, K, K, form1, xf1, rb1)
        q.qnn_quantize_form_sign_t(Wd, K, N, N, form1, wf1, rb1)
        q.qnn_tc_gemm(q.tc_operand(xf1, rb1, form1), q.tc_operand(wf1, rb1, form1), M, N, K, out, N)
    ms, best = _time_op(cold_direct, flush)
    rec("c1_layer_cold_weights_fp32_to_form", ms, best, bytes_=(M * K + K * N) * 4.0 + 2 * (M + N) * rb1 + M * N * 4, ops=2.0 * M * N * K,
        note="three launches: two quantisers that write the tensor-core form directly, then the product")
    ms, best = _time_op(lambda: q.qnn_quantize_form_sign_t(Wd, K, N, N, form1, wf1, rb1), flush)
    rec("c1_quantize_form_W_4096x4096_transposed", ms, best, bytes_=K * N * 4.5)
    # ... and as ONE pass over the fp32 weights: binarised while they stream, multiplied on the tensor cores
    wsf = torch.empty(q.qnn_fc_sign_f32_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    ms, best = _time_op(lambda: q.qnn_fc_sign_f32(Xd, M, K, K, Wd, N, N, out, N, wsf), flush)
    rec("c1_layer_cold_weights_one_pass", ms, best, bytes_=(M * K + K * N) * 4.0 + M * N * 4, ops=2.0 * M * N * K,
        note="qnn_fc_sign_f32: weights read once as fp32, nothing packed written; bytes = fp32 inputs + int32 output")

    # ... and 40 such passes back to back on four copies of the weights (268 MB, more than twice the L2: every pass reads
    # its weights from HBM) -- what the kernel sustains once the launch and the quantiser before it overlap the previous pass
    Wcopies = [Wd] + [Wd.clone() for _ in range(3)]

    def cold_many():
        for i in range(40):
            q.qnn_fc_sign_f32(Xd, M, K, K, Wcopies[i % 4], N, N, out, N, wsf)
    cold_many()
    torch.cuda.synchronize()
    tsm = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); cold_many(); e1.record()
        e1.synchronize()
        tsm.append(e0.elapsed_time(e1) / 40)
    rec("c1_layer_cold_weights_one_pass_x40_back_to_back", statistics.median(tsm), min(tsm), bytes_=(M * K + K * N) * 4.0 + M * N * 4,
        ops=2.0 * M * N * K, note="per pass; 40 passes in a row, weights rotating over four copies (268 MB) so that each pass reads them from HBM")
    del Wcopies

    # Items whose roofline time is below a few microseconds cannot approach it in a single launch (a launch alone costs
    # 3-5 us): the same calls 100 times back to back inside one CUDA graph show what is left without the launch latency.
    ms, best = _time_graph(lambda: q.qnn_quantize_pack_sign(Xd, M, K, K, a, ld), flush)
    rec("c1_pack_X_100x4096_x100_in_one_graph", ms, best, bytes_=M * K * 4.125, note="per call; 100 calls in one CUDA graph")
    ms, best = _time_graph(lambda: q.qnn_xnor_gemm(a, ld, b, ld, M, N, K, out, N, algo, ws), flush)
    rec("c1_xnor_gemm_100x4096x4096_x100_in_one_graph", ms, best, bytes_=(M + N) * ld * 4 + M * N * 4, ops=2.0 * M * N * K,
        note="per call; 100 calls in one CUDA graph")
    ms, best = _time_graph(warm_prepacked, flush)
    rec("c1_xnor_gemm_prepacked_weights_x100_in_one_graph", ms, best, bytes_=(M + N) * ld * 4 + M * N * 4, ops=2.0 * M * N * K,
        note="per call; 100 calls in one CUDA graph")
    del Xd, Wd

    # large row-major sign pack and standalone threshold pack (HBM-bound steps on tensors >= 32 MB)
    n = 8192
    big = torch.randn(n, n, device="cuda")
    pk = torch.zeros(n, n // 32, dtype=torch.int32, device="cuda")
    ms, best = _time_op(lambda: q.qnn_quantize_pack_sign(big, n, n, n, pk, n // 32), flush)
    rec("pack_sign_rowmajor_8192x8192", ms, best, bytes_=n * n * 4.125)
    ms, best = _time_op(lambda: q.qnn_quantize_pack_sign_t(big, n, n, n, pk, n // 32), flush)
    rec("pack_sign_transposed_8192x8192", ms, best, bytes_=n * n * 4.125)
    s = torch.randint(-100, 100, (BATCH, 4096), dtype=torch.int32, device="cuda")
    tb = torch.zeros(BATCH, 128, dtype=torch.int32, device="cuda")
    ms, best = _time_op(lambda: q.qnn_threshold_pack(s, BATCH, 4096, 4096, bench.thr[0], None, tb, 128), flush)
    rec("c2_threshold_pack_10000x4096", ms, best, bytes_=BATCH * 4096 * 4.125)
    del big, s
    ms, best = _time_op(lambda: q.qnn_pack_planes_u8(bench.x, BATCH, 784, 784, 8, bench.planes, bench.kw0,
                                                     BATCH * bench.kw0), flush)
    rec("c2_pack_planes_u8_10000x784", ms, best, bytes_=BATCH * 784 * 2.0, note="near launch latency")

    # config 3: 1-bit x 2-bit AlexNet FC layers
    wl3 = workloads.alexnet_fc()
    for i, (X, W) in enumerate(zip(wl3.Xs, wl3.Ws)):
        M, K = X.shape; N = W.shape[1]; ld = K // 32
        ap = torch.zeros(2, M, ld, dtype=torch.int32, device="cuda"); bp = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_kbit(X.cuda(), M, K, K, 2, 0.0, 1.0, ap, ld, M * ld)
        q.qnn_quantize_pack_sign_t(W.cuda(), K, N, N, bp, ld)
        o = torch.empty(M, N, dtype=torch.int32, device="cuda")
        w3 = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, N, K, 2, 1, algo), 256), dtype=torch.uint8, device="cuda")
        ms, best = _time_op(lambda: q.qnn_bitplane_gemm(ap, 2, q.QNN_MODE_U01, ld, M * ld, bp, 1, q.QNN_MODE_PM1, ld, 0,
                                                        M, N, K, o, N, algo, w3), flush)
        rec(f"c3_fc{6 + i}_2bit_x_1bit_{M}x{N}x{K}", ms, best, ops=2.0 * M * N * K * 2)
        f3 = q.qnn_tc_form(2, q.QNN_MODE_U01, 1, q.QNN_MODE_PM1, K)
        rb3 = q.qnn_tc_row_bytes(K, f3)
        wf3 = torch.empty(N, rb3, dtype=torch.uint8, device="cuda"); af3 = torch.empty(M, rb3, dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(bp, 1, q.QNN_MODE_PM1, ld, 0, N, K, f3, wf3, rb3)

        def fc_prepacked():
            q.qnn_tc_prepack(ap, 2, q.QNN_MODE_U01, ld, M * ld, M, K, f3, af3, rb3)
            q.qnn_tc_gemm(q.tc_operand(af3, rb3, f3, 2, q.QNN_MODE_U01), q.tc_operand(wf3, rb3, f3), M, N, K, o, N)
        ms, best = _time_op(fc_prepacked, flush)
        rec(f"c3_fc{6 + i}_prepacked_weights", ms, best, ops=2.0 * M * N * K * 2)

    # config 4: CIFAR conv
    wl4 = workloads.cifar_conv()
    B, C, H, Wd_ = wl4.X.shape; Co = wl4.W.shape[0]
    xb = torch.zeros(B, H, Wd_, C // 32, dtype=torch.int32, device="cuda")
    wb = torch.zeros(Co, 9 * C // 32, dtype=torch.int32, device="cuda")
    x4 = wl4.X.cuda()
    q.qnn_pack_conv_weights(wl4.W.cuda(), Co, C, 3, 3, wb)
    ms, best = _time_op(lambda: q.qnn_quantize_pack_sign_nchw(x4, B, C, H, Wd_, xb), flush)
    rec("c4_pack_sign_nchw_128x256x16x16", ms, best, bytes_=B * C * H * Wd_ * 4.125)
    o4 = torch.empty(B, Co, H, Wd_, dtype=torch.int32, device="cuda")
    ob = torch.zeros(B, H, Wd_, Co // 32, dtype=torch.int32, device="cuda")
    t4 = wl4.T.cuda()
    w4 = torch.empty(q.qnn_workspace_bytes(q.QNN_OP_CONV2D, B * H * Wd_, Co, 9 * C, 1, 1, algo), dtype=torch.uint8, device="cuda")
    ops4 = 2.0 * B * H * Wd_ * Co * 9 * C
    ms, best = _time_op(lambda: q.qnn_binary_conv2d(xb, B, C, H, Wd_, wb, Co, 3, 3, 1, 1, 1, o4, None, None, None, algo, w4), flush)
    rec("c4_conv3x3_int32_out", ms, best, ops=ops4)
    ms, best = _time_op(lambda: q.qnn_binary_conv2d(xb, B, C, H, Wd_, wb, Co, 3, 3, 1, 1, 1, None, t4, None, ob, algo, w4), flush)
    rec("c4_conv3x3_threshold_bits_out", ms, best, ops=ops4)
    prep = torch.empty(q.qnn_conv_prepared_bytes(Co, C, 3, 3, 1), dtype=torch.uint8, device="cuda")
    q.qnn_conv_prepare(wb, Co, C, 3, 3, 1, 1, prep)
    f4 = q.qnn_conv_form(C)
    xf4 = torch.empty(B * H * Wd_, q.qnn_tc_row_bytes(C, f4), dtype=torch.uint8, device="cuda")
    q.qnn_tc_prepack(xb, 1, q.QNN_MODE_PM1, C // 32, 0, B * H * Wd_, C, f4, xf4, xf4.shape[1])
    of4 = torch.empty(B * H * Wd_, q.qnn_tc_row_bytes(Co, f4), dtype=torch.uint8, device="cuda")
    ms, best = _time_op(lambda: q.qnn_binary_conv2d_prepared(xb, 0, B, C, H, Wd_, prep, Co, 3, 3, 1, out_nchw=o4, ws=w4), flush)
    rec("c4_conv3x3_prepared_filters_int32_out", ms, best, ops=ops4)
    ms, best = _time_op(lambda: q.qnn_binary_conv2d_prepared(xf4, f4, B, C, H, Wd_, prep, Co, 3, 3, 1, thr=t4, out_form=of4,
                                                              out_form_kind=f4), flush)
    rec("c4_conv3x3_prepared_filters_form_in_form_out", ms, best, ops=ops4, note="mid-network layer: activations arrive and leave in tensor-core form")

    # Algorithm 4 end to end from host buffers at small batches: call by call against one CUDA graph per pass
    for Bm in (100, 1000):
        mb = MlpBench(q, 0, algo, M=Bm)
        opsb = sum(_ops(Bm))
        ms, best = _time_op(mb.step_e2e_calls, flush)
        rec(f"mlp_e2e_batch{Bm}_call_by_call", ms, best, ops=opsb, note="qnn_mlp_forward_host: copies, kernels and the copy back issued one by one")
        ms, best = _time_op(mb.step_e2e, flush)
        rec(f"mlp_e2e_batch{Bm}_one_graph", ms, best, ops=opsb, note="the same pass replayed as one CUDA graph (qnn_mlp_graph_launch)")
        del mb
    ms, best = _time_op(bench.step_e2e_calls, flush)
    rec(f"mlp_e2e_batch{BATCH}_call_by_call", ms, best, ops=sum(_ops(BATCH)), note="qnn_mlp_forward_host, 2 chunks")

    # the whole CIFAR-10 ConvNet of Table 7 (first layer on 8-bit pixels, pooled thresholds, FC head), one call per pass
    for Bn in (128, 1024):
        convnet_record(q, Bn, flush, rec)

    # Algorithm 1's backward products of a 4096-unit hidden layer at batch 10000 with 6-bit logarithmic gradients
    # (Eq. 10, 31 exponents = 5 int8 groups): gradient x +-1 weights, and +-1 activations^T x gradient
    backward_records(q, flush, rec)

    # config 5: LSTM gate 4b x 4b and the square sweep
    wl5 = workloads.lstm_gate()
    M, K = wl5.X.shape; N = wl5.W.shape[1]; ld = K // 32
    ap = torch.zeros(4, M, ld, dtype=torch.int32, device="cuda"); bp = torch.zeros(4, N, ld, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_kbit(wl5.X.cuda(), M, K, K, 4, -1.0, 1.0, ap, ld, M * ld)
    q.qnn_quantize_pack_kbit_t(wl5.W.cuda(), K, N, N, 4, -1.0, 1.0, bp, ld, N * ld)
    o = torch.empty(M, N, dtype=torch.int32, device="cuda")
    w5 = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, N, K, 4, 4, algo), 256), dtype=torch.uint8, device="cuda")
    ms, best = _time_op(lambda: q.qnn_bitplane_gemm(ap, 4, q.QNN_MODE_PM1, ld, M * ld, bp, 4, q.QNN_MODE_PM1, ld, N * ld,
                                                    M, N, K, o, N, algo, w5), flush)
    rec("c5_lstm_gate_4bit_x_4bit_700x4096x2048", ms, best, ops=2.0 * M * N * K * 16)
    for n in (1024, 4096, 8192, 16384):
        ld = n // 32
        g = torch.Generator(device="cuda").manual_seed(4)
        a = torch.randint(-2**31, 2**31 - 1, (n, ld), dtype=torch.int32, device="cuda", generator=g)
        b = torch.randint(-2**31, 2**31 - 1, (n, ld), dtype=torch.int32, device="cuda", generator=g)
        o = torch.empty(n, n, dtype=torch.int32, device="cuda")
        wsq = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, n, n, n, 1, 1, algo), 256), dtype=torch.uint8, device="cuda")
        reps = 3 if n >= 8192 else 7
        ms, best = _time_op(lambda: q.qnn_xnor_gemm(a, ld, b, ld, n, n, n, o, n, algo, wsq), flush, reps=reps, warm=2)
        rec(f"c5_square_xnor_gemm_{n}", ms, best, bytes_=2 * n * ld * 4 + n * n * 4.0, ops=2.0 * n ** 3,
            note="random packed words (timing only; parity is covered by the tests)")
        del a, b, o, wsq
    return recs


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--algo", default="auto", choices=["auto", "popc", "tc_i8", "b1_mma", "tc_fp4"])
    ap.add_argument("--no-extras", action="store_true", help="skip the per-config extra records")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--convnet-only", type=int, default=0, metavar="BATCH",
                    help="time only the Table 7 ConvNet forward at this batch and print its record (one GPU)")
    ap.add_argument("--backward-only", action="store_true",
                    help="time only Algorithm 1's backward products with 6-bit logarithmic gradients and print their records (one GPU)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    from paper_1609_07061_b200 import binding as q
    if args.convnet_only > 0:
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

        def flush():
            flush_buf.fill_(1)
            flush_buf.sum()
        out = []
        convnet_record(q, args.convnet_only, flush, lambda name, ms, best, bytes_=None, ops=None, note=None: out.append(
            {"name": name, "ms": round(ms, 5), "ms_best": round(best, 5), "binary_Tops": round(ops / ms / 1e9, 2), "note": note}),
            reps=max(args.steps if args.steps != 200 else 7, 1))
        print(json.dumps(out[0]))
        return
    if args.backward_only:
        flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")

        def flush():
            flush_buf.fill_(1)
            flush_buf.sum()
        out = []

        def rec(name, ms, best, bytes_=None, ops=None, note=None):
            r = {"name": name, "ms": round(ms, 5), "ms_best": round(best, 5)}
            if bytes_ is not None:
                r["GBps"] = round(bytes_ / ms / 1e6, 1)
            if ops is not None:
                r["int8_Tops"] = round(ops / ms / 1e9, 2)
            r["note"] = note
            out.append(r)
        backward_records(q, flush, rec, reps=max(args.steps if args.steps != 200 else 5, 1))
        print(json.dumps(out))
        return
    rank, world, local = _dist_setup(args.gpus)
    algo = {"auto": q.QNN_ALGO_AUTO, "popc": q.QNN_ALGO_POPC, "tc_i8": q.QNN_ALGO_TC_I8, "b1_mma": q.QNN_ALGO_B1_MMA,
            "tc_fp4": q.QNN_ALGO_TC_FP4}[args.algo]
    peaks = _peaks()
    bench = MlpBench(q, rank, algo)
    per_layer = _ops(BATCH)
    ops_step = sum(per_layer)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident arm ----------------------------------------------------
    sampler = ClockSampler(local)
    sampler.start()
    for _ in range(args.warmup):
        bench.step_calls()
    barrier()
    t_begin = time.time()
    launches0 = q.qnn_launch_count()
    step_ev, dom_ev = [], []
    barrier()
    for _ in range(args.steps):
        bench.flush_l2()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(); d1.record()                         # creates the underlying handles; re-recorded by the library
        s.record()
        bench.step_calls(ev=(d0, d1))
        e.record()
        step_ev.append((s, e)); dom_ev.append((d0, d1))
    barrier()
    launches = q.qnn_launch_count() - launches0
    total_ms = sum(s.elapsed_time(e) for s, e in step_ev)
    dom_ms = sum(a.elapsed_time(b) for a, b in dom_ev) / args.steps
    if q.qnn_device_status() != 0:
        raise SystemExit("device status reports a bounded wait that ran out")

    # ---- end-to-end arm: host buffers through qnn_mlp_forward_host -------------
    for _ in range(3):
        bench.step_e2e()
    barrier()
    e2e_ev = []
    for _ in range(args.steps):
        bench.flush_l2()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record(); bench.step_e2e(); e.record()
        e2e_ev.append((s, e))
    barrier()
    e2e_ms = sum(s.elapsed_time(e) for s, e in e2e_ev)
    if os.environ.get("QNN_BENCH_DEBUG"):
        sys.stderr.write("e2e per step (ms): " + " ".join(f"{s.elapsed_time(e):.3f}" for s, e in e2e_ev) + "\n")
    t_end = time.time()
    clocks = sampler.stop(t_begin, t_end)
    same = bool(torch.equal(bench.scores_host, bench.scores.cpu()))

    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([total_ms, e2e_ms, dom_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms, dom_ms = (float(v) for v in t.cpu())
        ok = torch.tensor([1 if same else 0], device="cuda")
        dist.all_reduce(ok, op=dist.ReduceOp.MIN)
        same = bool(ok.item())

    if rank == 0:
        value = world * ops_step * args.steps / (total_ms / 1e3) / 1e12
        e2e_value = world * ops_step * args.steps / (e2e_ms / 1e3) / 1e12
        resolved = q.qnn_select_algo(BATCH, 4096, 4096, 1, 1, 1, 1) if algo == q.QNN_ALGO_AUTO else algo
        dom_ops = per_layer[1]
        achieved = dom_ops / (dom_ms / 1e3) / 1e12
        if resolved == q.QNN_ALGO_TC_FP4:
            # e2m1 tensor peak = measured bf16 peak x the nominal fp4:bf16 ratio (4).  The kernel is bracketed by its own
            # event pair inside a sub-millisecond step with idle gaps (L2 flush) around it, so it runs at burst clocks.
            bound, peak = "tensor", 4.0 * peaks["bf16_tflops"]
            peak_note = (f"4 x {peaks['source']} burst bf16 ({peaks['bf16_tflops']} TF/s; sustained "
                         f"{peaks['bf16_tflops_sustained']}); one e2m1 MAC = one +-1 product")
            kernel = "tcgen05 kind::mxf4 xnor product 10000x4096x4096, threshold epilogue (gemm_tc_kernel<FP4>)"
            dtype = "fp4 (e2m1 values, unit scales, fp32 accumulate: exact integers)"
        elif resolved == q.QNN_ALGO_TC_I8:
            bound, peak = "tensor", 2.0 * peaks["bf16_tflops"]
            peak_note = (f"2 x {peaks['source']} burst bf16 ({peaks['bf16_tflops']} TF/s; sustained "
                         f"{peaks['bf16_tflops_sustained']}); one int8 MAC = one +-1 product")
            kernel = "tcgen05 kind::i8 xnor product 10000x4096x4096, threshold epilogue (gemm_tc_kernel<I8>)"
            dtype = "int8"
        else:
            # xor+popc+add on the CUDA cores: the popc unit issues 16 lanes/clk/SM -> 148 SM x 16 x 64 binary ops/clk
            mhz = clocks["sm_max_mhz"] or peaks["sm_max_mhz"]
            bound, peak = "alu", 148 * 16 * 64 * mhz * 1e6 / 1e12
            peak_note = f"148 SMs x 16 popc/clk x 64 binary ops x {mhz:.0f} MHz (popc-pipe bound of the plain xor/popc/add loop)"
            kernel = "popc xnor product 10000x4096x4096" if resolved == q.QNN_ALGO_POPC else "b1 mma.sync product 10000x4096x4096"
            dtype = "u32"
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": dtype, "data": "synthetic",
            "config": {"workload": "MNIST-shaped binarised MLP 784-4096-4096-4096-10 (Algorithm 4), batch 10000 per GPU, "
                                   "8-bit inputs as 8 bit-planes (K 784 padded to 800+), thresholds in [-64,64], seed 1",
                       "global_batch": BATCH * world, "parallelism": f"dp{world} (independent batch shards, no collective)",
                       "algo": {0: "auto", 1: "popc", 2: "tc_i8", 3: "b1_mma", 4: "tc_fp4"}[resolved],
                       "l2": "flushed between steps (256 MiB device fill, then a 256 MiB read so no dirty lines remain; untimed)",
                       "weights": "packed and rewritten in tensor-core form once at load (not in the step)"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": BATCH * DIMS[0],
                    "d2h_bytes_per_step": BATCH * DIMS[-1] * 4, "ms_per_step": e2e_ms / args.steps,
                    "matches_device_arm": same,
                    "api": "qnn_mlp_forward_host (pinned host buffers in, pinned host scores out, two overlapped half-batches)"},
            "gpu_launches": int(launches),
            "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                       "samples": clocks["samples"]},
            "roofline": {"bound": bound, "achieved": achieved, "peak": peak, "unit": "Tops/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_BYTES.get(kernel), "kernel": kernel, "ms_per_launch": dom_ms,
                         "peak_note": peak_note},
            "per_layer_binary_ops": per_layer,
        }
        # the same step counted once per integer multiply-accumulate (layer 1's eight planes are one int8 product)
        int_ops_step = sum(_ops(BATCH, count_planes=False))
        line["int_ops_value"] = world * int_ops_step * args.steps / (total_ms / 1e3) / 1e12
        line["int_ops_unit"] = "Tops/s (2*M*N*K per layer: operations the tensor cores issue)"
        if world == 1:
            try:
                pk = pipe_peaks(q)
                line["pipe_peaks"] = pk
                key = {q.QNN_ALGO_TC_FP4: "e2m1_tensor", q.QNN_ALGO_TC_I8: "int8_tensor"}.get(resolved, "popc_alu")
                line["roofline"]["measured_pipe_peak"] = pk[key]["Tops"]
                line["roofline"]["frac_of_measured_pipe_peak"] = achieved / pk[key]["Tops"]
                line["roofline"]["pipe_peak_note"] = ("issue-only loop of the same instruction on resident shared-memory tiles, every SM, "
                                                      "measured in this run (no loads, no epilogue)")
            except Exception as ex:
                line["pipe_peaks_error"] = repr(ex)
        if not args.no_cpu_baseline and world == 1:
            cb = _cpu_baseline()
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
        if not args.no_extras and world == 1:
            try:
                line["extra"] = run_extras(q, bench, peaks, algo)
            except Exception as ex:  # extras never invalidate the headline record
                line["extra_error"] = repr(ex)
            try:
                line["algorithms"] = algo_matrix(q, bench.flush_l2)
            except Exception as ex:
                line["algorithms_error"] = repr(ex)
        line["paper_context"] = "paper: XNOR kernel 23x its own baseline kernel, 3.4x cuBLAS at 8192^3, MLP 7x, on a GTX750 (context only)"
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
