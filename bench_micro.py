"""Times single library calls on seeded paper-shaped inputs (device time, L2 flushed before every timed call).

    python bench_micro.py pack_sign 8192          # fp32 [n, n] -> packed bits, row-major
    python bench_micro.py pack_sign_t 8192        # the transposed (weight) packer
    python bench_micro.py threshold_pack 10000 4096
    python bench_micro.py conv_c4                 # 128 x 256 x 16 x 16, 3x3, prepared bank, form in / form out
    python bench_micro.py conv_c4 pool            # the same with 2x2 pooling inside the call
    python bench_micro.py xnor 4096 4096 4096 --algo popc   # one qnn_xnor_gemm call from packed bits under a forced algorithm
    python bench_micro.py mlp_layer1              # 10000 x 4096 x 784, uint8 codes x +-1 on the int8 tensor path, form out
    python bench_micro.py fc_cold                 # config 1 from fp32 activations and fp32 weights in one pass (qnn_fc_sign_f32)

Prints one JSON line.  Small enough to put under a profiler: one warm-up call and `--reps` timed ones.
"""
from __future__ import annotations

import argparse
import json
import statistics

import os
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1609_07061_b200 import binding as q          # noqa: E402
from paper_1609_07061_b200 import workloads             # noqa: E402


def _time(fn, reps):
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    fn()
    ts = []
    for _ in range(reps):
        flush.fill_(1)
        flush.sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); fn(); b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return statistics.median(ts)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op", choices=["pack_sign", "pack_sign_t", "threshold_pack", "conv_c4", "xnor", "mlp_layer1", "fc_cold"])
    ap.add_argument("args", nargs="*")
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--algo", default="auto", choices=["auto", "popc", "tc_i8", "b1_mma", "tc_fp4", "tc_packed"])
    a = ap.parse_args()
    rec = {"op": a.op}
    if a.op in ("pack_sign", "pack_sign_t"):
        n = int(a.args[0]) if a.args else 8192
        g = torch.Generator(device="cuda").manual_seed(0)
        x = torch.randn(n, n, device="cuda", generator=g)
        out = torch.zeros(n, n // 32, dtype=torch.int32, device="cuda")
        if a.op == "pack_sign":
            ms = _time(lambda: q.qnn_quantize_pack_sign(x, n, n, n, out, n // 32), a.reps)
        else:
            ms = _time(lambda: q.qnn_quantize_pack_sign_t(x, n, n, n, out, n // 32), a.reps)
        rec.update(shape=[n, n], ms=ms, GBps=n * n * 4.125 / ms / 1e6)
    elif a.op == "threshold_pack":
        M = int(a.args[0]) if a.args else 10000
        N = int(a.args[1]) if len(a.args) > 1 else 4096
        g = torch.Generator(device="cuda").manual_seed(0)
        s = torch.randint(-100, 100, (M, N), dtype=torch.int32, device="cuda", generator=g)
        thr = torch.randint(-64, 65, (N,), dtype=torch.int32, device="cuda", generator=g)
        out = torch.zeros(M, N // 32, dtype=torch.int32, device="cuda")
        ms = _time(lambda: q.qnn_threshold_pack(s, M, N, N, thr, None, out, N // 32), a.reps)
        rec.update(shape=[M, N], ms=ms, GBps=M * N * 4.125 / ms / 1e6)
    elif a.op == "xnor":
        M, N, K = (int(v) for v in a.args[:3]) if len(a.args) >= 3 else (4096, 4096, 4096)
        algo = {"auto": q.QNN_ALGO_AUTO, "popc": q.QNN_ALGO_POPC, "tc_i8": q.QNN_ALGO_TC_I8, "b1_mma": q.QNN_ALGO_B1_MMA,
                "tc_fp4": q.QNN_ALGO_TC_FP4, "tc_packed": q.QNN_ALGO_TC_PACKED}[a.algo]
        g = torch.Generator(device="cuda").manual_seed(4)
        ld = (K + 31) // 32
        x = torch.randint(-2**31, 2**31 - 1, (M, ld), dtype=torch.int32, device="cuda", generator=g)
        w = torch.randint(-2**31, 2**31 - 1, (N, ld), dtype=torch.int32, device="cuda", generator=g)
        if K % 32:
            x[:, -1] &= (1 << (K % 32)) - 1
            w[:, -1] &= (1 << (K % 32)) - 1
        o = torch.empty(M, N, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, M, N, K, 1, 1, algo), 256), dtype=torch.uint8, device="cuda")
        ms = _time(lambda: q.qnn_xnor_gemm(x, ld, w, ld, M, N, K, o, N, algo, ws), a.reps)
        rec.update(shape=[M, N, K], algo=a.algo, ms=ms, binary_Tops=2.0 * M * N * K / ms / 1e9)
    elif a.op == "fc_cold":
        wl = workloads.fc_single()
        M, K = wl.X.shape
        N = wl.W.shape[1]
        x, w = wl.X.cuda(), wl.W.cuda()
        o = torch.empty(M, N, dtype=torch.int32, device="cuda")
        ws = torch.empty(q.qnn_fc_sign_f32_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
        ms = _time(lambda: q.qnn_fc_sign_f32(x, M, K, K, w, N, N, o, N, ws), a.reps)
        rec.update(shape=[M, N, K], ms=ms, GBps=((M * K + K * N) * 4.0 + M * N * 4.0) / ms / 1e6)
    elif a.op == "mlp_layer1":
        M, N, K = 10000, 4096, 784
        g = torch.Generator(device="cuda").manual_seed(1)
        pitch = q.qnn_tc_row_bytes(K, q.QNN_FORM_I8)
        x = torch.randint(0, 256, (M, pitch), dtype=torch.uint8, device="cuda", generator=g)
        x[:, K:] = 0
        wbits = torch.randint(-2**31, 2**31 - 1, (N, (K + 31) // 32), dtype=torch.int32, device="cuda", generator=g)
        wbits[:, -1] &= (1 << (K % 32)) - 1
        wf = torch.empty(N, pitch, dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(wbits, 1, q.QNN_MODE_PM1, wbits.shape[1], 0, N, K, q.QNN_FORM_I8, wf, pitch)
        thr = torch.zeros(N, dtype=torch.int32, device="cuda")
        of = torch.empty(M, q.qnn_tc_row_bytes(N, q.QNN_FORM_FP4), dtype=torch.uint8, device="cuda")
        A = q.tc_operand(x, pitch, q.QNN_FORM_I8, 8, q.QNN_MODE_U01)
        Bo = q.tc_operand(wf, pitch, q.QNN_FORM_I8)
        ms = _time(lambda: q.qnn_tc_gemm(A, Bo, M, N, K, thr=thr, out_form=of, out_form_kind=q.QNN_FORM_FP4, ld_form_bytes=of.shape[1]), a.reps)
        rec.update(shape=[M, N, K], ms=ms, int_Tops=2.0 * M * N * K / ms / 1e9)
    else:
        pool = 1 if (a.args and a.args[0] == "pool") else 0
        wl = workloads.cifar_conv()
        B, C, H, W = wl.X.shape
        Co = wl.W.shape[0]
        xb = torch.zeros(B, H, W, C // 32, dtype=torch.int32, device="cuda")
        wb = torch.zeros(Co, 9 * C // 32, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_sign_nchw(wl.X.cuda(), B, C, H, W, xb)
        q.qnn_pack_conv_weights(wl.W.cuda(), Co, C, 3, 3, wb)
        prep = torch.empty(q.qnn_conv_prepared_bytes(Co, C, 3, 3, 1), dtype=torch.uint8, device="cuda")
        q.qnn_conv_prepare(wb, Co, C, 3, 3, 1, 1, prep)
        form = q.qnn_conv_form(C)
        xf = torch.empty(B * H * W, q.qnn_tc_row_bytes(C, form), dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(xb, 1, q.QNN_MODE_PM1, C // 32, 0, B * H * W, C, form, xf, xf.shape[1])
        rows = B * (H // 2) * (W // 2) if pool else B * H * W
        of = torch.empty(rows, q.qnn_tc_row_bytes(Co, form), dtype=torch.uint8, device="cuda")
        thr = wl.T.cuda()
        ms = _time(lambda: q.qnn_binary_conv2d_prepared(xf, form, B, C, H, W, prep, Co, 3, 3, 1, thr=thr, out_form=of, out_form_kind=form,
                                                        pool2x2=pool), a.reps)
        rec.update(shape=[B, C, H, W, Co], pool=pool, ms=ms, binary_Tops=2.0 * B * H * W * Co * 9 * C / ms / 1e9)
    print(json.dumps(rec))


if __name__ == "__main__":
    main()
