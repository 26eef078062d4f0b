"""GPU parity on the paper-shaped workloads: convolution, the Algorithm-4 MLP, k-bit FC layers, big squares."""
import numpy as np
import pytest
import torch

import oracle
from paper_1609_07061_b200 import workloads
from util import Guarded, as_i32_words, dev, pack_bits_ref, unpack_words, words_np, words_per_row

pytestmark = pytest.mark.gpu

ALGOS = [1, 2, 4, 0]       # POPC, TC_I8, TC_FP4, AUTO


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _skip_unsupported(q, e):
    if e.status == q.QNN_ERR_UNSUPPORTED:
        pytest.skip(str(e))
    raise e


def _conv_gpu(q, X, Wt, T, flip, stride, pad, pad_bit, algo, want_int=True, want_bits=True):
    B, C, H, W = X.shape
    Cout, _, KH, KW = Wt.shape
    Ho = (H + 2 * pad - KH) // stride + 1
    Wo = (W + 2 * pad - KW) // stride + 1
    cw = words_per_row(C)
    xb = torch.zeros(B, H, W, cw, dtype=torch.int32, device="cuda")
    wb = torch.zeros(Cout, KH * KW * cw, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign_nchw(dev(X), B, C, H, W, xb)
    q.qnn_pack_conv_weights(dev(Wt), Cout, C, KH, KW, wb)
    out = Guarded((B, Cout, Ho, Wo), torch.int32, fill=-7) if want_int else None
    bits = Guarded((B, Ho, Wo, words_per_row(Cout)), torch.int32, fill=0) if want_bits else None
    n = q.qnn_workspace_bytes(q.QNN_OP_CONV2D, B * Ho * Wo, Cout, KH * KW * 32 * cw, 1, 1, algo)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    try:
        q.qnn_binary_conv2d(xb, B, C, H, W, wb, Cout, KH, KW, stride, pad, pad_bit, out.t if out else None,
                            dev(T) if want_bits else None, dev(flip) if (want_bits and flip is not None) else None,
                            bits.t if bits else None, algo, ws)
    except q.QnnError as e:
        _skip_unsupported(q, e)
    torch.cuda.synchronize()
    if out: out.check()
    if bits: bits.check()
    return (out.t.cpu().numpy() if out else None), (words_np(bits.t) if bits else None)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("B,C,H,W,Co,KH,KW,stride,pad,pad_bit", [
    (2, 3, 5, 6, 4, 3, 3, 1, 1, 1), (1, 33, 4, 4, 5, 3, 3, 1, 1, 1), (2, 64, 8, 8, 70, 3, 3, 1, 1, 1),
    (2, 40, 7, 5, 33, 1, 1, 1, 0, 1), (1, 32, 9, 9, 16, 3, 3, 2, 1, 1), (1, 16, 6, 6, 8, 5, 3, 1, 2, 0),
    (3, 256, 16, 16, 256, 3, 3, 1, 1, 1),
    # geometries of the implicit tensor-core path: ragged tiles, W not dividing 128, -1 padding, 5x5, 7x7, one row per tile
    (2, 128, 13, 12, 70, 3, 3, 1, 1, 0), (1, 256, 7, 20, 33, 5, 5, 1, 2, 1), (2, 128, 5, 128, 16, 3, 3, 1, 1, 1),
    (1, 256, 40, 3, 8, 3, 3, 1, 1, 1), (2, 512, 9, 9, 40, 1, 1, 1, 0, 1), (1, 128, 6, 5, 9, 7, 7, 1, 3, 0),
    (5, 256, 3, 2, 300, 3, 3, 1, 1, 1)])
def test_conv2d(q, B, C, H, W, Co, KH, KW, stride, pad, pad_bit, algo):
    rng = np.random.default_rng(B + C + H + Co)
    X = rng.standard_normal((B, C, H, W)).astype(np.float32)
    Wt = rng.uniform(-1, 1, (Co, C, KH, KW)).astype(np.float32)
    T = rng.integers(-16, 17, Co).astype(np.int32)
    flip = rng.integers(0, 2, Co).astype(np.uint8)
    want = oracle.conv2d(oracle.sign(X), oracle.sign(Wt), stride, pad, 1 if pad_bit else -1)
    got, bits = _conv_gpu(q, X, Wt, T, flip, stride, pad, pad_bit, algo)
    np.testing.assert_array_equal(got, want)
    Bn, _, Ho, Wo = want.shape
    rows = want.transpose(0, 2, 3, 1).reshape(-1, Co)
    np.testing.assert_array_equal(unpack_words(bits.reshape(-1, words_per_row(Co)), Co), oracle.threshold(rows, T, flip))
    # bits-only and int-only calls agree with the combined call
    got2, _ = _conv_gpu(q, X, Wt, T, flip, stride, pad, pad_bit, algo, want_int=True, want_bits=False)
    _, bits2 = _conv_gpu(q, X, Wt, T, flip, stride, pad, pad_bit, algo, want_int=False, want_bits=True)
    np.testing.assert_array_equal(got2, want)
    np.testing.assert_array_equal(bits2, bits)


@pytest.mark.parametrize("algo", ALGOS)
def test_cifar_conv_config_sampled(q, algo):
    """Config 4 at full size on the GPU; the oracle checks sixteen whole images spread over the batch."""
    wl = workloads.cifar_conv()
    X, Wt, T = wl.X.numpy(), wl.W.numpy(), wl.T.numpy()
    got, bits = _conv_gpu(q, X, Wt, T, None, 1, 1, 1, algo)
    ws = oracle.sign(Wt)
    for b in (0, 1, 7, 8, 15, 16, 31, 32, 63, 64, 65, 95, 96, 120, 126, 127):
        want = oracle.conv2d(oracle.sign(X[b:b + 1]), ws, 1, 1, 1)
        np.testing.assert_array_equal(got[b:b + 1], want)
        rows = want.transpose(0, 2, 3, 1).reshape(-1, 256)
        np.testing.assert_array_equal(unpack_words(bits[b].reshape(-1, 8), 256), oracle.threshold(rows, T))
    # property over the whole output: parity and bound of a +-1 sum of 2304 terms
    assert np.all(np.abs(got) <= 2304) and np.all(got % 2 == 0)


def _mlp_gpu(q, wl, M, algo, host=False, in_bits=8, prepack=False):
    dims = wl.dims
    packed, ldws = [], []
    for W in wl.Ws:
        K, N = W.shape
        ld = (words_per_row(K) + 3) // 4 * 4
        out = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_sign_t(W.cuda(), K, N, N, out, ld)
        packed.append(out); ldws.append(ld)
    thr = [t.cuda() for t in wl.Ts]
    layers = q.make_mlp_layers(packed, ldws, dims[:-1], dims[1:], thr, [None] * len(thr))
    keep = q.prepack_mlp_weights(layers, packed, in_bits) if prepack else None   # noqa: F841 (keeps the buffers alive)
    n = q.qnn_mlp_workspace_bytes(M, in_bits, layers, algo, 1 if host else 0)
    ws = torch.empty(n, dtype=torch.uint8, device="cuda")
    try:
        if host:
            xh = wl.X[:M].contiguous().pin_memory()
            sh = torch.empty(M, dims[-1], dtype=torch.int32).pin_memory()
            q.qnn_mlp_forward_host(xh, M, in_bits, layers, sh, algo, ws)
            return sh.numpy().copy()
        scores = Guarded((M, dims[-1]), torch.int32, fill=-7)
        q.qnn_mlp_forward(wl.X[:M].cuda(), M, in_bits, layers, scores.t, algo, ws)
        torch.cuda.synchronize()
        scores.check()
        return scores.t.cpu().numpy()
    except q.QnnError as e:
        _skip_unsupported(q, e)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("M,dims", [(1, (784, 64, 10)), (37, (50, 40, 24, 10)), (200, (784, 512, 256, 10)),
                                    (130, (100, 300, 10)), (5, (33, 7))])
def test_mlp_forward_small(q, M, dims, algo):
    wl = workloads.mnist_mlp(M=M, dims=dims, seed=1)
    want = oracle.mlp_forward(wl.X.numpy().astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                              [t.numpy() for t in wl.Ts])
    np.testing.assert_array_equal(_mlp_gpu(q, wl, M, algo), want)
    np.testing.assert_array_equal(_mlp_gpu(q, wl, M, algo, host=True), want)


@pytest.mark.parametrize("algo", [2, 4, 0])
@pytest.mark.parametrize("M,dims,in_bits", [(37, (50, 40, 24, 10), 8), (300, (784, 512, 256, 10), 8), (130, (100, 300, 10), 8),
                                            (129, (96, 160, 33), 4), (2100, (784, 1024, 1024, 10), 8)])
def test_mlp_forward_prepacked_weights(q, M, dims, in_bits, algo):
    """Weights rewritten once in their layer's tensor-core form (w_tc) give the same scores as per-call rewriting,
    also when a layer is large enough for the automatic choice to take the tensor-core chain."""
    wl = workloads.mnist_mlp(M=M, dims=dims, seed=1)
    x = wl.X.numpy().astype(np.int32) & ((1 << in_bits) - 1)
    want = oracle.mlp_forward(x, [oracle.sign(w.numpy()) for w in wl.Ws], [t.numpy() for t in wl.Ts])
    np.testing.assert_array_equal(_mlp_gpu(q, wl, M, algo, in_bits=in_bits, prepack=True), want)
    np.testing.assert_array_equal(_mlp_gpu(q, wl, M, algo, host=True, in_bits=in_bits, prepack=True), want)


@pytest.mark.parametrize("prepack", [False, True])
def test_mnist_mlp_config_auto_chain(q, prepack):
    """Config 2 at full size on the automatic choice: uint8 input fed straight to the int8 product, hidden
    activations chained in e2m1 form, packed bits only in front of the 10-unit head."""
    wl = workloads.mnist_mlp()
    got = _mlp_gpu(q, wl, 10000, 0, prepack=prepack)
    rows = np.array([0, 1, 63, 64, 127, 128, 129, 255, 256, 1000, 4095, 4096, 5000, 7777, 9983, 9984, 9985, 9998, 9999])
    want = oracle.mlp_forward(wl.X.numpy()[rows].astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                              [t.numpy() for t in wl.Ts])
    np.testing.assert_array_equal(got[rows], want)
    assert q.qnn_device_status() == 0


def test_mnist_mlp_config_every_row(q):
    """Config 2 at full size, the launch configuration bench.py times (automatic choice, prepacked weights):
    ALL 10000 rows of scores against the oracle's Algorithm 4, so that one wrong bit in any layer of any row shows."""
    wl = workloads.mnist_mlp()
    got = _mlp_gpu(q, wl, 10000, 0, prepack=True)
    want = oracle.mlp_forward(wl.X.numpy().astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                              [t.numpy() for t in wl.Ts])
    np.testing.assert_array_equal(got, want)
    np.testing.assert_array_equal(_mlp_gpu(q, wl, 10000, 0, host=True, prepack=True), want)
    assert q.qnn_device_status() == 0


@pytest.mark.parametrize("algo", ALGOS)
def test_mnist_mlp_config_sampled(q, algo):
    """Config 2 at full size (batch 10000, the launch configuration bench.py times); batch rows are independent,
    so the oracle runs the whole network on a sample of rows spread over several tiles and the ragged tail."""
    wl = workloads.mnist_mlp()
    got = _mlp_gpu(q, wl, 10000, algo)
    rows = np.array([0, 1, 63, 64, 127, 128, 129, 255, 256, 1000, 4095, 4096, 5000, 7777, 9983, 9984, 9985, 9998, 9999])
    want = oracle.mlp_forward(wl.X.numpy()[rows].astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                              [t.numpy() for t in wl.Ts])
    np.testing.assert_array_equal(got[rows], want)
    # properties that hold for every row: scores have the parity of K = 4096 and are bounded by it
    assert np.all(got % 2 == 0) and np.all(np.abs(got) <= 4096)
    np.testing.assert_array_equal(_mlp_gpu(q, wl, 10000, algo, host=True), got)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("layer", [0, 1, 2])
def test_alexnet_fc_config(q, layer, algo):
    """Config 3: 2-bit activations on [0,1] x 1-bit weights, GPU quantisers + bit-plane product; oracle on sampled rows."""
    wl = workloads.alexnet_fc()
    X, W = wl.Xs[layer], wl.Ws[layer]
    M, K = X.shape
    N = W.shape[1]
    ld = words_per_row(K)
    ap = torch.zeros(2, M, ld, dtype=torch.int32, device="cuda")
    bp = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_kbit(X.cuda(), M, K, K, 2, 0.0, 1.0, ap, ld, M * ld)
    q.qnn_quantize_pack_sign_t(W.cuda(), K, N, N, bp, ld)
    out = Guarded((M, N), torch.int32, fill=-7)
    n = q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, N, K, 2, 1, algo)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")
    try:
        q.qnn_bitplane_gemm(ap, 2, q.QNN_MODE_U01, ld, M * ld, bp, 1, q.QNN_MODE_PM1, ld, 0, M, N, K, out.t, N, algo, ws)
    except q.QnnError as e:
        _skip_unsupported(q, e)
    torch.cuda.synchronize()
    out.check()
    rows = np.array([0, 1, 31, 64, 127, 128, 200, 255])
    codes = oracle.linear_quant_codes(X.numpy()[rows], 2, 0.0, 1.0)
    want = oracle.int_gemm(codes, oracle.sign(W.numpy()))
    np.testing.assert_array_equal(out.t.cpu().numpy()[rows], want)


@pytest.mark.parametrize("algo", ALGOS)
def test_lstm_gate_config(q, algo):
    """Config 5, recurrent part: 4-bit x 4-bit signed levels, 700 x 4096 x 2048; oracle on sampled rows."""
    wl = workloads.lstm_gate()
    M, K = wl.X.shape
    N = wl.W.shape[1]
    ld = words_per_row(K)
    ap = torch.zeros(4, M, ld, dtype=torch.int32, device="cuda")
    bp = torch.zeros(4, N, ld, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_kbit(wl.X.cuda(), M, K, K, 4, -1.0, 1.0, ap, ld, M * ld)
    q.qnn_quantize_pack_kbit_t(wl.W.cuda(), K, N, N, 4, -1.0, 1.0, bp, ld, N * ld)
    out = Guarded((M, N), torch.int32, fill=-7)
    n = q.qnn_workspace_bytes(q.QNN_OP_BITPLANE_GEMM, M, N, K, 4, 4, algo)
    ws = torch.empty(max(n, 256), dtype=torch.uint8, device="cuda")
    try:
        q.qnn_bitplane_gemm(ap, 4, q.QNN_MODE_PM1, ld, M * ld, bp, 4, q.QNN_MODE_PM1, ld, N * ld, M, N, K, out.t, N,
                            algo, ws)
    except q.QnnError as e:
        _skip_unsupported(q, e)
    torch.cuda.synchronize()
    out.check()
    rows = np.array([0, 1, 63, 64, 127, 128, 500, 639, 640, 698, 699])
    va = oracle.codes_to_symmetric(oracle.linear_quant_codes(wl.X.numpy()[rows], 4, -1.0, 1.0), 4)
    vb = oracle.codes_to_symmetric(oracle.linear_quant_codes(wl.W.numpy(), 4, -1.0, 1.0), 4)
    np.testing.assert_array_equal(out.t.cpu().numpy()[rows], oracle.int_gemm(va, vb))


def _square(q, n, algo):
    wl = workloads.square_gemm(n)
    ld = words_per_row(n)
    a = torch.zeros(n, ld, dtype=torch.int32, device="cuda")
    b = torch.zeros(n, ld, dtype=torch.int32, device="cuda")
    Xd = wl.X.cuda()
    q.qnn_quantize_pack_sign(Xd, n, n, n, a, ld)
    del Xd
    Wd = wl.W.cuda()
    q.qnn_quantize_pack_sign_t(Wd, n, n, n, b, ld)
    del Wd
    out = torch.empty(n, n, dtype=torch.int32, device="cuda")
    nws = q.qnn_workspace_bytes(q.QNN_OP_XNOR_GEMM, n, n, n, 1, 1, algo)
    ws = torch.empty(max(nws, 256), dtype=torch.uint8, device="cuda")
    try:
        q.qnn_xnor_gemm(a, ld, b, ld, n, n, n, out, n, algo, ws)
    except q.QnnError as e:
        _skip_unsupported(q, e)
    torch.cuda.synchronize()
    return wl, out


@pytest.mark.parametrize("algo", ALGOS)
def test_square_1024_full(q, algo):
    wl, out = _square(q, 1024, algo)
    np.testing.assert_array_equal(out.cpu().numpy(), oracle.xnor_gemm(wl.X.numpy(), wl.W.numpy()))


def _check_square_sampled_and_checksums(wl, got, n):
    """Exact oracle on sampled full rows and full columns, plus int64 row-sum and column-sum checksums that cover
    every output:  sum_n out[m,n] = a_m . (sum_n w_n)   and   sum_m out[m,n] = (sum_m a_m) . w_n .
    The sign matrices are walked in row blocks so that the 16384^2 case needs no int64 copy of them."""
    X, W = wl.X.numpy(), wl.W.numpy()
    rows = np.array([0, 1, 127, 128, n // 2 + 1, n - 129, n - 2, n - 1])
    cols = np.array([0, 5, 127, 128, 255, n // 2, n - 128, n - 1])
    np.testing.assert_array_equal(got[rows], oracle.xnor_gemm(X[rows], W))
    np.testing.assert_array_equal(got[:, cols], oracle.xnor_gemm(X, np.ascontiguousarray(W[:, cols])))
    blk = 1024
    w_rowsum = np.empty(n, np.int64)                 # sum_n sign(W)[k, n]
    a_colsum = np.zeros(n, np.int64)                 # sum_m sign(X)[m, k]
    for r0 in range(0, n, blk):
        w_rowsum[r0:r0 + blk] = oracle.sign(W[r0:r0 + blk]).sum(axis=1, dtype=np.int64)
        a_colsum += oracle.sign(X[r0:r0 + blk]).sum(axis=0, dtype=np.int64)
    want_rows = np.empty(n, np.int64)
    want_cols = np.zeros(n, np.int64)
    for r0 in range(0, n, blk):
        want_rows[r0:r0 + blk] = oracle.sign(X[r0:r0 + blk]).astype(np.int64) @ w_rowsum
        want_cols += a_colsum[r0:r0 + blk] @ oracle.sign(W[r0:r0 + blk]).astype(np.int64)
    np.testing.assert_array_equal(got.sum(axis=1, dtype=np.int64), want_rows)
    np.testing.assert_array_equal(got.sum(axis=0, dtype=np.int64), want_cols)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("n", [4096, 8192])
def test_square_large_sampled_and_checksums(q, n, algo):
    """Sizes where the scalar oracle cannot run whole: sampled rows / columns and full-coverage checksums."""
    wl, out = _square(q, n, algo)
    _check_square_sampled_and_checksums(wl, out.cpu().numpy(), n)


@pytest.mark.parametrize("algo", [0, 4])
def test_square_16384_sampled_and_checksums(q, algo):
    """The largest square of the scaling sweep (2^28 outputs, the CTA-pair kernel's tile arithmetic at its
    largest), on the algorithms the automatic choice can take there."""
    n = 16384
    wl, out = _square(q, n, algo)
    got = out.cpu().numpy()
    del out
    torch.cuda.empty_cache()
    assert q.qnn_device_status() == 0
    _check_square_sampled_and_checksums(wl, got, n)


@pytest.mark.parametrize("B,C,H,W,Co,KS,pad_bit", [(2, 256, 16, 16, 256, 3, 1), (2, 128, 13, 12, 70, 3, 0), (1, 256, 7, 20, 33, 5, 1),
                                                  (3, 512, 8, 8, 128, 1, 1)])
@pytest.mark.parametrize("x_as_form", [False, True])
def test_conv2d_prepared_filter_bank(q, B, C, H, W, Co, KS, pad_bit, x_as_form):
    """Filter bank prepared once (tensor-core form + border table), input as packed bits or already in form;
    int32, packed-bit and form outputs of one call against the oracle."""
    pad = KS // 2
    rng = np.random.default_rng(B + C + H + Co + KS)
    X = rng.standard_normal((B, C, H, W)).astype(np.float32)
    Wt = rng.uniform(-1, 1, (Co, C, KS, KS)).astype(np.float32)
    T = rng.integers(-16, 17, Co).astype(np.int32)
    flip = rng.integers(0, 2, Co).astype(np.uint8)
    want = oracle.conv2d(oracle.sign(X), oracle.sign(Wt), 1, pad, 1 if pad_bit else -1)
    cw = words_per_row(C)
    xb = torch.zeros(B, H, W, cw, dtype=torch.int32, device="cuda")
    wb = torch.zeros(Co, KS * KS * cw, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign_nchw(dev(X), B, C, H, W, xb)
    q.qnn_pack_conv_weights(dev(Wt), Co, C, KS, KS, wb)
    form = q.qnn_conv_form(C)
    assert form in (q.QNN_FORM_FP4, q.QNN_FORM_I8)
    prep = torch.empty(q.qnn_conv_prepared_bytes(Co, C, KS, KS, pad), dtype=torch.uint8, device="cuda")
    q.qnn_conv_prepare(wb, Co, C, KS, KS, pad, pad_bit, prep)
    pix_bytes = cw * (32 if form == q.QNN_FORM_I8 else 16)
    x_arg, x_form, ws = xb, 0, torch.empty(B * H * W * pix_bytes + 256, dtype=torch.uint8, device="cuda")
    if x_as_form:
        xf = torch.empty(B * H * W, pix_bytes, dtype=torch.uint8, device="cuda")
        q.qnn_tc_prepack(xb, 1, q.QNN_MODE_PM1, cw, 0, B * H * W, C, form, xf, pix_bytes)
        x_arg, x_form, ws = xf, form, None
    out = Guarded((B, Co, H, W), torch.int32, fill=-7)
    bits = Guarded((B, H, W, words_per_row(Co)), torch.int32, fill=0)
    oform = q.QNN_FORM_FP4
    onb = words_per_row(Co) * 16
    of = Guarded((B * H * W, onb), torch.uint8, fill=0x5C)
    q.qnn_binary_conv2d_prepared(x_arg, x_form, B, C, H, W, prep, Co, KS, KS, pad, out.t, dev(T), dev(flip), bits.t, of.t,
                                 oform, ws)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    rows = want.transpose(0, 2, 3, 1).reshape(-1, Co)
    wbits = oracle.threshold(rows, T, flip)
    np.testing.assert_array_equal(unpack_words(words_np(bits.t).reshape(-1, words_per_row(Co)), Co), wbits)
    # form output: e2m1 nibbles of the thresholded signs, pad columns zero
    E2M1 = {0: 0x0, 1: 0x2, -1: 0xA}
    vals = np.zeros((rows.shape[0], words_per_row(Co) * 32), np.int32)
    vals[:, :Co] = 2 * wbits.astype(np.int32) - 1
    nib = np.vectorize(E2M1.__getitem__)(vals).astype(np.uint8)
    np.testing.assert_array_equal(of.t.cpu().numpy(), (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8))
    for gbuf in (out, bits, of):
        gbuf.check()


def test_conv2d_prepared_chain_two_layers(q):
    """conv -> threshold -> conv with the activations handed over in tensor-core form (no packed bits in between)."""
    rng = np.random.default_rng(5)
    B, C, H, W, C1, C2 = 2, 256, 8, 8, 256, 40
    X = rng.standard_normal((B, C, H, W)).astype(np.float32)
    W1 = rng.uniform(-1, 1, (C1, C, 3, 3)).astype(np.float32)
    W2 = rng.uniform(-1, 1, (C2, C1, 3, 3)).astype(np.float32)
    T = rng.integers(-16, 17, C1).astype(np.int32)
    s1 = oracle.conv2d(oracle.sign(X), oracle.sign(W1), 1, 1, 1)
    h = np.where(s1 >= T[None, :, None, None], 1, -1).astype(np.int32)
    want = oracle.conv2d(h, oracle.sign(W2), 1, 1, 1)
    FP4 = q.QNN_FORM_FP4
    xb = torch.zeros(B, H, W, C // 32, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign_nchw(dev(X), B, C, H, W, xb)
    preps = []
    for Wt, (co, ci) in ((W1, (C1, C)), (W2, (C2, C1))):
        wb = torch.zeros(co, 9 * ci // 32, dtype=torch.int32, device="cuda")
        q.qnn_pack_conv_weights(dev(Wt), co, ci, 3, 3, wb)
        pr = torch.empty(q.qnn_conv_prepared_bytes(co, ci, 3, 3, 1), dtype=torch.uint8, device="cuda")
        q.qnn_conv_prepare(wb, co, ci, 3, 3, 1, 1, pr)
        preps.append(pr)
    hf = torch.empty(B * H * W, C1 // 2, dtype=torch.uint8, device="cuda")
    ws = torch.empty(B * H * W * C // 2 + 256, dtype=torch.uint8, device="cuda")
    q.qnn_binary_conv2d_prepared(xb, 0, B, C, H, W, preps[0], C1, 3, 3, 1, thr=dev(T), out_form=hf, out_form_kind=FP4, ws=ws)
    out = torch.empty(B, C2, H, W, dtype=torch.int32, device="cuda")
    q.qnn_binary_conv2d_prepared(hf, FP4, B, C1, H, W, preps[1], C2, 3, 3, 1, out_nchw=out)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0
    np.testing.assert_array_equal(out.cpu().numpy(), want)


@pytest.mark.parametrize("M,K,N,ldx,ldw", [(100, 4096, 4096, 4096, 4096), (1, 1, 1, 1, 1), (5, 31, 7, 33, 9), (37, 300, 130, 300, 132),
                                           (128, 256, 32, 256, 32), (129, 1000, 257, 1000, 260), (64, 513, 96, 516, 97), (300, 2048, 1000, 2048, 1000)])
def test_fc_sign_f32_weights_read_once(q, M, K, N, ldx, ldw):
    """The small-batch layer straight from fp32 activations and fp32 weights (config 1's shape first; then ragged M, N, K,
    unaligned leading dimensions, several row tiles): every output against the oracle's sign-then-multiply."""
    if (M, K, N) == (100, 4096, 4096):
        wl = workloads.fc_single()
        X, W = wl.X.numpy(), wl.W.numpy()
    else:
        rng = np.random.default_rng(M * 3 + K * 5 + N)
        X = rng.standard_normal((M, ldx)).astype(np.float32)
        W = rng.uniform(-1, 1, (K, ldw)).astype(np.float32)
        sp = np.array([0.0, -0.0, np.nan, np.inf, -np.inf, 1e-45, -1e-45], np.float32)
        W.reshape(-1)[:min(W.size, sp.size)] = sp[:min(W.size, sp.size)]
        X.reshape(-1)[:min(X.size, sp.size)] = sp[::-1][:min(X.size, sp.size)]
    out = Guarded((M, N + 3), torch.int32, fill=-7)
    ws = torch.empty(q.qnn_fc_sign_f32_workspace_bytes(M, K), dtype=torch.uint8, device="cuda")
    q.qnn_fc_sign_f32(dev(X), M, K, X.shape[1], dev(W), N, W.shape[1], out.t, N + 3, ws)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    got = out.t.cpu().numpy()
    np.testing.assert_array_equal(got[:, :N], oracle.xnor_gemm(X[:, :K], W[:, :N]))
    assert (got[:, N:] == -7).all()
    out.check()
    with pytest.raises(q.QnnError) as e:
        q.qnn_fc_sign_f32(dev(X), M, K, X.shape[1], dev(W), N, W.shape[1], out.t, N + 3, None)
    assert e.value.status == q.QNN_ERR_WORKSPACE


@pytest.mark.parametrize("M,dims,chunks", [(2100, (784, 1024, 1024, 10), 3), (300, (784, 512, 256, 10), 1), (5000, (784, 1024, 1024, 10), 4)])
def test_mlp_graph_from_host_buffers(q, M, dims, chunks):
    """The end-to-end pass (pinned host input -> scores in pinned host memory) as one CUDA graph: every replay, also
    with new inputs written into the same host buffer, must give the oracle's Algorithm-4 scores."""
    wl = workloads.mnist_mlp(M=M, dims=dims, seed=1)
    packed, ldws = [], []
    for W in wl.Ws:
        K, N = W.shape
        ld = (words_per_row(K) + 3) // 4 * 4
        o = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_sign_t(W.cuda(), K, N, N, o, ld)
        packed.append(o); ldws.append(ld)
    thr = [t.cuda() for t in wl.Ts]
    layers = q.make_mlp_layers(packed, ldws, dims[:-1], dims[1:], thr, [None] * len(thr))
    keep = q.prepack_mlp_weights(layers, packed, 8)                                   # noqa: F841
    ws = torch.empty(q.qnn_mlp_workspace_bytes(M, 8, layers, q.QNN_ALGO_AUTO, 1), dtype=torch.uint8, device="cuda")
    xh = wl.X.contiguous().pin_memory()
    sh = torch.full((M, dims[-1]), -7, dtype=torch.int32).pin_memory()
    g = q.MlpGraph(xh, M, 8, layers, sh, q.QNN_ALGO_AUTO, ws, chunks=chunks)
    Ws = [oracle.sign(w.numpy()) for w in wl.Ws]
    Ts = [t.numpy() for t in wl.Ts]
    want = oracle.mlp_forward(wl.X.numpy().astype(np.int32), Ws, Ts)
    for _ in range(2):
        sh.fill_(-7)
        g.launch()
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        np.testing.assert_array_equal(sh.numpy(), want)
    # new inputs through the same host buffer
    x2 = workloads.mnist_mlp(M=M, dims=dims, seed=1, stream=1).X
    xh.copy_(x2)
    g.launch()
    torch.cuda.synchronize()
    np.testing.assert_array_equal(sh.numpy(), oracle.mlp_forward(x2.numpy().astype(np.int32), Ws, Ts))
