"""GPU parity of the Table 7 layer types: first-layer convolution on pixel codes, pooled thresholds, the whole ConvNet."""
import numpy as np
import pytest
import torch

import oracle
from paper_1609_07061_b200 import workloads
from util import Guarded, dev, pack_bits_ref, unpack_words, words_np, words_per_row

pytestmark = pytest.mark.gpu

E2M1 = {0: 0x0, 1: 0x2, -1: 0xA}


@pytest.fixture(scope="module")
def q():
    import paper_1609_07061_b200.binding as b
    return b


def _form_bytes(bits01, C, kind, q):
    """Expected tensor-core form of rows of 0/1 bits: +-1 values, pad columns (up to whole words) zero."""
    rows = bits01.shape[0]
    vals = np.zeros((rows, words_per_row(C) * 32), np.int32)
    vals[:, :C] = 2 * bits01.astype(np.int32) - 1
    if kind == q.QNN_FORM_I8:
        return vals.astype(np.int8).view(np.uint8)
    nib = np.vectorize(E2M1.__getitem__)(vals).astype(np.uint8)
    return (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)


@pytest.mark.parametrize("B,C,H,W,Co,KS,pad,pad_code", [
    (2, 3, 32, 32, 128, 3, 1, 0), (1, 3, 9, 7, 40, 3, 1, 0), (2, 1, 8, 8, 33, 5, 2, 17), (1, 4, 6, 5, 16, 1, 0, 0),
    (1, 3, 8, 8, 8, 3, 0, 0), (3, 5, 11, 13, 70, 3, 1, 255)])
@pytest.mark.parametrize("kind", ["i8", "fp4"])
def test_conv2d_u8(q, B, C, H, W, Co, KS, pad, pad_code, kind):
    """8-bit codes x +-1 filters (Eq. 8 over the eight planes): int32, packed-bit and form outputs of one call."""
    rng = np.random.default_rng(B * 100 + C * 10 + H + Co)
    X = rng.integers(0, 256, (B, C, H, W)).astype(np.uint8)
    Wt = rng.uniform(-1, 1, (Co, C, KS, KS)).astype(np.float32)
    want = oracle.conv2d(X.astype(np.int32), oracle.sign(Wt), 1, pad, pad_code)
    Ho, Wo = want.shape[2], want.shape[3]
    span = int(np.abs(want).max()) // 2 + 1
    T = rng.integers(-span, span + 1, Co).astype(np.int32)
    flip = rng.integers(0, 2, Co).astype(np.uint8)
    wb = torch.zeros(Co, KS * KS * words_per_row(C), dtype=torch.int32, device="cuda")
    q.qnn_pack_conv_weights(dev(Wt), Co, C, KS, KS, wb)
    fk = q.QNN_FORM_I8 if kind == "i8" else q.QNN_FORM_FP4
    cwo = words_per_row(Co)
    out = Guarded((B, Co, Ho, Wo), torch.int32, fill=-7)
    bits = Guarded((B, Ho, Wo, cwo), torch.int32, fill=0)
    of = Guarded((B * Ho * Wo, cwo * (32 if kind == "i8" else 16)), torch.uint8, fill=0x5C)
    ws = torch.empty(q.qnn_conv2d_u8_workspace_bytes(B, C, H, W, Co, KS, KS, pad), dtype=torch.uint8, device="cuda")
    q.qnn_conv2d_u8(dev(X), B, C, H, W, wb, Co, KS, KS, pad, pad_code, out.t, dev(T), dev(flip), bits.t, of.t, fk, ws)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    np.testing.assert_array_equal(out.t.cpu().numpy(), want)
    rows = want.transpose(0, 2, 3, 1).reshape(-1, Co)
    wbits = oracle.threshold(rows, T, flip)
    np.testing.assert_array_equal(unpack_words(words_np(bits.t).reshape(-1, cwo), Co), wbits)
    np.testing.assert_array_equal(of.t.cpu().numpy(), _form_bytes(wbits, Co, fk, q))
    for g in (out, bits, of):
        g.check()


def test_conv2d_u8_argument_errors(q):
    x = torch.zeros(1, 3, 8, 8, dtype=torch.uint8, device="cuda")
    wb = torch.zeros(8, 9, dtype=torch.int32, device="cuda")
    out = torch.zeros(1, 8, 8, 8, dtype=torch.int32, device="cuda")
    ws = torch.empty(q.qnn_conv2d_u8_workspace_bytes(1, 3, 8, 8, 8, 3, 3, 1), dtype=torch.uint8, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_conv2d_u8(x, 1, 3, 8, 8, wb, 8, 3, 3, 1, 0, out_nchw=out, ws=None)
    assert e.value.status == q.QNN_ERR_WORKSPACE
    with pytest.raises(q.QnnError) as e:
        q.qnn_conv2d_u8(x, 1, 3, 8, 8, wb, 8, 3, 3, 1, 300, out_nchw=out, ws=ws)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    with pytest.raises(q.QnnError) as e:      # packed bits need thresholds
        q.qnn_conv2d_u8(x, 1, 3, 8, 8, wb, 8, 3, 3, 1, 0, out_bits=torch.zeros(64, dtype=torch.int32, device="cuda"), ws=ws)
    assert e.value.status == q.QNN_ERR_INVALID_ARG
    q.qnn_conv2d_u8(x, 0, 3, 8, 8, wb, 8, 3, 3, 1, 0, out_nchw=out, ws=ws)      # empty batch: nothing to do


@pytest.mark.parametrize("B,H,W,C", [(2, 8, 8, 128), (1, 7, 5, 40), (3, 2, 2, 33), (2, 16, 16, 256), (1, 32, 32, 512), (1, 4, 6, 7)])
@pytest.mark.parametrize("with_flip", [False, True])
def test_maxpool2x2_bits(q, B, H, W, C, with_flip):
    """Pooled bits must equal the threshold of the pooled integer sums (Table 7's order: pool, then batch norm + sign)."""
    rng = np.random.default_rng(B + H * 3 + W * 5 + C)
    s = rng.integers(-30, 30, (B, C, H, W)).astype(np.int32)
    T = rng.integers(-10, 11, C).astype(np.int32)
    flip = rng.integers(0, 2, C).astype(np.uint8) if with_flip else None
    rows = lambda t: t.transpose(0, 2, 3, 1).reshape(-1, C)
    want = oracle.threshold(rows(oracle.maxpool2x2(s)), T, flip)
    cw = words_per_row(C)
    in_bits = dev(pack_bits_ref(oracle.threshold(rows(s), T, flip)).view(np.int32).reshape(B, H, W, cw))
    Ho, Wo = H // 2, W // 2
    for fk, per_word in ((q.QNN_FORM_I8, 32), (q.QNN_FORM_FP4, 16)):
        ob = Guarded((B, Ho, Wo, cw), torch.int32, fill=0)
        of = Guarded((B * Ho * Wo, cw * per_word), torch.uint8, fill=0x5C)
        q.qnn_maxpool2x2_bits(in_bits, B, H, W, C, None if flip is None else dev(flip), ob.t, of.t, fk)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(unpack_words(words_np(ob.t).reshape(-1, cw), C), want)
        np.testing.assert_array_equal(of.t.cpu().numpy(), _form_bytes(want, C, fk, q))
        ob.check()
        of.check()


def _oracle_layers(wl):
    layers, t = [], 0
    for i, (Wc, pool) in enumerate(zip(wl.conv_W, wl.conv_pool)):
        layers.append(dict(kind="conv", W=oracle.sign(Wc.numpy()), pad=1, pad_value=0 if i == 0 else 1, pool=pool,
                           T=wl.Ts[t].numpy(), flip=wl.flips[t].numpy()))
        t += 1
    for j, Wf in enumerate(wl.fc_W):
        last = j == len(wl.fc_W) - 1
        layers.append(dict(kind="fc", W=oracle.sign(Wf.numpy()), T=None if last else wl.Ts[t].numpy(),
                           flip=None if last else wl.flips[t].numpy()))
        t += 0 if last else 1
    return layers


def _run_net(q, wl, B):
    H, W = wl.X.shape[2], wl.X.shape[3]
    net = q.ConvNet(wl.X.shape[1], H, W, wl.conv_W, wl.conv_pool, wl.fc_W, wl.Ts, wl.flips)
    ws = net.workspace(B)
    scores = Guarded((B, net.n_out), torch.int32, fill=-7)
    net.forward(wl.X[:B].cuda(), scores.t, ws)
    torch.cuda.synchronize()
    assert q.qnn_device_status() == 0, q.qnn_last_error()
    scores.check()
    return scores.t.cpu().numpy()


@pytest.mark.parametrize("B,H,W,widths,fc,thr", [
    (3, 8, 8, (8, 8, 16, 16), (24, 10), 3),                 # narrow layers: packed im2col path everywhere
    (2, 8, 8, (128, 128, 256, 256), (64, 10), 24),          # int8- and e2m1-form implicit convolutions, pooled hand-over
    (5, 12, 20, (128, 40, 40, 256, 256), (10,), 16),        # tensor-core and im2col layers mixed, odd sizes
    (1, 4, 4, (128, 128), (32, 16, 10), 16)])
def test_convnet_forward_small(q, B, H, W, widths, fc, thr):
    wl = workloads.cifar_convnet(B=B, H=H, W=W, widths=widths, fc=fc, seed=5, thr=thr)
    got = _run_net(q, wl, B)
    want = oracle.convnet_forward(wl.X.numpy().astype(np.int32), _oracle_layers(wl))
    np.testing.assert_array_equal(got, want)


def test_cifar_convnet_table7(q):
    """The full Table 7 network (2x128C3 - MP2 - 2x256C3 - MP2 - 2x512C3 - MP2 - 2x1024FC - 10) at batch 128;
    batch rows are independent, so the oracle checks a seeded sample of the images."""
    B = 128
    wl = workloads.cifar_convnet(B=B, seed=5)
    got = _run_net(q, wl, B)
    idx = np.sort(np.random.default_rng(0).choice(B, 8, replace=False))
    want = oracle.convnet_forward(wl.X.numpy().astype(np.int32)[idx], _oracle_layers(wl))
    np.testing.assert_array_equal(got[idx], want)
    # the same images in a smaller batch give the same scores (tiling does not leak between images)
    wl2 = workloads.cifar_convnet(B=B, seed=5)
    wl2.X = wl.X[torch.from_numpy(idx)]
    np.testing.assert_array_equal(_run_net(q, wl2, len(idx)), want)


def test_convnet_argument_errors(q):
    wl = workloads.cifar_convnet(B=2, H=8, W=8, widths=(8, 8), fc=(10,), seed=5, thr=3)
    net = q.ConvNet(3, 8, 8, wl.conv_W, wl.conv_pool, wl.fc_W, wl.Ts, wl.flips)
    scores = torch.zeros(2, 10, dtype=torch.int32, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_convnet_forward(wl.X.cuda(), 2, 8, 8, net.layers, net.prepared, scores, None)
    assert e.value.status == q.QNN_ERR_WORKSPACE
    # layers that do not chain: FC inputs must equal the feature map size
    net.layers[2].C = 77
    assert q.qnn_convnet_workspace_bytes(2, 8, 8, net.layers) == 0
    with pytest.raises(q.QnnError) as e:
        q.qnn_convnet_forward(wl.X.cuda(), 2, 8, 8, net.layers, net.prepared, scores, torch.empty(1 << 20, dtype=torch.uint8, device="cuda"))
    assert e.value.status == q.QNN_ERR_INVALID_ARG


def _capture(fn):
    """Runs fn() once eagerly (one-time kernel attributes), then captures a second call in a CUDA graph."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        fn()
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            fn()
    torch.cuda.synchronize()
    return g


def test_mlp_forward_replays_from_a_cuda_graph(q):
    """qnn_mlp_forward (Algorithm 4 as one call) is allocation-free and asynchronous: captured once in a CUDA
    graph, every replay must reproduce the oracle's scores, on the tensor-core chain with prepacked weights."""
    M, dims = 2100, (784, 1024, 1024, 10)
    wl = workloads.mnist_mlp(M=M, dims=dims, seed=1)
    packed, ldws = [], []
    for Wm in wl.Ws:
        K, N = Wm.shape
        ld = (words_per_row(K) + 3) // 4 * 4
        o = torch.zeros(N, ld, dtype=torch.int32, device="cuda")
        q.qnn_quantize_pack_sign_t(Wm.cuda(), K, N, N, o, ld)
        packed.append(o); ldws.append(ld)
    thr = [t.cuda() for t in wl.Ts]
    layers = q.make_mlp_layers(packed, ldws, dims[:-1], dims[1:], thr, [None] * len(thr))
    keep = q.prepack_mlp_weights(layers, packed, 8)                                   # noqa: F841
    assert q.qnn_select_algo(M, dims[2], dims[1], 1, 1, q.QNN_MODE_PM1, q.QNN_MODE_PM1) in (q.QNN_ALGO_TC_FP4, q.QNN_ALGO_TC_I8)
    ws = torch.empty(q.qnn_mlp_workspace_bytes(M, 8, layers, q.QNN_ALGO_AUTO, 0), dtype=torch.uint8, device="cuda")
    x = wl.X.cuda()
    scores = torch.zeros(M, dims[-1], dtype=torch.int32, device="cuda")
    g = _capture(lambda: q.qnn_mlp_forward(x, M, 8, layers, scores, q.QNN_ALGO_AUTO, ws))
    want = oracle.mlp_forward(wl.X.numpy().astype(np.int32), [oracle.sign(w.numpy()) for w in wl.Ws],
                              [t.numpy() for t in wl.Ts])
    for _ in range(3):
        scores.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        np.testing.assert_array_equal(scores.cpu().numpy(), want)


def test_convnet_forward_replays_from_a_cuda_graph(q):
    """qnn_convnet_forward likewise: captured once in a CUDA graph, a replay must reproduce the oracle's scores
    (the tensor-core kernels inside are launched with programmatic stream serialisation, which the capture has
    to carry over)."""
    B = 64
    wl = workloads.cifar_convnet(B=B, H=16, W=16, widths=(128, 128, 256, 256), fc=(256, 10), seed=5, thr=24)
    net = q.ConvNet(3, 16, 16, wl.conv_W, wl.conv_pool, wl.fc_W, wl.Ts, wl.flips)
    ws = net.workspace(B)
    x = wl.X.cuda()
    scores = torch.zeros(B, net.n_out, dtype=torch.int32, device="cuda")
    g = _capture(lambda: net.forward(x, scores, ws))
    want = oracle.convnet_forward(wl.X.numpy().astype(np.int32), _oracle_layers(wl))
    for _ in range(3):
        scores.fill_(-7)
        g.replay()
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        np.testing.assert_array_equal(scores.cpu().numpy(), want)


def test_degenerate_sizes(q):
    """Empty batches and images without a 2 x 2 window are valid no-ops; nothing is written."""
    wl = workloads.cifar_convnet(B=1, H=8, W=8, widths=(8, 8), fc=(10,), seed=5, thr=3)
    net = q.ConvNet(3, 8, 8, wl.conv_W, wl.conv_pool, wl.fc_W, wl.Ts, wl.flips)
    scores = Guarded((1, 10), torch.int32, fill=-7)
    q.qnn_convnet_forward(wl.X.cuda(), 0, 8, 8, net.layers, net.prepared, scores.t, None)       # B = 0: no workspace needed
    bits = torch.zeros(2, 1, 5, 1, dtype=torch.int32, device="cuda")
    ob = Guarded((2, 0, 2, 1), torch.int32, fill=0)
    q.qnn_maxpool2x2_bits(bits, 2, 1, 5, 8, None, ob.t, None, 0)                                 # a single row: no window
    q.qnn_maxpool2x2_bits(bits, 0, 4, 4, 8, None, ob.t, None, 0)
    out = Guarded((4, 32), torch.uint8, fill=0x5C)
    q.qnn_logquant_pack_i8(torch.zeros(4, 8, device="cuda"), 0, 8, 8, -1, 1, out.t, 32)
    q.qnn_logquant_pack_i8(torch.zeros(4, 8, device="cuda"), 4, 0, 8, -1, 1, out.t, 32)
    torch.cuda.synchronize()
    assert (scores.t.cpu().numpy() == -7).all() and (out.t.cpu().numpy() == 0x5C).all()
    for g in (scores, ob, out):
        g.check()


@pytest.mark.parametrize("B,C,H,W,Co", [(3, 256, 16, 16, 256), (5, 128, 8, 8, 70), (2, 128, 4, 4, 32), (2, 256, 6, 16, 40), (1, 512, 2, 2, 33),
                                         (9, 256, 8, 8, 64)])
def test_conv_with_pooling_inside_the_call(q, B, C, H, W, Co):
    """conv -> 2x2 max-pool -> threshold (Table 7's order) in one call: the epilogue pools the thresholded signs."""
    rng = np.random.default_rng(B + C + H + W + Co)
    X = rng.standard_normal((B, C, H, W)).astype(np.float32)
    Wt = rng.uniform(-1, 1, (Co, C, 3, 3)).astype(np.float32)
    T = (rng.integers(-24, 25, Co) + int(round((9 * C) ** 0.5))).astype(np.int32)
    flip = rng.integers(0, 2, Co).astype(np.uint8)
    s = oracle.conv2d(oracle.sign(X), oracle.sign(Wt), 1, 1, 1)
    pooled = oracle.maxpool2x2(s)
    want = oracle.threshold(pooled.transpose(0, 2, 3, 1).reshape(-1, Co), T, flip)
    assert 0.02 < want.mean() < 0.98                       # both outcomes occur, so the comparison means something
    cw, cwo = words_per_row(C), words_per_row(Co)
    xb = torch.zeros(B, H, W, cw, dtype=torch.int32, device="cuda")
    wb = torch.zeros(Co, 9 * cw, dtype=torch.int32, device="cuda")
    q.qnn_quantize_pack_sign_nchw(dev(X), B, C, H, W, xb)
    q.qnn_pack_conv_weights(dev(Wt), Co, C, 3, 3, wb)
    prep = torch.empty(q.qnn_conv_prepared_bytes(Co, C, 3, 3, 1), dtype=torch.uint8, device="cuda")
    q.qnn_conv_prepare(wb, Co, C, 3, 3, 1, 1, prep)
    assert q.qnn_conv_can_pool(H, W)
    ws = torch.empty(B * H * W * cw * 32 + 256, dtype=torch.uint8, device="cuda")
    Hp, Wp = H // 2, W // 2
    for fk, per_word in ((q.QNN_FORM_FP4, 16), (q.QNN_FORM_I8, 32)):
        bits = Guarded((B, Hp, Wp, cwo), torch.int32, fill=0)
        of = Guarded((B * Hp * Wp, cwo * per_word), torch.uint8, fill=0x5C)
        q.qnn_binary_conv2d_prepared(xb, 0, B, C, H, W, prep, Co, 3, 3, 1, thr=dev(T), flip=dev(flip), out_bits=bits.t, out_form=of.t,
                                     out_form_kind=fk, ws=ws, pool2x2=1)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        np.testing.assert_array_equal(unpack_words(words_np(bits.t).reshape(-1, cwo), Co), want)
        np.testing.assert_array_equal(of.t.cpu().numpy(), _form_bytes(want, Co, fk, q))
        bits.check()
        of.check()


def test_pooling_inside_the_call_is_refused_for_wide_images(q):
    assert not q.qnn_conv_can_pool(32, 32) and not q.qnn_conv_can_pool(7, 8)
    xb = torch.zeros(1, 32, 32, 4, dtype=torch.int32, device="cuda")
    wb = torch.zeros(32, 36, dtype=torch.int32, device="cuda")
    prep = torch.empty(q.qnn_conv_prepared_bytes(32, 128, 3, 3, 1), dtype=torch.uint8, device="cuda")
    q.qnn_conv_prepare(wb, 32, 128, 3, 3, 1, 1, prep)
    ws = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(q.QnnError) as e:
        q.qnn_binary_conv2d_prepared(xb, 0, 1, 128, 32, 32, prep, 32, 3, 3, 1, thr=torch.zeros(32, dtype=torch.int32, device="cuda"),
                                     out_bits=torch.zeros(256, dtype=torch.int32, device="cuda"), ws=ws, pool2x2=1)
    assert e.value.status == q.QNN_ERR_UNSUPPORTED


def test_back_to_back_passes_do_not_interfere(q):
    """Kernels of consecutive passes overlap their starts with the previous kernel's tail (programmatic stream
    serialisation) and share one workspace: many passes queued without synchronisation, on alternating inputs, must each
    give the result of a lone pass."""
    B = 32
    wl = workloads.cifar_convnet(B=B, H=16, W=16, widths=(128, 128, 256, 256), fc=(256, 10), seed=5, thr=24)
    net = q.ConvNet(3, 16, 16, wl.conv_W, wl.conv_pool, wl.fc_W, wl.Ts, wl.flips)
    ws = net.workspace(B)
    xs = [wl.X.cuda(), workloads.cifar_convnet(B=B, H=16, W=16, widths=(128, 128, 256, 256), fc=(256, 10), seed=5, thr=24,
                                               stream=1).X.cuda()]
    ref = []
    for x in xs:
        s = torch.zeros(B, 10, dtype=torch.int32, device="cuda")
        net.forward(x, s, ws)
        torch.cuda.synchronize()
        ref.append(s.clone())
    np.testing.assert_array_equal(ref[0].cpu().numpy(), oracle.convnet_forward(wl.X.numpy().astype(np.int32), _oracle_layers(wl)))
    assert not torch.equal(ref[0], ref[1])
    outs = [torch.zeros(B, 10, dtype=torch.int32, device="cuda") for _ in range(48)]
    for _ in range(3):
        for i, o in enumerate(outs):
            net.forward(xs[i & 1], o, ws)
        torch.cuda.synchronize()
        assert q.qnn_device_status() == 0, q.qnn_last_error()
        for i, o in enumerate(outs):
            assert torch.equal(o, ref[i & 1]), f"pass {i} differs"
            o.zero_()
